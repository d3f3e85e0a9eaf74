"""The benchmark configurations at their full sizes, in the launch configuration bench.py times.
The oracle cannot run these whole, so each test compares seeded SAMPLES of the outputs with the oracle
(sequences / rows it can compute one by one, from a host mirror that holds only their blocks) and checks
properties that hold at any size (bitwise reproducibility, chunked == one-shot, bit-identical outputs
across shrink/grow, elastic bytes read back exactly)."""
import math
import os
import sys

import numpy as np
import pytest
import torch

import ekv_inputs as I
import oracle
import paper_2608_23658_b200 as ekv
from helpers import bf16_bits

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
DEV = torch.device("cuda", 0)
MAX_ABS, MEAN_ABS = 2e-2, 2e-3
GiB = 1 << 30


def check_close(got_bf16, want_f64, what):
    got = got_bf16.detach().float().cpu().numpy().astype(np.float64)
    assert got.shape == want_f64.shape, (got.shape, want_f64.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite"
    err = np.abs(got - want_f64)
    assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, f"{what}: max-abs {err.max():.4g} mean-abs {err.mean():.4g}"


def host_mirror(seed, layer, tables, lengths, seq_ids, shape):
    cache, ctab, clen = I.compact_host_cache(seed, layer, tables, lengths, seq_ids, shape)
    return bf16_bits(cache).copy(), ctab, clen


# ------------------------------------------------------------------ configs[1]


def test_c2_llama8b_decode_step_sampled_against_oracle():
    sys.path.insert(0, ROOT)
    import bench
    cfg, s = I.C2, I.C2.shape
    wl = bench.DecodeWorkload(cfg, DEV)
    try:
        assert wl.B == 256 and int(wl.lengths.min()) >= 1024 and int(wl.lengths.max()) <= 8192
        wl.step_resident()
        torch.cuda.synchronize()
        first = wl.out.clone()
        wl.step_resident()
        torch.cuda.synchronize()
        assert torch.equal(first, wl.out), "the step is not bitwise reproducible"
        assert wl.pool.poll_status() == ekv.Status.OK
        order = torch.argsort(wl.lengths)
        ids = [int(order[0]), int(order[len(order) // 2]), int(order[-1])]
        cache, ctab, clen = host_mirror(cfg.seed, 0, wl.tables, wl.lengths, ids, s)
        # the device generator and its CPU regeneration agree on the sampled blocks
        nb0 = int(I.blocks_for(wl.lengths[ids[0]:ids[0] + 1], 16)[0])
        blk = wl.tables[ids[0], :nb0].long()
        dev_bits = bf16_bits(wl.pool.layer_tensor(0)[blk.to(DEV)].cpu()).reshape(-1)
        # (position L-1 of each sequence was overwritten by the step's ekv_write_kv: apply the same write on the host)
        slots = torch.stack([ctab[i, (int(clen[i]) - 1) // 16].long() * 16 + (int(clen[i]) - 1) % 16 for i in range(3)])
        assert oracle.write_kv(cache, int(ctab.max()) + 1, s.num_kv_heads, 16, s.head_dim, wl.h_k[ids], wl.h_v[ids], slots) == 0
        assert np.array_equal(dev_bits, cache[:nb0 * s.block_elems])
        want = oracle.attn_decode(cache, s.num_q_heads, s.num_kv_heads, 16, s.head_dim, wl.h_q[ids], ctab, clen, wl.scale)
        check_close(wl.out[ids], want, "C2 sampled sequences")
    finally:
        wl.close()


# ------------------------------------------------------------------ configs[2]


def test_c3_mixed_chunked_prefill_step():
    cfg, s = I.C3, I.C3.shape
    Lp = cfg.prompt_len
    lengths = I.decode_lengths(cfg)
    need = int(I.blocks_for(lengths, 16).sum()) + Lp // 16
    pool = ekv.Pool(num_q_heads=s.num_q_heads, num_kv_heads=s.num_kv_heads, head_dim=s.head_dim, base_blocks=int(need * 1.05))
    try:
        live = pool.info.live_blocks
        all_len = torch.cat([lengths, torch.tensor([Lp])])
        tables, _ = I.assign_blocks(cfg.seed, 12, all_len, 16, live)
        I.fill_pool_layer_(pool.layer_tensor(0), cfg.seed)
        d_tables = tables.to(DEV)
        dec_tables, prm_table = d_tables[:256].contiguous(), d_tables[256:257].contiguous()
        scale = 1 / math.sqrt(s.head_dim)
        n_kv = Lp * s.num_kv_heads * s.head_dim
        K = I.normal_bf16(cfg.seed, 7, 0, n_kv, device=DEV).view(Lp, s.num_kv_heads, s.head_dim)
        V = I.normal_bf16(cfg.seed, 8, 0, n_kv, device=DEV).view(Lp, s.num_kv_heads, s.head_dim)
        Q = I.normal_bf16(cfg.seed, 6, 0, Lp * s.num_q_heads * s.head_dim, device=DEV).view(Lp, s.num_q_heads, s.head_dim)
        qd = I.normal_bf16(cfg.seed, 3, 0, 256 * s.num_q_heads * s.head_dim, device=DEV).view(256, s.num_q_heads, s.head_dim)
        d_lens = lengths.to(torch.int32).to(DEV)
        slots = I.position_slots(tables[256], 0, Lp, 16).to(DEV)

        def step(start, c, out):
            """one engine step: write the chunk's K/V, chunk attention over prefix + itself, and the decode batch"""
            pool.write_kv(0, K[start:start + c], V[start:start + c], slots[start:start + c])
            cu = torch.tensor([0, c], dtype=torch.int32)
            pool.attn_prefill_chunk(0, Q[start:start + c], prm_table, cu.to(DEV), cu,
                                    torch.tensor([start + c], dtype=torch.int32, device=DEV), scale, out=out[start:start + c])
            return pool.attn_decode(0, qd, dec_tables, d_lens, scale)

        chunked, one = torch.empty_like(Q), torch.empty_like(Q)
        dec = [step(st, 8192, chunked) for st in range(0, Lp, 8192)]
        dec.append(step(0, Lp, one))
        torch.cuda.synchronize()
        assert pool.poll_status() == ekv.Status.OK
        for d in dec[1:]:
            assert torch.equal(dec[0], d)                       # the decode batch does not care about the prefill
        diff = (chunked.float() - one.float()).abs()
        assert diff.max().item() <= MAX_ABS and diff.mean().item() <= MEAN_ABS, "chunked vs one-shot"

        # oracle on a seeded sample of rows: first / last row of every chunk plus random ones, all heads
        rows = sorted(set([0, 1, 127, 128, 8191, 8192, 16383, 16384, 24575, 24576, Lp - 1] +
                          I.uniform_ints(cfg.seed, 31, 56, 0, Lp - 1).tolist()))
        nb = Lp // 16
        cache = np.zeros(nb * s.block_elems, dtype=np.uint16)
        ctab = torch.arange(nb, dtype=torch.int32)[None]
        assert oracle.write_kv(cache, nb, s.num_kv_heads, 16, s.head_dim, K.cpu(), V.cpu(), torch.arange(Lp)) == 0
        want = oracle.attn_prefill_chunk(cache, s.num_q_heads, s.num_kv_heads, 16, s.head_dim, Q.cpu(), ctab,
                                         np.array([0, Lp]), np.array([Lp]), scale, rows=np.array(rows))
        check_close(one[rows], want, "C3 one-shot rows")
        check_close(chunked[rows], want, "C3 chunked rows")
        # and two sampled decode sequences
        ids = [3, 200]
        dcache, dtab, dlen = host_mirror(cfg.seed, 0, tables, all_len, ids, s)
        wantd = oracle.attn_decode(dcache, s.num_q_heads, s.num_kv_heads, 16, s.head_dim, qd[ids].cpu(), dtab, dlen, scale)
        check_close(dec[0][ids], wantd, "C3 decode sample")
    finally:
        pool.close()


def test_prefill_chunk_over_a_128k_token_prefix():
    """The last 1024-token chunk of a 131072-token prompt (8192 blocks in the table, 1024 key tiles per query tile):
    the prefill kernel at the longest context of the configs, sampled rows against the oracle."""
    s = I.LLAMA8B
    Lp, c = 131072, 1024
    pool = ekv.Pool(num_q_heads=s.num_q_heads, num_kv_heads=s.num_kv_heads, head_dim=s.head_dim, base_blocks=Lp // 16 + 96)
    try:
        lengths = torch.tensor([Lp])
        tables, _ = I.assign_blocks(I.C4.seed, 21, lengths, 16, pool.info.live_blocks)
        I.fill_pool_layer_(pool.layer_tensor(0), I.C4.seed)
        Q = I.normal_bf16(I.C4.seed, 6, 0, c * s.num_q_heads * s.head_dim, device=DEV).view(c, s.num_q_heads, s.head_dim)
        cu = torch.tensor([0, c], dtype=torch.int32)
        scale = 1 / math.sqrt(s.head_dim)
        out = pool.attn_prefill_chunk(0, Q, tables.to(DEV), cu.to(DEV), cu, lengths.to(torch.int32).to(DEV), scale)
        again = pool.attn_prefill_chunk(0, Q, tables.to(DEV), cu.to(DEV), cu, lengths.to(torch.int32).to(DEV), scale)
        torch.cuda.synchronize()
        assert pool.poll_status() == ekv.Status.OK
        assert torch.equal(out, again)
        rows = [0, 1, 127, 128, 500, c - 1]
        cache, ctab, clen = host_mirror(I.C4.seed, 0, tables, lengths, [0], s)
        want = oracle.attn_prefill_chunk(cache, s.num_q_heads, s.num_kv_heads, 16, s.head_dim, Q.cpu(), ctab,
                                         np.array([0, c]), clen, scale, rows=np.array(rows))
        check_close(out[rows], want, "prefill over a 130048-token prefix")
    finally:
        pool.close()


# ------------------------------------------------------------------ configs[3]


def test_c4_long_context_70b_shape_with_elastic_blocks():
    cfg, s = I.C4, I.C4.shape
    lengths = I.decode_lengths(cfg)
    need = int(I.blocks_for(lengths, 16).sum())
    free, _ = torch.cuda.mem_get_info()
    budget = min(140 * GiB, free - 10 * GiB)                    # "sized to fill most of HBM"
    total = budget // s.block_bytes
    assert total > need * 1.02, f"pool of {budget / GiB:.1f} GiB cannot hold the draw ({need} blocks)"
    elastic = int(total * cfg.elastic_fraction)
    pool = ekv.Pool(num_q_heads=s.num_q_heads, num_kv_heads=s.num_kv_heads, head_dim=s.head_dim,
                    base_blocks=total - elastic, elastic_blocks=elastic, start_grown=True)
    try:
        info = pool.info
        live = info.live_blocks
        tables, _ = I.assign_blocks(cfg.seed, 12, lengths, 16, live)
        used = tables[tables >= 0]
        frac_elastic = float((used >= info.base_blocks).float().mean())
        assert 0.14 < frac_elastic < 0.18, frac_elastic          # ~16 % of every draw lives in the elastic range
        # only the blocks the batch touches need defined content: fill them (same function of the physical index)
        view = pool.layer_tensor(0)
        ids_sorted = torch.sort(used.long()).values.to(DEV)
        for o in range(0, len(ids_sorted), 4096):
            idx = ids_sorted[o:o + 4096]
            elem = (idx[:, None] * s.block_elems + torch.arange(s.block_elems, device=DEV)[None]).reshape(-1)
            vals = I.normal_bf16_at(cfg.seed, I.KV_STREAM, elem)
            view[idx] = vals.view(len(idx), 2, s.num_kv_heads, 16, s.head_dim)
        B = len(lengths)
        q = I.normal_bf16(cfg.seed, 3, 0, B * s.num_q_heads * s.head_dim, device=DEV).view(B, s.num_q_heads, s.head_dim)
        scale = 1 / math.sqrt(s.head_dim)
        d_tables, d_lens = tables.to(DEV), lengths.to(torch.int32).to(DEV)
        out = pool.attn_decode(0, q, d_tables, d_lens, scale)
        again = pool.attn_decode(0, q, d_tables, d_lens, scale)
        torch.cuda.synchronize()
        assert pool.poll_status() == ekv.Status.OK
        assert torch.equal(out, again)
        ids = [int(torch.argmin(lengths)), int(torch.argmax(lengths))]
        for b in ids:                                            # one mirror at a time: up to 0.5 GB each
            cache, ctab, clen = host_mirror(cfg.seed, 0, tables, lengths, [b], s)
            want = oracle.attn_decode(cache, s.num_q_heads, s.num_kv_heads, 16, s.head_dim, q[b:b + 1].cpu(), ctab, clen, scale)
            check_close(out[b:b + 1], want, f"C4 sequence {b} ({int(lengths[b])} keys)")
    finally:
        pool.close()


# ------------------------------------------------------------------ configs[4]


@pytest.mark.parametrize("fused", [False, True])
def test_c5_elastic_toggle_under_load(fused):
    """32 layers, batch 128, 1000 decode steps (EKV_C5_STEPS overrides), shrink/grow alternating every 50 steps.
    fused=True repeats the protocol (300 steps) on a pool with ONE range for all layers (EKV_FUSED_RANGE).
    112 tenants live in base blocks only; 16 'straddlers' take their new blocks from the elastic range while it
    is mapped and are drained to spare base blocks before every shrink."""
    cfg, s = I.C5, I.C5.shape
    steps = int(os.environ.get("EKV_C5_STEPS", 300 if fused else cfg.steps))
    NL, B, every = cfg.num_layers, cfg.decode.batch, cfg.toggle_every
    lengths = I.decode_lengths(cfg)
    elastic_blocks = cfg.elastic_total_bytes // NL // s.block_bytes
    end_blocks = int(I.blocks_for(lengths + steps, 16).sum())
    base_blocks = end_blocks + 512
    need_bytes = NL * (base_blocks + elastic_blocks) * s.block_bytes
    free, _ = torch.cuda.mem_get_info()
    assert need_bytes + 3 * GiB < free, f"configs[4] needs {need_bytes / GiB:.1f} GiB, device has {free / GiB:.1f} GiB free"
    pool = ekv.Pool(num_q_heads=s.num_q_heads, num_kv_heads=s.num_kv_heads, head_dim=s.head_dim, base_blocks=base_blocks,
                    elastic_blocks=elastic_blocks, num_layers=NL, start_grown=True, fused_range=fused)
    try:
        info = pool.info
        assert info.num_ranges == (1 if fused else NL)
        base, el = info.base_blocks, info.elastic_blocks
        for l in range(NL):
            I.fill_pool_layer_(pool.layer_tensor(l, 0, base), cfg.seed, layer=l)
        width = int(I.blocks_for(lengths + steps, 16).max())
        tables, spare = I.assign_blocks(cfg.seed, 12, lengths, 16, base, max_blocks_per_seq=width)
        free_base, free_el = spare.tolist(), list(range(base, base + el))
        straddler = torch.zeros(B, dtype=torch.bool)
        straddler[::8] = True                                    # 16 of 128
        tenants = torch.nonzero(~straddler).flatten()
        cur = lengths.clone()
        scale = 1 / math.sqrt(s.head_dim)
        q = I.normal_bf16(cfg.seed, 3, 0, B * s.num_q_heads * s.head_dim, device=DEV).view(B, s.num_q_heads, s.head_dim)
        ws = pool.workspace(B, width * 16)
        out = torch.empty_like(q)
        d_tables = tables.to(DEV)
        sample_b, sample_l = int(tenants[5]), 17                 # one base tenant, one layer: full oracle check at the end
        sample_rows = []
        grown, toggles = True, {"shrink": [], "grow": []}

        def new_rows(step):
            """K and V rows of this step's tokens for every layer: [NL, 2, B, Hkv, d]"""
            n = NL * 2 * B * s.num_kv_heads * s.head_dim
            return I.normal_bf16(cfg.seed, 100, step * n, n, device=DEV).view(NL, 2, B, s.num_kv_heads, s.head_dim)

        def probe(layer, who):
            """decode of frozen queries over the CURRENT contents for the given sequences"""
            return pool.attn_decode(layer, q[who].contiguous(), d_tables[who].contiguous(),
                                    cur[who].to(torch.int32).to(DEV), scale).clone()

        for step in range(steps):
            if step > 0 and step % every == 0:
                before = [probe(l, tenants) for l in (0, NL - 1)]
                if grown:
                    strad = torch.nonzero(straddler).flatten()
                    s_before = probe(3, strad)
                    # drain: move every elastic block of a straddler to a spare base block, all layers
                    moved = torch.nonzero(tables >= base)
                    olds = tables[moved[:, 0], moved[:, 1]].long()
                    news = torch.tensor([free_base.pop() for _ in range(len(olds))], dtype=torch.long)
                    for l in range(NL):
                        view = pool.layer_tensor(l)
                        view[news.to(DEV)] = view[olds.to(DEV)]
                    tables[moved[:, 0], moved[:, 1]] = news.to(torch.int32)
                    free_el += olds.tolist()
                    d_tables = tables.to(DEV)
                    toggles["shrink"].append(pool.shrink())
                    grown = False
                    assert pool.info.live_blocks == base
                    assert torch.equal(probe(3, strad), s_before), "drained straddlers changed"
                else:
                    toggles["grow"].append(pool.grow())
                    grown = True
                    # re-granted blocks read back exactly what is written after the remap
                    kv1 = new_rows(steps + step)
                    k1, v1 = kv1[0, 0], kv1[0, 1]
                    blk = base + (step // every) % el
                    pool.write_kv(5, k1[:1], v1[:1], torch.tensor([blk * 16 + 7], device=DEV))
                    got = pool.layer_tensor(5, blk, 1)
                    assert torch.equal(got[0, 0, :, 7, :], k1[0])
                    tbl = torch.tensor([[blk]], dtype=torch.int32, device=DEV)
                    pool.write_kv(5, k1[:1], v1[:1], torch.tensor([blk * 16], device=DEV))
                    o1 = pool.attn_decode(5, q[:1], tbl, torch.tensor([1], dtype=torch.int32, device=DEV), scale)
                    assert torch.equal(o1[0], v1[0].repeat_interleave(s.group, 0))
                after = [probe(l, tenants) for l in (0, NL - 1)]
                for a, b_ in zip(before, after):
                    assert torch.equal(a, b_), "base-resident outputs changed across a toggle"
            # append one token to every sequence
            pos = cur.clone()
            needs = torch.nonzero(pos % 16 == 0).flatten().tolist()
            for b in needs:
                pool_list = free_el if (grown and bool(straddler[b])) else free_base
                tables[b, int(pos[b]) // 16] = pool_list.pop()
            if needs:
                d_tables = tables.to(DEV)
            cur = cur + 1
            slots = (tables[torch.arange(B), pos // 16].long() * 16 + pos % 16).to(DEV)
            d_lens = cur.to(torch.int32).to(DEV)
            kv = new_rows(step)
            for l in range(NL):
                k, v = kv[l, 0], kv[l, 1]
                pool.write_kv(l, k, v, slots)
                pool.attn_decode(l, q, d_tables, d_lens, scale, out=out, workspace=ws)
                if l == sample_l:
                    sample_rows.append((k[sample_b].cpu(), v[sample_b].cpu()))
                    last = out[sample_b:sample_b + 1].clone()
        torch.cuda.synchronize()
        assert pool.poll_status() == ekv.Status.OK
        assert len(toggles["shrink"]) + len(toggles["grow"]) == (steps - 1) // every
        # full oracle check of one base tenant at one layer after all steps: initial fill + every appended row
        L0, L1 = int(lengths[sample_b]), int(cur[sample_b])
        nb = (L1 + 15) // 16
        row = tables[sample_b, :nb]
        assert (row >= 0).all() and (row < base).all()
        nb0 = (L0 + 15) // 16
        cache = np.zeros(nb * s.block_elems, dtype=np.uint16)
        cache[:nb0 * s.block_elems] = bf16_bits(I.host_blocks(cfg.seed, sample_l, row[:nb0].tolist(), s.block_elems)).reshape(-1)
        ks = torch.stack([r[0] for r in sample_rows])
        vs = torch.stack([r[1] for r in sample_rows])
        assert oracle.write_kv(cache, nb, s.num_kv_heads, 16, s.head_dim, ks, vs, torch.arange(L0, L1)) == 0
        want = oracle.attn_decode(cache, s.num_q_heads, s.num_kv_heads, 16, s.head_dim, q[sample_b:sample_b + 1].cpu(),
                                  torch.arange(nb, dtype=torch.int32)[None], np.array([L1]), scale)
        check_close(last, want, "C5 sampled tenant after all steps")
        ms = {k: [round(t[0], 2) for t in v] for k, v in toggles.items()}
        print(f"\nC5 toggles{' (fused range)' if fused else ''} (driver-call ms; the whole call also drains the queued steps), {NL} layers x "
              f"{el * s.block_bytes >> 20} MiB: {ms}")
    finally:
        pool.close()
