"""CUDA-graph replay across commit / decommit (the paper verifies its scheme with CUDA graphs enabled):
a decode step captured once keeps working, bit for bit, after ekv_shrink and ekv_grow, because nothing a
captured launch holds -- the layer pointer, the tensor map, the address of the live-limit word -- changes
when the elastic slice is mapped or unmapped.  The block table is a device buffer the graph re-reads, so a
drain (blocks moved, table rewritten in place) is picked up by the same graph."""
import math

import pytest
import torch

import ekv_inputs as I
import oracle
import paper_2608_23658_b200 as ekv
from helpers import assert_close, mirror_after_step

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_captured_decode_and_prefill_steps_replay_across_toggles():
    s = I.LLAMA8B
    NL = 4
    pool = ekv.Pool(num_q_heads=s.num_q_heads, num_kv_heads=s.num_kv_heads, head_dim=s.head_dim, base_blocks=512,
                    elastic_blocks=128, num_layers=NL, start_grown=True)
    try:
        info = pool.info
        base, el = info.base_blocks, info.elastic_blocks
        for l in range(NL):
            I.fill_pool_layer_(pool.layer_tensor(l), 9, layer=l)
        lengths = torch.tensor([900, 33, 1500, 257, 1024, 64])
        B = len(lengths)
        tables, spare = I.assign_blocks(9, 4, lengths, 16, base)                    # base tenants ...
        tables[2, 40:60] = torch.arange(base + 10, base + 30, dtype=torch.int32)     # ... and one straddler
        d_tables, d_lens = tables.to(DEV), lengths.to(torch.int32).to(DEV)
        q = I.normal_bf16(9, 3, 0, B * s.num_q_heads * s.head_dim, device=DEV).view(B, s.num_q_heads, s.head_dim)
        k = I.normal_bf16(9, 4, 0, B * s.num_kv_heads * s.head_dim, device=DEV).view(B, s.num_kv_heads, s.head_dim)
        v = I.normal_bf16(9, 5, 0, B * s.num_kv_heads * s.head_dim, device=DEV).view(B, s.num_kv_heads, s.head_dim)
        slots = I.last_token_slots(lengths, tables, 16).to(DEV)
        outs = [torch.empty_like(q) for _ in range(NL)]
        ws = pool.workspace(B, int(tables.shape[1]) * 16)
        c = 300
        qp = I.normal_bf16(9, 6, 0, c * s.num_q_heads * s.head_dim, device=DEV).view(c, s.num_q_heads, s.head_dim)
        outp = torch.empty_like(qp)
        cu = torch.tensor([0, c], dtype=torch.int32)
        d_cu, p_len = cu.to(DEV), torch.tensor([1500], dtype=torch.int32, device=DEV)
        scale = 1 / math.sqrt(s.head_dim)

        def step():
            for l in range(NL):
                pool.write_kv(l, k, v, slots)
                pool.attn_decode(l, q, d_tables, d_lens, scale, out=outs[l], workspace=ws)
            pool.attn_prefill_chunk(0, qp, d_tables[2:3], d_cu, cu, p_len, scale, out=outp)   # chunk of the straddler

        step()                                     # eager warm-up: first-call set-up happens outside the capture
        torch.cuda.synchronize()
        eager = [o.clone() for o in outs] + [outp.clone()]
        # the eager step against the oracle (every layer's decode of all six sequences, and the straddler's chunk);
        # the replays below are then pinned to it bit for bit
        for l in range(NL):
            cache, ctab, clen = mirror_after_step(9, l, tables, lengths, range(B), s, k.cpu(), v.cpu())
            want = oracle.attn_decode(cache, s.num_q_heads, s.num_kv_heads, 16, s.head_dim, q.cpu(), ctab, clen, scale)
            assert_close(eager[l], want, f"eager decode, layer {l}")
            if l == 0:
                wantp = oracle.attn_prefill_chunk(cache, s.num_q_heads, s.num_kv_heads, 16, s.head_dim, qp.cpu(), ctab[2:3],
                                                  cu, clen[2:3], scale)
                assert_close(eager[NL], wantp, "eager prefill chunk of the straddler")
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step()

        def replay():
            for o in outs:
                o.zero_()
            outp.zero_()
            graph.replay()
            torch.cuda.synchronize()
            return [o.clone() for o in outs] + [outp.clone()]

        for a, b in zip(replay(), eager):
            assert torch.equal(a, b)
        # drain the straddler to spare base blocks (table rewritten in place), then decommit
        src = tables[2, 40:60].to(DEV)
        dst = spare[:20].to(torch.int32).to(DEV)
        ekv.ekv_move_blocks(pool.handle, src, dst)
        d_tables[2, 40:60] = dst
        slots.copy_(I.last_token_slots(lengths, d_tables.cpu(), 16))
        pool.shrink()
        for a, b in zip(replay(), eager):
            assert torch.equal(a, b), "replay after decommit differs"
        pool.grow()
        for a, b in zip(replay(), eager):
            assert torch.equal(a, b), "replay after recommit differs"
        pool.shrink(keep_physical=True)
        pool.grow()
        for a, b in zip(replay(), eager):
            assert torch.equal(a, b)
        assert pool.poll_status() == ekv.Status.OK
        # what the graph buys on a launch-bound step (4 layers x 3 kernels + 2): eager vs replay
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        e0.record()
        for _ in range(20):
            step()
        e1.record()
        for _ in range(20):
            graph.replay()
        e2.record()
        torch.cuda.synchronize()
        print(f"\neager step {e0.elapsed_time(e1) / 20:.3f} ms, graph replay {e1.elapsed_time(e2) / 20:.3f} ms")
    finally:
        pool.close()
