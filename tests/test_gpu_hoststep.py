"""ekv_hoststep_*: a decode step driven from pinned host buffers gives exactly the bits of the device-resident
calls, for every step of a pipelined sequence of steps, and leaves the same bytes in the cache."""
import math

import pytest
import torch

import ekv_inputs as I
import oracle
from helpers import assert_close, bf16_bits

pytestmark = pytest.mark.gpu


def _pin(t):
    return t.contiguous().pin_memory()


@pytest.mark.parametrize("depth", [1, 2, 3])
def test_hoststep_matches_resident_calls_bitwise(depth):
    import paper_2608_23658_b200 as ekv
    dev = torch.device("cuda:0")
    s = I.LLAMA8B
    B, steps = 24, 7
    lengths0 = I.uniform_ints(91, 1, B, 200, 1500)
    max_len = int(lengths0.max()) + steps
    with ekv.Pool(num_q_heads=s.num_q_heads, num_kv_heads=s.num_kv_heads, head_dim=s.head_dim, base_blocks=4096) as pool, \
            ekv.Pool(num_q_heads=s.num_q_heads, num_kv_heads=s.num_kv_heads, head_dim=s.head_dim, base_blocks=4096) as ref:
        live = pool.info.live_blocks
        tables, _ = I.assign_blocks(91, 2, lengths0 + steps, s.block_size, live)
        for p in (pool, ref):
            I.fill_pool_layer_(p.layer_tensor(0), 91)
        scale = 1.0 / math.sqrt(s.head_dim)
        h_tables = _pin(tables)
        d_tables = tables.to(dev)
        ws = ref.workspace(B, int(tables.shape[1]) * s.block_size)
        hs = ekv.HostStep(pool, max_batch=B + 3, max_blocks_per_seq=int(tables.shape[1]), depth=depth)
        try:
            host_in, host_out, want = [], [], []
            for t in range(steps):
                lens = lengths0 + t + 1                       # the new token is the last key
                q = I.normal_bf16(91, 10 + t, 0, B * s.num_q_heads * s.head_dim).view(B, s.num_q_heads, s.head_dim)
                k = I.normal_bf16(91, 30 + t, 0, B * s.num_kv_heads * s.head_dim).view(B, s.num_kv_heads, s.head_dim)
                v = I.normal_bf16(91, 50 + t, 0, B * s.num_kv_heads * s.head_dim).view(B, s.num_kv_heads, s.head_dim)
                slots = I.last_token_slots(lens, tables, s.block_size)
                hb = dict(q=_pin(q), k=_pin(k), v=_pin(v), slots=_pin(slots), lens=_pin(lens.to(torch.int32)),
                          out=torch.empty(B, s.num_q_heads, s.head_dim, dtype=torch.bfloat16).pin_memory())
                host_in.append(hb)
                hs.decode(0, hb["q"], h_tables, hb["lens"], scale, hb["out"], h_k=hb["k"], h_v=hb["v"],
                          h_slot_mapping=hb["slots"])
                # the same step on the reference pool, device-resident
                ref.write_kv(0, k.to(dev), v.to(dev), slots.to(dev))
                want.append(ref.attn_decode(0, q.to(dev), d_tables, lens.to(torch.int32).to(dev), scale, workspace=ws).cpu())
            hs.flush()
            torch.cuda.synchronize(dev)
            for t in range(steps):
                assert torch.equal(host_in[t]["out"].view(torch.int16), want[t].view(torch.int16)), f"step {t}"
            assert torch.equal(pool.layer_tensor(0).view(torch.int16), ref.layer_tensor(0).view(torch.int16))
            # the last step against the oracle, on a host mirror built from the seeded fill plus every step's rows
            # (scattered by the oracle): all earlier writes of the pipeline must have landed for this to agree
            final = lengths0 + steps
            cache, ctab, _ = I.compact_host_cache(91, 0, tables, final, range(B), s)
            cache = bf16_bits(cache).copy()
            for t in range(steps):
                slots = I.last_token_slots(lengths0 + t + 1, ctab, s.block_size)
                assert oracle.write_kv(cache, cache.size // s.block_elems, s.num_kv_heads, s.block_size, s.head_dim,
                                       host_in[t]["k"], host_in[t]["v"], slots) == 0
            want_last = oracle.attn_decode(cache, s.num_q_heads, s.num_kv_heads, s.block_size, s.head_dim, host_in[-1]["q"],
                                           ctab, final, scale)
            assert_close(host_in[-1]["out"], want_last, "last pipelined step")
            # pure decode (no write) and a smaller batch reuse the same object
            hb = host_in[-1]
            out2 = torch.empty_like(hb["out"]).pin_memory()
            hs.decode(0, hb["q"][:5].contiguous().pin_memory(), _pin(tables[:5]), _pin(hb["lens"][:5]), scale, out2[:5])
            hs.flush()
            torch.cuda.synchronize(dev)
            assert torch.equal(out2[:5].view(torch.int16), want[-1][:5].view(torch.int16))
            # a batch AND a table width below the values the object was created with: the decode workspace sized at
            # creation must cover the split plan of this smaller shape too (a shorter table can need more key ranges)
            short = [b for b in range(B) if int(lengths0[b]) + steps <= 640][:3] or [int(torch.argmin(lengths0))]
            w = (int((lengths0 + steps)[short].max()) + s.block_size - 1) // s.block_size
            out3 = torch.empty(len(short), s.num_q_heads, s.head_dim, dtype=torch.bfloat16).pin_memory()
            hs.decode(0, _pin(hb["q"][short]), _pin(tables[short][:, :w]), _pin(hb["lens"][short]), scale, out3)
            hs.flush()
            torch.cuda.synchronize(dev)
            assert_close(out3, want_last[short], "narrow table, small batch")
            assert pool.poll_status() == ekv.Status.OK
        finally:
            hs.close()


def test_hoststep_argument_errors():
    import paper_2608_23658_b200 as ekv
    s = I.TINY
    with ekv.Pool(num_q_heads=s.num_q_heads, num_kv_heads=s.num_kv_heads, head_dim=s.head_dim, base_blocks=256) as pool:
        with pytest.raises(ekv.EkvError) as e:
            ekv.HostStep(pool, max_batch=0, max_blocks_per_seq=4)
        assert e.value.status == ekv.Status.ERR_INVALID
        with ekv.HostStep(pool, max_batch=4, max_blocks_per_seq=4) as hs:
            q = torch.zeros(5, s.num_q_heads, s.head_dim, dtype=torch.bfloat16).pin_memory()
            tables = torch.zeros(5, 4, dtype=torch.int32).pin_memory()
            lens = torch.ones(5, dtype=torch.int32).pin_memory()
            with pytest.raises(ekv.EkvError) as e:                       # batch above the capacity given at creation
                hs.decode(0, q, tables, lens, 1.0, torch.empty_like(q).pin_memory())
            assert e.value.status == ekv.Status.ERR_INVALID
            with pytest.raises(ekv.EkvError) as e:                       # k without v and slots
                hs.decode(0, q[:2].contiguous().pin_memory(), tables[:2].contiguous().pin_memory(),
                          lens[:2].contiguous().pin_memory(), 1.0, torch.empty(2, s.num_q_heads, s.head_dim,
                                                                            dtype=torch.bfloat16).pin_memory(),
                          h_k=torch.zeros(2, s.num_kv_heads, s.head_dim, dtype=torch.bfloat16).pin_memory())
            assert e.value.status == ekv.Status.ERR_INVALID
