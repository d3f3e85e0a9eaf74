"""EKV_FUSED_RANGE: one virtual range and two handles for the whole model, layers interleaved inside every block
id.  Every layer is still one pointer indexed by block id (a strided tensor), so the same kernels must give the
same results as with one range per layer, and the bytes of each layer must be exactly what was written."""
import math

import numpy as np
import pytest
import torch

import ekv_inputs as I
import oracle
import paper_2608_23658_b200 as ekv
from helpers import bf16_bits, empty_cache, place_sequence

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
MAX_ABS, MEAN_ABS = 2e-2, 2e-3
NL = 3


def check_close(got, want, what):
    err = np.abs(got.float().cpu().numpy().astype(np.float64) - want)
    assert np.isfinite(err).all() and err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (what, err.max(), err.mean())


@pytest.mark.parametrize("shape", [I.LLAMA8B, I.TINY])
def test_fused_range_pool_matches_oracle_and_per_layer_pool(shape):
    lengths = torch.tensor([700, 33, 1300, 1])
    chunk = (2, 300)                                      # request 2: last 300 rows as a prefill chunk
    need = int(I.blocks_for(lengths, 16).sum())
    pools = {fused: ekv.Pool(num_q_heads=shape.num_q_heads, num_kv_heads=shape.num_kv_heads, head_dim=shape.head_dim,
                             base_blocks=need // 2, elastic_blocks=need, num_layers=NL, start_grown=True, fused_range=fused)
             for fused in (True, False)}
    try:
        info = pools[True].info
        assert info.num_ranges == 1 and info.block_stride_bytes == NL * info.block_bytes
        assert pools[False].info.num_ranges == NL
        live = min(p.info.live_blocks for p in pools.values())
        tables, _ = I.assign_blocks(41, 4, lengths, 16, live)
        assert (tables >= info.base_blocks).any()
        scale = 1 / math.sqrt(shape.head_dim)
        q = I.normal_bf16(42, 3, 0, 4 * shape.num_q_heads * shape.head_dim).view(4, shape.num_q_heads, shape.head_dim)
        qc = I.normal_bf16(43, 3, 0, chunk[1] * shape.num_q_heads * shape.head_dim).view(chunk[1], shape.num_q_heads, shape.head_dim)
        cu = torch.tensor([0, chunk[1]], dtype=torch.int32)
        outs = {}
        for fused, pool in pools.items():
            for l in range(NL):
                pool.layer_tensor(l).view(torch.int16).fill_(0x7FC0)   # NaN patterns everywhere
            hosts = []
            for l in range(NL):
                host = empty_cache(pool.info.live_blocks, shape, fill=0x7FC0)
                for b, L in enumerate(lengths.tolist()):
                    n = L * shape.num_kv_heads * shape.head_dim
                    K = I.normal_bf16(500 + 10 * l + b, 1, 0, n).view(L, shape.num_kv_heads, shape.head_dim)
                    V = I.normal_bf16(500 + 10 * l + b, 2, 0, n).view(L, shape.num_kv_heads, shape.head_dim)
                    pool.write_kv(l, K.to(DEV), V.to(DEV), I.position_slots(tables[b], 0, L, 16).to(DEV))
                    place_sequence(host, shape, tables[b], K, V)
                hosts.append(host)
            torch.cuda.synchronize()
            for l in range(NL):                                                    # exact scatter, layer by layer
                assert np.array_equal(bf16_bits(pool.layer_tensor(l).cpu()).reshape(-1), hosts[l])
            res = []
            for l in range(NL):
                dec = pool.attn_decode(l, q.to(DEV), tables.to(DEV), lengths.to(torch.int32).to(DEV), scale)
                pre = pool.attn_prefill_chunk(l, qc.to(DEV), tables[chunk[0]:chunk[0] + 1].contiguous().to(DEV), cu.to(DEV), cu,
                                              lengths[chunk[0]:chunk[0] + 1].to(torch.int32).to(DEV), scale)
                wd = oracle.attn_decode(hosts[l], shape.num_q_heads, shape.num_kv_heads, 16, shape.head_dim, q, tables, lengths, scale)
                wp = oracle.attn_prefill_chunk(hosts[l], shape.num_q_heads, shape.num_kv_heads, 16, shape.head_dim, qc,
                                               tables[chunk[0]:chunk[0] + 1], cu, lengths[chunk[0]:chunk[0] + 1], scale)
                check_close(dec, wd, f"decode layer {l} fused={fused}")
                check_close(pre, wp, f"prefill layer {l} fused={fused}")
                res += [dec, pre]
            outs[fused] = res
            assert pool.poll_status() == ekv.Status.OK
        for a, b in zip(outs[True], outs[False]):
            assert torch.equal(a, b), "fused and per-layer ranges must give the same bits"
    finally:
        for p in pools.values():
            p.close()


def test_fused_range_toggle_moves_and_bytes():
    shape = I.LLAMA8B
    pool = ekv.Pool(num_q_heads=shape.num_q_heads, num_kv_heads=shape.num_kv_heads, head_dim=shape.head_dim, base_blocks=96,
                    elastic_blocks=64, num_layers=4, start_grown=True, fused_range=True)
    try:
        info = pool.info
        base, el = info.base_blocks, info.elastic_blocks
        ptrs = [pool.layer_ptr(l) for l in range(4)]
        assert ptrs == [ptrs[0] + l * info.block_bytes for l in range(4)]
        vals = {}
        for l in range(4):
            v = I.normal_bf16(60 + l, 1, 0, (base + el) * shape.block_elems).view(base + el, 2, shape.num_kv_heads, 16, shape.head_dim)
            pool.layer_tensor(l).copy_(v.to(DEV))
            vals[l] = v
        src = torch.tensor([base + 3, base + 60, 5], dtype=torch.int32, device=DEV)
        dst = torch.tensor([7, 90, base + 1], dtype=torch.int32, device=DEV)
        ekv.ekv_move_blocks(pool.handle, src, dst)
        for l in range(4):
            vals[l][dst.cpu().long()] = vals[l][src.cpu().long()].clone()
            assert torch.equal(pool.layer_tensor(l).cpu(), vals[l])
        ms = pool.shrink(keep_physical=True)
        assert pool.info.live_blocks == base and ms[0] >= 0
        for l in range(4):
            assert torch.equal(pool.layer_tensor(l).cpu(), vals[l][:base])
        pool.grow()
        assert [pool.layer_ptr(l) for l in range(4)] == ptrs
        for l in range(4):
            assert torch.equal(pool.layer_tensor(l).cpu(), vals[l])                # bytes survived the unmap
        free0 = torch.cuda.mem_get_info()[0]
        pool.shrink()
        assert torch.cuda.mem_get_info()[0] - free0 >= 0.9 * 4 * info.elastic_bytes
        pool.grow()
        assert pool.poll_status() == ekv.Status.OK
    finally:
        pool.close()
