"""KV-head (tensor-parallel) sharding of the path: attention is independent per kv-head, so a rank that owns
Hkv/tp kv-heads (and their query heads) of every block runs the very same kernels on a narrower pool and
produces exactly its slice of the heads; no exchange step lies on this path (the paper's tensor-parallel
discussion: the reserve is sharded, the per-rank KV stays).  One GPU plays the ranks one after the other."""
import math

import numpy as np
import pytest
import torch

import ekv_inputs as I
import oracle
import paper_2608_23658_b200 as ekv
from helpers import assert_close, empty_cache, place_sequence

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _run(shape, K, V, Q, Qp, lengths, tables, prefill_req, c):
    pool = ekv.Pool(num_q_heads=shape.num_q_heads, num_kv_heads=shape.num_kv_heads, head_dim=shape.head_dim,
                    base_blocks=int(tables.max()) + 1)
    try:
        for b, L in enumerate(lengths.tolist()):
            pool.write_kv(0, K[b].to(DEV), V[b].to(DEV), I.position_slots(tables[b], 0, L, 16).to(DEV))
        scale = 1 / math.sqrt(shape.head_dim)
        dec = pool.attn_decode(0, Q.to(DEV), tables.to(DEV), lengths.to(torch.int32).to(DEV), scale)
        cu = torch.tensor([0, c], dtype=torch.int32)
        pre = pool.attn_prefill_chunk(0, Qp.to(DEV), tables[prefill_req:prefill_req + 1].contiguous().to(DEV), cu.to(DEV), cu,
                                      lengths[prefill_req:prefill_req + 1].to(torch.int32).to(DEV), scale)
        torch.cuda.synchronize()
        assert pool.poll_status() == ekv.Status.OK
        return dec.float().cpu(), pre.float().cpu()
    finally:
        pool.close()


@pytest.mark.parametrize("tp", [2, 4])
def test_sharded_pools_reproduce_the_head_slices_of_the_full_pool(tp):
    full = I.LLAMA8B
    lengths = torch.tensor([700, 45, 2200, 1])
    tables, _ = I.assign_blocks(17, 4, lengths, 16, int(I.blocks_for(lengths, 16).sum()) + 9)
    K = [I.normal_bf16(170 + b, 1, 0, int(L) * 8 * 128).view(int(L), 8, 128) for b, L in enumerate(lengths)]
    V = [I.normal_bf16(170 + b, 2, 0, int(L) * 8 * 128).view(int(L), 8, 128) for b, L in enumerate(lengths)]
    Q = I.normal_bf16(18, 3, 0, 4 * 32 * 128).view(4, 32, 128)
    c = 260
    Qp = I.normal_bf16(19, 3, 0, c * 32 * 128).view(c, 32, 128)
    dec_full, pre_full = _run(full, K, V, Q, Qp, lengths, tables, 2, c)
    # the full pool against the oracle; the shards are then compared with the full pool
    host = empty_cache(int(tables.max()) + 1, full)
    for b in range(len(lengths)):
        place_sequence(host, full, tables[b], K[b], V[b])
    scale = 1 / math.sqrt(128)
    assert_close(dec_full, oracle.attn_decode(host, 32, 8, 16, 128, Q, tables, lengths, scale), "full-pool decode")
    cu = np.array([0, c], dtype=np.int32)
    assert_close(pre_full, oracle.attn_prefill_chunk(host, 32, 8, 16, 128, Qp, tables[2:3], cu, lengths[2:3], scale),
                 "full-pool prefill chunk")
    hk, hq = 8 // tp, 32 // tp
    for rank in range(tp):
        shard = I.Shape(hq, hk, 128)
        Ks = [k[:, rank * hk:(rank + 1) * hk].contiguous() for k in K]
        Vs = [v[:, rank * hk:(rank + 1) * hk].contiguous() for v in V]
        dec, pre = _run(shard, Ks, Vs, Q[:, rank * hq:(rank + 1) * hq].contiguous(), Qp[:, rank * hq:(rank + 1) * hq].contiguous(),
                        lengths, tables, 2, c)
        # prefill: one CTA per (query tile, head pair), no dependence on the head count -> the same bits
        assert torch.equal(pre, pre_full[:, rank * hq:(rank + 1) * hq])
        # decode: the split plan depends on B*Hkv, so the summation order may differ: tolerance
        d = (dec - dec_full[:, rank * hq:(rank + 1) * hq]).abs()
        assert d.max().item() <= 2e-2 and d.mean().item() <= 2e-3
        # and the shard on its own against the oracle run on the shard's heads only (a narrower cache)
        hosts = empty_cache(int(tables.max()) + 1, shard)
        for b in range(len(lengths)):
            place_sequence(hosts, shard, tables[b], Ks[b], Vs[b])
        want = oracle.attn_decode(hosts, hq, hk, 16, 128, Q[:, rank * hq:(rank + 1) * hq].contiguous(), tables, lengths, scale)
        assert_close(dec, want, f"decode of shard {rank}/{tp}")
