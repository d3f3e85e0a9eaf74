"""ekv_attn_decode_static_scratch: decode attention for callers that cannot allocate device memory
(an engine whose free memory all went to the KV pool, a host without an allocator, a path where
cudaMalloc must not be entered).  The scratch of the split pass is a fixed array inside the library;
this file checks, through the C ABI, that the call gives what ekv_attn_decode gives -- the same bits:
both run the same plan and kernels and differ only in where the partials live -- on two calls in a row
(the array is shared and keeps the previous call's contents), that this is also what the CPU oracle
computes, that the device's free memory and torch's own allocator do not move across a call, and that a
shape whose scratch need exceeds the array is refused.  It is collected last on purpose."""
import math

import pytest
import torch

import ekv_inputs as I
import oracle
import paper_2608_23658_b200 as ekv
from helpers import assert_close, mirror_after_step

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
MAX_ABS, MEAN_ABS = 2e-2, 2e-3


def _workload(pool, shape, lengths, seed):
    lengths = torch.as_tensor(lengths, dtype=torch.int64)
    live = pool.info.live_blocks
    tables, _ = I.assign_blocks(seed, 4, lengths, shape.block_size, live)
    I.fill_pool_layer_(pool.layer_tensor(0), seed)
    q = I.normal_bf16(seed, 3, 0, len(lengths) * shape.num_q_heads * shape.head_dim).view(
        len(lengths), shape.num_q_heads, shape.head_dim)
    cache, ctab, clen = mirror_after_step(seed, 0, tables, lengths, range(len(lengths)), shape)
    want = oracle.attn_decode(cache, shape.num_q_heads, shape.num_kv_heads, shape.block_size, shape.head_dim, q, ctab, clen,
                              1 / math.sqrt(shape.head_dim))
    return q.to(DEV), tables.to(DEV), lengths.to(torch.int32).to(DEV), want


def test_static_scratch_decode_matches_workspace_decode_twice_in_a_row():
    shape = I.LLAMA8B
    scale = 1 / math.sqrt(shape.head_dim)
    pool = ekv.Pool(num_q_heads=shape.num_q_heads, num_kv_heads=shape.num_kv_heads, head_dim=shape.head_dim,
                    base_blocks=1024)
    try:
        # two different shapes back to back: the second call finds the first call's partials in the array
        for lengths, seed in (([3000, 17, 1, 2048, 999, 4100], 5), ([64, 700], 6)):
            q, tables, lens, oracle_out = _workload(pool, shape, lengths, seed)
            want = pool.attn_decode(0, q, tables, lens, scale)              # existing entry point
            got = torch.full_like(q, float("nan"))
            ekv.ekv_attn_decode_static_scratch(pool.handle, 0, q, got, tables, lens, scale)
            again = torch.full_like(q, float("nan"))
            torch.cuda.synchronize()
            # the first call on the device has resolved the array's address; from here on a call must not
            # move the device's free memory nor enter torch's allocator
            free0, torch0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
            ekv.ekv_attn_decode_static_scratch(pool.handle, 0, q, again, tables, lens, scale)
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == torch0
            assert torch.equal(got, want) and torch.equal(again, want)
            assert_close(got, oracle_out, "static-scratch decode", MAX_ABS, MEAN_ABS)
        assert pool.poll_status() == ekv.Status.OK
    finally:
        pool.close()


def test_static_scratch_refuses_shapes_beyond_its_array():
    shape = I.LLAMA70B
    pool = ekv.Pool(num_q_heads=shape.num_q_heads, num_kv_heads=shape.num_kv_heads, head_dim=shape.head_dim,
                    base_blocks=64)
    try:
        B, max_blocks = 512, 8192   # 512 sequences of up to 131072 keys: far more partials than the array holds
        assert ekv.ekv_attn_workspace_bytes(pool.handle, B, max_blocks * 16) > ekv.EKV_STATIC_SCRATCH_BYTES
        q = torch.zeros(B, shape.num_q_heads, shape.head_dim, dtype=torch.bfloat16, device=DEV)
        tables = torch.zeros(B, max_blocks, dtype=torch.int32, device=DEV)
        lens = torch.ones(B, dtype=torch.int32, device=DEV)
        out = torch.full_like(q, 7.0)
        with pytest.raises(ekv.EkvError) as e:
            ekv.ekv_attn_decode_static_scratch(pool.handle, 0, q, out, tables, lens, 0.1)
        assert e.value.status == ekv.Status.ERR_WORKSPACE
        assert "bytes of scratch" in str(e.value)
        torch.cuda.synchronize()
        assert (out == 7.0).all()                                           # nothing was launched
    finally:
        pool.close()
