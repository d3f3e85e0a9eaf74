"""The alternative the paper rejects ("split the KV into two tensors and rewrite the kernel to read both"),
built to measure it: with the elastic blocks held in a separately allocated tensor the two-tensor kernel must
give the same bits as the single-range kernel on the same logical data, and its cost is reported."""
import math

import pytest
import torch

import ekv_inputs as I
import oracle
import paper_2608_23658_b200 as ekv
from helpers import assert_close, mirror_after_step

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_two_tensor_decode_matches_single_range_bitwise_and_reports_its_cost():
    s = I.LLAMA8B
    pool = ekv.Pool(num_q_heads=s.num_q_heads, num_kv_heads=s.num_kv_heads, head_dim=s.head_dim, base_blocks=12000,
                    elastic_blocks=2400, start_grown=True)
    try:
        info = pool.info
        base, el = info.base_blocks, info.elastic_blocks
        I.fill_pool_layer_(pool.layer_tensor(0), 23)
        lengths = I.uniform_ints(23, 11, 48, 1024, 6000)
        tables, _ = I.assign_blocks(23, 12, lengths, 16, base + el)           # ~1/6 of every sequence is elastic
        assert (tables >= base).any()
        B = len(lengths)
        q = I.normal_bf16(23, 3, 0, B * s.num_q_heads * s.head_dim, device=DEV).view(B, s.num_q_heads, s.head_dim)
        d_tables, d_lens = tables.to(DEV), lengths.to(torch.int32).to(DEV)
        scale = 1 / math.sqrt(s.head_dim)
        ws = pool.workspace(B, int(tables.shape[1]) * 16)
        single = pool.attn_decode(0, q, d_tables, d_lens, scale, workspace=ws)
        second = pool.layer_tensor(0, base, el).clone()                       # the elastic blocks as a tensor of their own
        two = torch.empty_like(q)
        ekv.ekv_attn_decode_two_tensor(pool.handle, 0, second, q, two, d_tables, d_lens, scale, ws)
        assert torch.equal(single, two)
        # the oracle on a sample of the sequences (longest, shortest, and the one with the most elastic blocks), so that
        # "same bits as the single-range kernel" also means "right"
        sample = sorted({int(lengths.argmax()), int(lengths.argmin()), int((tables >= base).sum(1).argmax()), 0})
        cache, ctab, clen = mirror_after_step(23, 0, tables, lengths, sample, s)
        want = oracle.attn_decode(cache, s.num_q_heads, s.num_kv_heads, 16, s.head_dim, q[sample].cpu(), ctab, clen, scale)
        assert_close(two[sample], want, "two-tensor decode")
        pool.shrink()                                                          # the two-tensor kernel needs no elastic range
        two2 = torch.empty_like(q)
        ekv.ekv_attn_decode_two_tensor(pool.handle, 0, second, q, two2, d_tables, d_lens, scale, ws)
        assert torch.equal(single, two2)
        bad = d_tables.clone()
        bad[0, 0] = base + el + 3
        ekv.ekv_attn_decode_two_tensor(pool.handle, 0, second, q, two2, bad, d_lens, scale, ws)
        torch.cuda.synchronize()
        st = pool.poll_status()
        assert st == ekv.Status.ERR_BLOCK_OOB, st
        pool.grow()
        I.fill_pool_layer_(pool.layer_tensor(0, base, el), 23, first_block=base)   # a releasing shrink loses the bytes

        def timed(fn):
            for _ in range(3):
                fn()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(20):
                fn()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / 20
        t1 = timed(lambda: pool.attn_decode(0, q, d_tables, d_lens, scale, out=two, workspace=ws))
        t2 = timed(lambda: ekv.ekv_attn_decode_two_tensor(pool.handle, 0, second, q, two2, d_tables, d_lens, scale, ws))
        assert torch.equal(two, two2)
        gb = I.decode_algorithmic_bytes(lengths, s) / 1e9
        print(f"\nsingle range {t1:.4f} ms ({gb / t1 * 1e3:.0f} GB/s), two tensors {t2:.4f} ms ({gb / t2 * 1e3:.0f} GB/s), "
              f"ratio {t2 / t1:.3f}")
    finally:
        pool.close()
