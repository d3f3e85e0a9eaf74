"""The kernels' bounded waits: a wait that nothing completes runs out, latches EKV_ERR_TIMEOUT, and the context
stays usable (no fault, no hang).  Driven by ekv_selftest_bounded_wait, which uses the kernels' own wait routine."""
import pytest
import torch

import ekv_inputs as I

pytestmark = pytest.mark.gpu


def test_wait_runs_out_latches_timeout_and_context_survives():
    import paper_2608_23658_b200 as ekv
    dev = torch.device("cuda:0")
    s = I.TINY
    with ekv.Pool(num_q_heads=s.num_q_heads, num_kv_heads=s.num_kv_heads, head_dim=s.head_dim, base_blocks=256) as pool:
        assert pool.poll_status() == ekv.Status.OK
        waited = torch.zeros(1, dtype=torch.int64, device=dev)
        ekv.ekv_selftest_bounded_wait(pool.handle, 2000, waited)        # 2 ms
        torch.cuda.synchronize(dev)
        ns = int(waited.item())
        assert 2_000_000 <= ns < 50_000_000, ns                          # gave up after the limit, not long after it
        assert pool.poll_status() == ekv.Status.ERR_TIMEOUT
        assert "bounded wait" in ekv.ekv_last_error()
        assert pool.poll_status() == ekv.Status.OK                       # read-and-clear
        # the context is intact: an ordinary call still gives the exact result
        k = I.normal_bf16(5, 1, 0, 3 * s.num_kv_heads * s.head_dim).view(3, s.num_kv_heads, s.head_dim).to(dev)
        v = I.normal_bf16(5, 2, 0, 3 * s.num_kv_heads * s.head_dim).view(3, s.num_kv_heads, s.head_dim).to(dev)
        slots = torch.tensor([0, 17, 40], dtype=torch.int64, device=dev)
        pool.write_kv(0, k, v, slots)
        q = torch.zeros(1, s.num_q_heads, s.head_dim, dtype=torch.bfloat16, device=dev)
        out = pool.attn_decode(0, q, torch.tensor([[0]], dtype=torch.int32, device=dev),
                               torch.tensor([1], dtype=torch.int32, device=dev), 1.0)
        torch.cuda.synchronize(dev)
        for h in range(s.num_q_heads):                                   # a single key returns its V row
            assert torch.equal(out[0, h].view(torch.int16), v[0, h // (s.num_q_heads // s.num_kv_heads)].view(torch.int16))
        assert pool.poll_status() == ekv.Status.OK
        with pytest.raises(ekv.EkvError) as e:
            ekv.ekv_selftest_bounded_wait(pool.handle, 0)
        assert e.value.status == ekv.Status.ERR_INVALID
