"""Pool state machine on a host without a GPU: rounding to granules, two-handles-one-range
bookkeeping, grow / shrink (releasing and keep-physical), unwinding after injected failures."""
import pytest

import paper_2608_23658_b200 as ekv
from fake_vmm import FakeVmm

MiB = 1 << 20


@pytest.fixture
def vmm():
    fake = FakeVmm()
    table = fake.table()
    ekv.ekv_set_vmm_backend(table)
    yield fake
    ekv.ekv_set_vmm_backend(None)
    assert fake.violations == []


def _create(**kw):
    args = dict(num_q_heads=32, num_kv_heads=8, head_dim=128, base_blocks=100, elastic_blocks=40)
    args.update(kw)
    return ekv.ekv_pool_create(**args)


def test_rounding_to_granules(vmm):
    # 8 kv-heads x 128 channels: block = 64 KiB, 32 blocks per 2 MiB granule
    pool = _create(base_blocks=100, elastic_blocks=40)
    info = ekv.ekv_pool_info(pool)
    assert info.granularity == 2 * MiB and info.block_bytes == 64 * 1024
    assert (info.base_blocks, info.elastic_blocks) == (128, 64)
    assert (info.base_bytes, info.elastic_bytes) == (8 * MiB, 4 * MiB)
    assert info.live_blocks == 128 and not info.grown and not info.physical_held
    ekv.ekv_pool_destroy(pool)
    # tiny geometry: 2 kv-heads x 64 channels: block = 8 KiB, 256 blocks per granule
    pool = _create(num_q_heads=4, num_kv_heads=2, head_dim=64, base_blocks=256, elastic_blocks=1)
    info = ekv.ekv_pool_info(pool)
    assert info.block_bytes == 8192 and (info.base_blocks, info.elastic_blocks) == (256, 256)
    ekv.ekv_pool_destroy(pool)
    assert not vmm.reserved and not vmm.handles and not vmm.mapped


def test_one_range_two_handles_per_layer(vmm):
    pool = _create(num_layers=3, flags=ekv.EKV_START_GROWN)
    info = ekv.ekv_pool_info(pool)
    assert info.grown and info.live_blocks == 192
    assert len(vmm.reserved) == 3 and len(vmm.handles) == 6 and len(vmm.mapped) == 6
    for layer in range(3):
        va = ekv.ekv_layer_ptr(pool, layer)
        assert vmm.reserved[va] == 12 * MiB                    # one range sized base + elastic
        assert vmm.mapped[va][0] == 8 * MiB                     # base at the bottom
        assert vmm.mapped[va + 8 * MiB][0] == 4 * MiB           # elastic at the top
        assert va in vmm.access and va + 8 * MiB in vmm.access
    ekv.ekv_pool_destroy(pool)
    assert not vmm.reserved and not vmm.handles and not vmm.mapped


def test_grow_shrink_cycle_and_constant_pointer(vmm):
    pool = _create(num_layers=2)
    ptrs = [ekv.ekv_layer_ptr(pool, l) for l in range(2)]
    base_handles = dict(vmm.handles)
    for cycle in range(3):
        ekv.ekv_grow(pool, host_only=True)
        info = ekv.ekv_pool_info(pool)
        assert info.grown and info.physical_held and info.live_blocks == 192
        assert len(vmm.mapped) == 4 and vmm.used() == 2 * 12 * MiB
        with pytest.raises(ekv.EkvError) as e:
            ekv.ekv_grow(pool, host_only=True)
        assert e.value.status == ekv.Status.ERR_STATE
        ekv.ekv_shrink(pool, host_only=True)                   # releasing shrink: memory goes back
        info = ekv.ekv_pool_info(pool)
        assert not info.grown and not info.physical_held and info.live_blocks == 128
        assert vmm.handles == base_handles and len(vmm.mapped) == 2
        with pytest.raises(ekv.EkvError) as e:
            ekv.ekv_shrink(pool, host_only=True)
        assert e.value.status == ekv.Status.ERR_STATE
        assert [ekv.ekv_layer_ptr(pool, l) for l in range(2)] == ptrs
    ekv.ekv_pool_destroy(pool)


def test_keep_physical_reuses_the_handle(vmm):
    pool = _create()
    ekv.ekv_grow(pool, host_only=True)
    elastic = set(vmm.handles) - {h for _, h in [vmm.mapped[ekv.ekv_layer_ptr(pool, 0)]]}
    ekv.ekv_shrink(pool, flags=ekv.EKV_KEEP_PHYSICAL, host_only=True)
    info = ekv.ekv_pool_info(pool)
    assert not info.grown and info.physical_held
    assert elastic <= set(vmm.handles) and len(vmm.mapped) == 1
    n_creates = sum(1 for e in vmm.log if e[0] == "create")
    ekv.ekv_grow(pool, host_only=True)
    assert sum(1 for e in vmm.log if e[0] == "create") == n_creates    # map only, no new allocation
    assert {h for _, h in vmm.mapped.values()} >= elastic
    ekv.ekv_pool_destroy(pool)
    assert not vmm.handles and not vmm.mapped and not vmm.reserved


@pytest.mark.parametrize("what", ["create", "map", "access"])
@pytest.mark.parametrize("layer", [0, 2, 3])
def test_failed_grow_unwinds_to_shrunk_state(vmm, what, layer):
    pool = _create(num_layers=4)
    before = (dict(vmm.handles), dict(vmm.mapped))
    setattr(vmm, f"fail_{what}_at", layer)
    with pytest.raises(ekv.EkvError) as e:
        ekv.ekv_grow(pool, host_only=True)
    assert e.value.status == (ekv.Status.ERR_OOM if what == "create" else ekv.Status.ERR_CUDA)
    assert f"layer {layer}" in str(e.value)
    info = ekv.ekv_pool_info(pool)
    assert not info.grown and not info.physical_held and info.live_blocks == info.base_blocks
    assert (vmm.handles, vmm.mapped) == before
    ekv.ekv_grow(pool, host_only=True)                         # and a later grow succeeds
    assert ekv.ekv_pool_info(pool).grown
    ekv.ekv_pool_destroy(pool)


def test_failed_grow_keeps_handles_held_before_the_call(vmm):
    pool = _create(num_layers=3)
    ekv.ekv_grow(pool, host_only=True)
    ekv.ekv_shrink(pool, flags=ekv.EKV_KEEP_PHYSICAL, host_only=True)
    held = dict(vmm.handles)
    vmm.fail_map_at = 1
    with pytest.raises(ekv.EkvError):
        ekv.ekv_grow(pool, host_only=True)
    assert vmm.handles == held and len(vmm.mapped) == 3
    assert ekv.ekv_pool_info(pool).physical_held
    ekv.ekv_pool_destroy(pool)


def test_capacity_oom_on_recommit(vmm):
    """The paper's recommit OOM: memory handed back at shrink may be gone when grow asks for it again."""
    vmm.capacity = 2 * 12 * MiB
    pool = _create(num_layers=2, flags=ekv.EKV_START_GROWN)
    ekv.ekv_shrink(pool, host_only=True)
    hog = [0]
    assert vmm.create(None, 6 * MiB, 0, hog) == 0               # somebody else takes the space
    with pytest.raises(ekv.EkvError) as e:
        ekv.ekv_grow(pool, host_only=True)
    assert e.value.status == ekv.Status.ERR_OOM
    assert not ekv.ekv_pool_info(pool).grown and len(vmm.mapped) == 2
    vmm.release(None, hog[0])
    ekv.ekv_grow(pool, host_only=True)
    ekv.ekv_pool_destroy(pool)


def test_failed_create_leaves_nothing_behind(vmm):
    vmm.fail_create_at = 2                                      # base handle of layer 2
    with pytest.raises(ekv.EkvError) as e:
        _create(num_layers=4)
    assert e.value.status == ekv.Status.ERR_OOM
    assert not vmm.reserved and not vmm.handles and not vmm.mapped


def test_argument_checks_and_host_only_refusal(vmm):
    for bad in (dict(head_dim=96), dict(block_size=32), dict(num_q_heads=12, num_kv_heads=8),
                dict(num_q_heads=72, num_kv_heads=8), dict(base_blocks=0), dict(elastic_blocks=-1), dict(flags=64)):
        with pytest.raises(ekv.EkvError) as e:
            _create(**bad)
        assert e.value.status == ekv.Status.ERR_INVALID
    vmm.gran = 96 * 1024                                        # not a multiple of the 64 KiB block
    with pytest.raises(ekv.EkvError) as e:
        _create()
    assert e.value.status == ekv.Status.ERR_INVALID
    vmm.gran = 2 * MiB
    pool = _create(elastic_blocks=0)
    with pytest.raises(ekv.EkvError) as e:
        ekv.ekv_grow(pool, host_only=True)                     # nothing to grow into
    assert e.value.status == ekv.Status.ERR_STATE
    assert ekv.ekv_attn_workspace_bytes(pool, 8, 4096) > 0
    import torch
    dummy = torch.zeros(16, dtype=torch.int64)
    st = ekv.load_library().ekv_write_kv(pool, 0, dummy.data_ptr(), dummy.data_ptr(), dummy.data_ptr(), 1, None)
    assert st == ekv.Status.ERR_STATE                           # no device state: compute refuses
    with pytest.raises(ekv.EkvError) as e:
        ekv.ekv_set_vmm_backend(None)                           # pools still exist
    assert e.value.status == ekv.Status.ERR_STATE
    ekv.ekv_pool_destroy(pool)


def test_fused_range_is_one_reservation_and_two_handles_for_all_layers(vmm):
    # 3 layers x 64 KiB blocks: a block id spans 192 KiB of the range, so counts round up to multiples of 32
    pool = _create(num_layers=3, base_blocks=100, elastic_blocks=40, flags=ekv.EKV_FUSED_RANGE)
    info = ekv.ekv_pool_info(pool)
    assert (info.base_blocks, info.elastic_blocks) == (128, 64)
    assert info.num_ranges == 1 and info.block_stride_bytes == 3 * 64 * 1024 and info.block_bytes == 64 * 1024
    assert len(vmm.reserved) == 1 and len(vmm.handles) == 1 and len(vmm.mapped) == 1
    (va, size), = vmm.reserved.items()
    assert size == (128 + 64) * 3 * 64 * 1024
    assert [ekv.ekv_layer_ptr(pool, l) for l in range(3)] == [va + l * 64 * 1024 for l in range(3)]
    n_calls = len(vmm.log)
    ekv.ekv_grow(pool, host_only=True)
    assert [e[0] for e in vmm.log[n_calls:]] == ["create", "map"]       # one create + one map for the whole model
    assert vmm.mapped[va + 128 * 3 * 64 * 1024][0] == 64 * 3 * 64 * 1024  # the elastic ids are the top of the range
    assert ekv.ekv_pool_info(pool).live_blocks == 192
    n_calls = len(vmm.log)
    ekv.ekv_shrink(pool, host_only=True)
    assert [e[0] for e in vmm.log[n_calls:]] == ["unmap", "release"]
    vmm.fail_map_at = 0
    with pytest.raises(ekv.EkvError):
        ekv.ekv_grow(pool, host_only=True)
    assert len(vmm.handles) == 1 and len(vmm.mapped) == 1 and not ekv.ekv_pool_info(pool).grown
    ekv.ekv_pool_destroy(pool)
    assert not vmm.reserved and not vmm.handles and not vmm.mapped


@pytest.mark.parametrize("k", [0, 1, 3])
@pytest.mark.parametrize("keep", [False, True])
def test_shrink_that_fails_half_way_keeps_books_and_mappings_in_step(vmm, k, keep):
    """The driver refuses the unmap of range k: ranges before k are unmapped (and released), the rest stay mapped,
    the pool still says grown while the live limit is already down; a second ekv_shrink finishes the job."""
    pool = _create(num_layers=4, flags=ekv.EKV_START_GROWN)
    flags = ekv.EKV_KEEP_PHYSICAL if keep else 0
    vmm.fail_unmap_at = k
    with pytest.raises(ekv.EkvError) as e:
        ekv.ekv_shrink(pool, flags=flags, host_only=True)
    assert e.value.status == ekv.Status.ERR_CUDA and f"layer {k}" in str(e.value)
    info = ekv.ekv_pool_info(pool)
    assert info.grown and info.live_blocks == info.base_blocks     # no kernel may reach the elastic ids any more
    assert len(vmm.mapped) == 4 + (4 - k)                           # base mappings + elastic ones from range k on
    assert len(vmm.handles) == (8 if keep else 8 - k)
    with pytest.raises(ekv.EkvError) as e:                         # still "grown": a grow is refused, not stacked on top
        ekv.ekv_grow(pool, host_only=True)
    assert e.value.status == ekv.Status.ERR_STATE
    ekv.ekv_shrink(pool, flags=flags, host_only=True)              # the retry touches only what is left
    info = ekv.ekv_pool_info(pool)
    assert not info.grown and len(vmm.mapped) == 4 and len(vmm.handles) == (8 if keep else 4)
    assert bool(info.physical_held) == keep
    ekv.ekv_grow(pool, host_only=True)                             # and the pool is fully usable afterwards
    assert ekv.ekv_pool_info(pool).live_blocks == 192 and len(vmm.mapped) == 8
    ekv.ekv_pool_destroy(pool)
    assert not vmm.reserved and not vmm.handles and not vmm.mapped


def test_live_limit_follows_every_toggle(vmm):
    pool = _create(num_layers=2)
    assert ekv.ekv_pool_info(pool).live_blocks == 128
    ekv.ekv_grow(pool, host_only=True)
    assert ekv.ekv_pool_info(pool).live_blocks == 192
    ekv.ekv_shrink(pool, flags=ekv.EKV_KEEP_PHYSICAL, host_only=True)
    assert ekv.ekv_pool_info(pool).live_blocks == 128
    vmm.fail_map_at = 1                                            # a grow that fails leaves the limit where it was
    with pytest.raises(ekv.EkvError):
        ekv.ekv_grow(pool, host_only=True)
    info = ekv.ekv_pool_info(pool)
    assert info.live_blocks == 128 and not info.grown and len(vmm.mapped) == 2
    ekv.ekv_pool_destroy(pool)


def test_workspace_bytes_cover_every_smaller_shape(vmm):
    """ekv_attn_workspace_bytes(max_batch, max_seq_len) promises room for EVERY call with B <= max_batch and a table
    no wider than max_seq_len allows -- a shorter table can be cut into more key ranges than a longer one, so the
    largest shape alone is not the bound.  Host-only pools plan for 148 SMs."""
    for heads in ((32, 8), (64, 8), (8, 8)):
        pool = _create(num_q_heads=heads[0], num_kv_heads=heads[1])
        for max_batch, max_blocks in ((1, 8192), (4, 1024), (3, 785), (37, 300), (256, 512), (2, 17), (5, 2353)):
            have = ekv.ekv_attn_workspace_bytes(pool, max_batch, max_blocks * 16)
            worst = 0
            for B in range(1, max_batch + 1):
                step = max(1, max_blocks // 700)
                for mb in list(range(1, max_blocks + 1, step)) + [max_blocks]:
                    chunk, nsplit, need = ekv.ekv_attn_decode_plan(pool, B, mb)
                    assert chunk % 64 == 0 and 64 <= chunk <= 2048 and (nsplit - 1) * chunk < mb * 16 <= nsplit * chunk
                    worst = max(worst, need)
            assert worst <= have, (heads, max_batch, max_blocks, worst, have)
            assert have <= 2 * worst + 4096                        # a bound, not a blank cheque
        ekv.ekv_pool_destroy(pool)
    # the two shapes a review found short by a few KiB with the plan of the largest shape alone (32q/8kv, d128, 148 SMs)
    pool = _create()
    assert ekv.ekv_attn_decode_plan(pool, 1, 2353)[2] <= ekv.ekv_attn_workspace_bytes(pool, 1, 8192 * 16)
    assert ekv.ekv_attn_decode_plan(pool, 3, 785)[2] <= ekv.ekv_attn_workspace_bytes(pool, 4, 1024 * 16)
    ekv.ekv_pool_destroy(pool)
