"""ekv: attention over a block-indexed KV cache in one elastic virtual range per layer (B200, sm_100a).

The Python layer only marshals arguments into the C ABI of ``libekv.so`` (see ``include/ekv.h``);
every step of the path runs in the library's CUDA kernels.  There is no CPU fallback: if the
library cannot be loaded, or no CUDA device exists, calls raise.
"""
from ._binding import (  # noqa: F401
    EKV_BF16, EKV_FUSED_RANGE, EKV_KEEP_PHYSICAL, EKV_PREFILL_ONE_HEAD, EKV_PREFILL_TWO_HEAD, EKV_PREFILL_WARP_MMA, EKV_START_GROWN, EkvError, PoolDesc, PoolInfo, VmmBackend, Status,
    EKV_STATIC_SCRATCH_BYTES, ekv_attn_decode, ekv_attn_decode_plan, ekv_attn_decode_static_scratch, ekv_attn_decode_two_tensor, ekv_attn_prefill_chunk, ekv_attn_workspace_bytes, ekv_grow, ekv_last_error, ekv_layer_ptr,
    ekv_poll_status, ekv_pool_create, ekv_pool_destroy, ekv_pool_info, ekv_set_vmm_backend, ekv_shrink,
    ekv_status_string, ekv_write_kv, library_path, load_library)
from ._binding import (  # noqa: F401,E402
    EKV_ACT_COMMIT, EKV_ACT_DECOMMIT, EKV_ACT_NONE, BlockPoolStats, ControllerStats, ekv_blockpool_admit_elastic,
    ekv_blockpool_alloc, ekv_blockpool_create, ekv_blockpool_destroy, ekv_blockpool_drain_commit, ekv_blockpool_drain_plan,
    ekv_blockpool_free, ekv_blockpool_gate_elastic, ekv_blockpool_stats, ekv_controller_create, ekv_controller_decide,
    ekv_controller_destroy, ekv_controller_stats, ekv_move_blocks)
from ._binding import (  # noqa: F401,E402
    ekv_hoststep_create, ekv_hoststep_decode, ekv_hoststep_destroy, ekv_hoststep_flush, ekv_selftest_bounded_wait)
from .pool import HostStep, Pool  # noqa: F401,E402
