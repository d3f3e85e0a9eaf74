"""ctypes binding of libekv.so: same names as the C ABI, argument marshalling only."""
from __future__ import annotations

import ctypes
import enum
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libekv.so")
_lib = None

EKV_BF16 = 0
EKV_START_GROWN = 1
EKV_KEEP_PHYSICAL = 2
EKV_FUSED_RANGE = 4
EKV_PREFILL_WARP_MMA = 8
EKV_PREFILL_ONE_HEAD = 16
EKV_PREFILL_TWO_HEAD = 32


class Status(enum.IntEnum):
    OK = 0
    ERR_INVALID = 1
    ERR_CUDA = 2
    ERR_OOM = 3
    ERR_STATE = 4
    ERR_BLOCK_OOB = 5
    ERR_TIMEOUT = 6
    ERR_WORKSPACE = 7


class EkvError(RuntimeError):
    def __init__(self, status: int, detail: str):
        self.status = Status(status) if status in Status._value2member_map_ else status
        super().__init__(f"{ekv_status_string(status)}: {detail}")


class PoolDesc(ctypes.Structure):
    _fields_ = [("device", ctypes.c_int32), ("num_layers", ctypes.c_int32), ("num_q_heads", ctypes.c_int32),
                ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("block_size", ctypes.c_int32),
                ("dtype", ctypes.c_int32), ("flags", ctypes.c_uint32), ("base_blocks", ctypes.c_int64),
                ("elastic_blocks", ctypes.c_int64)]


class BlockPoolStats(ctypes.Structure):
    _fields_ = [("base_blocks", ctypes.c_int64), ("elastic_blocks", ctypes.c_int64), ("free_base", ctypes.c_int64),
                ("free_elastic", ctypes.c_int64), ("elastic_in_use", ctypes.c_int64), ("num_gpu_blocks", ctypes.c_int64),
                ("admitted", ctypes.c_int32), ("draining", ctypes.c_int32)]


class ControllerDesc(ctypes.Structure):
    _fields_ = [("commit_after_decode_steps", ctypes.c_int32), ("reserve_prefill_tokens", ctypes.c_int32)]


class ControllerStats(ctypes.Structure):
    _fields_ = [("steps", ctypes.c_int64), ("commits", ctypes.c_int64), ("decommits", ctypes.c_int64),
                ("committed", ctypes.c_int32), ("decode_streak", ctypes.c_int32)]


EKV_ACT_NONE, EKV_ACT_COMMIT, EKV_ACT_DECOMMIT = 0, 1, 2


class PoolInfo(ctypes.Structure):
    _fields_ = [("granularity", ctypes.c_uint64), ("block_bytes", ctypes.c_uint64), ("base_bytes", ctypes.c_uint64),
                ("elastic_bytes", ctypes.c_uint64), ("base_blocks", ctypes.c_int64), ("elastic_blocks", ctypes.c_int64),
                ("live_blocks", ctypes.c_int64), ("grown", ctypes.c_int32), ("physical_held", ctypes.c_int32),
                ("num_layers", ctypes.c_int32), ("num_ranges", ctypes.c_int32), ("block_stride_bytes", ctypes.c_uint64)]


_u64p = ctypes.POINTER(ctypes.c_uint64)
_FN_GRAN = ctypes.CFUNCTYPE(ctypes.c_int, ctypes.c_void_p, ctypes.c_int, _u64p)
_FN_RESERVE = ctypes.CFUNCTYPE(ctypes.c_int, ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint64, _u64p)
_FN_VA_SIZE = ctypes.CFUNCTYPE(ctypes.c_int, ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint64)
_FN_CREATE = ctypes.CFUNCTYPE(ctypes.c_int, ctypes.c_void_p, ctypes.c_uint64, ctypes.c_int, _u64p)
_FN_RELEASE = ctypes.CFUNCTYPE(ctypes.c_int, ctypes.c_void_p, ctypes.c_uint64)
_FN_MAP = ctypes.CFUNCTYPE(ctypes.c_int, ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint64)
_FN_ACCESS = ctypes.CFUNCTYPE(ctypes.c_int, ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint64, ctypes.c_int)


class VmmBackend(ctypes.Structure):
    """Function table of ekv_set_vmm_backend; build one with VmmBackend.from_callables(...)."""
    _fields_ = [("user", ctypes.c_void_p), ("granularity", _FN_GRAN), ("reserve", _FN_RESERVE),
                ("unreserve", _FN_VA_SIZE), ("create", _FN_CREATE), ("release", _FN_RELEASE), ("map", _FN_MAP),
                ("unmap", _FN_VA_SIZE), ("set_access", _FN_ACCESS)]

    @classmethod
    def from_callables(cls, granularity, reserve, unreserve, create, release, map, unmap, set_access):
        return cls(None, _FN_GRAN(granularity), _FN_RESERVE(reserve), _FN_VA_SIZE(unreserve), _FN_CREATE(create),
                   _FN_RELEASE(release), _FN_MAP(map), _FN_VA_SIZE(unmap), _FN_ACCESS(set_access))


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Load libekv.so (built in-tree by paper_2608_23658_b200.build). Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: run `python -m paper_2608_23658_b200.build` "
                          "(there is no fallback implementation)")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, i32, i64, u32, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint32, ctypes.c_float
    sz = ctypes.c_size_t
    dblp = ctypes.POINTER(ctypes.c_double)
    sig = {
        "ekv_pool_create": (i32, [ctypes.POINTER(PoolDesc), ctypes.POINTER(vp)]),
        "ekv_pool_destroy": (i32, [vp]),
        "ekv_pool_info": (i32, [vp, ctypes.POINTER(PoolInfo)]),
        "ekv_layer_ptr": (i32, [vp, i32, ctypes.POINTER(vp)]),
        "ekv_grow": (i32, [vp, vp, u32, dblp]),
        "ekv_shrink": (i32, [vp, vp, u32, dblp]),
        "ekv_write_kv": (i32, [vp, i32, vp, vp, vp, i32, vp]),
        "ekv_attn_workspace_bytes": (sz, [vp, i32, i32]),
        "ekv_attn_decode_plan": (i32, [vp, i32, i32, ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(sz)]),
        "ekv_attn_decode": (i32, [vp, i32, vp, vp, vp, i32, vp, i32, f32, vp, sz, vp]),
        "ekv_attn_decode_two_tensor": (i32, [vp, i32, vp, i64, vp, vp, vp, i32, vp, i32, f32, vp, sz, vp]),
        "ekv_attn_decode_static_scratch": (i32, [vp, i32, vp, vp, vp, i32, vp, i32, f32, vp]),
        "ekv_attn_prefill_chunk": (i32, [vp, i32, vp, vp, vp, i32, vp, vp, vp, i32, f32, vp]),
        "ekv_hoststep_create": (i32, [vp, i32, i32, i32, ctypes.POINTER(vp)]),
        "ekv_hoststep_destroy": (i32, [vp]),
        "ekv_hoststep_decode": (i32, [vp, i32, vp, vp, vp, vp, vp, i32, vp, i32, f32, vp, vp]),
        "ekv_hoststep_flush": (i32, [vp, vp]),
        "ekv_selftest_bounded_wait": (i32, [vp, i32, vp, vp]),
        "ekv_poll_status": (i32, [vp]),
        "ekv_blockpool_create": (i32, [i64, i64, ctypes.POINTER(vp)]),
        "ekv_blockpool_destroy": (i32, [vp]),
        "ekv_blockpool_alloc": (i32, [vp, i64, vp]),
        "ekv_blockpool_free": (i32, [vp, vp, i64]),
        "ekv_blockpool_admit_elastic": (i32, [vp]),
        "ekv_blockpool_gate_elastic": (i32, [vp, ctypes.POINTER(i64)]),
        "ekv_blockpool_drain_plan": (i32, [vp, vp, vp, i64, ctypes.POINTER(i64)]),
        "ekv_blockpool_drain_commit": (i32, [vp]),
        "ekv_blockpool_stats": (i32, [vp, ctypes.POINTER(BlockPoolStats)]),
        "ekv_move_blocks": (i32, [vp, vp, vp, i32, vp]),
        "ekv_controller_create": (i32, [ctypes.POINTER(ControllerDesc), i32, ctypes.POINTER(vp)]),
        "ekv_controller_destroy": (i32, [vp]),
        "ekv_controller_decide": (i32, [vp, i32]),
        "ekv_controller_stats": (i32, [vp, ctypes.POINTER(ControllerStats)]),
        "ekv_status_string": (ctypes.c_char_p, [i32]),
        "ekv_last_error": (ctypes.c_char_p, []),
        "ekv_set_vmm_backend": (i32, [ctypes.POINTER(VmmBackend)]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    _lib = lib
    return lib


def _check(st: int):
    if st != 0:
        raise EkvError(st, ekv_last_error())


def _dptr(t):
    """Device (or host) address of a torch tensor / raw int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_contiguous(), "tensors passed to libekv must be contiguous"
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


def ekv_status_string(status: int) -> str:
    return load_library().ekv_status_string(int(status)).decode()


def ekv_last_error() -> str:
    return load_library().ekv_last_error().decode()


def ekv_set_vmm_backend(backend: VmmBackend | None):
    _check(load_library().ekv_set_vmm_backend(ctypes.byref(backend) if backend is not None else None))


def ekv_pool_create(*, device=0, num_layers=1, num_q_heads, num_kv_heads, head_dim, block_size=16, base_blocks,
                    elastic_blocks=0, flags=0, dtype=EKV_BF16) -> int:
    desc = PoolDesc(device, num_layers, num_q_heads, num_kv_heads, head_dim, block_size, dtype, flags, base_blocks,
                    elastic_blocks)
    out = ctypes.c_void_p()
    _check(load_library().ekv_pool_create(ctypes.byref(desc), ctypes.byref(out)))
    return out.value


def ekv_pool_destroy(pool: int):
    _check(load_library().ekv_pool_destroy(pool))


def ekv_pool_info(pool: int) -> PoolInfo:
    info = PoolInfo()
    _check(load_library().ekv_pool_info(pool, ctypes.byref(info)))
    return info


def ekv_layer_ptr(pool: int, layer: int) -> int:
    out = ctypes.c_void_p()
    _check(load_library().ekv_layer_ptr(pool, layer, ctypes.byref(out)))
    return out.value


def _toggle(fn, pool, stream, flags, host_only):
    ms = (ctypes.c_double * 2)()
    _check(fn(pool, None if host_only else _stream(stream), flags, ms))
    return float(ms[0]), float(ms[1])


def ekv_grow(pool: int, stream=None, flags: int = 0, host_only: bool = False):
    """Returns (driver-call ms, whole-call ms)."""
    return _toggle(load_library().ekv_grow, pool, stream, flags, host_only)


def ekv_shrink(pool: int, stream=None, flags: int = 0, host_only: bool = False):
    """Returns (driver-call ms, whole-call ms)."""
    return _toggle(load_library().ekv_shrink, pool, stream, flags, host_only)


def ekv_write_kv(pool: int, layer: int, k, v, slot_mapping, stream=None):
    T = int(slot_mapping.shape[0])
    _check(load_library().ekv_write_kv(pool, layer, _dptr(k), _dptr(v), _dptr(slot_mapping), T, _stream(stream)))


def ekv_attn_workspace_bytes(pool: int, max_batch: int, max_seq_len: int) -> int:
    return int(load_library().ekv_attn_workspace_bytes(pool, max_batch, max_seq_len))


def ekv_attn_decode_plan(pool: int, B: int, max_blocks_per_seq: int):
    """Returns (keys per range, ranges per sequence, scratch bytes) of a decode call of exactly this shape."""
    chunk, nsplit, need = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_size_t()
    _check(load_library().ekv_attn_decode_plan(pool, B, max_blocks_per_seq, ctypes.byref(chunk), ctypes.byref(nsplit),
                                               ctypes.byref(need)))
    return int(chunk.value), int(nsplit.value), int(need.value)


def ekv_attn_decode(pool: int, layer: int, q, out, block_tables, seq_lens, scale: float, workspace, stream=None):
    B = int(seq_lens.shape[0])
    max_blocks = int(block_tables.shape[1])
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load_library().ekv_attn_decode(pool, layer, _dptr(q), _dptr(out), _dptr(block_tables), max_blocks,
                                          _dptr(seq_lens), B, float(scale), _dptr(workspace), ws_bytes,
                                          _stream(stream)))


def ekv_attn_decode_two_tensor(pool: int, layer: int, second_tensor, q, out, block_tables, seq_lens, scale: float, workspace,
                               stream=None):
    """Decode over two tensors: ids below the pool's base_blocks address the pool, the others `second_tensor`
    (a torch tensor of whole blocks in the pool's block layout)."""
    B = int(seq_lens.shape[0])
    max_blocks = int(block_tables.shape[1])
    info = ekv_pool_info(pool)
    nbytes = second_tensor.numel() * second_tensor.element_size()
    assert nbytes % info.block_bytes == 0
    ws_bytes = workspace.numel() * workspace.element_size()
    _check(load_library().ekv_attn_decode_two_tensor(pool, layer, _dptr(second_tensor), nbytes // info.block_bytes, _dptr(q),
                                                     _dptr(out), _dptr(block_tables), max_blocks, _dptr(seq_lens), B,
                                                     float(scale), _dptr(workspace), ws_bytes, _stream(stream)))


EKV_STATIC_SCRATCH_BYTES = 64 << 20


def ekv_attn_decode_static_scratch(pool: int, layer: int, q, out, block_tables, seq_lens, scale: float, stream=None):
    """Decode attention for callers that cannot allocate: same result as ekv_attn_decode, scratch taken
    from the library's built-in device array (at most EKV_STATIC_SCRATCH_BYTES; larger shapes are refused)."""
    B = int(seq_lens.shape[0])
    max_blocks = int(block_tables.shape[1])
    _check(load_library().ekv_attn_decode_static_scratch(pool, layer, _dptr(q), _dptr(out), _dptr(block_tables),
                                                         max_blocks, _dptr(seq_lens), B, float(scale),
                                                         _stream(stream)))


def ekv_selftest_bounded_wait(pool: int, limit_us: int, waited_ns=None, stream=None):
    """Runs the kernels' bounded wait until it gives up (nothing arrives); latches EKV_ERR_TIMEOUT. Harmless."""
    _check(load_library().ekv_selftest_bounded_wait(pool, int(limit_us), _dptr(waited_ns), _stream(stream)))


def ekv_hoststep_create(pool: int, max_batch: int, max_blocks_per_seq: int, depth: int = 2) -> int:
    out = ctypes.c_void_p()
    _check(load_library().ekv_hoststep_create(pool, max_batch, max_blocks_per_seq, depth, ctypes.byref(out)))
    return out.value


def ekv_hoststep_destroy(step: int):
    _check(load_library().ekv_hoststep_destroy(step))


def ekv_hoststep_decode(step: int, layer: int, h_q, h_k, h_v, h_slot_mapping, h_block_tables, h_seq_lens, scale: float, h_out,
                        stream=None):
    """One decode step from HOST tensors (pinned for overlap); h_k / h_v / h_slot_mapping may all be None."""
    B = int(h_seq_lens.shape[0])
    max_blocks = int(h_block_tables.shape[1])
    for t in (h_q, h_k, h_v, h_slot_mapping, h_block_tables, h_seq_lens, h_out):
        assert t is None or not t.is_cuda, "ekv_hoststep_decode takes host tensors"
    _check(load_library().ekv_hoststep_decode(step, layer, _dptr(h_q), _dptr(h_k), _dptr(h_v), _dptr(h_slot_mapping),
                                              _dptr(h_block_tables), max_blocks, _dptr(h_seq_lens), B, float(scale),
                                              _dptr(h_out), _stream(stream)))


def ekv_hoststep_flush(step: int, stream=None):
    _check(load_library().ekv_hoststep_flush(step, _stream(stream)))


def ekv_attn_prefill_chunk(pool: int, layer: int, q, out, block_tables, cu_q_lens, cu_q_lens_host, seq_lens,
                           scale: float, stream=None):
    R = int(seq_lens.shape[0])
    max_blocks = int(block_tables.shape[1])
    assert cu_q_lens_host.device.type == "cpu" and cu_q_lens_host.numel() == R + 1
    _check(load_library().ekv_attn_prefill_chunk(pool, layer, _dptr(q), _dptr(out), _dptr(block_tables), max_blocks,
                                                 _dptr(cu_q_lens), _dptr(cu_q_lens_host), _dptr(seq_lens), R,
                                                 float(scale), _stream(stream)))


def ekv_poll_status(pool: int) -> Status:
    return Status(load_library().ekv_poll_status(pool))


# ---------------------------------------------------------------- block pool, drain, controller


def ekv_blockpool_create(base_blocks: int, elastic_blocks: int) -> int:
    out = ctypes.c_void_p()
    _check(load_library().ekv_blockpool_create(base_blocks, elastic_blocks, ctypes.byref(out)))
    return out.value


def ekv_blockpool_destroy(bp: int):
    _check(load_library().ekv_blockpool_destroy(bp))


def ekv_blockpool_alloc(bp: int, n: int) -> list:
    ids = (ctypes.c_int32 * max(n, 1))()
    _check(load_library().ekv_blockpool_alloc(bp, n, ids))
    return list(ids[:n])


def ekv_blockpool_free(bp: int, ids):
    arr = (ctypes.c_int32 * max(len(ids), 1))(*ids)
    _check(load_library().ekv_blockpool_free(bp, arr, len(ids)))


def ekv_blockpool_admit_elastic(bp: int):
    _check(load_library().ekv_blockpool_admit_elastic(bp))


def ekv_blockpool_gate_elastic(bp: int) -> int:
    n = ctypes.c_int64(0)
    _check(load_library().ekv_blockpool_gate_elastic(bp, ctypes.byref(n)))
    return int(n.value)


def ekv_blockpool_drain_plan(bp: int, capacity: int):
    """Returns (from_ids, to_ids)."""
    f = (ctypes.c_int32 * max(capacity, 1))()
    t = (ctypes.c_int32 * max(capacity, 1))()
    n = ctypes.c_int64(0)
    _check(load_library().ekv_blockpool_drain_plan(bp, f, t, capacity, ctypes.byref(n)))
    return list(f[:n.value]), list(t[:n.value])


def ekv_blockpool_drain_commit(bp: int):
    _check(load_library().ekv_blockpool_drain_commit(bp))


def ekv_blockpool_stats(bp: int) -> BlockPoolStats:
    st = BlockPoolStats()
    _check(load_library().ekv_blockpool_stats(bp, ctypes.byref(st)))
    return st


def ekv_move_blocks(pool: int, src_ids, dst_ids, stream=None):
    n = int(src_ids.shape[0])
    _check(load_library().ekv_move_blocks(pool, _dptr(src_ids), _dptr(dst_ids), n, _stream(stream)))


def ekv_controller_create(commit_after_decode_steps: int, reserve_prefill_tokens: int, initially_committed: bool = False) -> int:
    desc = ControllerDesc(commit_after_decode_steps, reserve_prefill_tokens)
    out = ctypes.c_void_p()
    _check(load_library().ekv_controller_create(ctypes.byref(desc), int(initially_committed), ctypes.byref(out)))
    return out.value


def ekv_controller_destroy(ctrl: int):
    _check(load_library().ekv_controller_destroy(ctrl))


def ekv_controller_decide(ctrl: int, next_prefill_tokens: int) -> int:
    return int(load_library().ekv_controller_decide(ctrl, next_prefill_tokens))


def ekv_controller_stats(ctrl: int) -> ControllerStats:
    st = ControllerStats()
    _check(load_library().ekv_controller_stats(ctrl, ctypes.byref(st)))
    return st
