"""CPU oracle for the elastic-KV attention path -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper over ``ekv_oracle.c`` (plain C, double precision, OpenMP over
independent rows).  Only tests, the smoke check and the benchmark's cpu_baseline /
reference legs may import this package; the CUDA library never does, and this
package never imports the CUDA binding.

bf16 tensors cross this boundary as their 16-bit patterns (numpy ``uint16`` or a
torch ``bfloat16`` CPU tensor, which is reinterpreted, not converted).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ekv_oracle.c")
_SO = os.path.join(_HERE, "libekv_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no CUDA involved). Returns the .so path."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-fno-fast-math",
             "-ffp-contract=off", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i32, i64, dbl, vp = ctypes.c_int, ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
        lib.ekv_oracle_elem_index.restype = i64
        lib.ekv_oracle_elem_index.argtypes = [i64, i32, i32, i32, i32, i32, i32, i32]
        lib.ekv_oracle_threads.restype = i32
        lib.ekv_oracle_write_kv.restype = None
        lib.ekv_oracle_write_kv.argtypes = [vp, i64, i32, i32, i32, vp, vp, vp, i32, vp]
        lib.ekv_oracle_attn_decode.restype = None
        lib.ekv_oracle_attn_decode.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, i32, vp, i32, dbl]
        lib.ekv_oracle_attn_prefill_chunk.restype = None
        lib.ekv_oracle_attn_prefill_chunk.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, i32, vp, vp,
                                                      i32, dbl, vp, i32]
        _lib = lib
    return _lib


def _bits(a) -> np.ndarray:
    """bf16 payload -> contiguous numpy uint16 view (no value conversion)."""
    if isinstance(a, np.ndarray):
        assert a.dtype == np.uint16, a.dtype
        return np.ascontiguousarray(a)
    import torch  # local: the oracle itself needs numpy only
    assert a.dtype == torch.bfloat16 and a.device.type == "cpu"
    return a.contiguous().view(torch.int16).numpy().view(np.uint16)


def _i32(a) -> np.ndarray:
    if not isinstance(a, np.ndarray):
        a = a.cpu().numpy()
    return np.ascontiguousarray(a, dtype=np.int32)


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def threads() -> int:
    """Number of host threads the attention loops will use."""
    return int(_load().ekv_oracle_threads())


def elem_index(n, kv, h, t, x, num_kv_heads, block_size, head_dim) -> int:
    return int(_load().ekv_oracle_elem_index(n, kv, h, t, x, num_kv_heads, block_size, head_dim))


def write_kv(cache, live_blocks, num_kv_heads, block_size, head_dim, k, v, slot_mapping) -> int:
    """Exact scatter into ``cache`` (numpy uint16, modified in place). Returns #out-of-range slots."""
    assert isinstance(cache, np.ndarray) and cache.dtype == np.uint16 and cache.flags.c_contiguous
    kb, vb = _bits(k), _bits(v)
    sm = slot_mapping if isinstance(slot_mapping, np.ndarray) else slot_mapping.cpu().numpy()
    sm = np.ascontiguousarray(sm, dtype=np.int64)
    T = int(sm.shape[0])
    assert kb.size == T * num_kv_heads * head_dim == vb.size
    oob = ctypes.c_int64(0)
    _load().ekv_oracle_write_kv(_ptr(cache), int(live_blocks), num_kv_heads, block_size, head_dim,
                                _ptr(kb), _ptr(vb), _ptr(sm), T, ctypes.byref(oob))
    return int(oob.value)


def attn_decode(cache, num_q_heads, num_kv_heads, block_size, head_dim, q, block_tables, seq_lens,
                scale) -> np.ndarray:
    """Returns float64 [B, Hq, d]."""
    cb, qb = _bits(cache), _bits(q)
    bt, sl = _i32(block_tables), _i32(seq_lens)
    B = int(sl.shape[0])
    assert bt.ndim == 2 and bt.shape[0] == B
    assert qb.size == B * num_q_heads * head_dim
    out = np.empty((B, num_q_heads, head_dim), dtype=np.float64)
    _load().ekv_oracle_attn_decode(_ptr(cb), num_q_heads, num_kv_heads, block_size, head_dim, _ptr(qb),
                                   _ptr(out), _ptr(bt), int(bt.shape[1]), _ptr(sl), B, float(scale))
    return out


def attn_prefill_chunk(cache, num_q_heads, num_kv_heads, block_size, head_dim, q, block_tables,
                       cu_q_lens, seq_lens, scale, rows=None) -> np.ndarray:
    """Returns float64 [T, Hq, d], or [len(rows), Hq, d] when a row sample is given."""
    cb, qb = _bits(cache), _bits(q)
    bt, cu, sl = _i32(block_tables), _i32(cu_q_lens), _i32(seq_lens)
    R = int(sl.shape[0])
    assert bt.ndim == 2 and bt.shape[0] == R and cu.shape[0] == R + 1
    T = int(cu[R])
    assert qb.size == T * num_q_heads * head_dim
    if rows is None:
        rp, n = None, 0
        out = np.empty((T, num_q_heads, head_dim), dtype=np.float64)
    else:
        rows = _i32(rows)
        assert rows.size == 0 or (rows.min() >= 0 and rows.max() < T)
        rp, n = _ptr(rows), int(rows.size)
        out = np.empty((n, num_q_heads, head_dim), dtype=np.float64)
    _load().ekv_oracle_attn_prefill_chunk(_ptr(cb), num_q_heads, num_kv_heads, block_size, head_dim,
                                          _ptr(qb), _ptr(out), _ptr(bt), int(bt.shape[1]), _ptr(cu),
                                          _ptr(sl), R, float(scale), rp, n)
    return out
