"""Test-side helpers: cache construction by array views (an independent statement of the KV
layout: a layer is a [blocks, 2, Hkv, block_size, d] array) and bf16 bit handling."""
import numpy as np
import torch


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_f64(a: np.ndarray) -> np.ndarray:
    return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f64_of(t: torch.Tensor) -> np.ndarray:
    return t.to(torch.float64).numpy()


def empty_cache(pool_blocks, shape, fill=0):
    return np.full(pool_blocks * shape.block_elems, fill, dtype=np.uint16)


def cache_view(cache, shape):
    return cache.reshape(-1, 2, shape.num_kv_heads, shape.block_size, shape.head_dim)


def place_sequence(cache, shape, table_row, K, V):
    """K, V: bf16 torch [L, Hkv, d] -> scattered into the blocks table_row names."""
    view = cache_view(cache, shape)
    kb, vb = bf16_bits(K), bf16_bits(V)
    L = kb.shape[0]
    for j in range(L):
        n, t = int(table_row[j // shape.block_size]), j % shape.block_size
        view[n, 0, :, t, :] = kb[j]
        view[n, 1, :, t, :] = vb[j]
