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


def mirror_after_step(seed, layer, tables, lengths, seq_ids, shape, k=None, v=None):
    """Host mirror of the listed sequences of a pool filled by ekv_inputs.fill_pool_layer_(seed, layer), after a
    decode step has written the rows k[b], v[b] (bf16 [B, Hkv, d], indexed like `lengths`) at position L_b - 1.
    Returns (cache uint16, compact tables, lengths); the scatter is done by the oracle."""
    import ekv_inputs as I
    import oracle
    cache, ctab, clen = I.compact_host_cache(seed, layer, tables, lengths, seq_ids, shape)
    cache = bf16_bits(cache).copy()
    if k is not None:
        ids = list(seq_ids)
        slots = I.last_token_slots(clen, ctab, shape.block_size)
        oob = oracle.write_kv(cache, cache.size // shape.block_elems, shape.num_kv_heads, shape.block_size, shape.head_dim,
                              k[ids].contiguous(), v[ids].contiguous(), slots)
        assert oob == 0
    return cache, ctab, clen


def assert_close(got_bf16, want_f64, what="", max_abs=2e-2, mean_abs=2e-3):
    got = got_bf16.detach().float().cpu().numpy().astype(np.float64)
    assert got.shape == want_f64.shape, (got.shape, want_f64.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    err = np.abs(got - want_f64)
    assert err.max() <= max_abs and err.mean() <= mean_abs, f"{what}: max-abs {err.max():.4g}, mean-abs {err.mean():.4g}"
