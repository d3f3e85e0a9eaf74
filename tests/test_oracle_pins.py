"""Pins for the CPU oracle: everything here checks oracle/ against something other than itself --
a float64 NumPy restatement on brute-force inputs, torch's scaled_dot_product_attention on
contiguous KV, closed forms, and invariants of the definition.  No GPU, no CUDA library."""
import os

import numpy as np
import pytest
import torch

import ekv_inputs as I
import oracle
from helpers import bf16_bits, bits_to_f64, cache_view, empty_cache, f64_of, place_sequence

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
SH = I.TINY


def _seq(seed, L, shape=SH):
    n = L * shape.num_kv_heads * shape.head_dim
    K = I.normal_bf16(seed, 1, 0, n).view(L, shape.num_kv_heads, shape.head_dim)
    V = I.normal_bf16(seed, 2, 0, n).view(L, shape.num_kv_heads, shape.head_dim)
    return K, V


def _q(seed, rows, shape=SH):
    return I.normal_bf16(seed, 3, 0, rows * shape.num_q_heads * shape.head_dim).view(
        rows, shape.num_q_heads, shape.head_dim)


def _brute(q_row, K, V, g, scale):
    """float64 restatement: softmax(scale * q K^T) V for one head, keys = all rows of K."""
    s = scale * (f64_of(K[:, g, :]) @ f64_of(q_row))
    p = np.exp(s - s.max())
    return (p[:, None] * f64_of(V[:, g, :])).sum(0) / p.sum()


def _pool(lengths, shape=SH, seed=5, slack=7):
    lengths = torch.as_tensor(lengths, dtype=torch.int64)
    need = int(I.blocks_for(lengths, shape.block_size).sum())
    tables, _ = I.assign_blocks(seed, 4, lengths, shape.block_size, need + slack)
    return tables, need + slack


# ------------------------------------------------------------------ layout


def test_layout_golden_offsets():
    """Hand-computed element indices for the documented layout (block, K|V, head, token, channel)."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "layout_offsets.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) >= 8
    for r in rows:
        n, kv, h, t, x, hkv, bs, d, want = map(int, r)
        assert oracle.elem_index(n, kv, h, t, x, hkv, bs, d) == want


def test_layout_matches_array_view():
    shape = I.Shape(8, 4, 32, 16)
    cache = np.arange(6 * shape.block_elems, dtype=np.uint32)
    view = cache.reshape(6, 2, shape.num_kv_heads, shape.block_size, shape.head_dim)
    for (n, kv, h, t, x) in [(0, 0, 0, 0, 0), (5, 1, 3, 15, 31), (2, 1, 0, 7, 5), (3, 0, 2, 1, 30)]:
        assert view[n, kv, h, t, x] == oracle.elem_index(n, kv, h, t, x, 4, 16, 32)


# ------------------------------------------------------------------ write_kv (exact scatter)


def test_write_kv_scatter_roundtrip_and_canaries():
    pool = 12
    cache = empty_cache(pool, SH, fill=0xBEEF)
    T = 40
    K, V = _seq(11, T)
    slots = I.permutation(3, 1, pool * SH.block_size)[:T].clone()
    slots[5] = -1
    slots[17] = -7
    oob = oracle.write_kv(cache, pool, SH.num_kv_heads, SH.block_size, SH.head_dim, K, V, slots)
    assert oob == 0
    view = cache_view(cache, SH)
    touched = np.zeros(view.shape, dtype=bool)
    kb, vb = bf16_bits(K), bf16_bits(V)
    for i, s in enumerate(slots.tolist()):
        if s < 0:
            continue
        n, t = divmod(s, SH.block_size)
        assert np.array_equal(view[n, 0, :, t, :], kb[i])
        assert np.array_equal(view[n, 1, :, t, :], vb[i])
        touched[n, :, :, t, :] = True
    assert np.all(view[~touched] == 0xBEEF)
    assert touched.sum() == (T - 2) * 2 * SH.num_kv_heads * SH.head_dim


def test_write_kv_live_limit_and_last_writer():
    pool, live = 8, 5
    cache = empty_cache(pool, SH, fill=0x1234)
    K, V = _seq(12, 4)
    slots = torch.tensor([3 * 16 + 2, 6 * 16 + 1, 3 * 16 + 2, 5 * 16], dtype=torch.int64)
    oob = oracle.write_kv(cache, live, SH.num_kv_heads, SH.block_size, SH.head_dim, K, V, slots)
    assert oob == 2  # blocks 6 and 5 are >= live
    view = cache_view(cache, SH)
    assert np.array_equal(view[3, 0, :, 2, :], bf16_bits(K)[2])  # token 2 overwrote token 0
    assert np.all(view[5:] == 0x1234)


# ------------------------------------------------------------------ attention: brute force + library


@pytest.mark.parametrize("shape", [I.TINY, I.Shape(8, 2, 32, 16), I.Shape(6, 6, 16, 16)])
def test_decode_matches_float64_brute_force(shape):
    lengths = [1, 2, 15, 16, 17, 33, 70]
    tables, pool = _pool(lengths, shape)
    cache = empty_cache(pool, shape)
    seqs = [_seq(100 + b, L, shape) for b, L in enumerate(lengths)]
    for b, (K, V) in enumerate(seqs):
        place_sequence(cache, shape, tables[b], K, V)
    q = _q(7, len(lengths), shape)
    scale = 1.0 / np.sqrt(shape.head_dim)
    out = oracle.attn_decode(cache, shape.num_q_heads, shape.num_kv_heads, shape.block_size, shape.head_dim,
                             q, tables, torch.tensor(lengths), scale)
    for b, (K, V) in enumerate(seqs):
        for h in range(shape.num_q_heads):
            want = _brute(q[b, h], K, V, h // shape.group, scale)
            assert np.abs(out[b, h] - want).max() < 1e-12


def test_prefill_matches_float64_brute_force():
    chunks = [(0, 5), (16, 20), (37, 1), (3, 30)]  # (prefix, chunk rows)
    lengths = [p + c for p, c in chunks]
    tables, pool = _pool(lengths)
    cache = empty_cache(pool, SH)
    seqs = [_seq(200 + r, L) for r, L in enumerate(lengths)]
    for r, (K, V) in enumerate(seqs):
        place_sequence(cache, SH, tables[r], K, V)
    cu = np.cumsum([0] + [c for _, c in chunks]).astype(np.int32)
    q = _q(8, int(cu[-1]))
    scale = 0.2
    out = oracle.attn_prefill_chunk(cache, SH.num_q_heads, SH.num_kv_heads, SH.block_size, SH.head_dim, q,
                                    tables, cu, np.array(lengths), scale)
    for r, (p, c) in enumerate(chunks):
        K, V = seqs[r]
        for i in range(c):
            row = cu[r] + i
            for h in range(SH.num_q_heads):
                want = _brute(q[row, h], K[:p + i + 1], V[:p + i + 1], h // SH.group, scale)
                assert np.abs(out[row, h] - want).max() < 1e-12
    # the row-sample form returns the same rows
    rows = np.array([0, 4, 5, 24, 25, int(cu[-1]) - 1], dtype=np.int32)
    sub = oracle.attn_prefill_chunk(cache, SH.num_q_heads, SH.num_kv_heads, SH.block_size, SH.head_dim, q,
                                    tables, cu, np.array(lengths), scale, rows=rows)
    assert np.array_equal(sub, out[rows])


def test_contiguous_kv_reduces_to_torch_sdpa():
    """Identity block table + one sequence = ordinary attention: compare with the library routine."""
    shape = I.Shape(8, 2, 64, 16)
    p, c = 48, 37
    L = p + c
    K, V = _seq(31, L, shape)
    nb = (L + 15) // 16
    table = torch.arange(nb, dtype=torch.int32)[None]
    cache = empty_cache(nb, shape)
    place_sequence(cache, shape, table[0], K, V)
    q = _q(9, c, shape)
    scale = 1.0 / np.sqrt(shape.head_dim)
    out = oracle.attn_prefill_chunk(cache, shape.num_q_heads, shape.num_kv_heads, shape.block_size,
                                    shape.head_dim, q, table, np.array([0, c]), np.array([L]), scale)
    qq = q.double().permute(1, 0, 2)[None]                                   # [1, Hq, c, d]
    kk = K.double().permute(1, 0, 2).repeat_interleave(shape.group, 0)[None]  # [1, Hq, L, d]
    vv = V.double().permute(1, 0, 2).repeat_interleave(shape.group, 0)[None]
    mask = torch.arange(L)[None, :] <= (p + torch.arange(c))[:, None]         # lower-right causal
    ref = torch.nn.functional.scaled_dot_product_attention(qq, kk, vv, attn_mask=mask, scale=scale)
    ref = ref[0].permute(1, 0, 2).numpy()
    assert np.abs(out - ref).max() < 1e-10
    # decode = last row
    dec = oracle.attn_decode(cache, shape.num_q_heads, shape.num_kv_heads, shape.block_size, shape.head_dim,
                             q[-1:], table, np.array([L]), scale)
    assert np.abs(dec[0] - ref[-1]).max() < 1e-10


# ------------------------------------------------------------------ closed forms


def test_single_key_returns_its_v_row_exactly():
    K, V = _seq(41, 1)
    tables, pool = _pool([1])
    cache = empty_cache(pool, SH)
    place_sequence(cache, SH, tables[0], K, V)
    out = oracle.attn_decode(cache, 4, 2, 16, 64, _q(1, 1), tables, np.array([1]), 0.125)
    for h in range(4):
        assert np.array_equal(out[0, h], f64_of(V[0, h // 2]))


def test_identical_keys_return_mean_of_v():
    L = 40
    K, V = _seq(42, L)
    K[:] = K[0]
    tables, pool = _pool([L])
    cache = empty_cache(pool, SH)
    place_sequence(cache, SH, tables[0], K, V)
    out = oracle.attn_decode(cache, 4, 2, 16, 64, _q(2, 1), tables, np.array([L]), 0.125)
    for h in range(4):
        assert np.abs(out[0, h] - f64_of(V[:, h // 2]).mean(0)).max() < 1e-13


def test_zero_query_gives_causal_running_mean():
    p, c = 10, 25
    K, V = _seq(43, p + c)
    tables, pool = _pool([p + c])
    cache = empty_cache(pool, SH)
    place_sequence(cache, SH, tables[0], K, V)
    q = torch.zeros(c, 4, 64, dtype=torch.bfloat16)
    out = oracle.attn_prefill_chunk(cache, 4, 2, 16, 64, q, tables, np.array([0, c]), np.array([p + c]), 0.3)
    run = np.cumsum(f64_of(V), 0) / np.arange(1, p + c + 1)[:, None, None]
    for i in range(c):
        for h in range(4):
            assert np.abs(out[i, h] - run[p + i, h // 2]).max() < 1e-13


def test_dominant_key_selects_its_v_row():
    L, star = 50, 23
    K, V = _seq(44, L)
    K[:] = 0
    q = torch.zeros(1, 4, 64, dtype=torch.bfloat16)
    q[..., 0] = 8.0
    K[star, :, 0] = 8.0  # score 64*scale above the rest
    tables, pool = _pool([L])
    cache = empty_cache(pool, SH)
    place_sequence(cache, SH, tables[0], K, V)
    out = oracle.attn_decode(cache, 4, 2, 16, 64, q, tables, np.array([L]), 1.0)
    for h in range(4):
        assert np.abs(out[0, h] - f64_of(V[star, h // 2])).max() < 1e-6


# ------------------------------------------------------------------ invariants


def _decode_case(seed=50):
    lengths = torch.tensor([5, 64, 100, 31])
    seqs = [_seq(seed + b, int(L)) for b, L in enumerate(lengths)]
    q = _q(seed, len(lengths))
    return lengths, seqs, q


def test_block_permutation_invariance_is_bitwise():
    lengths, seqs, q = _decode_case()
    outs = []
    for perm_seed in (1, 2):
        tables, _ = I.assign_blocks(perm_seed, 9, lengths, 16, 40)
        cache = empty_cache(40, SH, fill=0x7FC0)  # unused blocks hold NaN patterns
        for b, (K, V) in enumerate(seqs):
            place_sequence(cache, SH, tables[b], K, V)
        outs.append(oracle.attn_decode(cache, 4, 2, 16, 64, q, tables, lengths, 0.125))
    assert np.array_equal(outs[0], outs[1])
    assert np.isfinite(outs[0]).all()


def test_chunked_prefill_equals_one_shot_and_decode_is_last_row():
    L = 90
    K, V = _seq(60, L)
    tables, pool = _pool([L])
    cache = empty_cache(pool, SH)
    place_sequence(cache, SH, tables[0], K, V)
    q = _q(61, L)
    args = (cache, 4, 2, 16, 64)
    one = oracle.attn_prefill_chunk(*args, q, tables, np.array([0, L]), np.array([L]), 0.125)
    parts, start = [], 0
    for c in (1, 16, 30, 43):
        parts.append(oracle.attn_prefill_chunk(*args, q[start:start + c], tables, np.array([0, c]),
                                               np.array([start + c]), 0.125))
        start += c
    assert start == L
    assert np.array_equal(np.concatenate(parts), one)
    for pos in (0, 15, 16, 89):
        dec = oracle.attn_decode(*args, q[pos:pos + 1], tables, np.array([pos + 1]), 0.125)
        assert np.array_equal(dec[0], one[pos])


def test_gqa_group_structure():
    L = 37
    K, V = _seq(70, L)
    tables, pool = _pool([L])
    cache = empty_cache(pool, SH)
    place_sequence(cache, SH, tables[0], K, V)
    q = _q(71, 1)
    q[0, 1] = q[0, 0]  # heads 0,1 share kv-head 0
    q[0, 2] = q[0, 0]  # head 2 reads kv-head 1
    base = oracle.attn_decode(cache, 4, 2, 16, 64, q, tables, np.array([L]), 0.125)
    assert np.array_equal(base[0, 0], base[0, 1])
    assert not np.array_equal(base[0, 0], base[0, 2])
    K2 = K.clone()
    K2[:, 1] = -K2[:, 1]  # perturb kv-head 1 only
    cache2 = empty_cache(pool, SH)
    place_sequence(cache2, SH, tables[0], K2, V)
    pert = oracle.attn_decode(cache2, 4, 2, 16, 64, q, tables, np.array([L]), 0.125)
    assert np.array_equal(pert[0, :2], base[0, :2])
    assert not np.array_equal(pert[0, 2:], base[0, 2:])


def test_output_is_convex_combination_and_ignores_table_tail():
    lengths, seqs, q = _decode_case(80)
    tables, _ = I.assign_blocks(3, 9, lengths, 16, 40, max_blocks_per_seq=12)
    cache = empty_cache(40, SH, fill=0x7FC0)
    for b, (K, V) in enumerate(seqs):
        place_sequence(cache, SH, tables[b], K, V)
    out = oracle.attn_decode(cache, 4, 2, 16, 64, q, tables, lengths, 0.125)
    for b, (K, V) in enumerate(seqs):
        v = f64_of(V)
        for h in range(4):
            assert (out[b, h] <= v[:, h // 2].max(0) + 1e-12).all()
            assert (out[b, h] >= v[:, h // 2].min(0) - 1e-12).all()
    garbage = tables.clone()
    garbage[garbage < 0] = 39  # entries past ceil(L/bs) must never be read
    assert np.array_equal(out, oracle.attn_decode(cache, 4, 2, 16, 64, q, garbage, lengths, 0.125))


def test_scale_and_sign_sensitivity():
    """A dropped scale or a swapped K/V operand cannot pass: compare two scales analytically."""
    L = 2
    K = torch.zeros(L, 2, 64, dtype=torch.bfloat16)
    V = torch.zeros(L, 2, 64, dtype=torch.bfloat16)
    K[1, :, 0] = 1.0
    V[0, :, :] = 1.0
    V[1, :, :] = 3.0
    q = torch.zeros(1, 4, 64, dtype=torch.bfloat16)
    q[..., 0] = 2.0
    tables, pool = _pool([L])
    cache = empty_cache(pool, SH)
    place_sequence(cache, SH, tables[0], K, V)
    for scale in (0.5, 1.0, -1.0):
        out = oracle.attn_decode(cache, 4, 2, 16, 64, q, tables, np.array([L]), scale)
        w = 1.0 / (1.0 + np.exp(-2.0 * scale))  # weight of key 1
        assert np.abs(out - (1.0 + 2.0 * w)).max() < 1e-14
