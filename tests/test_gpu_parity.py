"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs.  Bit-exact for the KV write and pool bytes; max-abs 2e-2 / mean-abs 2e-3 for bf16-in,
fp32-accumulate attention outputs."""
import math

import numpy as np
import pytest
import torch

import ekv_inputs as I
import oracle
import paper_2608_23658_b200 as ekv
from helpers import bf16_bits, cache_view, empty_cache, place_sequence

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 2e-2, 2e-3
DEV = "cuda:0"


def check_close(got_bf16: torch.Tensor, want_f64: np.ndarray, what=""):
    got = got_bf16.detach().float().cpu().numpy().astype(np.float64)
    assert got.shape == want_f64.shape, (got.shape, want_f64.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    err = np.abs(got - want_f64)
    assert err.max() <= MAX_ABS, f"{what}: max-abs {err.max():.4g}"
    assert err.mean() <= MEAN_ABS, f"{what}: mean-abs {err.mean():.4g}"


def seq_kv(seed, L, shape):
    n = L * shape.num_kv_heads * shape.head_dim
    K = I.normal_bf16(seed, 1, 0, n).view(L, shape.num_kv_heads, shape.head_dim)
    V = I.normal_bf16(seed, 2, 0, n).view(L, shape.num_kv_heads, shape.head_dim)
    return K, V


def rand_q(seed, rows, shape):
    return I.normal_bf16(seed, 3, 0, rows * shape.num_q_heads * shape.head_dim).view(
        rows, shape.num_q_heads, shape.head_dim)


# Which prefill kernel the pools of a test ask for (see the `prefill_kernel` fixture): nothing = the library's own
# choice by shape and chunk length; otherwise one of the pool flags that pin it.
_PREFILL_FLAGS = {}


def make_pool(shape, base_blocks, elastic_blocks=0, grown=False, layers=1):
    return ekv.Pool(num_q_heads=shape.num_q_heads, num_kv_heads=shape.num_kv_heads, head_dim=shape.head_dim,
                    base_blocks=base_blocks, elastic_blocks=elastic_blocks, num_layers=layers, start_grown=grown,
                    **_PREFILL_FLAGS)


@pytest.fixture(params=["auto", "one_head", "two_head", "warp_mma"])
def prefill_kernel(request):
    """Runs a prefill test once per kernel family: the library's own choice, then each family pinned through its pool
    flag (two_head falls back to one_head on shapes it cannot take: head_dim 64, a query group of one)."""
    _PREFILL_FLAGS.clear()
    if request.param != "auto":
        _PREFILL_FLAGS["prefill_" + request.param] = True
    yield request.param
    _PREFILL_FLAGS.clear()


class Case:
    """A set of sequences placed in a pool (through ekv_write_kv) and mirrored on the host."""

    def __init__(self, shape, lengths, pool_blocks, seed, pool=None, elastic_blocks=0, id_lo=0, perm_seed=None,
                 max_blocks_per_seq=None, fill_bits=0x7FC0):
        self.shape = shape
        self.lengths = torch.as_tensor(lengths, dtype=torch.int64)
        self.own_pool = pool is None
        self.pool = pool or make_pool(shape, pool_blocks - elastic_blocks, elastic_blocks, grown=elastic_blocks > 0)
        info = self.pool.info
        self.live = info.live_blocks
        usable = self.live - id_lo if pool_blocks is None else pool_blocks
        self.tables, self.free_ids = I.assign_blocks(seed if perm_seed is None else perm_seed, 4, self.lengths,
                                                     shape.block_size, usable, id_lo=id_lo,
                                                     max_blocks_per_seq=max_blocks_per_seq)
        self.seqs = [seq_kv(seed * 1000 + b, int(L), shape) for b, L in enumerate(self.lengths)]
        # device: poison every live block with NaN patterns, then scatter through the library
        view = self.pool.layer_tensor(0)
        view.view(torch.int16).fill_(np.array(fill_bits, dtype=np.uint16).view(np.int16).item())
        self.host = empty_cache(self.live, shape, fill=fill_bits)
        for b, (K, V) in enumerate(self.seqs):
            L = int(self.lengths[b])
            if L == 0:
                continue
            slots = I.position_slots(self.tables[b], 0, L, shape.block_size)
            self.pool.write_kv(0, K.to(DEV), V.to(DEV), slots.to(DEV))
            place_sequence(self.host, shape, self.tables[b], K, V)
        torch.cuda.synchronize()
        self.d_tables = self.tables.to(DEV)
        self.d_lengths = self.lengths.to(torch.int32).to(DEV)

    def close(self):
        if self.own_pool:
            self.pool.close()

    def decode(self, q, scale):
        return self.pool.attn_decode(0, q.to(DEV), self.d_tables, self.d_lengths, scale)

    def oracle_decode(self, q, scale):
        s = self.shape
        return oracle.attn_decode(self.host, s.num_q_heads, s.num_kv_heads, s.block_size, s.head_dim, q,
                                  self.tables, self.lengths, scale)


# --------------------------------------------------------------------------- KV write


def test_write_kv_is_an_exact_scatter():
    shape = I.TINY
    pool = make_pool(shape, 256, 256, grown=True)
    try:
        info = pool.info
        assert info.live_blocks == 512
        view = pool.layer_tensor(0)
        view.view(torch.int16).fill_(0x1234)
        T = 777
        K, V = seq_kv(5, T, shape)
        slots = I.permutation(9, 1, 512 * 16)[:T].clone()
        slots[::50] = -1
        pool.write_kv(0, K.to(DEV), V.to(DEV), slots.to(DEV))
        torch.cuda.synchronize()
        assert pool.poll_status() == ekv.Status.OK
        host = empty_cache(512, shape, fill=0x1234)
        assert oracle.write_kv(host, 512, shape.num_kv_heads, 16, shape.head_dim, K, V, slots) == 0
        got = bf16_bits(view.cpu()).reshape(-1)
        assert np.array_equal(got, host)
    finally:
        pool.close()


def test_write_kv_llama_shape_and_live_limit():
    shape = I.LLAMA8B
    pool = make_pool(shape, 64, 32, grown=False)  # elastic range exists but is NOT mapped
    try:
        info = pool.info
        assert (info.base_blocks, info.elastic_blocks, info.live_blocks) == (64, 32, 64)
        view = pool.layer_tensor(0)
        view.view(torch.int16).fill_(0x0BAD)
        T = 300
        K, V = seq_kv(6, T, shape)
        slots = I.permutation(10, 1, 64 * 16)[:T].clone()
        slots[7] = 70 * 16 + 3      # a block in the unmapped elastic range: must be skipped, not touched
        slots[9] = 5000 * 16        # far outside
        pool.write_kv(0, K.to(DEV), V.to(DEV), slots.to(DEV))
        torch.cuda.synchronize()
        assert pool.poll_status() == ekv.Status.ERR_BLOCK_OOB
        assert pool.poll_status() == ekv.Status.OK  # read-and-clear
        host = empty_cache(64, shape, fill=0x0BAD)
        assert oracle.write_kv(host, 64, shape.num_kv_heads, 16, shape.head_dim, K, V, slots) == 2
        assert np.array_equal(bf16_bits(view.cpu()).reshape(-1), host)
    finally:
        pool.close()


# --------------------------------------------------------------------------- decode


def test_decode_c1_tiny_paged_step():
    """configs[0]: 4/2 heads, d64, 512 blocks (256 base + 256 elastic, grown), 8 sequences U[1,512]."""
    cfg = I.C1
    lengths = I.decode_lengths(cfg)
    case = Case(cfg.shape, lengths, 512, cfg.seed, elastic_blocks=256)
    try:
        assert (case.tables >= 256).any() and ((case.tables >= 0) & (case.tables < 256)).any()
        q = rand_q(cfg.seed, len(lengths), cfg.shape)
        scale = 1 / math.sqrt(cfg.shape.head_dim)
        out = case.decode(q, scale)
        check_close(out, case.oracle_decode(q, scale), "C1 decode")
        assert case.pool.poll_status() == ekv.Status.OK
    finally:
        case.close()


@pytest.mark.parametrize("shape,lengths", [
    (I.LLAMA8B, [1, 15, 16, 17, 64, 65, 1000, 2049, 3333]),
    (I.LLAMA70B, [1, 16, 33, 500, 1025, 2500]),
    (I.Shape(8, 8, 128), [3, 200, 1100]),       # MHA: group of 1
    (I.Shape(16, 8, 64), [7, 129, 2100]),
])
def test_decode_matches_oracle_across_tiles_and_tails(shape, lengths):
    need = int(I.blocks_for(torch.tensor(lengths), 16).sum())
    case = Case(shape, lengths, need + 37, 21)
    try:
        q = rand_q(22, len(lengths), shape)
        scale = 1 / math.sqrt(shape.head_dim)
        out = case.decode(q, scale)
        check_close(out, case.oracle_decode(q, scale), f"decode {shape}")
        again = case.decode(q, scale)
        assert torch.equal(out, again), "decode is not bitwise reproducible"
        assert case.pool.poll_status() == ekv.Status.OK
    finally:
        case.close()


def test_decode_closed_forms_and_empty_sequence():
    shape = I.LLAMA8B
    lengths = [1, 0, 40, 1]
    case = Case(shape, lengths, 16, 31)
    try:
        # sequence 2: identical keys -> mean of V
        K, V = case.seqs[2]
        K[:] = K[0]
        slots = I.position_slots(case.tables[2], 0, 40, 16)
        case.pool.write_kv(0, K.to(DEV), V.to(DEV), slots.to(DEV))
        q = rand_q(32, 4, shape)
        out = case.decode(q, 0.09).float().cpu()
        for b in (0, 3):  # one key: its V row, exactly
            want = case.seqs[b][1][0].float().repeat_interleave(shape.group, 0)
            assert torch.equal(out[b], want)
        assert torch.equal(out[1], torch.zeros_like(out[1]))  # no keys: zeros
        mean_v = V.double().mean(0).repeat_interleave(shape.group, 0).numpy()
        assert np.abs(out[2].double().numpy() - mean_v).max() < 4e-3
    finally:
        case.close()


def test_decode_block_permutation_and_elastic_placement_are_bitwise_invariant():
    """Same logical data, different physical blocks (all-base, all-elastic, mixed): identical bits."""
    shape = I.LLAMA8B
    lengths = [700, 33, 2100, 1]
    need = int(I.blocks_for(torch.tensor(lengths), 16).sum())
    pool = make_pool(shape, 256, 256, grown=True)
    try:
        info = pool.info
        q = rand_q(41, len(lengths), shape)
        outs = []
        for id_lo, span, perm_seed in [(0, info.base_blocks, 1), (info.base_blocks, info.elastic_blocks, 2),
                                       (0, info.live_blocks, 3), (0, info.live_blocks, 4)]:
            assert need <= span
            case = Case(shape, lengths, span, 40, pool=pool, id_lo=id_lo, perm_seed=perm_seed)
            outs.append(case.decode(q, 0.088))
            if id_lo == 0 and span == info.live_blocks:
                assert (case.tables >= info.base_blocks).any(), "mixed case must straddle the base/elastic line"
        for o in outs[1:]:
            assert torch.equal(outs[0], o)
        check_close(outs[0], case.oracle_decode(q, 0.088), "straddling decode")
    finally:
        pool.close()


def test_decode_out_of_range_block_id_is_skipped_and_latched():
    shape = I.LLAMA8B
    pool = make_pool(shape, 64, 32, grown=False)
    try:
        lengths = [100, 50]
        case = Case(shape, lengths, 64, 51, pool=pool)
        q = rand_q(52, 2, shape)
        good = case.decode(q, 0.088)
        assert pool.poll_status() == ekv.Status.OK
        bad = case.tables.clone()
        bad[0, 2] = 80                      # inside the reserved range but NOT live (unmapped)
        bad[1, 1] = -5
        out = pool.attn_decode(0, q.to(DEV), bad.to(DEV), case.d_lengths, 0.088)
        torch.cuda.synchronize()
        assert pool.poll_status() == ekv.Status.ERR_BLOCK_OOB
        assert torch.isfinite(out.float()).all()
        # the skipped block's keys are simply absent: oracle on the shortened key set
        s = shape
        K, V = case.seqs[0]
        keep = torch.cat([torch.arange(0, 32), torch.arange(48, 100)])
        host = empty_cache(8, s)
        tbl = torch.arange(8, dtype=torch.int32)[None]
        place_sequence(host, s, tbl[0], K[keep], V[keep])
        want = oracle.attn_decode(host, s.num_q_heads, s.num_kv_heads, 16, s.head_dim, q[:1], tbl,
                                  torch.tensor([len(keep)]), 0.088)
        check_close(out[:1], want, "decode with a skipped block")
        assert torch.equal(pool.attn_decode(0, q.to(DEV), case.d_tables, case.d_lengths, 0.088), good)
    finally:
        pool.close()
    # long sequences: every warp walks many blocks, so the stage a skipped block would have used is reused
    pool = make_pool(shape, 512, 32, grown=False)
    try:
        lengths = [3000, 2500]
        case = Case(shape, lengths, 512, 53, pool=pool)
        q = rand_q(54, 2, shape)
        bad = case.tables.clone()
        skip = [0, 5, 6, 40, 187]                               # first block, neighbours, middle, the last one
        for j in skip:
            bad[0, j] = 530
        out = pool.attn_decode(0, q.to(DEV), bad.to(DEV), case.d_lengths, 0.088)
        torch.cuda.synchronize()
        assert pool.poll_status() == ekv.Status.ERR_BLOCK_OOB   # and not a timeout
        K, V = case.seqs[0]
        keep = torch.tensor([t for t in range(3000) if t // 16 not in skip])
        nb = (len(keep) + 15) // 16
        host = empty_cache(nb, shape)
        tbl = torch.arange(nb, dtype=torch.int32)[None]
        place_sequence(host, shape, tbl[0], K[keep], V[keep])
        want = oracle.attn_decode(host, shape.num_q_heads, shape.num_kv_heads, 16, shape.head_dim, q[:1], tbl,
                                  torch.tensor([len(keep)]), 0.088)
        check_close(out[:1], want, "long decode with skipped blocks")
        good = pool.attn_decode(0, q.to(DEV), case.d_tables, case.d_lengths, 0.088)
        check_close(good, case.oracle_decode(q, 0.088), "long decode")
        assert torch.equal(out[1], good[1])
    finally:
        pool.close()


def test_decode_argument_errors():
    shape = I.TINY
    pool = make_pool(shape, 256)
    try:
        q = torch.zeros(2, 4, 64, dtype=torch.bfloat16, device=DEV)
        bt = torch.zeros(2, 4, dtype=torch.int32, device=DEV)
        sl = torch.ones(2, dtype=torch.int32, device=DEV)
        small = torch.empty(256, dtype=torch.uint8, device=DEV)
        with pytest.raises(ekv.EkvError) as e:
            pool.attn_decode(0, q, bt, sl, 1.0, workspace=small)
        assert e.value.status == ekv.Status.ERR_WORKSPACE
        with pytest.raises(ekv.EkvError) as e:
            pool.attn_decode(3, q, bt, sl, 1.0)
        assert e.value.status == ekv.Status.ERR_INVALID
    finally:
        pool.close()


# --------------------------------------------------------------------------- prefill chunk


def run_prefill(case, q, chunks, scale):
    """chunks: list of (request index, first row of the chunk in the prompt, rows)."""
    s = case.shape
    outs = []
    for (r, start, c) in chunks:
        cu = torch.tensor([0, c], dtype=torch.int32)
        out = case.pool.attn_prefill_chunk(0, q[r][start:start + c].contiguous().to(DEV), case.d_tables[r:r + 1].contiguous(),
                                           cu.to(DEV), cu, torch.tensor([start + c], dtype=torch.int32, device=DEV),
                                           scale)
        outs.append(out)
    return outs


def test_prefill_c1_chunk_over_cached_prefix(prefill_kernel):
    """configs[0]: one 256-token chunk over a 256-token cached prefix."""
    cfg = I.C1
    case = Case(cfg.shape, [512], 512, cfg.seed + 100, elastic_blocks=256)
    try:
        s = cfg.shape
        q = rand_q(cfg.seed + 1, 256, s)
        scale = 1 / math.sqrt(s.head_dim)
        (out,) = run_prefill(case, [torch.cat([torch.zeros(256, s.num_q_heads, s.head_dim, dtype=torch.bfloat16), q])],
                             [(0, 256, 256)], scale)
        want = oracle.attn_prefill_chunk(case.host, s.num_q_heads, s.num_kv_heads, 16, s.head_dim, q, case.tables,
                                         np.array([0, 256]), np.array([512]), scale)
        check_close(out, want, "C1 prefill chunk")
        assert case.pool.poll_status() == ekv.Status.OK
    finally:
        case.close()


@pytest.mark.parametrize("shape", [I.LLAMA8B, I.TINY, I.LLAMA70B, I.Shape(12, 4, 128), I.Shape(28, 4, 128), I.Shape(4, 4, 128),
                                   I.Shape(6, 2, 64)])
def test_prefill_batched_ragged_requests_match_oracle(shape, prefill_kernel):
    chunks = [(0, 1), (0, 100), (37, 64), (500, 129), (130, 300), (1000, 17)]  # (prefix, rows)
    lengths = [p + c for p, c in chunks]
    need = int(I.blocks_for(torch.tensor(lengths), 16).sum())
    case = Case(shape, lengths, need + 11, 61)
    try:
        cu = torch.tensor(np.cumsum([0] + [c for _, c in chunks]), dtype=torch.int32)
        T = int(cu[-1])
        q = rand_q(62, T, shape)
        scale = 1 / math.sqrt(shape.head_dim)
        out = case.pool.attn_prefill_chunk(0, q.to(DEV), case.d_tables, cu.to(DEV), cu, case.d_lengths, scale)
        want = oracle.attn_prefill_chunk(case.host, shape.num_q_heads, shape.num_kv_heads, 16, shape.head_dim, q,
                                         case.tables, cu, case.lengths, scale)
        check_close(out, want, f"batched prefill {shape}")
        assert torch.equal(out, case.pool.attn_prefill_chunk(0, q.to(DEV), case.d_tables, cu.to(DEV), cu,
                                                             case.d_lengths, scale))
        assert case.pool.poll_status() == ekv.Status.OK
    finally:
        case.close()


@pytest.mark.parametrize("shape,R", [(I.LLAMA8B, 60), (I.TINY, 60), (I.LLAMA8B, 300), (I.Shape(28, 4, 128), 150), (I.Shape(20, 4, 128), 60),
                                     (I.Shape(6, 2, 128), 300)])
def test_prefill_many_requests_find_their_tiles(shape, R, prefill_kernel):
    """Many short requests in one call, some of them empty: every query tile must find its request (up to 256
    requests by bisection over a prefix table in the kernel parameters, more by walking cu_q_lens)."""
    rows = I.uniform_ints(71, 1, R, 0, 150)                  # chunk lengths, zeros included
    rows[R // 2] = 0
    prefix = I.uniform_ints(71, 2, R, 0, 90)
    lengths = rows + prefix
    need = int(I.blocks_for(lengths, 16).sum())
    case = Case(shape, lengths.tolist(), need + 7, 72)
    try:
        cu = torch.cat([torch.zeros(1, dtype=torch.int64), torch.cumsum(rows, 0)]).to(torch.int32)
        q = rand_q(73, int(cu[-1]), shape)
        scale = 1 / math.sqrt(shape.head_dim)
        out = case.pool.attn_prefill_chunk(0, q.to(DEV), case.d_tables, cu.to(DEV), cu, case.d_lengths, scale)
        want = oracle.attn_prefill_chunk(case.host, shape.num_q_heads, shape.num_kv_heads, 16, shape.head_dim, q,
                                         case.tables, cu, case.lengths, scale)
        check_close(out, want, f"{R} requests, {shape}")
        assert case.pool.poll_status() == ekv.Status.OK
    finally:
        case.close()


@pytest.mark.parametrize("shape", [I.LLAMA8B, I.TINY])
@pytest.mark.parametrize("mult", [4, 16])
def test_sharp_softmax_large_scores(shape, mult, prefill_kernel):
    """Queries 4x and 16x larger than the configs draw them: scores spread over tens of units, a row's running
    maximum jumps far between key tiles (the rescale paths of both kernels run), and nearly all the weight sits on a
    few keys.  Still inside the tolerance."""
    lengths = [1500, 333, 64]
    case = Case(shape, lengths, 140, 77)
    try:
        scale = 1 / math.sqrt(shape.head_dim)
        q = (rand_q(78, 3, shape).float() * mult).to(torch.bfloat16)      # exact: a power of two
        check_close(case.decode(q, scale), case.oracle_decode(q, scale), f"decode, q x{mult}")
        cu = torch.tensor(np.cumsum([0] + lengths), dtype=torch.int32)
        qp = (rand_q(79, int(cu[-1]), shape).float() * mult).to(torch.bfloat16)
        out = case.pool.attn_prefill_chunk(0, qp.to(DEV), case.d_tables, cu.to(DEV), cu, case.d_lengths, scale)
        want = oracle.attn_prefill_chunk(case.host, shape.num_q_heads, shape.num_kv_heads, 16, shape.head_dim, qp,
                                         case.tables, cu, case.lengths, scale)
        check_close(out, want, f"prefill, q x{mult}")
        assert case.pool.poll_status() == ekv.Status.OK
    finally:
        case.close()


@pytest.mark.parametrize("shape", [I.LLAMA8B, I.TINY])
def test_scores_that_rise_along_the_sequence_force_a_rescale_at_every_tile(shape, prefill_kernel):
    """Keys grow along the sequence so that each 16-token block scores about 2 units (log2) above the one before: a
    row's running maximum rises by far more than the lazy-rescale threshold at every key tile, the accumulated output
    is scaled down by 2^-16 or less each time, and nearly all the weight sits on the last visible block."""
    L, d = 1024, shape.head_dim
    case = Case(shape, [L], 80, 81)
    try:
        ramp = (torch.arange(L) // 16).float() / 64.0                      # multiples of 1/64: exact in bf16
        K = (ramp[:, None, None] * torch.ones(1, shape.num_kv_heads, d)).to(torch.bfloat16)
        V = case.seqs[0][1]
        slots = I.position_slots(case.tables[0], 0, L, shape.block_size)
        case.pool.write_kv(0, K.to(DEV), V.to(DEV), slots.to(DEV))
        place_sequence(case.host, shape, case.tables[0], K, V)
        scale = 1 / math.sqrt(d)
        qmag = 8.0 * 128 / d                                               # same score slope for both head sizes
        q = torch.full((L, shape.num_q_heads, d), qmag, dtype=torch.bfloat16)
        cu = torch.tensor([0, L], dtype=torch.int32)
        out = case.pool.attn_prefill_chunk(0, q.to(DEV), case.d_tables, cu.to(DEV), cu, case.d_lengths, scale)
        want = oracle.attn_prefill_chunk(case.host, shape.num_q_heads, shape.num_kv_heads, 16, d, q, case.tables, cu,
                                         case.lengths, scale)
        check_close(out, want, "prefill over rising scores")
        dec = case.pool.attn_decode(0, q[-1:].to(DEV), case.d_tables, case.d_lengths, scale)
        check_close(dec, want[-1:], "decode over rising scores")
        assert case.pool.poll_status() == ekv.Status.OK
    finally:
        case.close()


def test_prefill_chunked_equals_one_shot_and_decode_equals_last_row(prefill_kernel):
    shape = I.LLAMA8B
    L = 1500
    case = Case(shape, [L], 120, 71)
    try:
        q = rand_q(72, L, shape)
        scale = 1 / math.sqrt(shape.head_dim)
        (one,) = run_prefill(case, [q], [(0, 0, L)], scale)
        parts = run_prefill(case, [q], [(0, 0, 1), (0, 1, 500), (0, 501, 487), (0, 988, 512)], scale)
        chunked = torch.cat(parts)
        d = (one.float() - chunked.float()).abs()
        assert d.max() <= MAX_ABS and d.mean() <= MEAN_ABS
        want = oracle.attn_prefill_chunk(case.host, shape.num_q_heads, shape.num_kv_heads, 16, shape.head_dim, q,
                                         case.tables, np.array([0, L]), np.array([L]), scale)
        check_close(one, want, "one-shot prefill")
        check_close(chunked, want, "chunked prefill")
        dec = case.pool.attn_decode(0, q[-1:].to(DEV), case.d_tables, case.d_lengths, scale)
        check_close(dec, want[-1:], "decode vs last prefill row")
    finally:
        case.close()


# --------------------------------------------------------------------------- elastic range


def test_elastic_toggle_bytes_pointer_and_outputs():
    """Outputs for base-resident blocks are bit-identical across shrink/grow; with kept physical
    memory the elastic bytes read back exactly; the layer pointer never moves."""
    shape = I.LLAMA8B
    pool = make_pool(shape, 128, 1024, grown=True, layers=2)
    try:
        info = pool.info
        base, el = info.base_blocks, info.elastic_blocks
        ptrs = [pool.layer_ptr(l) for l in range(2)]
        lengths = [900, 77]
        case = Case(shape, lengths, base, 81, pool=pool)          # tenants of the base range only
        q = rand_q(82, 2, shape)
        ref = case.decode(q, 0.088)
        # seeded bytes into the elastic blocks of both layers
        for l in range(2):
            I.fill_normal_bf16_(pool.layer_tensor(l, base, el), 83, 10 + l)
        before = [pool.layer_tensor(l, base, el).cpu() for l in range(2)]

        ms = pool.shrink(keep_physical=True)
        assert ms[0] >= 0 and ms[1] >= ms[0]
        assert not pool.info.grown and pool.info.physical_held and pool.info.live_blocks == base
        assert torch.equal(case.decode(q, 0.088), ref)
        pool.grow()
        assert [pool.layer_ptr(l) for l in range(2)] == ptrs
        for l in range(2):
            assert torch.equal(pool.layer_tensor(l, base, el).cpu(), before[l])   # bytes survived the unmap
        assert torch.equal(case.decode(q, 0.088), ref)

        torch.cuda.synchronize()
        free0 = torch.cuda.mem_get_info()[0]
        pool.shrink()                                               # releasing shrink: memory returns
        free1 = torch.cuda.mem_get_info()[0]
        assert not pool.info.physical_held
        assert free1 - free0 >= 2 * info.elastic_bytes * 0.9
        assert torch.equal(case.decode(q, 0.088), ref)
        with pytest.raises(ValueError):
            pool.layer_tensor(0, base, el)                          # the wrapper refuses unmapped views
        free2 = torch.cuda.mem_get_info()[0]
        pool.grow()
        assert torch.cuda.mem_get_info()[0] <= free2 - 2 * info.elastic_bytes * 0.9
        # re-granted blocks read back exactly what is written after the remap, K through a copy and
        # V through the kernel (a one-key sequence returns its V row exactly)
        K, V = seq_kv(84, 1, shape)
        blk = base + 5
        pool.write_kv(1, K.to(DEV), V.to(DEV), torch.tensor([blk * 16], device=DEV))
        got = pool.layer_tensor(1, blk, 1).cpu()
        assert torch.equal(got[0, 0, :, 0, :], K[0]) and torch.equal(got[0, 1, :, 0, :], V[0])
        out = pool.attn_decode(1, q[:1].to(DEV), torch.tensor([[blk]], dtype=torch.int32, device=DEV),
                               torch.tensor([1], dtype=torch.int32, device=DEV), 0.088)
        assert torch.equal(out[0].cpu(), V[0].repeat_interleave(shape.group, 0))
        assert torch.equal(case.decode(q, 0.088), ref)
        assert pool.poll_status() == ekv.Status.OK
    finally:
        pool.close()


def test_prefill_edge_cases_bad_ids_empty_requests_negative_scale(prefill_kernel):
    """Out-of-range block ids inside a prompt are skipped and latched (every prefill kernel); requests with zero
    rows are legal; a negative scale is served (by the warp-level kernel) whatever the pool asks for."""
    shape = I.LLAMA8B
    pool = make_pool(shape, 128, 32, grown=False)
    try:
        chunks = [(0, 0), (200, 150), (0, 0), (64, 1)]               # (prefix, rows); two empty requests
        lengths = [p + c for p, c in chunks]
        case = Case(shape, lengths, 128, 91, pool=pool)
        cu = torch.tensor(np.cumsum([0] + [c for _, c in chunks]), dtype=torch.int32)
        q = rand_q(92, int(cu[-1]), shape)
        scale = 1 / math.sqrt(shape.head_dim)
        out = pool.attn_prefill_chunk(0, q.to(DEV), case.d_tables, cu.to(DEV), cu, case.d_lengths, scale)
        want = oracle.attn_prefill_chunk(case.host, shape.num_q_heads, shape.num_kv_heads, 16, shape.head_dim, q, case.tables,
                                         cu, case.lengths, scale)
        check_close(out, want, "prefill with empty requests")
        assert pool.poll_status() == ekv.Status.OK
        # a block of the prompt points into the unmapped elastic range: its 16 keys are skipped
        bad = case.tables.clone()
        bad[1, 3] = 140
        outb = pool.attn_prefill_chunk(0, q.to(DEV), bad.to(DEV), cu.to(DEV), cu, case.d_lengths, scale)
        torch.cuda.synchronize()
        assert pool.poll_status() == ekv.Status.ERR_BLOCK_OOB
        K, V = case.seqs[1]
        keep = torch.cat([torch.arange(0, 48), torch.arange(64, 350)])
        nb = (len(keep) + 15) // 16
        # oracle with the 16 keys removed: rows keep their causal limits, so restate them as shifted positions
        host = empty_cache(nb + 1, shape)
        tbl = torch.arange(nb, dtype=torch.int32)[None]
        place_sequence(host, shape, tbl[0], K[keep], V[keep])
        qs = q[int(cu[1]):int(cu[2])]
        wantb = oracle.attn_prefill_chunk(host, shape.num_q_heads, shape.num_kv_heads, 16, shape.head_dim, qs, tbl,
                                          np.array([0, 150]), np.array([len(keep)]), scale)
        check_close(outb[int(cu[1]):int(cu[2])], wantb, "prefill with a skipped block")
        # negative scale takes the warp-MMA kernel; compare with the oracle too
        outn = pool.attn_prefill_chunk(0, q.to(DEV), case.d_tables, cu.to(DEV), cu, case.d_lengths, -scale)
        wantn = oracle.attn_prefill_chunk(case.host, shape.num_q_heads, shape.num_kv_heads, 16, shape.head_dim, q,
                                          case.tables, cu, case.lengths, -scale)
        check_close(outn, wantn, "prefill with a negative scale")
        assert pool.poll_status() == ekv.Status.OK
    finally:
        pool.close()


def test_prefill_request_with_fewer_keys_than_rows_is_zeroed_and_latched(prefill_kernel):
    """A request whose seq_len is smaller than its chunk (no valid prefix) is invalid: its rows come out as zeros,
    EKV_ERR_BLOCK_OOB is latched, and the requests around it are served as usual (every prefill kernel)."""
    shape = I.LLAMA8B
    chunks = [(20, 140), (0, 200), (300, 129)]                    # (prefix, rows)
    lengths = [p + c for p, c in chunks]
    case = Case(shape, lengths, int(I.blocks_for(torch.tensor(lengths), 16).sum()) + 9, 101)
    try:
        cu = torch.tensor(np.cumsum([0] + [c for _, c in chunks]), dtype=torch.int32)
        q = rand_q(102, int(cu[-1]), shape)
        scale = 1 / math.sqrt(shape.head_dim)
        want = oracle.attn_prefill_chunk(case.host, shape.num_q_heads, shape.num_kv_heads, 16, shape.head_dim, q, case.tables,
                                         cu, case.lengths, scale)
        short = case.d_lengths.clone()
        short[1] = 150                                             # 200 rows over 150 keys
        out = torch.full((int(cu[-1]), shape.num_q_heads, shape.head_dim), 7.0, dtype=torch.bfloat16, device=DEV)
        case.pool.attn_prefill_chunk(0, q.to(DEV), case.d_tables, cu.to(DEV), cu, short, scale, out=out)
        torch.cuda.synchronize()
        assert case.pool.poll_status() == ekv.Status.ERR_BLOCK_OOB
        a, b = int(cu[1]), int(cu[2])
        assert torch.equal(out[a:b], torch.zeros_like(out[a:b]))
        check_close(out[:a], want[:a], "request before the invalid one")
        check_close(out[b:], want[b:], "request after the invalid one")
    finally:
        case.close()


@pytest.mark.parametrize("shape", [I.LLAMA8B, I.Shape(28, 4, 128)])
def test_prefill_many_invalid_requests_among_valid_ones(shape, prefill_kernel):
    """A batch of short requests in which about a third have fewer keys than rows, often several in a row: the
    persistent kernels walk lists in which items without work follow each other, and must neither stall nor mix up
    the others (rows of invalid requests are zeros, the rest matches the oracle, EKV_ERR_BLOCK_OOB is latched)."""
    R = 400
    rows = I.uniform_ints(111, 1, R, 2, 140)
    prefix = I.uniform_ints(111, 2, R, 0, 40)
    lengths = rows + prefix
    case = Case(shape, lengths.tolist(), int(I.blocks_for(lengths, 16).sum()) + 5, 112)
    try:
        cu = torch.cat([torch.zeros(1, dtype=torch.int64), torch.cumsum(rows, 0)]).to(torch.int32)
        q = rand_q(113, int(cu[-1]), shape)
        scale = 1 / math.sqrt(shape.head_dim)
        want = oracle.attn_prefill_chunk(case.host, shape.num_q_heads, shape.num_kv_heads, 16, shape.head_dim, q, case.tables,
                                         cu, case.lengths, scale)
        pick = I.uniform_ints(111, 3, R, 0, 99)
        invalid = [r for r in range(R) if int(pick[r]) < 35 or 100 <= r < 112]       # a third of them, and a run of twelve
        short = case.d_lengths.clone()
        for r in invalid:
            short[r] = int(rows[r]) - 1
        out = torch.full((int(cu[-1]), shape.num_q_heads, shape.head_dim), 7.0, dtype=torch.bfloat16, device=DEV)
        for _ in range(2):
            case.pool.attn_prefill_chunk(0, q.to(DEV), case.d_tables, cu.to(DEV), cu, short, scale, out=out)
        torch.cuda.synchronize()
        assert case.pool.poll_status() == ekv.Status.ERR_BLOCK_OOB
        got = out.float().cpu().numpy().astype(np.float64)
        bad = set(invalid)
        for r in range(R):
            a, b = int(cu[r]), int(cu[r + 1])
            if r in bad:
                assert not got[a:b].any(), f"request {r}: rows of an invalid request must be zeros"
            else:
                err = np.abs(got[a:b] - want[a:b])
                assert err.max() <= MAX_ABS, f"request {r}: max-abs {err.max():.4g}"
    finally:
        case.close()


@pytest.mark.parametrize("seed", range(8))
def test_prefill_random_batches_match_oracle_and_repeat_bit_for_bit(seed):
    """Seeded random batches (head layout, number of requests, chunk and prefix lengths, empty and invalid requests):
    the library's own kernel choice against the oracle, and the same call twice must give the same bits (a race between
    the roles of a persistent CTA shows up as a difference between runs long before it shows up as a wrong value)."""
    hq, hkv = [(32, 8), (28, 4), (12, 4), (8, 8), (20, 4), (64, 8), (6, 2), (16, 8)][seed]
    shape = I.Shape(hq, hkv, 128)
    R = [1, 3, 17, 40, 90, 150, 60, 25][seed]
    rows = I.uniform_ints(500 + seed, 1, R, 0, [900, 400, 300, 200, 140, 60, 129, 260][seed])
    prefix = I.uniform_ints(500 + seed, 2, R, 0, [1500, 700, 300, 200, 60, 130, 10, 400][seed])
    rows[0] = max(int(rows[0]), 1)
    lengths = rows + prefix
    case = Case(shape, lengths.tolist(), int(I.blocks_for(lengths, 16).sum()) + 3, 600 + seed)
    try:
        cu = torch.cat([torch.zeros(1, dtype=torch.int64), torch.cumsum(rows, 0)]).to(torch.int32)
        q = rand_q(700 + seed, int(cu[-1]), shape)
        scale = 1 / math.sqrt(shape.head_dim)
        pick = I.uniform_ints(500 + seed, 3, R, 0, 99)
        invalid = [r for r in range(1, R) if int(pick[r]) < 12 and int(rows[r]) > 1]
        seq = case.d_lengths.clone()
        for r in invalid:
            seq[r] = int(rows[r]) - 1
        outs = [case.pool.attn_prefill_chunk(0, q.to(DEV), case.d_tables, cu.to(DEV), cu, seq, scale).clone() for _ in range(3)]
        torch.cuda.synchronize()
        assert case.pool.poll_status() == (ekv.Status.ERR_BLOCK_OOB if invalid else ekv.Status.OK)
        assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])
        want = oracle.attn_prefill_chunk(case.host, shape.num_q_heads, shape.num_kv_heads, 16, shape.head_dim, q, case.tables,
                                         cu, case.lengths, scale)
        got = outs[0].float().cpu().numpy().astype(np.float64)
        for r in invalid:
            a, b = int(cu[r]), int(cu[r + 1])
            assert not got[a:b].any()
            want[a:b] = 0.0
        check_close(outs[0], want, f"random batch {seed}, {hq}q/{hkv}kv, {R} requests")
    finally:
        case.close()


def test_prefill_calls_in_flight_on_two_streams_keep_their_own_work_lists():
    """Two chunked-prefill calls of one pool running at the same time (two streams, different requests): the persistent
    kernel hands out its work items from a counter in device memory, and every launch must have its own."""
    shape = I.LLAMA8B
    case = Case(shape, [3000, 2500], 400, 97)
    try:
        scale = 1 / math.sqrt(shape.head_dim)
        cus = [torch.tensor([0, 3000], dtype=torch.int32), torch.tensor([0, 2500], dtype=torch.int32)]
        qs = [rand_q(98, 3000, shape).to(DEV), rand_q(99, 2500, shape).to(DEV)]
        tabs = [case.d_tables[0:1].contiguous(), case.d_tables[1:2].contiguous()]
        lens = [case.d_lengths[0:1].contiguous(), case.d_lengths[1:2].contiguous()]
        dcu = [c.to(DEV) for c in cus]
        alone = [case.pool.attn_prefill_chunk(0, qs[i], tabs[i], dcu[i], cus[i], lens[i], scale) for i in range(2)]
        torch.cuda.synchronize()
        streams = [torch.cuda.Stream(), torch.cuda.Stream()]
        outs = [torch.empty_like(q) for q in qs]
        for rep in range(3):
            for o in outs:
                o.zero_()
            torch.cuda.synchronize()
            for i in range(2):
                with torch.cuda.stream(streams[i]):
                    case.pool.attn_prefill_chunk(0, qs[i], tabs[i], dcu[i], cus[i], lens[i], scale, out=outs[i], stream=streams[i])
            torch.cuda.synchronize()
            for i in range(2):
                assert torch.equal(outs[i], alone[i]), f"call {i}, repetition {rep}"
        assert case.pool.poll_status() == ekv.Status.OK
    finally:
        case.close()


def test_prefill_kernel_families_agree_on_the_same_call():
    """The same call through each kernel family (pinned by its pool flag), each against the oracle and against the
    others."""
    shape = I.LLAMA8B
    outs = {}
    for impl in ("warp_mma", "two_head", "one_head"):
        pool = ekv.Pool(num_q_heads=shape.num_q_heads, num_kv_heads=shape.num_kv_heads, head_dim=shape.head_dim,
                        base_blocks=64, **{"prefill_" + impl: True})
        try:
            case = Case(shape, [700, 45], 64, 93, pool=pool)
            cu = torch.tensor([0, 300, 345], dtype=torch.int32)
            q = rand_q(94, 345, shape)
            out = pool.attn_prefill_chunk(0, q.to(DEV), case.d_tables, cu.to(DEV), cu, case.d_lengths, 0.088)
            want = oracle.attn_prefill_chunk(case.host, 32, 8, 16, 128, q, case.tables, cu, case.lengths, 0.088)
            check_close(out, want, impl + " prefill kernel")
            outs[impl] = out.float().cpu()
            assert pool.poll_status() == ekv.Status.OK
        finally:
            pool.close()
    for a, b in (("warp_mma", "two_head"), ("warp_mma", "one_head"), ("two_head", "one_head")):
        diff = (outs[a] - outs[b]).abs()
        assert diff.max().item() <= MAX_ABS and diff.mean().item() <= MEAN_ABS, (a, b)
    assert not torch.equal(outs["warp_mma"], outs["two_head"]), "different kernels are expected to round differently somewhere"


def test_recommit_out_of_memory_leaves_the_pool_shrunk_and_usable():
    """The paper's recommit OOM (the memory lent back may be gone when the controller wants it again): a grow
    whose physical allocation cannot be satisfied returns EKV_ERR_OOM, the pool stays shrunk, and attention over
    base blocks is unaffected.  The elastic range asked for is larger than the whole device, so creation fails at
    once without filling the memory."""
    shape = I.LLAMA8B
    total = torch.cuda.mem_get_info()[1]
    huge_blocks = int(2 * total // shape.block_bytes)
    pool = make_pool(shape, 128, huge_blocks, grown=False)        # reserving address space costs no memory
    try:
        case = Case(shape, [500, 70], 128, 95, pool=pool)
        q = rand_q(96, 2, shape)
        ref = case.decode(q, 0.088)
        free0 = torch.cuda.mem_get_info()[0]
        with pytest.raises(ekv.EkvError) as e:
            pool.grow()
        assert e.value.status == ekv.Status.ERR_OOM
        info = pool.info
        assert not info.grown and not info.physical_held and info.live_blocks == info.base_blocks
        assert abs(torch.cuda.mem_get_info()[0] - free0) < (64 << 20)   # nothing left allocated
        assert torch.equal(case.decode(q, 0.088), ref)
        assert pool.poll_status() == ekv.Status.OK
    finally:
        pool.close()
    with pytest.raises(ekv.EkvError) as e:                       # a base range that cannot be backed: nothing is left behind
        make_pool(shape, huge_blocks, 0)
    assert e.value.status == ekv.Status.ERR_OOM


def test_empty_calls_are_no_ops():
    """T = 0, B = 0 and R = 0 are legal and launch nothing."""
    shape = I.LLAMA8B
    pool = make_pool(shape, 64)
    try:
        view = pool.layer_tensor(0)
        view.view(torch.int16).fill_(0x3C00)
        before = view.cpu()
        z_kv = torch.empty(0, shape.num_kv_heads, shape.head_dim, dtype=torch.bfloat16, device=DEV)
        pool.write_kv(0, z_kv, z_kv, torch.empty(0, dtype=torch.int64, device=DEV))
        z_q = torch.empty(0, shape.num_q_heads, shape.head_dim, dtype=torch.bfloat16, device=DEV)
        out = pool.attn_decode(0, z_q, torch.empty(0, 4, dtype=torch.int32, device=DEV),
                               torch.empty(0, dtype=torch.int32, device=DEV), 0.1,
                               workspace=torch.empty(256, dtype=torch.uint8, device=DEV))
        assert out.shape == z_q.shape
        cu = torch.zeros(1, dtype=torch.int32)
        outp = pool.attn_prefill_chunk(0, z_q, torch.empty(0, 4, dtype=torch.int32, device=DEV), cu.to(DEV), cu,
                                       torch.empty(0, dtype=torch.int32, device=DEV), 0.1)
        assert outp.shape == z_q.shape
        ekv.ekv_move_blocks(pool.handle, torch.empty(0, dtype=torch.int32, device=DEV),
                            torch.empty(0, dtype=torch.int32, device=DEV))
        torch.cuda.synchronize()
        assert pool.poll_status() == ekv.Status.OK
        assert torch.equal(view.cpu(), before)
    finally:
        pool.close()


def test_decode_single_split_path_writes_final_rows_directly():
    """Many short sequences: one key range per sequence, so the split kernel finishes the rows itself (no combine
    pass).  Includes empty sequences, which must still come out as zero rows."""
    shape = I.LLAMA8B
    lengths = [int(x) for x in I.uniform_ints(97, 11, 200, 0, 500)]
    lengths[3] = 0
    lengths[77] = 0
    need = int(I.blocks_for(torch.tensor(lengths), 16).sum())
    case = Case(shape, lengths, need + 8, 97, max_blocks_per_seq=32)   # 32 blocks = 512 keys = one range
    try:
        q = rand_q(98, len(lengths), shape)
        out = torch.full((len(lengths), shape.num_q_heads, shape.head_dim), float("nan"), dtype=torch.bfloat16, device=DEV)
        case.pool.attn_decode(0, q.to(DEV), case.d_tables, case.d_lengths, 0.088, out=out)
        check_close(out, case.oracle_decode(q, 0.088), "single-split decode")
        assert (out[3] == 0).all() and (out[77] == 0).all()
        assert case.pool.poll_status() == ekv.Status.OK
    finally:
        case.close()
