"""Seeded synthetic inputs for the elastic-KV attention path.

This module is the only code the CUDA tests/benchmark and the CPU oracle tests
share.  It holds NO attention / scatter arithmetic: only a counter-based integer
generator (so the same bits come out on a CPU and on a GPU, and any sub-range can
be regenerated without materialising the rest), length / block-table draws and
the descriptions of the five benchmark configurations.

Value recipe ("~N(0,1) bf16"): splitmix64 of (key, element index) gives two 64-bit
words = eight 16-bit uniforms; their sum, centred, times one float32 constant, is
rounded to bf16 (round-to-nearest-even).  This is a central-limit approximation
of N(0,1): unit variance, support clipped at about +-4.9 sigma.
"""
from __future__ import annotations

import dataclasses
import math

import torch

BASE_SEED = 260823658

_M64 = (1 << 64) - 1


def _s64(x: int) -> int:
    """Python int -> the int64 with the same low 64 bits."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLD = _s64(0x9E3779B97F4A7C15)
_MUL1 = _s64(0xBF58476D1CE4E5B9)
_MUL2 = _s64(0x94D049BB133111EB)


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    return (z >> s) & ((1 << (64 - s)) - 1)


def mix64(x: torch.Tensor) -> torch.Tensor:
    """splitmix64 output function on int64 tensors (two's-complement wraparound)."""
    z = x + _GOLD
    z = (z ^ _lsr(z, 30)) * _MUL1
    z = (z ^ _lsr(z, 27)) * _MUL2
    return z ^ _lsr(z, 31)


def _key(seed: int, stream: int) -> int:
    k = torch.tensor([_s64(seed * 0x100000001B3 + stream)], dtype=torch.int64)
    return int(mix64(mix64(k) + stream)[0])


_SIGMA8 = math.sqrt(8.0 * (65536.0 ** 2 - 1.0) / 12.0)
_INV_SIGMA8 = float(torch.tensor(1.0 / _SIGMA8, dtype=torch.float32))


def _normal_from_idx(key: int, idx: torch.Tensor) -> torch.Tensor:
    total = torch.zeros_like(idx)
    for half in range(2):
        w = mix64((idx * 2 + half) ^ key)
        for f in range(4):
            total += _lsr(w, 16 * f) & 0xFFFF
    centred = (total - 4 * 65535).to(torch.float32)  # |.| < 2^24: exact
    return (centred * _INV_SIGMA8).to(torch.bfloat16)


def normal_bf16(seed: int, stream: int, start: int, count: int, device="cpu") -> torch.Tensor:
    """bf16 values ~N(0,1) for element indices start .. start+count-1 of (seed, stream).

    Element i depends only on (seed, stream, i); identical bits on every device."""
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    return _normal_from_idx(_key(seed, stream), idx)


def normal_bf16_at(seed: int, stream: int, idx: torch.Tensor) -> torch.Tensor:
    """The same values at arbitrary element indices (int64 tensor, any device)."""
    return _normal_from_idx(_key(seed, stream), idx)


def fill_normal_bf16_(dst: torch.Tensor, seed: int, stream: int, start: int = 0,
                      chunk: int = 1 << 24) -> torch.Tensor:
    """In-place fill of a flat bf16 tensor with normal_bf16(seed, stream, start + i)."""
    flat = dst.view(-1)
    n = flat.numel()
    for o in range(0, n, chunk):
        c = min(chunk, n - o)
        flat[o:o + c] = normal_bf16(seed, stream, start + o, c, device=dst.device)
    return dst


def uniform_ints(seed: int, stream: int, count: int, lo: int, hi: int) -> torch.Tensor:
    """count integers uniform on [lo, hi] inclusive (int64, CPU)."""
    key = _key(seed, stream)
    idx = torch.arange(count, dtype=torch.int64)
    w = _lsr(mix64(idx ^ key), 1)  # non-negative
    return lo + w % (hi - lo + 1)


def permutation(seed: int, stream: int, n: int) -> torch.Tensor:
    """Seeded permutation of 0..n-1 (int64, CPU): argsort of per-index hash words."""
    key = _key(seed, stream)
    w = mix64(torch.arange(n, dtype=torch.int64) ^ key)
    return torch.argsort(w, stable=True)


# --------------------------------------------------------------------------- shapes


@dataclasses.dataclass(frozen=True)
class Shape:
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    block_size: int = 16

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    @property
    def token_bytes(self) -> int:  # K and V of one token, all kv heads, one layer
        return 2 * self.num_kv_heads * self.head_dim * 2

    @property
    def block_bytes(self) -> int:
        return self.block_size * self.token_bytes

    @property
    def block_elems(self) -> int:
        return self.block_bytes // 2


TINY = Shape(4, 2, 64)
LLAMA8B = Shape(32, 8, 128)
LLAMA70B = Shape(64, 8, 128)


def blocks_for(lengths: torch.Tensor, block_size: int) -> torch.Tensor:
    return (lengths + block_size - 1) // block_size


def assign_blocks(seed: int, stream: int, lengths: torch.Tensor, block_size: int, pool_blocks: int,
                  id_lo: int = 0, max_blocks_per_seq: int | None = None):
    """Scatter sequences over a pool: a seeded permutation of ids id_lo..id_lo+pool_blocks-1 is cut
    into consecutive runs, one run per sequence.  Returns (block_tables int32 [B, max_blocks],
    unused ids int64).  Unused table entries hold -1."""
    nb = blocks_for(lengths, block_size)
    need = int(nb.sum())
    if need > pool_blocks:
        raise ValueError(f"workload needs {need} blocks, pool has {pool_blocks}")
    perm = permutation(seed, stream, pool_blocks) + id_lo
    width = int(nb.max()) if max_blocks_per_seq is None else max_blocks_per_seq
    tables = torch.full((len(lengths), width), -1, dtype=torch.int32)
    o = 0
    for b, n in enumerate(nb.tolist()):
        tables[b, :n] = perm[o:o + n].to(torch.int32)
        o += n
    return tables, perm[o:]


def last_token_slots(lengths: torch.Tensor, tables: torch.Tensor, block_size: int) -> torch.Tensor:
    """Slot (block*block_size + offset) of position L-1 of every sequence (int64)."""
    pos = lengths - 1
    blk = tables[torch.arange(len(lengths)), pos // block_size].to(torch.int64)
    return blk * block_size + pos % block_size


def position_slots(table_row: torch.Tensor, start: int, count: int, block_size: int) -> torch.Tensor:
    """Slots of positions start..start+count-1 of one sequence (int64)."""
    pos = torch.arange(start, start + count, dtype=torch.int64)
    return table_row[pos // block_size].to(torch.int64) * block_size + pos % block_size


# ------------------------------------------------------------------ the five configurations


@dataclasses.dataclass(frozen=True)
class DecodeSet:
    batch: int
    len_lo: int
    len_hi: int


@dataclasses.dataclass(frozen=True)
class Config:
    name: str
    shape: Shape
    seed: int
    num_layers: int = 1
    decode: DecodeSet | None = None
    prompt_len: int = 0            # one synthetic prompt (0 = none)
    chunk_lens: tuple = ()         # chunkings of that prompt to run
    elastic_fraction: float = 0.0  # share of pool blocks in the elastic sub-range
    elastic_total_bytes: int = 0   # or: absolute elastic reserve summed over layers
    steps: int = 1
    toggle_every: int = 0


C1 = Config("c1_tiny_paged_step", TINY, BASE_SEED + 1, decode=DecodeSet(8, 1, 512), prompt_len=512,
            chunk_lens=(256,), elastic_fraction=0.5)
C2 = Config("c2_llama8b_decode", LLAMA8B, BASE_SEED + 2, decode=DecodeSet(256, 1024, 8192))
C3 = Config("c3_llama8b_mixed_prefill", LLAMA8B, BASE_SEED + 3, decode=DecodeSet(256, 2048, 8192),
            prompt_len=32768, chunk_lens=(8192, 32768))
C4 = Config("c4_llama70b_long_context", LLAMA70B, BASE_SEED + 4, decode=DecodeSet(64, 32768, 131072),
            elastic_fraction=0.16)
C5 = Config("c5_elastic_toggle", LLAMA8B, BASE_SEED + 5, num_layers=32, decode=DecodeSet(128, 1024, 16384),
            elastic_total_bytes=3 << 30, steps=1000, toggle_every=50)

CONFIGS = {c.name: c for c in (C1, C2, C3, C4, C5)}


def decode_lengths(cfg: Config, batch: int | None = None) -> torch.Tensor:
    d = cfg.decode
    return uniform_ints(cfg.seed, 11, d.batch if batch is None else batch, d.len_lo, d.len_hi)


# ------------------------------------------------------------------ physical fills and host mirrors

KV_STREAM = 21  # stream id of "pool content as a function of the physical element index"


def fill_pool_layer_(layer_view: torch.Tensor, seed: int, layer: int = 0, first_block: int = 0, chunk: int = 1 << 24) -> None:
    """Fill a [blocks, 2, Hkv, bs, d] bf16 view of a layer (starting at physical block first_block)
    so that element e of the layer holds normal_bf16(seed, KV_STREAM + layer, e).  The view may be strided
    between blocks (a layer of a fused range); each block itself is dense."""
    block_elems = layer_view[0].numel()
    if layer_view.is_contiguous():
        fill_normal_bf16_(layer_view, seed, KV_STREAM + layer, start=first_block * block_elems, chunk=chunk)
        return
    per = max(1, chunk // block_elems)
    for b0 in range(0, layer_view.shape[0], per):
        b1 = min(layer_view.shape[0], b0 + per)
        vals = normal_bf16(seed, KV_STREAM + layer, (first_block + b0) * block_elems, (b1 - b0) * block_elems,
                           device=layer_view.device)
        layer_view[b0:b1] = vals.view(b1 - b0, *layer_view.shape[1:])


def host_blocks(seed: int, layer: int, block_ids, block_elems: int, device="cpu") -> torch.Tensor:
    """Regeneration, in host memory, of the listed physical blocks of a fill_pool_layer_ pool: bf16 [n, block_elems].
    The generator itself may run on another torch device (same bits everywhere); the result is returned on the CPU."""
    out = torch.empty(len(block_ids), block_elems, dtype=torch.bfloat16)
    if torch.device(device).type == "cpu":
        for i, n in enumerate(block_ids):
            out[i] = normal_bf16(seed, KV_STREAM + layer, int(n) * block_elems, block_elems)
        return out
    ids = torch.as_tensor(block_ids, dtype=torch.int64, device=device)
    ar = torch.arange(block_elems, dtype=torch.int64, device=device)[None]
    per = max(1, (1 << 25) // block_elems)
    for o in range(0, len(ids), per):
        idx = (ids[o:o + per, None] * block_elems + ar).reshape(-1)
        out[o:o + per] = normal_bf16_at(seed, KV_STREAM + layer, idx).view(-1, block_elems).cpu()
    return out


def compact_host_cache(seed: int, layer: int, tables: torch.Tensor, lengths: torch.Tensor, seq_ids, shape: Shape,
                       device="cpu"):
    """Host mirror holding only the blocks of the listed sequences, renumbered 0..n-1.
    Returns (cache bf16 [n*block_elems], compact tables int32 [len(seq_ids), width], lengths).
    `device`: where the value generator runs (the mirror always ends up in host memory)."""
    nb = blocks_for(lengths, shape.block_size)
    width = int(nb[list(seq_ids)].max())
    ctab = torch.full((len(seq_ids), width), -1, dtype=torch.int32)
    ids = []
    for i, b in enumerate(seq_ids):
        n = int(nb[b])
        ctab[i, :n] = torch.arange(len(ids), len(ids) + n, dtype=torch.int32)
        ids += tables[b, :n].tolist()
    cache = host_blocks(seed, layer, ids, shape.block_elems, device=device).view(-1)
    return cache, ctab, lengths[list(seq_ids)].clone()


def decode_algorithmic_bytes(lengths: torch.Tensor, shape: Shape) -> int:
    """Bytes a decode step must move: every cached K and V element once, Q in, O out, block table."""
    B = len(lengths)
    kv = int(lengths.sum()) * shape.token_bytes
    qo = 2 * B * shape.num_q_heads * shape.head_dim * 2
    table = int(blocks_for(lengths, shape.block_size).sum()) * 4
    return kv + qo + table


def write_algorithmic_bytes(T: int, shape: Shape) -> int:
    return 2 * T * shape.token_bytes + 8 * T


def prefill_flops(chunk: int, prefix: int, shape: Shape) -> int:
    """Causal-exact FLOPs of both contractions: 4*d*Hq per (query row, visible key) pair."""
    pairs = chunk * prefix + chunk * (chunk + 1) // 2
    return 4 * shape.head_dim * shape.num_q_heads * pairs
