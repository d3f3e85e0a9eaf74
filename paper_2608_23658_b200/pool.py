"""Convenience wrapper over the C ABI: owns a pool handle, hands out zero-copy torch views of the
mapped part of a layer's range and keeps a decode workspace.  No arithmetic happens here."""
from __future__ import annotations

import torch

from . import _binding as B


class _RawCuda:
    """Minimal __cuda_array_interface__ carrier for a raw device range (int16 elements)."""

    def __init__(self, ptr: int, nelem: int):
        self.__cuda_array_interface__ = {"shape": (nelem,), "typestr": "<i2", "data": (ptr, False), "version": 3,
                                         "strides": None}


class Pool:
    def __init__(self, *, num_q_heads, num_kv_heads, head_dim, base_blocks, elastic_blocks=0, num_layers=1,
                 block_size=16, device=0, start_grown=False, fused_range=False, prefill_warp_mma=False,
                 prefill_one_head=False, prefill_two_head=False):
        self.device = torch.device("cuda", device)
        torch.cuda.set_device(self.device)
        self.handle = B.ekv_pool_create(device=device, num_layers=num_layers, num_q_heads=num_q_heads,
                                        num_kv_heads=num_kv_heads, head_dim=head_dim, block_size=block_size,
                                        base_blocks=base_blocks, elastic_blocks=elastic_blocks,
                                        flags=(B.EKV_START_GROWN if start_grown else 0) | (B.EKV_FUSED_RANGE if fused_range else 0) |
                                        (B.EKV_PREFILL_WARP_MMA if prefill_warp_mma else 0) |
                                        (B.EKV_PREFILL_ONE_HEAD if prefill_one_head else 0) |
                                        (B.EKV_PREFILL_TWO_HEAD if prefill_two_head else 0))
        self.num_q_heads, self.num_kv_heads, self.head_dim, self.block_size = num_q_heads, num_kv_heads, head_dim, block_size
        self.num_layers = num_layers
        self._ws = None

    # -- lifetime
    def close(self):
        if self.handle:
            torch.cuda.synchronize(self.device)
            B.ekv_pool_destroy(self.handle)
            self.handle = None
            self._ws = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- state
    @property
    def info(self) -> B.PoolInfo:
        return B.ekv_pool_info(self.handle)

    def layer_ptr(self, layer: int) -> int:
        return B.ekv_layer_ptr(self.handle, layer)

    def layer_tensor(self, layer: int, first_block: int = 0, num_blocks: int | None = None) -> torch.Tensor:
        """bf16 view [blocks, 2, Hkv, block_size, head_dim] of blocks first_block.. of a layer.
        Only LIVE blocks may be viewed: unmapped elastic addresses fault when touched."""
        info = self.info
        if num_blocks is None:
            num_blocks = info.live_blocks - first_block
        if first_block < 0 or first_block + num_blocks > info.live_blocks:
            raise ValueError("view would reach past the live (mapped) blocks")
        elems = info.block_bytes // 2
        stride = info.block_stride_bytes // 2      # elements between consecutive block ids of this layer
        span = (num_blocks - 1) * stride + elems if num_blocks > 0 else 0
        raw = _RawCuda(self.layer_ptr(layer) + first_block * info.block_stride_bytes, max(span, 1))
        flat = torch.as_tensor(raw, device=self.device).view(torch.bfloat16)
        d, bs, hk = self.head_dim, self.block_size, self.num_kv_heads
        # dense when stride == elems (one range per layer); a strided view over the fused range otherwise
        return torch.as_strided(flat, (num_blocks, 2, hk, bs, d), (stride, hk * bs * d, bs * d, d, 1))

    def grow(self, stream=None):
        return B.ekv_grow(self.handle, stream)

    def shrink(self, keep_physical: bool = False, stream=None):
        return B.ekv_shrink(self.handle, stream, B.EKV_KEEP_PHYSICAL if keep_physical else 0)

    def poll_status(self) -> B.Status:
        return B.ekv_poll_status(self.handle)

    # -- compute (argument marshalling only)
    def write_kv(self, layer, k, v, slot_mapping, stream=None):
        B.ekv_write_kv(self.handle, layer, k, v, slot_mapping, stream)

    def workspace(self, batch: int, max_seq_len: int) -> torch.Tensor:
        need = B.ekv_attn_workspace_bytes(self.handle, batch, max_seq_len)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=self.device)
        return self._ws

    def attn_decode(self, layer, q, block_tables, seq_lens, scale, out=None, workspace=None, stream=None):
        if out is None:
            out = torch.empty_like(q)
        if workspace is None:
            workspace = self.workspace(int(seq_lens.shape[0]), int(block_tables.shape[1]) * self.block_size)
        B.ekv_attn_decode(self.handle, layer, q, out, block_tables, seq_lens, scale, workspace, stream)
        return out

    def attn_prefill_chunk(self, layer, q, block_tables, cu_q_lens, cu_q_lens_host, seq_lens, scale, out=None,
                           stream=None):
        if out is None:
            out = torch.empty_like(q)
        B.ekv_attn_prefill_chunk(self.handle, layer, q, out, block_tables, cu_q_lens, cu_q_lens_host, seq_lens,
                                 scale, stream)
        return out


class HostStep:
    """Decode steps driven from pinned host tensors (ekv_hoststep_*): copies in, write_kv + decode, copy out,
    double-buffered on the library's own copy streams.  Close it before its pool."""

    def __init__(self, pool: Pool, max_batch: int, max_blocks_per_seq: int, depth: int = 2):
        self.pool = pool
        self.handle = B.ekv_hoststep_create(pool.handle, max_batch, max_blocks_per_seq, depth)

    def decode(self, layer, h_q, h_block_tables, h_seq_lens, scale, h_out, h_k=None, h_v=None, h_slot_mapping=None,
               stream=None):
        B.ekv_hoststep_decode(self.handle, layer, h_q, h_k, h_v, h_slot_mapping, h_block_tables, h_seq_lens, scale, h_out,
                              stream)

    def flush(self, stream=None):
        B.ekv_hoststep_flush(self.handle, stream)

    def close(self):
        if self.handle:
            B.ekv_hoststep_destroy(self.handle)
            self.handle = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()
