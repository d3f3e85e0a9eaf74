// Internal declarations shared by the translation units of libekv (not part of the ABI).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/ekv.h"

// Bits latched by kernels into the pool's status word (host-mapped, read by ekv_poll_status).
#define EKV_DEV_FLAG_OOB 1u
#define EKV_DEV_FLAG_TIMEOUT 2u

// Prefill launches of one pool that may be in flight at the same time (each owns one device word while it runs).
#define EKV_LAUNCH_SLOTS 64

struct ekv_pool {
    ekv_pool_desc_t desc;
    ekv_vmm_backend_t be;
    bool host_only;  // created through a replacement VMM backend: no device state, no compute

    // A "range" is one virtual address reservation with one base mapping and one elastic mapping.  Default: one
    // range per layer (the paper's arrangement).  EKV_FUSED_RANGE: a single range for all layers, block n of
    // layer l at (n*num_layers + l)*block_bytes, so a toggle is one map / unmap instead of one per layer.
    int num_ranges;
    bool fused;
    uint64_t granularity, block_bytes, block_stride;  // block_stride: bytes between consecutive block ids of one layer
    uint64_t base_bytes, elastic_bytes;               // per RANGE
    int64_t base_blocks, elastic_blocks;              // per layer
    bool grown;

    std::vector<uint64_t> va;              // per range: start of the reserved range
    std::vector<uint64_t> base_handle;     // per range
    std::vector<uint64_t> elastic_handle;  // per range, valid while elastic_held
    std::vector<char> elastic_held;        // per range: the elastic handle exists
    std::vector<char> elastic_mapped;      // per range: the elastic handle is mapped at the top of the range
    int64_t live_limit;                    // the live limit last published to the device (host-only pools: last decided)

    uint64_t layer_base(int layer) const { return fused ? va[0] + (uint64_t)layer * block_bytes : va[layer]; }

    // device state (absent when host_only)
    long long *d_live;      // device words: [0] number of block ids kernels may dereference; [1 .. kLaunchSlots] one word per
                            // prefill launch in flight: low half = abort flag, high half = next item number
    unsigned launch_seq;    // prefill launches so far (picks the slot)
    unsigned *h_status;     // pinned, host-mapped status word
    unsigned *d_status;     // its device alias
    unsigned long long *d_layer_base;  // device array: start address of every layer's range
    std::vector<CUtensorMap> kv_map;  // per layer: 3-D view (channel, row in block, block id), box 64 x block_size x 1, 128B swizzle
    int sm_count;
};

namespace ekv {

void set_error(const char *fmt, ...);
ekv_status_t cuda_fail(cudaError_t e, const char *what);

// Checks shared by the compute entry points; sets the device current.
ekv_status_t check_compute(ekv_pool *pool, int32_t layer, const char *who);

// Split plan of the decode pass: depends only on the call's shape arguments.
struct DecodePlan {
    int chunk_tokens;  // keys per split (multiple of 64)
    int nsplit;        // splits per (sequence, kv-head) at the maximum length
};
DecodePlan plan_decode(const ekv_pool *pool, int B, int max_blocks_per_seq);

ekv_status_t launch_set_live(ekv_pool *pool, long long value, cudaStream_t stream);

// Tensor map over a KV tensor of `blocks` blocks that are `block_stride` bytes apart, each laid out
// (K|V, kv-head, token, channel): dims (channel, row in block, block), box 64 x block_size x 1, 128-byte swizzle.
ekv_status_t encode_kv_map(void *base, uint64_t blocks, uint64_t block_stride, int num_kv_heads, int head_dim, int block_size,
                           CUtensorMap *out);

// Tensor map over a query tensor [tokens, num_q_heads, head_dim] bf16: dims (channel, head, token), box 64 channels x
// 1 head x box_rows tokens, 128-byte swizzle: one box lands as the K-major [row][128 B] half tile the MMAs read.
// Tokens past the end read as zero.
ekv_status_t encode_q_map(const void *q, uint64_t tokens, int num_q_heads, int head_dim, int box_rows, CUtensorMap *out);

}  // namespace ekv
