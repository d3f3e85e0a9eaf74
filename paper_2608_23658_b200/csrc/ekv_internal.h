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

struct ekv_pool {
    ekv_pool_desc_t desc;
    ekv_vmm_backend_t be;
    bool host_only;  // created through a replacement VMM backend: no device state, no compute

    uint64_t granularity, block_bytes, base_bytes, elastic_bytes;
    int64_t base_blocks, elastic_blocks;
    bool grown;

    std::vector<uint64_t> va;              // per layer: start of the reserved range
    std::vector<uint64_t> base_handle;     // per layer
    std::vector<uint64_t> elastic_handle;  // per layer, valid while elastic_held
    std::vector<char> elastic_held;        // per layer: the elastic handle exists

    // device state (absent when host_only)
    long long *d_live;      // device words: [0] number of block ids kernels may dereference, [1] abort word
    unsigned *h_status;     // pinned, host-mapped status word
    unsigned *d_status;     // its device alias
    unsigned long long *d_layer_base;  // device array: start address of every layer's range
    std::vector<CUtensorMap> kv_map;  // per layer: 2-D view [rows of head_dim bf16], box 64 x block_size, 128B swizzle
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

// Tensor map over a KV tensor laid out like a layer range (box 64 channels x block_size tokens, 128-byte swizzle).
ekv_status_t encode_kv_map(void *base, uint64_t rows, int head_dim, int block_size, CUtensorMap *out);

}  // namespace ekv
