// Host-side block pool with a gated elastic id range, the one-step-ahead controller, and the device
// kernel that moves blocks out of the elastic range before a decommit ("drain").
//
// Follows the paper's section "An Elastic KV Mechanism".  The pool is a free list of integer ids
// and nothing else.  Ids above base_blocks belong to the elastic slice and leave the list only while
// that slice is committed (paragraph "Two handles, one virtual range").  The controller lends the
// slice out while steps only decode and reclaims it just before a step that prefills, waiting a few
// quiet steps before lending again; reclaiming means: move live data off the elastic ids, wait for
// the device, unmap (paragraph "Controller").
#include <string.h>

#include <new>
#include <vector>

#include "ekv_internal.h"

struct ekv_blockpool {
    int64_t base, elastic;
    bool admitted;                     // elastic ids may be handed out
    std::vector<int32_t> free_base;    // stack: back() is handed out next
    std::vector<int32_t> free_elastic;
    std::vector<uint8_t> in_use;       // per id: 0 free, 1 allocated, 3 allocated and part of the outstanding drain plan
    int64_t elastic_in_use;
    // drain in progress: pairs handed out by ekv_blockpool_drain_plan, settled by ekv_blockpool_drain_commit
    std::vector<int32_t> drain_from, drain_to;
};

struct ekv_controller {
    ekv_controller_desc_t desc;
    bool committed;
    int32_t decode_streak;
    int64_t commits, decommits, steps;
};

using namespace ekv;

extern "C" {

ekv_status_t ekv_blockpool_create(int64_t base_blocks, int64_t elastic_blocks, ekv_blockpool_t **out) {
    if (!out || base_blocks < 1 || elastic_blocks < 0 || base_blocks + elastic_blocks > 0x7fffffffLL) {
        set_error("ekv_blockpool_create: bad argument (base %lld, elastic %lld)", (long long)base_blocks, (long long)elastic_blocks);
        return EKV_ERR_INVALID;
    }
    ekv_blockpool *bp = new (std::nothrow) ekv_blockpool();
    if (!bp) {
        set_error("ekv_blockpool_create: host allocation failed");
        return EKV_ERR_OOM;
    }
    bp->base = base_blocks;
    bp->elastic = elastic_blocks;
    bp->admitted = false;
    bp->elastic_in_use = 0;
    bp->in_use.assign((size_t)(base_blocks + elastic_blocks), 0);
    bp->free_base.reserve((size_t)base_blocks);
    for (int64_t i = base_blocks - 1; i >= 0; --i) bp->free_base.push_back((int32_t)i);  // lowest id first
    bp->free_elastic.reserve((size_t)elastic_blocks);
    for (int64_t i = base_blocks + elastic_blocks - 1; i >= base_blocks; --i) bp->free_elastic.push_back((int32_t)i);
    *out = bp;
    return EKV_OK;
}

ekv_status_t ekv_blockpool_destroy(ekv_blockpool_t *bp) {
    delete bp;
    return EKV_OK;
}

ekv_status_t ekv_blockpool_alloc(ekv_blockpool_t *bp, int64_t n, int32_t *ids_out) {
    if (!bp || n < 0 || (n > 0 && !ids_out)) {
        set_error("ekv_blockpool_alloc: bad argument");
        return EKV_ERR_INVALID;
    }
    const int64_t avail = (int64_t)bp->free_base.size() + (bp->admitted ? (int64_t)bp->free_elastic.size() : 0);
    if (n > avail) {
        set_error("ekv_blockpool_alloc: %lld blocks requested, %lld available (%s)", (long long)n, (long long)avail,
                  bp->admitted ? "elastic range admitted" : "elastic range gated");
        return EKV_ERR_OOM;  // all-or-nothing: nothing was handed out
    }
    for (int64_t i = 0; i < n; ++i) {
        int32_t id;
        if (!bp->free_base.empty()) {  // base ids first: elastic blocks are the ones that must be drained later
            id = bp->free_base.back();
            bp->free_base.pop_back();
        } else {
            id = bp->free_elastic.back();
            bp->free_elastic.pop_back();
            ++bp->elastic_in_use;
        }
        bp->in_use[(size_t)id] = 1;
        ids_out[i] = id;
    }
    return EKV_OK;
}

ekv_status_t ekv_blockpool_free(ekv_blockpool_t *bp, const int32_t *ids, int64_t n) {
    if (!bp || n < 0 || (n > 0 && !ids)) {
        set_error("ekv_blockpool_free: bad argument");
        return EKV_ERR_INVALID;
    }
    for (int64_t i = 0; i < n; ++i) {  // validate everything first: a bad id changes nothing
        const int64_t id = ids[i];
        if (id < 0 || id >= bp->base + bp->elastic || bp->in_use[(size_t)id] != 1) {
            for (int64_t k = 0; k < i; ++k) bp->in_use[(size_t)ids[k]] = 1;  // undo the duplicate marks
            if (id >= 0 && id < bp->base + bp->elastic && bp->in_use[(size_t)id] == 3) {
                set_error("ekv_blockpool_free: id %lld belongs to the outstanding drain plan; commit the drain first", (long long)id);
                return EKV_ERR_STATE;
            }
            set_error("ekv_blockpool_free: id %lld is not an allocated block (or is listed twice)", (long long)id);
            return EKV_ERR_INVALID;
        }
        bp->in_use[(size_t)id] = 2;  // marks duplicates inside this call
    }
    for (int64_t i = 0; i < n; ++i) {
        const int32_t id = ids[i];
        bp->in_use[(size_t)id] = 0;
        if (id < bp->base) {
            bp->free_base.push_back(id);
        } else {
            bp->free_elastic.push_back(id);
            --bp->elastic_in_use;
        }
    }
    return EKV_OK;
}

ekv_status_t ekv_blockpool_admit_elastic(ekv_blockpool_t *bp) {
    if (!bp) {
        set_error("ekv_blockpool_admit_elastic: NULL pool");
        return EKV_ERR_INVALID;
    }
    if (!bp->drain_from.empty()) {
        set_error("ekv_blockpool_admit_elastic: a drain is in progress");
        return EKV_ERR_STATE;
    }
    bp->admitted = true;
    return EKV_OK;
}

ekv_status_t ekv_blockpool_gate_elastic(ekv_blockpool_t *bp, int64_t *elastic_in_use) {
    if (!bp) {
        set_error("ekv_blockpool_gate_elastic: NULL pool");
        return EKV_ERR_INVALID;
    }
    bp->admitted = false;
    if (elastic_in_use) *elastic_in_use = bp->elastic_in_use;
    return EKV_OK;
}

ekv_status_t ekv_blockpool_drain_plan(ekv_blockpool_t *bp, int32_t *from_ids, int32_t *to_ids, int64_t capacity, int64_t *n_out) {
    if (!bp || !n_out || capacity < 0 || (capacity > 0 && (!from_ids || !to_ids))) {
        set_error("ekv_blockpool_drain_plan: bad argument");
        return EKV_ERR_INVALID;
    }
    if (bp->admitted || !bp->drain_from.empty()) {
        set_error("ekv_blockpool_drain_plan: %s", bp->admitted ? "gate the elastic range first" : "a drain is already in progress");
        return EKV_ERR_STATE;
    }
    const int64_t n = bp->elastic_in_use;
    *n_out = n;
    if (n > capacity) {
        set_error("ekv_blockpool_drain_plan: %lld pairs needed, arrays hold %lld", (long long)n, (long long)capacity);
        return EKV_ERR_INVALID;
    }
    if (n > (int64_t)bp->free_base.size()) {
        set_error("ekv_blockpool_drain_plan: %lld elastic blocks in use but only %zu base blocks free (preempt requests first)",
                  (long long)n, bp->free_base.size());
        return EKV_ERR_OOM;
    }
    int64_t k = 0;
    for (int64_t id = bp->base; id < bp->base + bp->elastic && k < n; ++id) {
        if (bp->in_use[(size_t)id] == 0) continue;
        const int32_t to = bp->free_base.back();
        bp->free_base.pop_back();
        bp->in_use[(size_t)to] = 3;
        bp->in_use[(size_t)id] = 3;
        from_ids[k] = (int32_t)id;
        to_ids[k] = to;
        bp->drain_from.push_back((int32_t)id);
        bp->drain_to.push_back(to);
        ++k;
    }
    return EKV_OK;
}

ekv_status_t ekv_blockpool_drain_commit(ekv_blockpool_t *bp) {
    if (!bp) {
        set_error("ekv_blockpool_drain_commit: NULL pool");
        return EKV_ERR_INVALID;
    }
    for (int32_t id : bp->drain_from) {
        bp->in_use[(size_t)id] = 0;
        bp->free_elastic.push_back(id);
        --bp->elastic_in_use;
    }
    for (int32_t id : bp->drain_to) bp->in_use[(size_t)id] = 1;  // an ordinary allocated block from now on
    bp->drain_from.clear();
    bp->drain_to.clear();
    return EKV_OK;
}

ekv_status_t ekv_blockpool_stats(const ekv_blockpool_t *bp, ekv_blockpool_stats_t *out) {
    if (!bp || !out) {
        set_error("ekv_blockpool_stats: NULL argument");
        return EKV_ERR_INVALID;
    }
    out->base_blocks = bp->base;
    out->elastic_blocks = bp->elastic;
    out->free_base = (int64_t)bp->free_base.size();
    out->free_elastic = (int64_t)bp->free_elastic.size();
    out->elastic_in_use = bp->elastic_in_use;
    out->num_gpu_blocks = bp->base + (bp->admitted ? bp->elastic : 0);
    out->admitted = bp->admitted ? 1 : 0;
    out->draining = bp->drain_from.empty() ? 0 : 1;
    return EKV_OK;
}

// ------------------------------------------------------------------ controller

ekv_status_t ekv_controller_create(const ekv_controller_desc_t *desc, int32_t initially_committed, ekv_controller_t **out) {
    if (!desc || !out || desc->commit_after_decode_steps < 1 || desc->reserve_prefill_tokens < 1) {
        set_error("ekv_controller_create: bad argument");
        return EKV_ERR_INVALID;
    }
    ekv_controller *c = new (std::nothrow) ekv_controller();
    if (!c) {
        set_error("ekv_controller_create: host allocation failed");
        return EKV_ERR_OOM;
    }
    c->desc = *desc;
    c->committed = initially_committed != 0;
    c->decode_streak = 0;
    c->commits = c->decommits = c->steps = 0;
    *out = c;
    return EKV_OK;
}

ekv_status_t ekv_controller_destroy(ekv_controller_t *c) {
    delete c;
    return EKV_OK;
}

ekv_action_t ekv_controller_decide(ekv_controller_t *c, int32_t next_prefill_tokens) {
    if (!c) return EKV_ACT_NONE;
    ++c->steps;
    if (next_prefill_tokens >= c->desc.reserve_prefill_tokens) {
        // the next step needs the activation reserve back: give it back NOW, before the step runs
        c->decode_streak = 0;
        if (c->committed) {
            c->committed = false;
            ++c->decommits;
            return EKV_ACT_DECOMMIT;
        }
        return EKV_ACT_NONE;
    }
    if (c->decode_streak < 0x7fffffff) ++c->decode_streak;
    if (!c->committed && c->decode_streak >= c->desc.commit_after_decode_steps) {
        c->committed = true;
        ++c->commits;
        return EKV_ACT_COMMIT;
    }
    return EKV_ACT_NONE;
}

ekv_status_t ekv_controller_stats(const ekv_controller_t *c, ekv_controller_stats_t *out) {
    if (!c || !out) {
        set_error("ekv_controller_stats: NULL argument");
        return EKV_ERR_INVALID;
    }
    out->steps = c->steps;
    out->commits = c->commits;
    out->decommits = c->decommits;
    out->committed = c->committed ? 1 : 0;
    out->decode_streak = c->decode_streak;
    return EKV_OK;
}

}  // extern "C"

// ------------------------------------------------------------------ drain copy on the device

namespace ekv {

// One CTA per (pair, layer): copies block src -> dst (block_bytes, 16-byte pieces).  HBM-bound copy.
__global__ void __launch_bounds__(256) move_blocks_kernel(const unsigned long long *__restrict__ layer_base, int num_layers,
                                                          const int *__restrict__ src_ids, const int *__restrict__ dst_ids,
                                                          int pieces_per_block, long long block_stride_pieces,
                                                          const long long *__restrict__ live_ptr, unsigned *status) {
    const int pair = blockIdx.x, layer = blockIdx.y;
    const long long live = *live_ptr;
    const long long s = src_ids[pair], d = dst_ids[pair];
    if (s < 0 || d < 0 || s >= live || d >= live) {
        if (threadIdx.x == 0) atomicOr(status, EKV_DEV_FLAG_OOB);
        return;
    }
    const uint4 *src = reinterpret_cast<const uint4 *>(layer_base[layer]) + s * block_stride_pieces;
    uint4 *dst = reinterpret_cast<uint4 *>(layer_base[layer]) + d * block_stride_pieces;
    for (int i = threadIdx.x; i < pieces_per_block; i += blockDim.x) dst[i] = src[i];
}

}  // namespace ekv

extern "C" ekv_status_t ekv_move_blocks(ekv_pool_t *pool, const int32_t *src_ids, const int32_t *dst_ids, int32_t n, void *stream) {
    ekv_status_t st = check_compute(pool, 0, "ekv_move_blocks");
    if (st != EKV_OK) return st;
    if (n < 0 || n > 0x7fffffff / 2 || (n > 0 && (!src_ids || !dst_ids)) || pool->desc.num_layers > 65535) {
        set_error("ekv_move_blocks: bad argument (n=%d)", n);
        return EKV_ERR_INVALID;
    }
    if (n == 0) return EKV_OK;
    dim3 grid((unsigned)n, (unsigned)pool->desc.num_layers);
    move_blocks_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>(pool->d_layer_base, pool->desc.num_layers, src_ids, dst_ids,
                                                               (int)(pool->block_bytes / 16), (long long)(pool->block_stride / 16),
                                                               pool->d_live, pool->d_status);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "ekv_move_blocks launch");
    return EKV_OK;
}
