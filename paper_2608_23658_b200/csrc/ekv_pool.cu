// Elastic KV pool: one virtual range per layer, a base handle that is always mapped and an
// elastic handle that is mapped / unmapped at the top of the range (the paper's "Two handles,
// one virtual range").  Host code only, plus a one-thread kernel that publishes the live limit.
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <chrono>
#include <mutex>
#include <new>
#include <numeric>

#include "ekv_internal.h"

namespace ekv {

static thread_local char g_err[512] = "";

void set_error(const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
}

ekv_status_t cuda_fail(cudaError_t e, const char *what) {
    set_error("%s: %s", what, cudaGetErrorString(e));
    return e == cudaErrorMemoryAllocation ? EKV_ERR_OOM : EKV_ERR_CUDA;
}

// ------------------------------------------------------------------ CUDA driver VMM backend

typedef CUresult (*pfn_granularity)(size_t *, const CUmemAllocationProp *, CUmemAllocationGranularity_flags);
typedef CUresult (*pfn_reserve)(CUdeviceptr *, size_t, size_t, CUdeviceptr, unsigned long long);
typedef CUresult (*pfn_addr_free)(CUdeviceptr, size_t);
typedef CUresult (*pfn_create)(CUmemGenericAllocationHandle *, size_t, const CUmemAllocationProp *, unsigned long long);
typedef CUresult (*pfn_release)(CUmemGenericAllocationHandle);
typedef CUresult (*pfn_map)(CUdeviceptr, size_t, size_t, CUmemGenericAllocationHandle, unsigned long long);
typedef CUresult (*pfn_unmap)(CUdeviceptr, size_t);
typedef CUresult (*pfn_set_access)(CUdeviceptr, size_t, const CUmemAccessDesc *, size_t);
typedef CUresult (*pfn_encode_tiled)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                     const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                     CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                     CUtensorMapFloatOOBfill);

struct Driver {
    bool tried = false, ok = false;
    pfn_granularity granularity;
    pfn_reserve reserve;
    pfn_addr_free addr_free;
    pfn_create create;
    pfn_release release;
    pfn_map map;
    pfn_unmap unmap;
    pfn_set_access set_access;
    pfn_encode_tiled encode_tiled;
};
static Driver g_drv;
static std::mutex g_mu;

static bool load_one(const char *name, void **fn) {
    cudaDriverEntryPointQueryResult q;
    cudaError_t e = cudaGetDriverEntryPoint(name, fn, cudaEnableDefault, &q);
    if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || *fn == nullptr) {
        set_error("CUDA driver entry point %s unavailable (%s)", name, cudaGetErrorString(e));
        (void)cudaGetLastError();
        return false;
    }
    return true;
}

static bool load_driver() {
    std::lock_guard<std::mutex> lk(g_mu);
    if (g_drv.tried) return g_drv.ok;
    g_drv.tried = true;
    g_drv.ok = load_one("cuMemGetAllocationGranularity", (void **)&g_drv.granularity) &&
               load_one("cuMemAddressReserve", (void **)&g_drv.reserve) &&
               load_one("cuMemAddressFree", (void **)&g_drv.addr_free) &&
               load_one("cuMemCreate", (void **)&g_drv.create) &&
               load_one("cuMemRelease", (void **)&g_drv.release) &&
               load_one("cuMemMap", (void **)&g_drv.map) &&
               load_one("cuMemUnmap", (void **)&g_drv.unmap) &&
               load_one("cuMemSetAccess", (void **)&g_drv.set_access) &&
               load_one("cuTensorMapEncodeTiled", (void **)&g_drv.encode_tiled);
    return g_drv.ok;
}

static int cu_code(CUresult r) { return r == CUDA_SUCCESS ? 0 : (r == CUDA_ERROR_OUT_OF_MEMORY ? 2 : 1000 + (int)r); }

static CUmemAllocationProp device_prop(int device) {
    CUmemAllocationProp p;
    memset(&p, 0, sizeof p);
    p.type = CU_MEM_ALLOCATION_TYPE_PINNED;
    p.location.type = CU_MEM_LOCATION_TYPE_DEVICE;
    p.location.id = device;
    return p;
}

static int drv_granularity(void *, int device, uint64_t *bytes) {
    CUmemAllocationProp p = device_prop(device);
    size_t g = 0;
    CUresult r = g_drv.granularity(&g, &p, CU_MEM_ALLOC_GRANULARITY_MINIMUM);
    *bytes = g;
    return cu_code(r);
}
static int drv_reserve(void *, uint64_t size, uint64_t alignment, uint64_t *va) {
    CUdeviceptr p = 0;
    CUresult r = g_drv.reserve(&p, size, alignment, 0, 0);
    *va = (uint64_t)p;
    return cu_code(r);
}
static int drv_unreserve(void *, uint64_t va, uint64_t size) { return cu_code(g_drv.addr_free((CUdeviceptr)va, size)); }
static int drv_create(void *, uint64_t size, int device, uint64_t *handle) {
    CUmemAllocationProp p = device_prop(device);
    CUmemGenericAllocationHandle h = 0;
    CUresult r = g_drv.create(&h, size, &p, 0);
    *handle = (uint64_t)h;
    return cu_code(r);
}
static int drv_release(void *, uint64_t handle) { return cu_code(g_drv.release((CUmemGenericAllocationHandle)handle)); }
static int drv_map(void *, uint64_t va, uint64_t size, uint64_t handle) {
    return cu_code(g_drv.map((CUdeviceptr)va, size, 0, (CUmemGenericAllocationHandle)handle, 0));
}
static int drv_unmap(void *, uint64_t va, uint64_t size) { return cu_code(g_drv.unmap((CUdeviceptr)va, size)); }
static int drv_set_access(void *, uint64_t va, uint64_t size, int device) {
    CUmemAccessDesc d;
    memset(&d, 0, sizeof d);
    d.location.type = CU_MEM_LOCATION_TYPE_DEVICE;
    d.location.id = device;
    d.flags = CU_MEM_ACCESS_FLAGS_PROT_READWRITE;
    return cu_code(g_drv.set_access((CUdeviceptr)va, size, &d, 1));
}

static const ekv_vmm_backend_t k_driver_backend = {nullptr,    drv_granularity, drv_reserve, drv_unreserve, drv_create,
                                                   drv_release, drv_map,         drv_unmap,   drv_set_access};
static ekv_vmm_backend_t g_backend = k_driver_backend;
static bool g_backend_replaced = false;
static int g_live_pools = 0;

static ekv_status_t be_status(int rc, const char *what, int layer) {
    if (rc == 0) return EKV_OK;
    set_error("%s failed at layer %d (backend code %d)", what, layer, rc);
    return rc == 2 ? EKV_ERR_OOM : EKV_ERR_CUDA;
}

// ------------------------------------------------------------------ live-limit publication

__global__ void set_live_kernel(long long *live, long long value) { *live = value; }

ekv_status_t launch_set_live(ekv_pool *pool, long long value, cudaStream_t stream) {
    if (!pool->host_only) {
        set_live_kernel<<<1, 1, 0, stream>>>(pool->d_live, value);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return cuda_fail(e, "publish live limit");
    }
    pool->live_limit = value;
    return EKV_OK;
}

ekv_status_t check_compute(ekv_pool *pool, int32_t layer, const char *who) {
    if (!pool) {
        set_error("%s: pool is NULL", who);
        return EKV_ERR_INVALID;
    }
    if (pool->host_only) {
        set_error("%s: pool was created through a replacement VMM backend and holds no device state", who);
        return EKV_ERR_STATE;
    }
    if (layer < 0 || layer >= pool->desc.num_layers) {
        set_error("%s: layer %d outside [0, %d)", who, layer, pool->desc.num_layers);
        return EKV_ERR_INVALID;
    }
    cudaError_t e = cudaSetDevice(pool->desc.device);
    if (e != cudaSuccess) return cuda_fail(e, who);
    return EKV_OK;
}

ekv_status_t encode_kv_map(void *base, uint64_t blocks, uint64_t block_stride, int num_kv_heads, int head_dim, int block_size,
                           CUtensorMap *out) {
    if (!load_driver()) return EKV_ERR_CUDA;
    cuuint64_t gdim[3] = {(cuuint64_t)head_dim, (cuuint64_t)2 * num_kv_heads * block_size, (cuuint64_t)blocks};
    cuuint64_t gstride[2] = {(cuuint64_t)head_dim * 2, (cuuint64_t)block_stride};
    cuuint32_t box[3] = {64, (cuuint32_t)block_size, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_drv.encode_tiled(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, gdim, gstride, box, estr,
                                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error("cuTensorMapEncodeTiled failed (CUresult %d) for a KV tensor at %p with %llu blocks, block stride %llu", (int)r, base,
                  (unsigned long long)blocks, (unsigned long long)block_stride);
        return EKV_ERR_CUDA;
    }
    return EKV_OK;
}

ekv_status_t encode_q_map(const void *q, uint64_t tokens, int num_q_heads, int head_dim, int box_rows, CUtensorMap *out) {
    if (!load_driver()) return EKV_ERR_CUDA;
    cuuint64_t gdim[3] = {(cuuint64_t)head_dim, (cuuint64_t)num_q_heads, (cuuint64_t)tokens};
    cuuint64_t gstride[2] = {(cuuint64_t)head_dim * 2, (cuuint64_t)num_q_heads * head_dim * 2};
    cuuint32_t box[3] = {64, 1, (cuuint32_t)box_rows};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_drv.encode_tiled(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(q), gdim, gstride, box, estr,
                                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error("cuTensorMapEncodeTiled failed (CUresult %d) for a query tensor at %p with %llu tokens", (int)r, q,
                  (unsigned long long)tokens);
        return EKV_ERR_CUDA;
    }
    return EKV_OK;
}

static uint64_t round_up(uint64_t x, uint64_t m) { return (x + m - 1) / m * m; }

static double now_ms() {
    using namespace std::chrono;
    return duration<double, std::milli>(steady_clock::now().time_since_epoch()).count();
}

// Undo helper: unmap / release / unreserve whatever a partially built pool holds.
static void teardown(ekv_pool *p) {
    const uint64_t layer_bytes = p->base_bytes + p->elastic_bytes;  // bytes of one range
    for (size_t l = 0; l < p->va.size(); ++l) {
        if (p->elastic_mapped[l]) p->be.unmap(p->be.user, p->va[l] + p->base_bytes, p->elastic_bytes);
        if (p->elastic_held[l]) p->be.release(p->be.user, p->elastic_handle[l]);
        if (p->base_handle[l] != ~0ull) {
            p->be.unmap(p->be.user, p->va[l], p->base_bytes);
            p->be.release(p->be.user, p->base_handle[l]);
        }
        p->be.unreserve(p->be.user, p->va[l], layer_bytes);
    }
    if (p->d_live) cudaFree(p->d_live);
    if (p->d_layer_base) cudaFree(p->d_layer_base);
    if (p->h_status) cudaFreeHost(p->h_status);
}

// Undo of a grow that failed part of the way: unmap what it mapped, release what it created.  The error
// text of the failure is kept.
static void unmap_elastic_after_failure(ekv_pool *p, const std::vector<char> &mapped, const std::vector<char> &created) {
    char keep[sizeof g_err];
    memcpy(keep, g_err, sizeof keep);
    for (int l = 0; l < p->num_ranges; ++l) {
        if (mapped[l]) {
            p->be.unmap(p->be.user, p->va[l] + p->base_bytes, p->elastic_bytes);
            p->elastic_mapped[l] = 0;
        }
        if (created[l]) {
            p->be.release(p->be.user, p->elastic_handle[l]);
            p->elastic_held[l] = 0;
        }
    }
    memcpy(g_err, keep, sizeof keep);
}

// Map (creating where not held) the elastic handle of every layer.  On failure everything this
// call mapped or created is undone.  `created_out` (may be NULL) receives which handles this call created.
static ekv_status_t map_elastic(ekv_pool *p, std::vector<char> *created_out = nullptr) {
    const int L = p->num_ranges;
    std::vector<char> created(L, 0), mapped(L, 0);
    ekv_status_t st = EKV_OK;
    for (int l = 0; l < L && st == EKV_OK; ++l) {
        const uint64_t va = p->va[l] + p->base_bytes;
        if (!p->elastic_held[l]) {
            uint64_t h = 0;
            st = be_status(p->be.create(p->be.user, p->elastic_bytes, p->desc.device, &h), "create elastic handle", l);
            if (st != EKV_OK) break;
            p->elastic_handle[l] = h;
            p->elastic_held[l] = 1;
            created[l] = 1;
        }
        st = be_status(p->be.map(p->be.user, va, p->elastic_bytes, p->elastic_handle[l]), "map elastic handle", l);
        if (st != EKV_OK) break;
        mapped[l] = 1;
        p->elastic_mapped[l] = 1;
        st = be_status(p->be.set_access(p->be.user, va, p->elastic_bytes, p->desc.device), "grant elastic access", l);
    }
    if (st != EKV_OK) unmap_elastic_after_failure(p, mapped, created);
    else if (created_out) *created_out = created;
    return st;
}

}  // namespace ekv

using namespace ekv;

extern "C" {

const char *ekv_last_error(void) { return g_err; }

const char *ekv_status_string(ekv_status_t s) {
    switch (s) {
        case EKV_OK: return "EKV_OK";
        case EKV_ERR_INVALID: return "EKV_ERR_INVALID";
        case EKV_ERR_CUDA: return "EKV_ERR_CUDA";
        case EKV_ERR_OOM: return "EKV_ERR_OOM";
        case EKV_ERR_STATE: return "EKV_ERR_STATE";
        case EKV_ERR_BLOCK_OOB: return "EKV_ERR_BLOCK_OOB";
        case EKV_ERR_TIMEOUT: return "EKV_ERR_TIMEOUT";
        case EKV_ERR_WORKSPACE: return "EKV_ERR_WORKSPACE";
    }
    return "EKV_ERR_UNKNOWN";
}

ekv_status_t ekv_set_vmm_backend(const ekv_vmm_backend_t *backend) {
    std::lock_guard<std::mutex> lk(g_mu);
    if (g_live_pools != 0) {
        set_error("ekv_set_vmm_backend: %d pool(s) still exist", g_live_pools);
        return EKV_ERR_STATE;
    }
    if (backend == nullptr) {
        g_backend = k_driver_backend;
        g_backend_replaced = false;
        return EKV_OK;
    }
    if (!backend->granularity || !backend->reserve || !backend->unreserve || !backend->create || !backend->release ||
        !backend->map || !backend->unmap || !backend->set_access) {
        set_error("ekv_set_vmm_backend: every function of the table must be set");
        return EKV_ERR_INVALID;
    }
    g_backend = *backend;
    g_backend_replaced = true;
    return EKV_OK;
}

ekv_status_t ekv_pool_create(const ekv_pool_desc_t *desc, ekv_pool_t **out) {
    if (!desc || !out) {
        set_error("ekv_pool_create: NULL argument");
        return EKV_ERR_INVALID;
    }
    *out = nullptr;
    const ekv_pool_desc_t d = *desc;
    if (d.num_layers < 1 || d.num_kv_heads < 1 || d.num_q_heads < d.num_kv_heads || d.num_q_heads % d.num_kv_heads != 0 ||
        d.num_q_heads / d.num_kv_heads > 8 || (d.head_dim != 64 && d.head_dim != 128) || d.block_size != 16 ||
        d.dtype != EKV_BF16 || d.base_blocks < 1 || d.elastic_blocks < 0 || d.device < 0 ||
        (d.flags & ~(uint32_t)(EKV_START_GROWN | EKV_FUSED_RANGE | EKV_PREFILL_WARP_MMA | EKV_PREFILL_ONE_HEAD | EKV_PREFILL_TWO_HEAD)) != 0) {
        set_error("ekv_pool_create: unsupported geometry (layers %d, heads %d/%d, head_dim %d, block_size %d, dtype %d, "
                  "blocks %lld+%lld, flags 0x%x)",
                  d.num_layers, d.num_q_heads, d.num_kv_heads, d.head_dim, d.block_size, d.dtype, (long long)d.base_blocks,
                  (long long)d.elastic_blocks, d.flags);
        return EKV_ERR_INVALID;
    }

    bool replaced;
    ekv_vmm_backend_t be;
    {
        std::lock_guard<std::mutex> lk(g_mu);
        replaced = g_backend_replaced;
        be = g_backend;
    }
    cudaDeviceProp prop;
    memset(&prop, 0, sizeof prop);
    if (!replaced) {
        cudaError_t e = cudaSetDevice(d.device);
        if (e == cudaSuccess) e = cudaFree(0);
        if (e != cudaSuccess) return cuda_fail(e, "ekv_pool_create: select device");
        if (!load_driver()) return EKV_ERR_CUDA;
        e = cudaGetDeviceProperties(&prop, d.device);
        if (e != cudaSuccess) return cuda_fail(e, "ekv_pool_create: device properties");
    }

    ekv_pool *p = new (std::nothrow) ekv_pool();
    if (!p) {
        set_error("ekv_pool_create: host allocation failed");
        return EKV_ERR_OOM;
    }
    p->desc = d;
    p->be = be;
    p->host_only = replaced;
    p->grown = false;
    p->live_limit = 0;
    p->launch_seq = 0;
    p->d_live = nullptr;
    p->h_status = nullptr;
    p->d_status = nullptr;
    p->d_layer_base = nullptr;
    p->sm_count = replaced ? 148 : prop.multiProcessorCount;
    p->block_bytes = 2ull * d.num_kv_heads * d.block_size * d.head_dim * 2ull;

    uint64_t gran = 0;
    int rc = be.granularity(be.user, d.device, &gran);
    if (rc != 0 || gran == 0) {
        set_error("ekv_pool_create: granularity query failed (backend code %d)", rc);
        delete p;
        return EKV_ERR_CUDA;
    }
    if (gran % p->block_bytes != 0) {
        set_error("ekv_pool_create: granularity %llu is not a multiple of block_bytes %llu", (unsigned long long)gran,
                  (unsigned long long)p->block_bytes);
        delete p;
        return EKV_ERR_INVALID;
    }
    p->granularity = gran;
    p->fused = (d.flags & EKV_FUSED_RANGE) != 0;
    p->num_ranges = p->fused ? 1 : d.num_layers;
    const uint64_t per_block = p->fused ? (uint64_t)d.num_layers * p->block_bytes : p->block_bytes;  // range bytes per block id
    p->block_stride = per_block;
    // round the block counts UP until a range's base part and elastic part are whole granules
    uint64_t step = gran / std::gcd((uint64_t)gran, per_block);  // block counts must be multiples of this
    p->base_blocks = (int64_t)round_up((uint64_t)d.base_blocks, step);
    p->elastic_blocks = (int64_t)round_up((uint64_t)d.elastic_blocks, step);
    p->base_bytes = (uint64_t)p->base_blocks * per_block;
    p->elastic_bytes = (uint64_t)p->elastic_blocks * per_block;
    const uint64_t layer_bytes = p->base_bytes + p->elastic_bytes;  // bytes of one range
    if ((uint64_t)(p->base_blocks + p->elastic_blocks) >= (1ull << 31)) {
        set_error("ekv_pool_create: %lld block ids per layer exceed the 2^31 addressing limit",
                  (long long)(p->base_blocks + p->elastic_blocks));
        delete p;
        return EKV_ERR_INVALID;
    }

    ekv_status_t st = EKV_OK;
    for (int l = 0; l < p->num_ranges && st == EKV_OK; ++l) {
        uint64_t va = 0;
        st = be_status(be.reserve(be.user, layer_bytes, gran, &va), "reserve virtual range", l);
        if (st != EKV_OK) break;
        p->va.push_back(va);
        p->base_handle.push_back(~0ull);
        p->elastic_handle.push_back(0);
        p->elastic_held.push_back(0);
        p->elastic_mapped.push_back(0);
        uint64_t h = 0;
        st = be_status(be.create(be.user, p->base_bytes, d.device, &h), "create base handle", l);
        if (st != EKV_OK) break;
        st = be_status(be.map(be.user, va, p->base_bytes, h), "map base handle", l);
        if (st != EKV_OK) {
            be.release(be.user, h);
            break;
        }
        p->base_handle[l] = h;
        st = be_status(be.set_access(be.user, va, p->base_bytes, d.device), "grant base access", l);
    }
    if (st == EKV_OK && (d.flags & EKV_START_GROWN) && p->elastic_bytes > 0) {
        st = map_elastic(p);
        if (st == EKV_OK) p->grown = true;
    }

    p->live_limit = p->base_blocks + (p->grown ? p->elastic_blocks : 0);
    if (st == EKV_OK && !p->host_only) {
        cudaError_t e = cudaMalloc((void **)&p->d_live, (1 + EKV_LAUNCH_SLOTS) * sizeof(long long));  // [0] live limit, then launch words
        if (e == cudaSuccess) e = cudaMemset(p->d_live, 0, (1 + EKV_LAUNCH_SLOTS) * sizeof(long long));
        if (e == cudaSuccess) e = cudaHostAlloc((void **)&p->h_status, sizeof(unsigned), cudaHostAllocMapped);
        if (e == cudaSuccess) {
            *p->h_status = 0;
            e = cudaHostGetDevicePointer((void **)&p->d_status, p->h_status, 0);
        }
        if (e == cudaSuccess) {
            long long live = p->base_blocks + (p->grown ? p->elastic_blocks : 0);
            e = cudaMemcpy(p->d_live, &live, sizeof live, cudaMemcpyHostToDevice);
        }
        if (e == cudaSuccess) e = cudaMalloc((void **)&p->d_layer_base, sizeof(unsigned long long) * d.num_layers);
        if (e == cudaSuccess) {
            std::vector<unsigned long long> bases(d.num_layers);
            for (int l = 0; l < d.num_layers; ++l) bases[l] = p->layer_base(l);
            e = cudaMemcpy(p->d_layer_base, bases.data(), sizeof(unsigned long long) * d.num_layers, cudaMemcpyHostToDevice);
        }
        if (e != cudaSuccess) st = cuda_fail(e, "ekv_pool_create: device state");
        // One tensor map per layer over ALL its block ids (base + elastic).  Encoding reads no memory,
        // and the map never changes when the elastic slice is mapped or unmapped.
        for (int l = 0; l < d.num_layers && st == EKV_OK; ++l) {
            CUtensorMap m;
            st = encode_kv_map((void *)p->layer_base(l), (uint64_t)(p->base_blocks + p->elastic_blocks), p->block_stride,
                               d.num_kv_heads, d.head_dim, d.block_size, &m);
            if (st != EKV_OK) break;
            p->kv_map.push_back(m);
        }
    }

    if (st != EKV_OK) {
        char keep[sizeof g_err];
        memcpy(keep, g_err, sizeof keep);
        teardown(p);
        delete p;
        memcpy(g_err, keep, sizeof keep);
        return st;
    }
    {
        std::lock_guard<std::mutex> lk(g_mu);
        ++g_live_pools;
    }
    *out = p;
    return EKV_OK;
}

ekv_status_t ekv_pool_destroy(ekv_pool_t *pool) {
    if (!pool) return EKV_OK;
    if (!pool->host_only) {
        cudaSetDevice(pool->desc.device);
        cudaDeviceSynchronize();
    }
    teardown(pool);
    delete pool;
    std::lock_guard<std::mutex> lk(g_mu);
    --g_live_pools;
    return EKV_OK;
}

ekv_status_t ekv_pool_info(const ekv_pool_t *pool, ekv_pool_info_t *info) {
    if (!pool || !info) {
        set_error("ekv_pool_info: NULL argument");
        return EKV_ERR_INVALID;
    }
    memset(info, 0, sizeof *info);
    info->granularity = pool->granularity;
    info->block_bytes = pool->block_bytes;
    info->base_bytes = (uint64_t)pool->base_blocks * pool->block_bytes;        // per layer
    info->elastic_bytes = (uint64_t)pool->elastic_blocks * pool->block_bytes;  // per layer
    info->block_stride_bytes = pool->block_stride;
    info->num_ranges = pool->num_ranges;
    info->base_blocks = pool->base_blocks;
    info->elastic_blocks = pool->elastic_blocks;
    info->live_blocks = pool->live_limit;
    info->grown = pool->grown ? 1 : 0;
    int held = 0;
    for (char c : pool->elastic_held) held |= c;
    info->physical_held = held;
    info->num_layers = pool->desc.num_layers;
    return EKV_OK;
}

ekv_status_t ekv_layer_ptr(const ekv_pool_t *pool, int32_t layer, void **dptr) {
    if (!pool || !dptr || layer < 0 || layer >= pool->desc.num_layers) {
        set_error("ekv_layer_ptr: bad argument");
        return EKV_ERR_INVALID;
    }
    *dptr = (void *)pool->layer_base(layer);
    return EKV_OK;
}

ekv_status_t ekv_grow(ekv_pool_t *pool, void *stream, uint32_t flags, double *ms_out) {
    if (!pool || flags != 0) {
        set_error("ekv_grow: bad argument");
        return EKV_ERR_INVALID;
    }
    if (pool->grown || pool->elastic_bytes == 0) {
        set_error("ekv_grow: %s", pool->grown ? "already grown" : "pool has no elastic range");
        return EKV_ERR_STATE;
    }
    const double t0 = now_ms();
    if (!pool->host_only) {
        cudaError_t e = cudaSetDevice(pool->desc.device);
        if (e != cudaSuccess) return cuda_fail(e, "ekv_grow");
    }
    const double t1 = now_ms();
    std::vector<char> created;
    ekv_status_t st = map_elastic(pool, &created);
    const double t2 = now_ms();
    if (st != EKV_OK) return st;
    st = launch_set_live(pool, pool->base_blocks + pool->elastic_blocks, (cudaStream_t)stream);
    if (st == EKV_OK && !pool->host_only) {
        cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
        if (e != cudaSuccess) st = cuda_fail(e, "ekv_grow: stream sync");
    }
    if (st != EKV_OK) {
        // The range is mapped but the kernels were not told: back to the shrunk state.  The limit is put back
        // first (best effort: whatever broke the stream may refuse this too; the host copy is what ekv_pool_info reports).
        char keep[sizeof g_err];
        memcpy(keep, g_err, sizeof keep);
        (void)launch_set_live(pool, pool->base_blocks, (cudaStream_t)stream);
        if (!pool->host_only) (void)cudaDeviceSynchronize();
        pool->live_limit = pool->base_blocks;
        memcpy(g_err, keep, sizeof keep);
        unmap_elastic_after_failure(pool, std::vector<char>(pool->num_ranges, 1), created);
        return st;
    }
    pool->grown = true;
    if (ms_out) {
        ms_out[0] = t2 - t1;
        ms_out[1] = now_ms() - t0;
    }
    return st;
}

ekv_status_t ekv_shrink(ekv_pool_t *pool, void *stream, uint32_t flags, double *ms_out) {
    if (!pool || (flags & ~(uint32_t)EKV_KEEP_PHYSICAL) != 0) {
        set_error("ekv_shrink: bad argument");
        return EKV_ERR_INVALID;
    }
    if (!pool->grown) {
        set_error("ekv_shrink: not grown");
        return EKV_ERR_STATE;
    }
    const double t0 = now_ms();
    if (!pool->host_only) {
        // Order: lower the limit on the caller's stream, then wait for EVERY stream of the device,
        // so no kernel that may still read an elastic block is in flight when the range goes away.
        cudaError_t e = cudaSetDevice(pool->desc.device);
        if (e != cudaSuccess) return cuda_fail(e, "ekv_shrink");
        ekv_status_t st = launch_set_live(pool, pool->base_blocks, (cudaStream_t)stream);
        if (st != EKV_OK) return st;
        e = cudaDeviceSynchronize();
        if (e != cudaSuccess) return cuda_fail(e, "ekv_shrink: device sync");
    }
    else pool->live_limit = pool->base_blocks;
    const double t1 = now_ms();
    ekv_status_t st = EKV_OK;
    for (int l = 0; l < pool->num_ranges; ++l) {
        if (pool->elastic_mapped[l]) {  // a range can be unmapped already: this call may be the retry of one that failed half way
            st = be_status(pool->be.unmap(pool->be.user, pool->va[l] + pool->base_bytes, pool->elastic_bytes), "unmap elastic range", l);
            if (st != EKV_OK) return st;  // this range and the later ones stay mapped; the pool stays "grown" with the limit at base
            pool->elastic_mapped[l] = 0;
        }
        if (!(flags & EKV_KEEP_PHYSICAL) && pool->elastic_held[l]) {
            // The handle is dropped from the books whatever the driver answers: it is unmapped, and a second
            // release of a handle the driver may already have let go would be worse than a leak.
            ekv_status_t s2 = be_status(pool->be.release(pool->be.user, pool->elastic_handle[l]), "release elastic handle", l);
            if (s2 != EKV_OK && st == EKV_OK) st = s2;
            pool->elastic_held[l] = 0;
        }
    }
    const double t2 = now_ms();
    pool->grown = false;
    if (ms_out) {
        ms_out[0] = t2 - t1;
        ms_out[1] = t2 - t0;
    }
    return st;
}

ekv_status_t ekv_poll_status(ekv_pool_t *pool) {
    if (!pool) {
        set_error("ekv_poll_status: pool is NULL");
        return EKV_ERR_INVALID;
    }
    if (pool->host_only) return EKV_OK;
    unsigned v = __atomic_exchange_n(pool->h_status, 0u, __ATOMIC_ACQ_REL);
    if (v & EKV_DEV_FLAG_TIMEOUT) {
        set_error("ekv_poll_status: a kernel gave up a bounded wait since the last poll%s",
                  (v & EKV_DEV_FLAG_OOB) ? " (and skipped a block id outside the live range)" : "");
        return EKV_ERR_TIMEOUT;
    }
    if (v & EKV_DEV_FLAG_OOB) {
        set_error("ekv_poll_status: a kernel skipped a block id (or slot) outside the live range since the last poll");
        return EKV_ERR_BLOCK_OOB;
    }
    return EKV_OK;
}

}  // extern "C"
