// Chunked-prefill attention, warp-level tensor path (mma.sync m16n8k16).  Used for head_dim 64,
// where the query tile of the tcgen05 kernel does not apply, and as the in-library cross-check of
// the tcgen05 kernel in the GPU tests (pools created with EKV_PREFILL_WARP_MMA).
//
// CTA = 4 warps = 64 query rows of one (request, q-head); KV tiles of 64 tokens (4 blocks) arrive
// through a 2-stage ring of TMA box loads (128-byte swizzle) on mbarriers.  Per warp: S(16x64) =
// Q K^T from register-resident Q fragments and ldmatrix'ed K; online softmax on the C fragments,
// which are re-packed in place as the A fragments of O += P V (V through ldmatrix.trans).
#pragma once
#include <cuda_bf16.h>
#include <math.h>

#include "ekv_internal.h"
#include "ptx.cuh"

namespace ekv {

struct PrefillParams {
    const __nv_bfloat16 *q;
    __nv_bfloat16 *out;
    const int *block_tables;
    const int *cu_q_lens;
    const int *seq_lens;
    const long long *live;
    unsigned *status;
    int *abort_word;  // device word: a CTA of this launch gave up on a wait (tcgen05 kernel)
    int max_blocks, num_q_heads, num_kv_heads, group, R;
    int q_tiles;      // query tiles of the call (of the launching kernel's tile height)
    float scale_log2;
    // tile_prefix[r] = query tiles of requests 0..r-1 (filled by the host when R <= kPrefixMax, else n_prefix = 0):
    // lets a CTA find its request by bisection in the parameter bank instead of walking cu_q_lens
    int n_prefix;
    int tile_prefix[257];
};
static constexpr int kPrefixMax = 256;

// Which request owns query tile `tile_idx` (tiles of `bm` rows, requests in order)?  Returns false if none.
__device__ __forceinline__ bool find_request(const PrefillParams &p, int tile_idx, int bm, int &req, int &first_tile, int &q0,
                                             int &c_r) {
    if (p.n_prefix) {
        if (tile_idx >= p.tile_prefix[p.R]) return false;
        int lo = 0, hi = p.R;  // invariant: tile_prefix[lo] <= tile_idx < tile_prefix[hi]
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (p.tile_prefix[mid] <= tile_idx) lo = mid;
            else hi = mid;
        }
        req = lo;
        first_tile = p.tile_prefix[lo];
        q0 = p.cu_q_lens[req];
        c_r = p.cu_q_lens[req + 1] - q0;
        return true;
    }
    int acc = 0;
    for (req = 0; req < p.R; ++req) {
        q0 = p.cu_q_lens[req];
        c_r = p.cu_q_lens[req + 1] - q0;
        const int nt = (c_r + bm - 1) / bm;
        if (tile_idx < acc + nt) {
            first_tile = acc;
            return true;
        }
        acc += nt;
    }
    return false;
}

static constexpr int kPmBM = 64;      // query rows per CTA
static constexpr int kPmBN = 64;      // keys per tile
static constexpr int kPmStages = 2;
static constexpr int kPmIdCache = 256;  // block ids cached per refill (64 tiles)

template <int D>
__global__ void __launch_bounds__(128, 2) prefill_mma_kernel(const __grid_constant__ CUtensorMap kvmap,
                                                             const PrefillParams p) {
    constexpr int BOXES = D / 64;
    constexpr int TILE_BYTES = BOXES * 2048;         // one 16-token block of K (or V)
    constexpr int KV_BYTES = 4 * TILE_BYTES;         // 64 tokens of K (or V)
    constexpr int STAGE_BYTES = 2 * KV_BYTES;
    constexpr int KSTEPS = D / 16;
    constexpr int NT_O = D / 8;
    constexpr unsigned FULL = 0xffffffffu;

    // ---- which (request, row range) is this CTA?  Heaviest (latest) tiles first.
    const int tile_idx = gridDim.x - 1 - blockIdx.x;
    const int h = blockIdx.y;
    const int g = h / p.group;
    int req = 0, acc = 0, c_r = 0, q0 = 0;
    if (!find_request(p, tile_idx, kPmBM, req, acc, q0, c_r)) return;
    const int row0 = (tile_idx - acc) * kPmBM;
    const int L = min(p.seq_lens[req], p.max_blocks * 16);
    const int prefix = L - c_r;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = lane >> 2, c = lane & 3;
    const int rows_here = min(kPmBM, c_r - row0);
    __nv_bfloat16 *out_base = p.out + ((size_t)(q0 + row0) * p.num_q_heads + h) * D;
    const size_t row_stride = (size_t)p.num_q_heads * D;

    if (prefix < 0) {  // malformed request: zero rows, latch
        if (threadIdx.x == 0) atomicOr(p.status, EKV_DEV_FLAG_OOB);
        for (int e = threadIdx.x; e < rows_here * D; e += 128)
            out_base[(size_t)(e / D) * row_stride + (e % D)] = __float2bfloat16_rn(0.f);
        return;
    }

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_u32 = smem_u32(smem_raw);
    const uint32_t base_u32 = (raw_u32 + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base_u32 - raw_u32);
    const uint32_t bars = base_u32 + kPmStages * STAGE_BYTES;
    int *ids = reinterpret_cast<int *>(base_ptr + kPmStages * STAGE_BYTES + 64);  // [kPmIdCache]

    const int kv_end = min(L, prefix + min(c_r, row0 + kPmBM));  // keys any row of this tile may see
    const int n_tiles = (kv_end + kPmBN - 1) / kPmBN;
    const int n_blocks = (kv_end + 15) >> 4;
    const long long live = *p.live;
    const int *bt = p.block_tables + (size_t)req * p.max_blocks;

    if (threadIdx.x == 0) {
        prefetch_tensormap(&kvmap);
        for (int s = 0; s < kPmStages; ++s) mbar_init(bars + 8 * s, 1);
        mbar_fence_init();
    }
    auto refill_ids = [&](int first_block) {  // all threads; caller syncs
        for (int e = threadIdx.x; e < kPmIdCache; e += 128) {
            const int bi = first_block + e;
            int id = -1;
            if (bi < n_blocks) {
                id = bt[bi];
                if (id < 0 || (long long)id >= live) {
                    id = -1;
                    atomicOr(p.status, EKV_DEV_FLAG_OOB);
                }
            }
            ids[e] = id;
        }
    };
    refill_ids(0);
    __syncthreads();

    auto issue = [&](int t) {  // thread 0 only
        const int stage = t % kPmStages;
        const uint32_t bar = bars + 8 * stage;
        const uint32_t dst = base_u32 + stage * STAGE_BYTES;
        mbar_expect_tx(bar, STAGE_BYTES);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int id = ids[(t * 4 + j) % kPmIdCache];
            if (id < 0) id = 0;  // masked below; block 0 is always mapped
            const int row_k = g * 16;  // row inside the block: (K|V, kv-head, token)
            const int row_v = row_k + p.num_kv_heads * 16;
#pragma unroll
            for (int x = 0; x < BOXES; ++x) {
                tma_load_3d(dst + j * TILE_BYTES + x * 2048, &kvmap, 64 * x, row_k, id, bar);
                tma_load_3d(dst + KV_BYTES + j * TILE_BYTES + x * 2048, &kvmap, 64 * x, row_v, id, bar);
            }
        }
    };
    if (threadIdx.x == 0 && n_tiles > 0) issue(0);

    // ---- Q fragments: rows warp*16 + r and + 8.
    uint32_t qa[KSTEPS][4];
    const int qr0 = row0 + warp * 16 + r, qr1 = qr0 + 8;
    {
        const __nv_bfloat16 *q0p = p.q + ((size_t)(q0 + qr0) * p.num_q_heads + h) * D;
        const __nv_bfloat16 *q1p = p.q + ((size_t)(q0 + qr1) * p.num_q_heads + h) * D;
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
            qa[ks][0] = qr0 < c_r ? *reinterpret_cast<const uint32_t *>(q0p + 16 * ks + 2 * c) : 0u;
            qa[ks][1] = qr1 < c_r ? *reinterpret_cast<const uint32_t *>(q1p + 16 * ks + 2 * c) : 0u;
            qa[ks][2] = qr0 < c_r ? *reinterpret_cast<const uint32_t *>(q0p + 16 * ks + 8 + 2 * c) : 0u;
            qa[ks][3] = qr1 < c_r ? *reinterpret_cast<const uint32_t *>(q1p + 16 * ks + 8 + 2 * c) : 0u;
        }
    }
    // last key each of my two rows may see (rows past the chunk reuse the last real row's limit)
    const int lim0 = prefix + min(qr0, c_r - 1), lim1 = prefix + min(qr1, c_r - 1);

    const int mi = lane >> 3, rr = lane & 7;
    const uint32_t k_row_off = (8 * (mi >> 1) + rr) * 128;  // K: matrices (tok lo, ch), (tok lo, ch+1), (tok hi, ch), ...
    const int k_par = mi & 1;
    const uint32_t v_row_off = (8 * (mi & 1) + rr) * 128;   // V: matrices (tok lo, ch), (tok hi, ch), (tok lo, ch+1), ...
    const int v_par = mi >> 1;

    float o[NT_O][4];
#pragma unroll
    for (int n = 0; n < NT_O; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    int failed_at = -1;

    for (int t = 0; t < n_tiles; ++t) {
        const int stage = t % kPmStages;
        const int tok0 = t * kPmBN;
        int bad_blocks = 0;  // read before the id cache may be refilled below
#pragma unroll
        // invalid ids AND blocks past the last visible key: both were loaded from a stand-in block whose rows may
        // hold anything, so their scores are masked and their V rows zeroed (0 * NaN must not reach O)
        for (int j = 0; j < 4; ++j) bad_blocks |= (ids[(t * 4 + j) % kPmIdCache] < 0) ? (1 << j) : 0;
        // all warps are past tile t-1 here, so its stage may be refilled with tile t+1
        if (t + 1 < n_tiles) {
            if (((t + 1) * 4) % kPmIdCache == 0) {
                __syncthreads();
                refill_ids((t + 1) * 4);
                __syncthreads();
            }
            if (threadIdx.x == 0) issue(t + 1);
        }
        const bool got = mbar_wait(bars + 8 * stage, (uint32_t)((t / kPmStages) & 1));
        if (__syncthreads_or(!got)) {
            failed_at = t;
            break;
        }
        const uint32_t kbase = base_u32 + stage * STAGE_BYTES;
        const uint32_t vbase = kbase + KV_BYTES;

        float s[8][4];
#pragma unroll
        for (int n = 0; n < 8; ++n) s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
#pragma unroll
            for (int ks = 0; ks < KSTEPS; ++ks) {
                const int chunk = 2 * ks + k_par;
                const uint32_t addr = kbase + j * TILE_BYTES + (chunk >> 3) * 2048 + k_row_off + (((chunk & 7) ^ rr) << 4);
                uint32_t k0, k1, k2, k3;
                ldmatrix_x4(addr, k0, k1, k2, k3);
                mma_bf16_16816(s[2 * j], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], k0, k1);
                mma_bf16_16816(s[2 * j + 1], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], k2, k3);
            }
        }
        const bool need_mask = (tok0 + kPmBN - 1 > prefix + row0) || bad_blocks != 0;
        const bool need_vmask = (tok0 + kPmBN > L) || bad_blocks != 0;
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int n = 0; n < 8; ++n) {
#pragma unroll
            for (int e = 0; e < 4; ++e) s[n][e] *= p.scale_log2;
            if (need_mask) {
                const int tk = tok0 + 8 * n + 2 * c;
                const bool bad = (bad_blocks >> (n >> 1)) & 1;
                if (tk > lim0 || bad) s[n][0] = -INFINITY;
                if (tk + 1 > lim0 || bad) s[n][1] = -INFINITY;
                if (tk > lim1 || bad) s[n][2] = -INFINITY;
                if (tk + 1 > lim1 || bad) s[n][3] = -INFINITY;
            }
            mx0 = fmaxf(mx0, fmaxf(s[n][0], s[n][1]));
            mx1 = fmaxf(mx1, fmaxf(s[n][2], s[n][3]));
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(FULL, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(FULL, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(FULL, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(FULL, mx1, 2));
        const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
        const float ms0 = mn0 == -INFINITY ? 0.f : mn0, ms1 = mn1 == -INFINITY ? 0.f : mn1;  // fully masked so far
        const float a0 = fast_exp2(m0 - ms0), a1 = fast_exp2(m1 - ms1);
        m0 = mn0;
        m1 = mn1;
        float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
        for (int n = 0; n < 8; ++n) {
            s[n][0] = fast_exp2(s[n][0] - ms0);
            s[n][1] = fast_exp2(s[n][1] - ms0);
            s[n][2] = fast_exp2(s[n][2] - ms1);
            s[n][3] = fast_exp2(s[n][3] - ms1);
            sum0 += s[n][0] + s[n][1];
            sum1 += s[n][2] + s[n][3];
        }
        l0 = l0 * a0 + sum0;
        l1 = l1 * a1 + sum1;
#pragma unroll
        for (int n = 0; n < NT_O; ++n) {
            o[n][0] *= a0;
            o[n][1] *= a0;
            o[n][2] *= a1;
            o[n][3] *= a1;
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {  // 16 keys per step
            const uint32_t pa0 = pack_bf16x2(s[2 * j][0], s[2 * j][1]);
            const uint32_t pa1 = pack_bf16x2(s[2 * j][2], s[2 * j][3]);
            const uint32_t pa2 = pack_bf16x2(s[2 * j + 1][0], s[2 * j + 1][1]);
            const uint32_t pa3 = pack_bf16x2(s[2 * j + 1][2], s[2 * j + 1][3]);
            uint32_t mlo = 0xffffffffu, mhi = 0xffffffffu;
            if (need_vmask) {
                const int tk = tok0 + 16 * j + 2 * c;
                const bool bad = (bad_blocks >> j) & 1;
                mlo = ((tk < L && !bad) ? 0x0000ffffu : 0u) | ((tk + 1 < L && !bad) ? 0xffff0000u : 0u);
                mhi = ((tk + 8 < L && !bad) ? 0x0000ffffu : 0u) | ((tk + 9 < L && !bad) ? 0xffff0000u : 0u);
            }
#pragma unroll
            for (int qq = 0; qq < NT_O / 2; ++qq) {
                const int chunk = 2 * qq + v_par;
                const uint32_t addr = vbase + j * TILE_BYTES + (chunk >> 3) * 2048 + v_row_off + (((chunk & 7) ^ rr) << 4);
                uint32_t v0, v1, v2, v3;
                ldmatrix_x4_trans(addr, v0, v1, v2, v3);
                if (need_vmask) {
                    v0 &= mlo;
                    v1 &= mhi;
                    v2 &= mlo;
                    v3 &= mhi;
                }
                mma_bf16_16816(o[2 * qq], pa0, pa1, pa2, pa3, v0, v1);
                mma_bf16_16816(o[2 * qq + 1], pa0, pa1, pa2, pa3, v2, v3);
            }
        }
        __syncthreads();  // stage fully consumed
    }

    if (failed_at >= 0) {
        if (threadIdx.x == 0) atomicOr(p.status, EKV_DEV_FLAG_TIMEOUT);
        // give the copies still in flight a bounded chance to land before the CTA's memory goes away
        for (int t = failed_at; t < n_tiles && t <= failed_at + 1; ++t)
            (void)mbar_wait(bars + 8 * (t % kPmStages), (uint32_t)((t / kPmStages) & 1), 100000000ull);
        return;
    }

    l0 += __shfl_xor_sync(FULL, l0, 1);
    l0 += __shfl_xor_sync(FULL, l0, 2);
    l1 += __shfl_xor_sync(FULL, l1, 1);
    l1 += __shfl_xor_sync(FULL, l1, 2);
    const float i0 = l0 > 0.f ? 1.f / l0 : 0.f, i1 = l1 > 0.f ? 1.f / l1 : 0.f;
    const int lr0 = warp * 16 + r, lr1 = lr0 + 8;
#pragma unroll
    for (int n = 0; n < NT_O; ++n) {
        if (lr0 < rows_here)
            *reinterpret_cast<uint32_t *>(out_base + (size_t)lr0 * row_stride + 8 * n + 2 * c) =
                pack_bf16x2(o[n][0] * i0, o[n][1] * i0);
        if (lr1 < rows_here)
            *reinterpret_cast<uint32_t *>(out_base + (size_t)lr1 * row_stride + 8 * n + 2 * c) =
                pack_bf16x2(o[n][2] * i1, o[n][3] * i1);
    }
}

template <int D>
static ekv_status_t launch_prefill_mma(ekv_pool *pool, int layer, const PrefillParams &p, int q_tiles,
                                       cudaStream_t stream) {
    constexpr int STAGE_BYTES = 2 * 4 * (D / 64) * 2048;
    const int smem = kPmStages * STAGE_BYTES + 1024 + 64 + kPmIdCache * 4;
    static bool attr_set[64] = {false};
    const int dev = pool->desc.device;
    if (dev >= 64 || !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(prefill_mma_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return cuda_fail(e, "ekv_attn_prefill_chunk: shared-memory attribute");
        if (dev < 64) attr_set[dev] = true;
    }
    dim3 grid(q_tiles, pool->desc.num_q_heads);
    prefill_mma_kernel<D><<<grid, 128, smem, stream>>>(pool->kv_map[layer], p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "ekv_attn_prefill_chunk: launch");
    return EKV_OK;
}

}  // namespace ekv
