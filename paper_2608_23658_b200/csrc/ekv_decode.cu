// ekv_attn_decode: GQA decode attention over the block-indexed KV range, HBM-bandwidth bound.
//
// Split pass.  One CTA per (sequence, kv-head, key range of `chunk_tokens`).  Each of the 4 warps
// owns every 4th 16-token block of the range and its own ring of shared-memory stages; lane 0
// feeds the ring with TMA tile loads (one 64-channel x 16-token box per 2 KiB, 128-byte swizzle)
// that complete on per-stage mbarriers, so ~24 KiB per warp can be in flight with no register
// cost.  The whole query group (<= 8 heads) of the kv-head is processed against each K/V tile,
// so KV bytes are read from HBM exactly once:
//     S^T-free formulation on the warp-level tensor path (M is tiny, tcgen05 does not apply):
//       S[head, token]  = Q[head, :] . K[token, :]      mma m16n8k16, heads padded to 16 rows
//       O^T[d, head]   += V^T[d, token] P^T[token, head] mma m16n8k16, V via ldmatrix.trans
//     The C fragment of S is exactly the B fragment P^T needs, so no shuffle sits between them.
// Online softmax keeps a running max per head (quad shuffles) in the exp2 domain.  The 4 warps
// merge through shared memory and write one fp32 partial (m, l, o[d]) per (sequence, head, split).
//
// Combine pass.  One CTA per (sequence, q-head): log-sum-exp merge of the partials -> bf16.
//
// The plan (chunk_tokens) depends only on the call's shape arguments and the summation order only
// on logical key positions, so results are bitwise reproducible and independent of which physical
// blocks (base or elastic) hold the data.
#include <cuda_bf16.h>
#include <math.h>

#include "ekv_internal.h"
#include "ptx.cuh"

namespace ekv {

static constexpr int kDecodeWarps = 4;
static constexpr int kDecodeStages = 3;
static constexpr int kBoxBytes = 16 * 128;  // 16 tokens x 64 bf16 channels
static constexpr int kChunkMaxLimit = 2048; // 32 blocks per warp: one block id per lane

struct DecodeParams {
    const __nv_bfloat16 *q;
    const int *block_tables;
    const int *seq_lens;
    const long long *live;
    unsigned *status;
    float *part_o;   // [B*Hq*nsplit, D]
    float2 *part_ml; // [B*Hq*nsplit]
    __nv_bfloat16 *out;
    int max_blocks, num_q_heads, num_kv_heads, group;
    int chunk_tokens, nsplit;
    float scale_log2;
    long long first_tensor_blocks;  // two-tensor variant only: ids below this live in the first tensor
    long long total_blocks;         // two-tensor variant only: ids at or above this are invalid
};

// kTwo = false: the paper's arrangement, one tensor map over the layer's single virtual range.
// kTwo = true: the alternative the paper rejected (two tensors, the kernel reads both): ids at or above
// p.first_tensor_blocks address a second, separately allocated tensor through kvmap2.
template <int D, bool kTwo>
__global__ void __launch_bounds__(kDecodeWarps * 32, 2)
decode_split_kernel(const __grid_constant__ CUtensorMap kvmap, const __grid_constant__ CUtensorMap kvmap2, const DecodeParams p) {
    constexpr int BOXES = D / 64;
    constexpr int TILE_BYTES = BOXES * kBoxBytes;
    constexpr int STAGE_BYTES = 2 * TILE_BYTES;
    constexpr int KSTEPS = D / 16;
    constexpr unsigned FULL = 0xffffffffu;

    const int split = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = lane >> 2, c = lane & 3;

    int L = p.seq_lens[b];
    L = max(0, min(L, p.max_blocks * 16));
    const int t_begin = split * p.chunk_tokens;
    if (t_begin >= L) {  // whole CTA leaves before any barrier exists
        if (p.nsplit == 1)  // no combine pass will run: an empty sequence gets its zero rows here
            for (int e = threadIdx.x; e < p.group * D; e += kDecodeWarps * 32)
                p.out[((size_t)b * p.num_q_heads + (size_t)g * p.group) * D + e] = __float2bfloat16_rn(0.f);
        return;
    }
    const int t_end = min(L, t_begin + p.chunk_tokens);
    const int nblk = (t_end - t_begin + 15) >> 4;
    const int nw = max(0, (nblk - warp + kDecodeWarps - 1) / kDecodeWarps);  // blocks this warp owns (<= 32)

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_u32 = smem_u32(smem_raw);
    const uint32_t base_u32 = (raw_u32 + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base_u32 - raw_u32);
    const uint32_t my_stages = base_u32 + warp * kDecodeStages * STAGE_BYTES;
    const uint32_t my_bars = base_u32 + kDecodeWarps * kDecodeStages * STAGE_BYTES + warp * kDecodeStages * 8;

    if (lane == 0) {
        prefetch_tensormap(&kvmap);
        if (kTwo) prefetch_tensormap(&kvmap2);
        for (int s = 0; s < kDecodeStages; ++s) mbar_init(my_bars + 8 * s, 1);
        mbar_fence_init();
    }
    __syncwarp();

    // Block ids of this warp's blocks: lane i holds the id of its i-th block.
    const long long live = kTwo ? p.total_blocks : *p.live;
    const int *bt = p.block_tables + (size_t)b * p.max_blocks + (t_begin >> 4) + warp;
    int my_id = (lane < nw) ? bt[lane * kDecodeWarps] : 0;
    const bool my_ok = (lane < nw) && my_id >= 0 && (long long)my_id < live;
    const unsigned valid_mask = __ballot_sync(FULL, my_ok);
    if (lane < nw && !my_ok) atomicOr(p.status, EKV_DEV_FLAG_OOB);

    const uint64_t policy = policy_evict_first();
    auto issue = [&](int i) {
        int id = __shfl_sync(FULL, my_id, i);
        if (lane == 0 && ((valid_mask >> i) & 1u)) {
            const int stage = i % kDecodeStages;
            const uint32_t bar = my_bars + 8 * stage;
            const uint32_t dst = my_stages + stage * STAGE_BYTES;
            const CUtensorMap *map = &kvmap;
            if (kTwo && id >= p.first_tensor_blocks) {  // the extra work of the two-tensor arrangement
                map = &kvmap2;
                id -= (int)p.first_tensor_blocks;
            }
            const int row_k = g * 16;  // row inside the block: (K|V, kv-head, token)
            const int row_v = row_k + p.num_kv_heads * 16;
            mbar_expect_tx(bar, STAGE_BYTES);
#pragma unroll
            for (int x = 0; x < BOXES; ++x) {
                tma_load_3d_hint(dst + x * kBoxBytes, map, 64 * x, row_k, id, bar, policy);
                tma_load_3d_hint(dst + TILE_BYTES + x * kBoxBytes, map, 64 * x, row_v, id, bar, policy);
            }
        }
    };
    for (int s = 0; s < kDecodeStages && s < nw; ++s) issue(s);

    // Q fragments (A operand): rows = heads of the group (r < group), zero above.
    uint32_t qa[KSTEPS][2];
    {
        const __nv_bfloat16 *qrow = p.q + ((size_t)b * p.num_q_heads + (size_t)g * p.group + r) * D;
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
            qa[ks][0] = (r < p.group) ? *reinterpret_cast<const uint32_t *>(qrow + 16 * ks + 2 * c) : 0u;
            qa[ks][1] = (r < p.group) ? *reinterpret_cast<const uint32_t *>(qrow + 16 * ks + 8 + 2 * c) : 0u;
        }
    }

    // ldmatrix lane addressing inside one swizzled tile: matrix mi = lane/8, row rr = lane%8.
    const int mi = lane >> 3, rr = lane & 7;
    const uint32_t lane_row_off = (8 * (mi >> 1) + rr) * 128;
    const int lane_par = mi & 1;

    float o[KSTEPS][4];
#pragma unroll
    for (int mt = 0; mt < KSTEPS; ++mt) o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f;
    float m_run = -INFINITY, l_run = 0.f;
    bool failed = false;

    // Phase parity per stage.  A skipped (invalid) block neither issues a copy nor waits, so the parity of a
    // stage advances only with the copies that really went through it, not with the iteration count.
    uint32_t stage_parity = 0;
    int i = 0;
    for (; i < nw; ++i) {
        const int stage = i % kDecodeStages;
        if ((valid_mask >> i) & 1u) {
            const bool got = mbar_wait(my_bars + 8 * stage, (stage_parity >> stage) & 1u);
            stage_parity ^= 1u << stage;
            if (__any_sync(FULL, !got)) {
                failed = true;
                break;
            }
            const uint32_t kbase = my_stages + stage * STAGE_BYTES;
            const uint32_t vbase = kbase + TILE_BYTES;
            const int tok0 = t_begin + (warp + kDecodeWarps * i) * 16;
            const bool partial = tok0 + 16 > L;

            float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int ks = 0; ks < KSTEPS; ++ks) {
                const int chunk = 2 * ks + lane_par;
                const uint32_t addr = kbase + (chunk >> 3) * kBoxBytes + lane_row_off + (((chunk & 7) ^ rr) << 4);
                uint32_t k0, k1, k2, k3;
                ldmatrix_x4(addr, k0, k1, k2, k3);
                mma_bf16_16816(s0, qa[ks][0], 0u, qa[ks][1], 0u, k0, k1);
                mma_bf16_16816(s1, qa[ks][0], 0u, qa[ks][1], 0u, k2, k3);
            }
            float x0 = s0[0] * p.scale_log2, x1 = s0[1] * p.scale_log2;
            float x2 = s1[0] * p.scale_log2, x3 = s1[1] * p.scale_log2;
            uint32_t mask_lo = 0xffffffffu, mask_hi = 0xffffffffu;
            if (partial) {
                const int t = tok0 + 2 * c;
                if (t >= L) x0 = -INFINITY;
                if (t + 1 >= L) x1 = -INFINITY;
                if (t + 8 >= L) x2 = -INFINITY;
                if (t + 9 >= L) x3 = -INFINITY;
                mask_lo = (t < L ? 0x0000ffffu : 0u) | (t + 1 < L ? 0xffff0000u : 0u);
                mask_hi = (t + 8 < L ? 0x0000ffffu : 0u) | (t + 9 < L ? 0xffff0000u : 0u);
            }
            float mx = fmaxf(fmaxf(x0, x1), fmaxf(x2, x3));
            mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, 2));
            const float m_new = fmaxf(m_run, mx);  // finite: token tok0 < L is never masked
            const float alpha = fast_exp2(m_run - m_new);
            const float p0 = fast_exp2(x0 - m_new), p1 = fast_exp2(x1 - m_new);
            const float p2 = fast_exp2(x2 - m_new), p3 = fast_exp2(x3 - m_new);
            l_run = l_run * alpha + ((p0 + p1) + (p2 + p3));
            m_run = m_new;
            if (__any_sync(FULL, alpha != 1.f)) {
                const float a_lo = __shfl_sync(FULL, alpha, 8 * c);
                const float a_hi = __shfl_sync(FULL, alpha, 8 * c + 4);
#pragma unroll
                for (int mt = 0; mt < KSTEPS; ++mt) {
                    o[mt][0] *= a_lo;
                    o[mt][1] *= a_hi;
                    o[mt][2] *= a_lo;
                    o[mt][3] *= a_hi;
                }
            }
            const uint32_t pb0 = pack_bf16x2(p0, p1), pb1 = pack_bf16x2(p2, p3);
#pragma unroll
            for (int mt = 0; mt < KSTEPS; ++mt) {
                const int chunk = 2 * mt + lane_par;
                const uint32_t addr = vbase + (chunk >> 3) * kBoxBytes + lane_row_off + (((chunk & 7) ^ rr) << 4);
                uint32_t v0, v1, v2, v3;
                ldmatrix_x4_trans(addr, v0, v1, v2, v3);
                if (partial) {  // unwritten slots may hold NaN patterns: 0 * NaN must not reach O
                    v0 &= mask_lo;
                    v1 &= mask_lo;
                    v2 &= mask_hi;
                    v3 &= mask_hi;
                }
                mma_bf16_16816(o[mt], v0, v1, v2, v3, pb0, pb1);
            }
        }
        __syncwarp();  // every lane is done reading the stage before it is refilled
        if (i + kDecodeStages < nw) issue(i + kDecodeStages);
    }

    if (failed) {
        // A copy barrier never completed.  Latch the error, give copies still in flight a bounded
        // chance to land (their destination must stay allocated), and contribute nothing.
        if (lane == 0) atomicOr(p.status, EKV_DEV_FLAG_TIMEOUT);
        stage_parity ^= 1u << (i % kDecodeStages);  // the wait that failed belongs to a copy still outstanding
        for (int j = i; j < nw && j < i + kDecodeStages; ++j)
            if ((valid_mask >> j) & 1u)
                (void)mbar_wait(my_bars + 8 * (j % kDecodeStages), (stage_parity >> (j % kDecodeStages)) & 1u, 200000000ull);
        m_run = -INFINITY;
        l_run = 0.f;
#pragma unroll
        for (int mt = 0; mt < KSTEPS; ++mt) o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f;
    }

    l_run += __shfl_xor_sync(FULL, l_run, 1);
    l_run += __shfl_xor_sync(FULL, l_run, 2);

    // Merge the 4 warps through shared memory (each warp reuses its own, now idle, first stage).
    float *wo = reinterpret_cast<float *>(base_ptr + warp * kDecodeStages * STAGE_BYTES);  // [8][D]
    float *wm = wo + 8 * D;                                                                // [8] m, [8] l
#pragma unroll
    for (int mt = 0; mt < KSTEPS; ++mt) {
        wo[(2 * c) * D + 16 * mt + r] = o[mt][0];
        wo[(2 * c + 1) * D + 16 * mt + r] = o[mt][1];
        wo[(2 * c) * D + 16 * mt + 8 + r] = o[mt][2];
        wo[(2 * c + 1) * D + 16 * mt + 8 + r] = o[mt][3];
    }
    if (c == 0) {
        wm[r] = m_run;
        wm[8 + r] = l_run;
    }
    __syncthreads();

    for (int e = threadIdx.x; e < p.group * D; e += kDecodeWarps * 32) {
        const int h = e / D, x = e % D;
        float mw[kDecodeWarps], mstar = -INFINITY;
#pragma unroll
        for (int w = 0; w < kDecodeWarps; ++w) {
            mw[w] = reinterpret_cast<const float *>(base_ptr + w * kDecodeStages * STAGE_BYTES)[8 * D + h];
            mstar = fmaxf(mstar, mw[w]);
        }
        float acc = 0.f, lsum = 0.f;
        if (mstar > -INFINITY) {
#pragma unroll
            for (int w = 0; w < kDecodeWarps; ++w) {
                const float *src = reinterpret_cast<const float *>(base_ptr + w * kDecodeStages * STAGE_BYTES);
                const float wgt = (mw[w] > -INFINITY) ? fast_exp2(mw[w] - mstar) : 0.f;
                acc += wgt * src[h * D + x];
                lsum += wgt * src[8 * D + 8 + h];
            }
        }
        const size_t slot = ((size_t)b * p.num_q_heads + (size_t)g * p.group + h) * p.nsplit + split;
        if (p.nsplit == 1) {  // the only split of every sequence: finish here, no partials, no combine pass
            p.out[slot * D + x] = __float2bfloat16_rn(lsum > 0.f ? acc / lsum : 0.f);
        } else {
            p.part_o[slot * D + x] = acc;
            if (x == 0) p.part_ml[slot] = make_float2(mstar, lsum);
        }
    }
}

// Block-wide max / sum over D threads (D = 64 or 128), fixed order: bitwise reproducible.
template <int D, bool kMax>
__device__ __forceinline__ float block_reduce(float v, float *scratch) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float u = __shfl_xor_sync(0xffffffffu, v, o);
        v = kMax ? fmaxf(v, u) : v + u;
    }
    __syncthreads();  // scratch may still be read from an earlier reduction
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = scratch[0];
#pragma unroll
    for (int w = 1; w < D / 32; ++w) r = kMax ? fmaxf(r, scratch[w]) : r + scratch[w];
    return r;
}

// One CTA per (sequence, q-head), one thread per output channel.  The splits are walked in parallel: the
// statistics (m, l) are reduced across the block, and the weighted sum of partial rows is taken in tiles of D
// splits whose weights sit in shared memory, so that a long sequence with hundreds of splits costs a few
// rounds of independent loads instead of hundreds of dependent ones.
template <int D>
__global__ void __launch_bounds__(D) decode_combine_kernel(const DecodeParams p) {
    __shared__ float scratch[D / 32];
    __shared__ float w_tile[D];
    const int bh = blockIdx.x;
    const int b = bh / p.num_q_heads;
    const int x = threadIdx.x;
    int L = p.seq_lens[b];
    L = max(0, min(L, p.max_blocks * 16));
    const int ns = (L + p.chunk_tokens - 1) / p.chunk_tokens;
    const float2 *ml = p.part_ml + (size_t)bh * p.nsplit;
    const float *po = p.part_o + (size_t)bh * p.nsplit * D;
    float mloc = -INFINITY;
    for (int s = x; s < ns; s += D) mloc = fmaxf(mloc, ml[s].x);
    const float mstar = block_reduce<D, true>(mloc, scratch);
    float acc = 0.f, lloc = 0.f;
    if (mstar > -INFINITY) {  // block-uniform
        for (int s0 = 0; s0 < ns; s0 += D) {
            const int s = s0 + x;
            float w = 0.f;
            if (s < ns) {
                const float2 v = ml[s];
                w = (v.x > -INFINITY) ? fast_exp2(v.x - mstar) : 0.f;
                lloc += w * v.y;
            }
            __syncthreads();  // the previous tile's weights are no longer needed
            w_tile[x] = w;
            __syncthreads();
            const int n = min(D, ns - s0);
            const float *src = po + (size_t)s0 * D + x;
            int i = 0;
            for (; i + 4 <= n; i += 4) {
                const float o0 = src[(size_t)i * D], o1 = src[(size_t)(i + 1) * D];
                const float o2 = src[(size_t)(i + 2) * D], o3 = src[(size_t)(i + 3) * D];
                acc += w_tile[i] * o0;
                acc += w_tile[i + 1] * o1;
                acc += w_tile[i + 2] * o2;
                acc += w_tile[i + 3] * o3;
            }
            for (; i < n; ++i) acc += w_tile[i] * src[(size_t)i * D];
        }
    }
    const float lsum = block_reduce<D, false>(lloc, scratch);
    p.out[(size_t)bh * D + x] = __float2bfloat16_rn(lsum > 0.f ? acc / lsum : 0.f);
}

static constexpr int kChunkMin = 256;  // 4 blocks per warp: below that the fixed cost of a CTA dominates

// Key ranges per (sequence, kv-head) that would fill the machine: 2 CTAs resident per SM, about 4 waves.
static long long wanted_splits(const ekv_pool *pool, int B) {
    const long long units = (long long)B * pool->desc.num_kv_heads;
    const long long target = (long long)pool->sm_count * 2 * 4;
    const long long want = (target + units - 1) / units;
    return want < 1 ? 1 : want;
}

DecodePlan plan_decode(const ekv_pool *pool, int B, int max_blocks_per_seq) {
    const int max_len = max_blocks_per_seq * pool->desc.block_size;
    const long long want = wanted_splits(pool, B);
    long long chunk = (max_len + want - 1) / want;
    chunk = (chunk + 63) / 64 * 64;
    if (chunk > kChunkMaxLimit) chunk = kChunkMaxLimit;
    const long long cmin = max_len >= kChunkMin ? kChunkMin : (max_len + 63) / 64 * 64;
    if (chunk < cmin) chunk = cmin;
    DecodePlan plan;
    plan.chunk_tokens = (int)chunk;
    plan.nsplit = (int)((max_len + chunk - 1) / chunk);
    if (plan.nsplit < 1) plan.nsplit = 1;
    return plan;
}

static size_t decode_workspace_need(const ekv_pool *pool, int B, int nsplit) {
    const size_t parts = (size_t)B * pool->desc.num_q_heads * nsplit;
    const size_t ml = (parts * sizeof(float2) + 255) / 256 * 256;
    return ml + parts * pool->desc.head_dim * sizeof(float);
}

template <int D, bool kTwo>
static ekv_status_t launch_decode_impl(ekv_pool *pool, const CUtensorMap &map, const CUtensorMap &map2, const DecodeParams &p, int B,
                                      cudaStream_t stream) {
    constexpr int STAGE_BYTES = 2 * (D / 64) * kBoxBytes;
    const int smem = kDecodeWarps * kDecodeStages * STAGE_BYTES + 1024 + kDecodeWarps * kDecodeStages * 8;
    static bool attr_set[64] = {false};
    const int dev = pool->desc.device;
    if (dev >= 64 || !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(decode_split_kernel<D, kTwo>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return cuda_fail(e, "ekv_attn_decode: shared-memory attribute");
        if (dev < 64) attr_set[dev] = true;
    }
    dim3 grid(p.nsplit, pool->desc.num_kv_heads, B);
    decode_split_kernel<D, kTwo><<<grid, kDecodeWarps * 32, smem, stream>>>(map, map2, p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "ekv_attn_decode: split launch");
    if (p.nsplit == 1) return EKV_OK;  // the split kernel wrote the final rows itself
    decode_combine_kernel<D><<<B * pool->desc.num_q_heads, D, 0, stream>>>(p);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "ekv_attn_decode: combine launch");
    return EKV_OK;
}

template <int D>
static ekv_status_t launch_decode(ekv_pool *pool, int layer, const DecodeParams &p, int B, cudaStream_t stream) {
    return launch_decode_impl<D, false>(pool, pool->kv_map[layer], pool->kv_map[layer], p, B, stream);
}


// Argument checks shared by the three decode entry points.
static ekv_status_t check_decode_args(const char *who, const void *q, const void *out, const int32_t *block_tables,
                                      int32_t max_blocks_per_seq, const int32_t *seq_lens, int32_t B) {
    if (B < 0 || max_blocks_per_seq < 1 || max_blocks_per_seq > (1 << 26) || B > 65535 ||
        (B > 0 && (!q || !out || !block_tables || !seq_lens)) || ((uintptr_t)q & 15) || ((uintptr_t)out & 15)) {
        set_error("%s: bad argument (B=%d, max_blocks_per_seq=%d)", who, B, max_blocks_per_seq);
        return EKV_ERR_INVALID;
    }
    return EKV_OK;
}

// Kernel parameters of one call; `scratch` holds the (m, l) pairs first, then the partial rows.
static DecodeParams make_decode_params(const ekv_pool *pool, const DecodePlan &plan, const void *q, void *out,
                                       const int32_t *block_tables, int32_t max_blocks_per_seq, const int32_t *seq_lens, int32_t B,
                                       float scale, void *scratch) {
    const size_t parts = (size_t)B * pool->desc.num_q_heads * plan.nsplit;
    DecodeParams p;
    p.q = (const __nv_bfloat16 *)q;
    p.block_tables = block_tables;
    p.seq_lens = seq_lens;
    p.live = pool->d_live;
    p.status = pool->d_status;
    p.part_ml = (float2 *)scratch;
    p.part_o = (float *)((uint8_t *)scratch + (parts * sizeof(float2) + 255) / 256 * 256);
    p.out = (__nv_bfloat16 *)out;
    p.max_blocks = max_blocks_per_seq;
    p.num_q_heads = pool->desc.num_q_heads;
    p.num_kv_heads = pool->desc.num_kv_heads;
    p.group = pool->desc.num_q_heads / pool->desc.num_kv_heads;
    p.chunk_tokens = plan.chunk_tokens;
    p.nsplit = plan.nsplit;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.first_tensor_blocks = p.total_blocks = 0;
    return p;
}

static ekv_status_t dispatch_decode(ekv_pool *pool, int layer, const DecodeParams &p, int B, cudaStream_t stream) {
    if (pool->desc.head_dim == 128) return launch_decode<128>(pool, layer, p, B, stream);
    return launch_decode<64>(pool, layer, p, B, stream);
}
}  // namespace ekv

using namespace ekv;

// Upper bound of plan_decode(pool, B, m).nsplit over every table width m <= max_blocks.  A shorter table can be cut
// into MORE ranges than the longest one (the range length is rounded up to 64 keys and floored at kChunkMin), so
// the plan of the largest shape alone is not a bound.  Three regimes of plan_decode:
//   range length not clamped, or raised to the floor: it is >= len/want, so nsplit <= want; and it is >= kChunkMin
//     (or covers the whole of a shorter table), so nsplit <= ceil(len / kChunkMin);
//   range length cut down to kChunkMaxLimit: nsplit = ceil(len / kChunkMaxLimit), largest at the largest len.
static long long nsplit_bound(const ekv_pool *pool, int B, int max_blocks) {
    const long long max_len = (long long)max_blocks * pool->desc.block_size;
    const long long by_floor = (max_len + kChunkMin - 1) / kChunkMin;
    const long long by_cap = (max_len + kChunkMaxLimit - 1) / kChunkMaxLimit;
    long long n = wanted_splits(pool, B);
    if (n > by_floor) n = by_floor;
    if (n < by_cap) n = by_cap;
    return n < 1 ? 1 : n;
}

extern "C" size_t ekv_attn_workspace_bytes(const ekv_pool_t *pool, int32_t max_batch, int32_t max_seq_len) {
    if (!pool || max_batch < 1 || max_seq_len < 1) return 0;
    const int max_blocks = (max_seq_len + pool->desc.block_size - 1) / pool->desc.block_size;
    size_t need = 0;
    for (int B = 1; B <= max_batch; ++B) {
        const size_t n = decode_workspace_need(pool, B, (int)nsplit_bound(pool, B, max_blocks));
        if (n > need) need = n;
    }
    return need;
}

extern "C" ekv_status_t ekv_attn_decode_plan(const ekv_pool_t *pool, int32_t B, int32_t max_blocks_per_seq, int32_t *chunk_tokens,
                                             int32_t *nsplit, size_t *workspace_bytes) {
    if (!pool || B < 1 || B > 65535 || max_blocks_per_seq < 1 || max_blocks_per_seq > (1 << 26)) {
        set_error("ekv_attn_decode_plan: bad argument (B=%d, max_blocks_per_seq=%d)", B, max_blocks_per_seq);
        return EKV_ERR_INVALID;
    }
    const DecodePlan plan = plan_decode(pool, B, max_blocks_per_seq);
    if (chunk_tokens) *chunk_tokens = plan.chunk_tokens;
    if (nsplit) *nsplit = plan.nsplit;
    if (workspace_bytes) *workspace_bytes = decode_workspace_need(pool, B, plan.nsplit);
    return EKV_OK;
}

extern "C" ekv_status_t ekv_attn_decode(ekv_pool_t *pool, int32_t layer, const void *q, void *out,
                                        const int32_t *block_tables, int32_t max_blocks_per_seq, const int32_t *seq_lens,
                                        int32_t B, float scale, void *workspace, size_t workspace_bytes, void *stream) {
    ekv_status_t st = check_compute(pool, layer, "ekv_attn_decode");
    if (st == EKV_OK) st = check_decode_args("ekv_attn_decode", q, out, block_tables, max_blocks_per_seq, seq_lens, B);
    if (st != EKV_OK) return st;
    if (B == 0) return EKV_OK;
    const DecodePlan plan = plan_decode(pool, B, max_blocks_per_seq);
    const size_t need = decode_workspace_need(pool, B, plan.nsplit);
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < need) {
        set_error("ekv_attn_decode: workspace %p of %zu bytes; need %zu bytes, 256-byte aligned", workspace, workspace_bytes,
                  need);
        return EKV_ERR_WORKSPACE;
    }
    const DecodeParams p = make_decode_params(pool, plan, q, out, block_tables, max_blocks_per_seq, seq_lens, B, scale, workspace);
    return dispatch_decode(pool, layer, p, B, (cudaStream_t)stream);
}

// ------------------------------------------------------------------------------------------------
// Decode attention for callers that cannot allocate.
//
// Some users of this library have no allocator to turn to when they need the split pass's scratch:
// a serving engine that, once started, has handed every free byte of the device to the KV pool (a
// cudaMalloc then fails or eats the reserve the elastic range gives back), a plain-C host that
// links no tensor library, or code running where the CUDA allocator must not be entered (inside a
// stream capture, from a callback).  For them the scratch lives in the library image itself: a
// fixed device array that every GPU loading the library carries until the process exits.
// ------------------------------------------------------------------------------------------------
namespace ekv {

static __device__ __align__(256) unsigned char g_decode_static_scratch[EKV_STATIC_SCRATCH_BYTES];

// In host code the array's name is only a handle for the runtime, not a device address; the address
// kernels may use is looked up once per device (with that device current) and cached here.
static void *g_decode_static_scratch_addr[64] = {nullptr};

static ekv_status_t static_scratch_address(int device, void **addr) {
    if (device < 0 || device >= 64) {
        set_error("ekv_attn_decode_static_scratch: device ordinal %d is outside the supported 0..63", device);
        return EKV_ERR_INVALID;
    }
    void *ptr = __atomic_load_n(&g_decode_static_scratch_addr[device], __ATOMIC_ACQUIRE);
    if (ptr == nullptr) {
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_decode_static_scratch);
        if (e != cudaSuccess) return cuda_fail(e, "ekv_attn_decode_static_scratch: cudaGetSymbolAddress");
        if (ptr == nullptr || ((uintptr_t)ptr & 255) != 0) {
            set_error("ekv_attn_decode_static_scratch: scratch symbol resolved to an unusable address %p", ptr);
            return EKV_ERR_CUDA;
        }
        __atomic_store_n(&g_decode_static_scratch_addr[device], ptr, __ATOMIC_RELEASE);
    }
    *addr = ptr;
    return EKV_OK;
}

}  // namespace ekv

extern "C" ekv_status_t ekv_attn_decode_static_scratch(ekv_pool_t *pool, int32_t layer, const void *q, void *out,
                                                       const int32_t *block_tables, int32_t max_blocks_per_seq,
                                                       const int32_t *seq_lens, int32_t B, float scale, void *stream) {
    ekv_status_t st = check_compute(pool, layer, "ekv_attn_decode_static_scratch");  // makes the pool's device current
    if (st == EKV_OK) st = check_decode_args("ekv_attn_decode_static_scratch", q, out, block_tables, max_blocks_per_seq, seq_lens, B);
    if (st != EKV_OK) return st;
    if (B == 0) return EKV_OK;
    const DecodePlan plan = plan_decode(pool, B, max_blocks_per_seq);
    const size_t need = decode_workspace_need(pool, B, plan.nsplit);
    if (need > (size_t)EKV_STATIC_SCRATCH_BYTES) {
        set_error("ekv_attn_decode_static_scratch: this call needs %zu bytes of scratch but the built-in array holds %zu "
                  "(B=%d, max_blocks_per_seq=%d); use ekv_attn_decode with a caller-provided workspace",
                  need, (size_t)EKV_STATIC_SCRATCH_BYTES, B, max_blocks_per_seq);
        return EKV_ERR_WORKSPACE;
    }
    void *scratch = nullptr;
    st = static_scratch_address(pool->desc.device, &scratch);
    if (st != EKV_OK) return st;
    const DecodeParams p = make_decode_params(pool, plan, q, out, block_tables, max_blocks_per_seq, seq_lens, B, scale, scratch);
    return dispatch_decode(pool, layer, p, B, (cudaStream_t)stream);
}

// ------------------------------------------------------------------------------------------------
// The two-tensor alternative (paper, "The contiguity constraint": split the KV into two tensors and
// rewrite the kernel to read both -- prototyped there and rejected).  Built here only to put a number on
// what the single-range design avoids: the same split kernel with a second tensor map and a per-block
// choice between the two.
// ------------------------------------------------------------------------------------------------
extern "C" ekv_status_t ekv_attn_decode_two_tensor(ekv_pool_t *pool, int32_t layer, const void *second_tensor,
                                                   int64_t second_blocks, const void *q, void *out, const int32_t *block_tables,
                                                   int32_t max_blocks_per_seq, const int32_t *seq_lens, int32_t B, float scale,
                                                   void *workspace, size_t workspace_bytes, void *stream) {
    ekv_status_t st = check_compute(pool, layer, "ekv_attn_decode_two_tensor");
    if (st == EKV_OK) st = check_decode_args("ekv_attn_decode_two_tensor", q, out, block_tables, max_blocks_per_seq, seq_lens, B);
    if (st != EKV_OK) return st;
    if (second_blocks < 1 || second_blocks >= (1ll << 31) || !second_tensor || ((uintptr_t)second_tensor & 15)) {
        set_error("ekv_attn_decode_two_tensor: bad second tensor (%p, %lld blocks)", second_tensor, (long long)second_blocks);
        return EKV_ERR_INVALID;
    }
    if (B == 0) return EKV_OK;
    const DecodePlan plan = plan_decode(pool, B, max_blocks_per_seq);
    const size_t need = decode_workspace_need(pool, B, plan.nsplit);
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < need) {
        set_error("ekv_attn_decode_two_tensor: workspace %p of %zu bytes; need %zu bytes, 256-byte aligned", workspace,
                  workspace_bytes, need);
        return EKV_ERR_WORKSPACE;
    }
    CUtensorMap map2;
    st = encode_kv_map(const_cast<void *>(second_tensor), (uint64_t)second_blocks, pool->block_bytes, pool->desc.num_kv_heads,
                       pool->desc.head_dim, pool->desc.block_size, &map2);
    if (st != EKV_OK) return st;
    DecodeParams p = make_decode_params(pool, plan, q, out, block_tables, max_blocks_per_seq, seq_lens, B, scale, workspace);
    p.first_tensor_blocks = pool->base_blocks;  // the first tensor is the pool's base range, whatever the elastic state
    p.total_blocks = pool->base_blocks + second_blocks;
    if (pool->desc.head_dim == 128)
        return launch_decode_impl<128, true>(pool, pool->kv_map[layer], map2, p, B, (cudaStream_t)stream);
    return launch_decode_impl<64, true>(pool, pool->kv_map[layer], map2, p, B, (cudaStream_t)stream);
}
