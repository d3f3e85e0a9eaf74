// Chunked-prefill attention on the 5th-generation tensor cores, ONE query head per CTA, two CTAs per SM.
//
// The two-head kernel (ekv_prefill_tc.cuh) owns a whole SM: 512 TMEM columns, 198 KB of shared memory, every
// register.  That is the right trade for a long prompt, where a CTA walks hundreds of key tiles and each K/V tile
// it stages feeds two heads.  For a batch of SHORT prompts a CTA sees one to four key tiles, most of its life is
// fixed cost (TMEM allocation, the Q tile, the first K/V tile, a strictly serial QK -> softmax -> PV -> write-out),
// and with one CTA per SM nothing overlaps that.  This kernel halves the footprint -- 128 query rows of one head,
// 256 TMEM columns (S 128 + O head_dim), about 97 KB of shared memory, 256 threads -- so that two CTAs share an SM
// and one's fixed cost and softmax hide behind the other's MMAs.  It is also the tcgen05 path for head_dim 64 and
// for odd query groups, which the two-head kernel cannot take.
//
//   warp 0        TMA producer of K and V tiles (16-token x 64-channel boxes gathered through the block table)
//   warp 1        TMEM allocation; MMA issuer: S = Q K^T (both operands from shared memory) and
//                 O += P V (P read from TMEM, V from shared memory, MN-major)
//   warps 2-3     idle (they complete the utility warpgroup, see the register note below)
//   warps 4-7     softmax, one thread per query row (= TMEM lane); same lazy-rescaling scheme as the two-head kernel
//
// One K and one V stage at head_dim 128 (two at 64): K(j+1) is loaded while softmax(j) and PV(j) run, V(j+1) while
// QK(j+1) and softmax(j+1) run, and the other CTA of the SM fills the tensor pipe meanwhile.
#pragma once
#include "ekv_prefill_tc.cuh"

namespace ekv {
namespace tc1 {

namespace cp = cuda::ptx;
using tc::fence_after;
using tc::fence_before;

static constexpr int kBM = 128, kBN = 128;
static constexpr int kThreads = 256;
static constexpr int kHalfBytes = 128 * 128;  // [128 rows][64 bf16], 128-byte swizzle
static constexpr int kTmemCols = 256;
static constexpr uint32_t kColS = 0, kColO = 128;
// Registers: two CTAs per SM leave 128 per thread at launch.  Warps 0-3 (producer, MMA issuer, two idle warps) form one
// warpgroup and drop to kRegsUtil, warps 4-7 (softmax) form the other and rise to kRegsSoftmax.  setmaxnreg must be
// executed by whole warpgroups (four consecutive warps from a multiple of four) that all ask for the same thing -- a
// warpgroup whose warps disagree blocks without bound -- which is why the CTA carries two idle warps.
static constexpr int kLaunchRegs = 128, kRegsUtil = 40, kRegsSoftmax = 216;
static_assert(128 * kRegsUtil + 128 * kRegsSoftmax <= kLaunchRegs * kThreads, "setmaxnreg split exceeds the CTA's registers");
static_assert(2 * kLaunchRegs * kThreads <= 65536 && kRegsUtil % 8 == 0 && kRegsSoftmax % 8 == 0, "two CTAs per SM");
static_assert(kRegsUtil == 40 && kRegsSoftmax == 216 && kThreads == 256, "the setmaxnreg instructions and the role split in the kernel carry these numbers as literals");

template <int D>
struct Geo {
    static constexpr int kHalves = D / 64;
    static constexpr int kTileBytes = kHalves * kHalfBytes;  // a Q, K or V tile
    static constexpr int kStages = D == 64 ? 2 : 1;
    static constexpr int kOffQ = 0;
    static constexpr int kOffK = kTileBytes;
    static constexpr int kOffV = kOffK + kStages * kTileBytes;
    static constexpr int kOffBar = kOffV + kStages * kTileBytes;
    static constexpr int kSmemBytes = kOffBar + 256 + 1024;
    // barrier slots
    static constexpr int Q_READY = 0, K_FULL = 1, K_EMPTY = K_FULL + kStages, V_FULL = K_EMPTY + kStages,
                         V_EMPTY = V_FULL + kStages, S_READY = V_EMPTY + kStages, P_PART = S_READY + 1, P_READY = P_PART + 1,
                         DRAIN = P_READY + 1, NBAR = DRAIN + 1;
    static_assert(8 * NBAR + 32 <= 256, "barrier area");
    // kind::f16 instruction descriptors: D = f32, A = B = bf16, M = 128
    static constexpr uint32_t kIdescQK = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
    static constexpr uint32_t kIdescPV = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | (((uint32_t)D >> 3) << 17) | ((128u >> 4) << 24);
};

template <int D>
struct Smem {
    uint32_t base;
    uint8_t *ptr;
    __device__ __forceinline__ uint32_t bar(int i) const { return base + Geo<D>::kOffBar + 8 * i; }
    __device__ __forceinline__ volatile int *abort_flag() const { return (volatile int *)(ptr + Geo<D>::kOffBar + 8 * Geo<D>::NBAR); }
    __device__ __forceinline__ uint32_t *tmem_slot() const { return (uint32_t *)(ptr + Geo<D>::kOffBar + 8 * Geo<D>::NBAR + 8); }
    // ring of 4: the producer may be a few tiles ahead of the softmax warps that read the mask
    __device__ __forceinline__ volatile int *bad_mask(int tile) const {
        return (volatile int *)(ptr + Geo<D>::kOffBar + 8 * Geo<D>::NBAR + 16 + 4 * (tile & 3));
    }
};

// Bounded wait that also gives up as soon as another role has flagged an abort (same contract as the two-head kernel).
template <int D>
__device__ __forceinline__ bool wait_or_abort(const Smem<D> &sh, int bar, uint32_t parity, unsigned *status, int *abort_word) {
    const uint32_t b = sh.bar(bar);
    if (mbar_try_wait(b, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    for (uint32_t i = 1;; ++i) {
        if (mbar_try_wait(b, parity)) return true;
        if ((i & 31u) == 0u) {
            if (*sh.abort_flag()) return false;
            if (global_timer_ns() - t0 > 2000000000ull) {
                *sh.abort_flag() = 1;
                *(volatile int *)abort_word = 1;
                atomicOr(status, EKV_DEV_FLAG_TIMEOUT);
                return false;
            }
        }
    }
}
template <int D>
__device__ __forceinline__ bool wait_warp(const Smem<D> &sh, int bar, uint32_t parity, unsigned *status, int *abort_word) {
    return __all_sync(0xffffffffu, wait_or_abort<D>(sh, bar, parity, status, abort_word));
}

template <int D>
__global__ void __launch_bounds__(kThreads, 2) prefill_tc1_kernel(const __grid_constant__ CUtensorMap kvmap, const PrefillParams p) {
    using G = Geo<D>;
    constexpr int kStages = G::kStages;
    constexpr int kPieces = D / 8;               // 16-byte pieces per row of Q / O
    constexpr int kRowsPerInst = 32 / kPieces;   // rows one warp-wide 16-byte access covers
    if (*(volatile int *)p.abort_word) return;   // an earlier CTA of this launch timed out

    // ---- which (request, 128-row tile, head)?  Heaviest (latest) tiles first.
    const int tile_idx = gridDim.x - 1 - blockIdx.x;
    const int head = blockIdx.y;
    const int g = head / p.group;
    int req = 0, acc_tiles = 0, c_r = 0, q0 = 0;
    if (!find_request(p, tile_idx, kBM, req, acc_tiles, q0, c_r)) return;
    const int row0 = (tile_idx - acc_tiles) * kBM;
    const int L = min(p.seq_lens[req], p.max_blocks * 16);
    const int prefix = L - c_r;
    const int rows_here = min(kBM, c_r - row0);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const size_t row_stride = (size_t)p.num_q_heads * D;

    if (prefix < 0) {  // malformed request: zero rows, latch
        if (threadIdx.x == 0) atomicOr(p.status, EKV_DEV_FLAG_OOB);
        for (int e = threadIdx.x; e < rows_here * D; e += kThreads)
            p.out[((size_t)(q0 + row0 + e / D)) * row_stride + (size_t)head * D + e % D] = __float2bfloat16_rn(0.f);
        return;
    }
    const int kv_end = min(L, prefix + row0 + rows_here);  // keys any row of this tile may see
    const int n_tiles = (kv_end + kBN - 1) / kBN;
    const int n_blocks = (kv_end + 15) >> 4;

    extern __shared__ uint8_t smem_raw[];
    Smem<D> sh;
    {
        const uint32_t raw = smem_u32(smem_raw);
        sh.base = (raw + 1023u) & ~1023u;
        sh.ptr = smem_raw + (sh.base - raw);
    }
    if (threadIdx.x == 0) {
        prefetch_tensormap(&kvmap);
        mbar_init(sh.bar(G::Q_READY), 4);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(sh.bar(G::K_FULL + s), 1);
            mbar_init(sh.bar(G::K_EMPTY + s), 1);
            mbar_init(sh.bar(G::V_FULL + s), 1);
            mbar_init(sh.bar(G::V_EMPTY + s), 1);
        }
        mbar_init(sh.bar(G::S_READY), 1);
        mbar_init(sh.bar(G::P_PART), 4);
        mbar_init(sh.bar(G::P_READY), 4);
        mbar_init(sh.bar(G::DRAIN), 1);
        *sh.abort_flag() = 0;
        mbar_fence_init();
    }
    if (warp == 1) {
        cp::tcgen05_alloc(cp::cta_group_1, sh.tmem_slot(), kTmemCols);
        cp::tcgen05_relinquish_alloc_permit(cp::cta_group_1);
    }
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem = *sh.tmem_slot();

    if (warp < 4) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 40;");
        if (warp == 0) {
            // =========================== TMA producer: K(j), then V(j) ===========================
            const long long live = *p.live;
            const int *bt = p.block_tables + (size_t)req * p.max_blocks;
            auto load_id = [&](int j) {  // lane l: id of block 8j + l%8 (-1 past the end, -2 invalid)
                int id = -1;
                const int bi = 8 * j + (lane & 7);
                if (bi < n_blocks) {
                    id = bt[bi];
                    if (id < 0 || (long long)id >= live) id = -2;
                }
                return id;
            };
            int id_next = load_id(0);
            bool ok = true;
            for (int j = 0; j < n_tiles && ok; ++j) {
                const int s = j % kStages;
                const int id_raw = id_next;
                if (j + 1 < n_tiles) id_next = load_id(j + 1);
                const unsigned oob = __ballot_sync(0xffffffffu, id_raw == -2) & 0xffu;
                // blocks whose smem rows will hold stand-in data: invalid ids and blocks past the last visible key
                const unsigned bad = __ballot_sync(0xffffffffu, id_raw < 0) & 0xffu;
                const int id = id_raw < 0 ? 0 : id_raw;  // masked later; block 0 is always mapped
                // box b of a tile: block b / kHalves, channel half b % kHalves  ->  [half][block][16 rows][128 B]
                const int b = lane % (8 * G::kHalves), blk = b / G::kHalves, half = b % G::kHalves;
                const int my_id = __shfl_sync(0xffffffffu, id, blk);
                const uint32_t ph = (uint32_t)(((j / kStages) - 1) & 1);
#pragma unroll
                for (int kv = 0; kv < 2; ++kv) {
                    const int FULL = kv ? G::V_FULL : G::K_FULL, EMPTY = kv ? G::V_EMPTY : G::K_EMPTY;
                    const uint32_t tile_base = sh.base + (kv ? G::kOffV : G::kOffK) + s * G::kTileBytes;
                    const int row = g * 16 + (kv ? p.num_kv_heads * 16 : 0);  // row inside the block: (K|V, kv-head, token)
                    if (j >= kStages && !wait_warp<D>(sh, EMPTY + s, ph, p.status, p.abort_word)) {
                        ok = false;
                        break;
                    }
                    if (lane == 0) {
                        if (!kv) {
                            if (oob) atomicOr(p.status, EKV_DEV_FLAG_OOB);
                            *sh.bad_mask(j) = (int)bad;
                        }
                        mbar_expect_tx(sh.bar(FULL + s), G::kTileBytes);
                    }
                    __syncwarp();
                    if (lane < 8 * G::kHalves)
                        tma_load_3d(tile_base + half * kHalfBytes + blk * 2048, &kvmap, 64 * half, row, my_id, sh.bar(FULL + s));
                }
            }
        } else if (warp == 1) {
            // =========================== MMA issuer ===========================
            const uint32_t q_lo = tc::desc_lo(sh.base + G::kOffQ, 16);
            const uint32_t k_lo0 = tc::desc_lo(sh.base + G::kOffK, 16), v_lo0 = tc::desc_lo(sh.base + G::kOffV, kHalfBytes);
            auto issue_qk = [&](int s) {  // S = Q K(s)^T
                const uint32_t k_lo = k_lo0 + (uint32_t)s * (G::kTileBytes >> 4);
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t off = ((k >> 2) * kHalfBytes + (k & 3) * 32) >> 4;
                    if (k == 0) tc::mma_ss_lo<false>(tmem + kColS, q_lo + off, k_lo + off, G::kIdescQK);
                    else tc::mma_ss_lo<true>(tmem + kColS, q_lo + off, k_lo + off, G::kIdescQK);
                }
            };
            auto issue_pv = [&](int s, bool acc, int k0, int k1) {  // O (+)= P[:, 16k0:16k1] V(s)[16k0:16k1, :]
                const uint32_t v_lo = v_lo0 + (uint32_t)s * (G::kTileBytes >> 4);
#pragma unroll
                for (int k = k0; k < k1; ++k)
                    tc::mma_ts_lo_dyn(tmem + kColO, tmem + kColS + 8 * k, v_lo + ((k * 2048) >> 4), G::kIdescPV, (acc || k > 0) ? 1u : 0u);
            };
            bool ok = wait_warp<D>(sh, G::Q_READY, 0, p.status, p.abort_word) && wait_warp<D>(sh, G::K_FULL + 0, 0, p.status, p.abort_word);
            if (ok) {
                fence_after();
                issue_qk(0);
                tc::mma_commit(sh.bar(G::K_EMPTY + 0));
                tc::mma_commit(sh.bar(G::S_READY));
                for (int j = 0; j < n_tiles && ok; ++j) {
                    const int s = j % kStages, s1 = (j + 1) % kStages;
                    const bool more = j + 1 < n_tiles;
                    ok = wait_warp<D>(sh, G::V_FULL + s, (uint32_t)((j / kStages) & 1), p.status, p.abort_word);
                    if (ok) ok = wait_warp<D>(sh, G::P_PART, (uint32_t)(j & 1), p.status, p.abort_word);
                    if (!ok) break;
                    fence_after();
                    issue_pv(s, j > 0, 0, tc::kPartSteps);  // keys 0..95 while the softmax warps finish the rest
                    ok = wait_warp<D>(sh, G::P_READY, (uint32_t)(j & 1), p.status, p.abort_word);
                    if (!ok) break;
                    fence_after();
                    issue_pv(s, true, tc::kPartSteps, kBN / 16);
                    tc::mma_commit(sh.bar(G::V_EMPTY + s));
                    if (more) {
                        ok = wait_warp<D>(sh, G::K_FULL + s1, (uint32_t)(((j + 1) / kStages) & 1), p.status, p.abort_word);
                        if (!ok) break;
                        fence_after();
                        issue_qk(s1);
                        tc::mma_commit(sh.bar(G::K_EMPTY + s1));
                    }
                    tc::mma_commit(sh.bar(G::S_READY));
                }
            }
            // every MMA this thread issued must be finished before TMEM is released
            tc::mma_commit(sh.bar(G::DRAIN));
            (void)wait_warp<D>(sh, G::DRAIN, 0, p.status, p.abort_word);
        }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
        // =========================== softmax + epilogue ===========================
        const int quarter = warp & 3;                    // TMEM lanes 32*quarter .. +31 belong to this warp
        const int wrow0 = quarter << 5;
        const int row = wrow0 | lane;                    // query row in the tile = TMEM lane
        const uint32_t lane_base = (uint32_t)wrow0 << 16;
        const uint32_t t_s = tmem + lane_base + kColS;
        const uint32_t t_o = tmem + lane_base + kColO;

        // ---- stage the Q tile (128-byte swizzle): each warp brings in its own 32 rows, kRowsPerInst rows per
        // instruction, so that a warp-wide load covers whole contiguous rows
        {
            uint8_t *qdst = sh.ptr + G::kOffQ;
            const int piece = lane % kPieces, sub = lane / kPieces;
            const __nv_bfloat16 *src = p.q + ((size_t)(q0 + row0)) * row_stride + (size_t)head * D + piece * 8;
            uint4 v[kPieces];
#pragma unroll
            for (int it = 0; it < 32 / kRowsPerInst; ++it) {
                const int rr = wrow0 + kRowsPerInst * it + sub;
                v[it] = rr < rows_here ? *reinterpret_cast<const uint4 *>(src + (size_t)rr * row_stride) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int it = 0; it < 32 / kRowsPerInst; ++it) {
                const int rr = wrow0 + kRowsPerInst * it + sub;
                *reinterpret_cast<uint4 *>(qdst + (piece >> 3) * kHalfBytes + rr * 128 + (((piece & 7) ^ (rr & 7)) << 4)) = v[it];
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(sh.bar(G::Q_READY));
        }

        const int lim = prefix + row0 + min(row, rows_here - 1);  // last key this row may see
        float m_run = -INFINITY, l_run = 0.f;
        bool ok = true;
        auto publish = [&](int bar) {  // this warp's 32 rows of P are in TMEM: one lane tells the MMA warp
            cp::tcgen05_wait_st();
            fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(sh.bar(bar));
        };
        for (int j = 0; j < n_tiles; ++j) {
            const int s = j % kStages;
            ok = wait_warp<D>(sh, G::S_READY, (uint32_t)(j & 1), p.status, p.abort_word);
            if (!ok) break;
            fence_after();
            const int key0 = j * kBN;
            const int bad = *sh.bad_mask(j);
            const bool need_mask = (key0 + kBN - 1 > prefix + row0) || bad != 0;
            // keys of this tile that lie past the sequence end, or in a skipped block, may hold anything
            // (unwritten slots): their V rows must not reach the tensor pipe, because 0 * NaN = NaN
            const bool dirty_v = (key0 + kBN > L) || bad != 0;
            if (dirty_v) {
                ok = wait_warp<D>(sh, G::V_FULL + s, (uint32_t)((j / kStages) & 1), p.status, p.abort_word);
                if (!ok) break;
                uint8_t *vdst = sh.ptr + G::kOffV + s * G::kTileBytes;
                if ((key0 + row >= L) || ((bad >> (row >> 4)) & 1)) {  // thread `row` owns key row `row` of the tile
#pragma unroll
                    for (int h2 = 0; h2 < G::kHalves; ++h2)
#pragma unroll
                        for (int c16 = 0; c16 < 8; ++c16)
                            *reinterpret_cast<uint4 *>(vdst + h2 * kHalfBytes + row * 128 + c16 * 16) = make_uint4(0u, 0u, 0u, 0u);
                }
                fence_proxy_async_smem();
            }

            // ---- the whole score row into registers (one TMEM read), masked entries become -inf
            float sv[128];
            {
                uint32_t(&r)[128] = reinterpret_cast<uint32_t(&)[128]>(sv);
                cp::tcgen05_ld_32x32b(reinterpret_cast<uint32_t(&)[32]>(r[0]), t_s);
                cp::tcgen05_ld_32x32b(reinterpret_cast<uint32_t(&)[32]>(r[32]), t_s + 32);
                cp::tcgen05_ld_32x32b(reinterpret_cast<uint32_t(&)[32]>(r[64]), t_s + 64);
                cp::tcgen05_ld_32x32b(reinterpret_cast<uint32_t(&)[32]>(r[96]), t_s + 96);
                cp::tcgen05_wait_ld();
            }
            if (need_mask) {
#pragma unroll
                for (int i = 0; i < 128; ++i)
                    if (key0 + i > lim || ((bad >> (i >> 4)) & 1)) sv[i] = -INFINITY;
            }
            float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
            for (int i = 0; i < 128; i += 4) {
                mx0 = fmaxf(mx0, sv[i]);
                mx1 = fmaxf(mx1, sv[i + 1]);
                mx2 = fmaxf(mx2, sv[i + 2]);
                mx3 = fmaxf(mx3, sv[i + 3]);
            }
            const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
            const float m_tile = mx * p.scale_log2;  // scale > 0 on this path
            // ---- lazy rescale: raise the reference max only when it is far behind
            const bool raise = m_tile > m_run + tc::kRescaleThreshold;  // also true for the first finite tile
            if (__any_sync(0xffffffffu, raise)) {
                const float m_new = raise ? m_tile : m_run;
                const float alpha = (raise && m_run > -INFINITY) ? fast_exp2(m_run - m_new) : (raise ? 0.f : 1.f);
                m_run = m_new;
                l_run *= alpha;
                if (j > 0) {  // O holds the sum over earlier tiles and no MMA touches it right now
#pragma unroll
                    for (int cc = 0; cc < D / 32; ++cc) {
                        float ov[32];
                        tc::tmem_ld32(ov, t_o + 32 * cc);
#pragma unroll
                        for (int i = 0; i < 32; ++i) ov[i] *= alpha;
                        tc::tmem_st32(t_o + 32 * cc, ov);
                    }
                }
            }
            const float m_use = m_run > -INFINITY ? m_run : 0.f;
            // ---- P = exp2(S*scale - m) (a masked -inf gives 0), row sum, bf16 pairs into the S columns
            // P of the first 96 keys is published early so the PV MMA overlaps the last quarter of this loop.
            float2 acc_a = make_float2(0.f, 0.f), acc_b = make_float2(0.f, 0.f);
            const float2 sc2 = make_float2(p.scale_log2, p.scale_log2), nm2 = make_float2(-m_use, -m_use);
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                    const float2 xa = __ffma2_rn(make_float2(sv[32 * cc + i], sv[32 * cc + i + 1]), sc2, nm2);
                    const float2 xb = __ffma2_rn(make_float2(sv[32 * cc + i + 2], sv[32 * cc + i + 3]), sc2, nm2);
                    const float2 pa = make_float2(fast_exp2(xa.x), fast_exp2(xa.y));
                    const float2 pb = make_float2(fast_exp2(xb.x), fast_exp2(xb.y));
                    acc_a = __fadd2_rn(acc_a, pa);
                    acc_b = __fadd2_rn(acc_b, pb);
                    pk[i >> 1] = pack_bf16x2(pa.x, pa.y);
                    pk[(i >> 1) + 1] = pack_bf16x2(pb.x, pb.y);
                }
                cp::tcgen05_st_32x32b(t_s + 16 * cc, pk);
                if (cc == tc::kPartSteps / 2 - 1) publish(G::P_PART);  // 96 keys stored
            }
            l_run += (acc_a.x + acc_a.y) + (acc_b.x + acc_b.y);
            publish(G::P_READY);
        }

        // ---- epilogue: O / l -> bf16 -> the (now idle) Q tile in shared memory -> global, whole rows per instruction.
        // Only the warp that wrote a row reads it: __syncwarp suffices.
        if (ok) ok = wait_warp<D>(sh, G::S_READY, (uint32_t)(n_tiles & 1), p.status, p.abort_word);
        if (ok) {
            fence_after();  // every MMA that read the Q tile or wrote O has completed (the commit covers all earlier ones)
            const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
            uint8_t *stage = sh.ptr + G::kOffQ;
#pragma unroll
            for (int cc = 0; cc < D / 32; ++cc) {
                float ov[32];
                tc::tmem_ld32(ov, t_o + 32 * cc);
#pragma unroll
                for (int i = 0; i < 32; i += 8) {
                    uint4 v;
                    v.x = pack_bf16x2(ov[i] * inv, ov[i + 1] * inv);
                    v.y = pack_bf16x2(ov[i + 2] * inv, ov[i + 3] * inv);
                    v.z = pack_bf16x2(ov[i + 4] * inv, ov[i + 5] * inv);
                    v.w = pack_bf16x2(ov[i + 6] * inv, ov[i + 7] * inv);
                    const int piece = cc * 4 + (i >> 3);
                    *reinterpret_cast<uint4 *>(stage + row * (D * 2) + ((piece ^ (row & (kPieces - 1))) << 4)) = v;
                }
            }
            __syncwarp();
            const int piece = lane % kPieces, sub = lane / kPieces;
            __nv_bfloat16 *dst = p.out + ((size_t)(q0 + row0)) * row_stride + (size_t)head * D + piece * 8;
#pragma unroll
            for (int it = 0; it < 32 / kRowsPerInst; ++it) {
                const int rr = wrow0 + kRowsPerInst * it + sub;
                const uint4 v = *reinterpret_cast<const uint4 *>(stage + rr * (D * 2) + ((piece ^ (rr & (kPieces - 1))) << 4));
                if (rr < rows_here) *reinterpret_cast<uint4 *>(dst + (size_t)rr * row_stride) = v;
            }
        }
    }

    // ---- teardown: everybody meets, copies in flight get a bounded chance to land, TMEM goes back
    fence_before();
    __syncthreads();
    fence_after();
    if (warp == 0 && *sh.abort_flag()) {
        for (int j = max(0, n_tiles - kStages); j < n_tiles; ++j) {
            (void)mbar_wait(sh.bar(G::K_FULL + j % kStages), (uint32_t)((j / kStages) & 1), 100000000ull);
            (void)mbar_wait(sh.bar(G::V_FULL + j % kStages), (uint32_t)((j / kStages) & 1), 100000000ull);
        }
    }
    __syncthreads();
    if (warp == 1) cp::tcgen05_dealloc(cp::cta_group_1, tmem, kTmemCols);
}

template <int D>
static ekv_status_t launch_prefill_tc1(ekv_pool *pool, int layer, const PrefillParams &p, int q_tiles, cudaStream_t stream) {
    static bool attr_set[64] = {false};
    const int dev = pool->desc.device;
    if (dev >= 64 || !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(prefill_tc1_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, Geo<D>::kSmemBytes);
        if (e == cudaSuccess)  // two CTAs of ~97 KB each must fit: ask for the largest shared-memory carve-out
            e = cudaFuncSetAttribute(prefill_tc1_kernel<D>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return cuda_fail(e, "ekv_attn_prefill_chunk: shared-memory attributes");
        if (dev < 64) attr_set[dev] = true;
    }
    dim3 grid(q_tiles, pool->desc.num_q_heads);
    cudaError_t e0 = cudaMemsetAsync(p.abort_word, 0, sizeof(int), stream);
    if (e0 != cudaSuccess) return cuda_fail(e0, "ekv_attn_prefill_chunk: clear abort word");
    prefill_tc1_kernel<D><<<grid, kThreads, Geo<D>::kSmemBytes, stream>>>(pool->kv_map[layer], p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "ekv_attn_prefill_chunk: launch");
    return EKV_OK;
}

}  // namespace tc1
}  // namespace ekv
