// Chunked-prefill attention on the 5th-generation tensor cores (tcgen05.mma, accumulators in TMEM),
// head_dim 128, even query group.
//
// One CTA = 128 query positions of one request x TWO query heads (A, B) that share a kv-head, so
// every K/V tile staged in shared memory feeds two 128x128 score tiles (ping-pong: while the
// softmax warps work on one head's scores the tensor pipe runs the other head's MMAs).
//
//   warp 0        TMA producer: 16-token x 64-channel boxes (128-byte swizzle) of K and V blocks,
//                 gathered through the block table into 128-key tiles, 2 stages each for K and V
//   warp 1        MMA issuer (whole warp converged, one elected lane issues): S = Q K^T (A, B from shared memory, K-major) and
//                 O += P V (A = P read from TMEM, B = V from shared memory, MN-major)
//   warp 2        TMEM allocation / release (512 columns: S_A S_B O_A O_B, P aliases S)
//   warps 4-7     softmax of head A: one thread per query row (= TMEM lane)
//   warps 8-11    softmax of head B
//
// Softmax is online in the exp2 domain with LAZY rescaling: the running reference max of a row is
// only raised (and O, l rescaled in TMEM) when a tile's max exceeds it by more than 2^8, so P stays
// below 256 and most tiles need no pass over O.  All mbarrier waits are bounded; a wait that runs
// out latches EKV_ERR_TIMEOUT, makes every role leave its loop, and the CTA still drains its
// copies, releases TMEM and exits.
#pragma once
#include <cuda/ptx>
#include <cuda_bf16.h>
#include <math.h>

#include "ekv_internal.h"
#include "ekv_prefill_mma.cuh"  // PrefillParams
#include "ptx.cuh"

namespace ekv {
namespace tc {

namespace cp = cuda::ptx;

static constexpr int kBM = 128;          // query rows per head tile
static constexpr int kBN = 128;          // keys per KV tile
static constexpr int kD = 128;           // head_dim
static constexpr int kHalfBytes = 128 * 128;           // [128 rows][64 bf16]: one swizzled half tile
static constexpr int kTileBytes = 2 * kHalfBytes;       // 32 KiB: a Q, K or V tile
static constexpr int kStages = 2;
static constexpr int kThreads = 384;
static constexpr float kRescaleThreshold = 8.f;        // log2 units
// Register re-partition (setmaxnreg): the CTA owns kLaunchRegs x kThreads registers.  Warps 0-3 drop to
// kRegsUtil, warps 4-11 rise to kRegsSoftmax.  The raise BLOCKS until the pool has the registers, so
// the split must fit the CTA's own allocation exactly -- nothing else bounds that wait.
static constexpr int kLaunchRegs = 168, kRegsUtil = 72, kRegsSoftmax = 216;
static_assert(128 * kRegsUtil + 256 * kRegsSoftmax <= kLaunchRegs * kThreads, "setmaxnreg split exceeds the CTA's registers");
static_assert(kLaunchRegs * kThreads <= 65536 && kRegsUtil % 8 == 0 && kRegsSoftmax % 8 == 0, "register split");

// shared-memory map (offsets from the 1024-byte aligned base)
static constexpr int kOffQ = 0;                                   // Q_A, Q_B
static constexpr int kOffK = kOffQ + 2 * kTileBytes;              // K stages
static constexpr int kOffV = kOffK + kStages * kTileBytes;        // V stages
static constexpr int kOffBar = kOffV + kStages * kTileBytes;      // mbarriers
static constexpr int kSmemBytes = kOffBar + 256 + 1024;           // + alignment slack

// barrier slots (8 bytes each)
enum Bar { Q_READY = 0, K_FULL = 1, K_EMPTY = 3, V_FULL = 5, V_EMPTY = 7, S_READY = 9, P_READY = 11, DRAIN = 13, P_PART = 14, NBAR = 16 };

// TMEM columns
__device__ __forceinline__ constexpr uint32_t col_s(int x) { return 128u * (uint32_t)x; }
__device__ __forceinline__ constexpr uint32_t col_o(int x) { return 256u + 128u * (uint32_t)x; }

// kind::f16 instruction descriptor: D = f32, A = B = bf16, M = 128, N = 128
static constexpr uint32_t kIdescBase = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
static constexpr uint32_t kIdescQK = kIdescBase;               // A, B both K-major
static constexpr uint32_t kIdescPV = kIdescBase | (1u << 16);  // B (= V) is MN-major

// The single MMA-issuing thread is the pace-setter of the whole CTA, so its instruction count per MMA matters:
// every shared-memory descriptor used here has the same upper word (stride byte offset 1024, version 1, 128-byte
// swizzle), and the lower word is (address >> 4) | (leading byte offset >> 4) << 16, so stepping through a tile
// is one 32-bit add per operand.
static constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t desc_lo(uint32_t addr, uint32_t lbo_bytes) {
    return ((addr >> 4) & 0x3FFFu) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
}
// These three are executed by the WHOLE (converged) issuing warp with warp-uniform operands; one lane, picked by
// elect.sync inside the block, issues the instruction.  Written this way the operands can live in uniform
// registers; wrapped in `if (lane == 0)` they are per-thread values that have to be moved over one by one.
template <bool kAcc>
__device__ __forceinline__ void mma_ss_lo(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc) {
    asm volatile(
        "{\n\t.reg .pred p, e;\n\t.reg .b64 da, db;\n\telect.sync _|e, 0xffffffff;\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
        "@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(kDescHi), "r"(idesc), "n"(kAcc ? 1 : 0)
        : "memory");
}
__device__ __forceinline__ void mma_ts_lo_dyn(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p, e;\n\t.reg .b64 db;\n\telect.sync _|e, 0xffffffff;\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(kDescHi), "r"(idesc), "r"(acc)
        : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile(
        "{\n\t.reg .pred e;\n\telect.sync _|e, 0xffffffff;\n\t"
        "@e tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}" ::"r"(bar)
        : "memory");
}
__device__ __forceinline__ void fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld32(float (&v)[32], uint32_t taddr) {
    uint32_t r[32];
    cp::tcgen05_ld_32x32b(r, taddr);
    cp::tcgen05_wait_ld();
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&v)[32]) {
    uint32_t r[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(v[i]);
    cp::tcgen05_st_32x32b(taddr, r);
}

static constexpr int kPartSteps = 6;  // PV k-steps (16 keys each) covered by the early P_PART arrival (even, 2..6)

struct Shared {
    uint32_t base;      // shared-window address of the aligned base
    uint8_t *ptr;       // generic pointer to the same place
    __device__ __forceinline__ uint32_t bar(int i) const { return base + kOffBar + 8 * i; }
    __device__ __forceinline__ volatile int *abort_flag() const { return (volatile int *)(ptr + kOffBar + 8 * NBAR); }
    __device__ __forceinline__ uint32_t *tmem_slot() const { return (uint32_t *)(ptr + kOffBar + 8 * NBAR + 8); }
    // Per-tile mask of key blocks whose shared-memory rows hold stand-in data.  Ring of 4: the K producer
    // may run two tiles ahead of the softmax warps (it only waits for the QK MMAs), so a slot per STAGE
    // would be overwritten before the softmax of the older tile has read it.
    __device__ __forceinline__ volatile int *bad_mask(int tile) const { return (volatile int *)(ptr + kOffBar + 8 * NBAR + 16 + 4 * (tile & 3)); }
};

// Bounded wait that also gives up as soon as another role has flagged an abort.
__device__ __forceinline__ bool wait_or_abort(const Shared &sh, int bar, uint32_t parity, unsigned *status, int *abort_word) {
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

// Warp-uniform form: every lane polls, all lanes agree on the outcome (the roles use warp-collective
// instructions afterwards, so a warp must leave its loop as a whole).
__device__ __forceinline__ bool wait_warp(const Shared &sh, int bar, uint32_t parity, unsigned *status, int *abort_word) {
    return __all_sync(0xffffffffu, wait_or_abort(sh, bar, parity, status, abort_word));
}

__global__ void __launch_bounds__(kThreads, 1) prefill_tc_kernel(const __grid_constant__ CUtensorMap kvmap,
                                                                 const PrefillParams p) {
    // a CTA of an earlier wave of this launch already timed out: do not start more work (the flag lives
    // in device memory and is cleared by the launcher; the host-mapped status word is never polled here)
    if (*(volatile int *)p.abort_word) return;

    // ---- which (request, 128-row tile, head pair)?  Heaviest (latest) tiles first.
    const int tile_idx = gridDim.x - 1 - blockIdx.x;
    const int pair = blockIdx.y;
    const int head0 = 2 * pair;
    const int g = head0 / p.group;
    int req = 0, acc_tiles = 0, c_r = 0, q0 = 0;
    if (!find_request(p, tile_idx, kBM, req, acc_tiles, q0, c_r)) return;
    const int row0 = (tile_idx - acc_tiles) * kBM;
    const int L = min(p.seq_lens[req], p.max_blocks * 16);
    const int prefix = L - c_r;
    const int rows_here = min(kBM, c_r - row0);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const size_t row_stride = (size_t)p.num_q_heads * kD;

    if (prefix < 0) {  // malformed request: zero rows, latch
        if (threadIdx.x == 0) atomicOr(p.status, EKV_DEV_FLAG_OOB);
        for (int e = threadIdx.x; e < rows_here * 2 * kD; e += kThreads) {
            const int row = e / (2 * kD), x = e % (2 * kD);
            p.out[((size_t)(q0 + row0 + row)) * row_stride + (size_t)head0 * kD + x] = __float2bfloat16_rn(0.f);
        }
        return;
    }
    const int kv_end = min(L, prefix + row0 + rows_here);  // keys any row of this tile may see
    const int n_tiles = (kv_end + kBN - 1) / kBN;
    const int n_blocks = (kv_end + 15) >> 4;

    extern __shared__ uint8_t smem_raw[];
    Shared sh;
    {
        const uint32_t raw = smem_u32(smem_raw);
        sh.base = (raw + 1023u) & ~1023u;
        sh.ptr = smem_raw + (sh.base - raw);
    }

    if (threadIdx.x == 0) {
        prefetch_tensormap(&kvmap);
        mbar_init(sh.bar(Q_READY), 256);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(sh.bar(K_FULL + s), 1);
            mbar_init(sh.bar(K_EMPTY + s), 1);
            mbar_init(sh.bar(V_FULL + s), 1);
            mbar_init(sh.bar(V_EMPTY + s), 1);
        }
        for (int x = 0; x < 2; ++x) {
            mbar_init(sh.bar(S_READY + x), 1);
            mbar_init(sh.bar(P_READY + x), 128);
            mbar_init(sh.bar(P_PART + x), 128);
        }
        mbar_init(sh.bar(DRAIN), 1);
        *sh.abort_flag() = 0;
        mbar_fence_init();
    }
    if (warp == 2) {
        cp::tcgen05_alloc(cp::cta_group_1, sh.tmem_slot(), 512);
        cp::tcgen05_relinquish_alloc_permit(cp::cta_group_1);
    }
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem = *sh.tmem_slot();

    if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
    if (warp == 0 || warp == 2) {
        // =========================== TMA producers: warp 0 feeds K tiles, warp 2 feeds V tiles ===========
        // (a TMA issue costs the issuing warp ~100 cycles, 16 boxes per tile: two warps keep up with the MMAs)
        const bool is_v = warp == 2;
        const int FULL = is_v ? V_FULL : K_FULL, EMPTY = is_v ? V_EMPTY : K_EMPTY;
        const uint32_t tile_base = sh.base + (is_v ? kOffV : kOffK);
        const int kv_row_off = is_v ? p.num_kv_heads * 16 : 0;
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
        for (int j = 0; j < n_tiles; ++j) {
            const int s = j % kStages;
            const int id_raw = id_next;
            if (j + 1 < n_tiles) id_next = load_id(j + 1);
            const unsigned oob = __ballot_sync(0xffffffffu, id_raw == -2) & 0xffu;
            // blocks whose smem rows will hold stand-in data: invalid ids and blocks past the last visible key
            const unsigned bad = __ballot_sync(0xffffffffu, id_raw < 0) & 0xffu;
            const int id = id_raw < 0 ? 0 : id_raw;  // masked later; block 0 is always mapped
            // box b of a tile: block b/2, channel half b%2  ->  [half][block][16 rows][128 B]
            const int b = lane & 15, blk = b >> 1, half = b & 1;
            const int my_id = __shfl_sync(0xffffffffu, id, blk);
            const int row = g * 16 + kv_row_off;  // row inside the block: (K|V, kv-head, token)
            if (j >= kStages && !wait_warp(sh, EMPTY + s, (uint32_t)(((j / kStages) - 1) & 1), p.status, p.abort_word)) break;
            if (lane == 0) {
                if (!is_v) {
                    if (oob) atomicOr(p.status, EKV_DEV_FLAG_OOB);
                    *sh.bad_mask(j) = (int)bad;
                }
                mbar_expect_tx(sh.bar(FULL + s), kTileBytes);
            }
            __syncwarp();
            if (lane < 16)
                tma_load_3d(tile_base + s * kTileBytes + half * kHalfBytes + blk * 2048, &kvmap, 64 * half, row, my_id, sh.bar(FULL + s));
        }
    } else if (warp == 1) {
        // =========================== MMA issuer ===========================
        // descriptor low words of the tile origins; stepping inside a tile adds a compile-time constant
        const uint32_t q_lo[2] = {desc_lo(sh.base + kOffQ, 16), desc_lo(sh.base + kOffQ + kTileBytes, 16)};
        const uint32_t k_lo0 = desc_lo(sh.base + kOffK, 16), v_lo0 = desc_lo(sh.base + kOffV, kHalfBytes);
        auto issue_qk = [&](int x, int s) {  // S_x = Q_x K(s)^T
            const uint32_t k_lo = k_lo0 + (uint32_t)s * (kTileBytes >> 4);
#pragma unroll
            for (int k = 0; k < kD / 16; ++k) {
                const uint32_t off = ((k >> 2) * kHalfBytes + (k & 3) * 32) >> 4;
                if (k == 0) mma_ss_lo<false>(tmem + col_s(x), q_lo[x] + off, k_lo + off, kIdescQK);
                else mma_ss_lo<true>(tmem + col_s(x), q_lo[x] + off, k_lo + off, kIdescQK);
            }
        };
        auto issue_pv = [&](int x, int s, bool acc, int k0, int k1) {  // O_x (+)= P_x[:, 16k0:16k1] V(s)[16k0:16k1, :]
            const uint32_t v_lo = v_lo0 + (uint32_t)s * (kTileBytes >> 4);
#pragma unroll
            for (int k = k0; k < k1; ++k)
                mma_ts_lo_dyn(tmem + col_o(x), tmem + col_s(x) + 8 * k, v_lo + ((k * 2048) >> 4), kIdescPV, (acc || k > 0) ? 1u : 0u);
        };
        bool ok = wait_warp(sh, Q_READY, 0, p.status, p.abort_word) && wait_warp(sh, K_FULL + 0, 0, p.status, p.abort_word);
        if (ok) {
            fence_after();
            issue_qk(0, 0);
            mma_commit(sh.bar(S_READY + 0));
            issue_qk(1, 0);
            mma_commit(sh.bar(K_EMPTY + 0));
            mma_commit(sh.bar(S_READY + 1));
            for (int j = 0; j < n_tiles && ok; ++j) {
                const int s = j % kStages, s1 = (j + 1) % kStages;
                const bool more = j + 1 < n_tiles;
                ok = wait_warp(sh, V_FULL + s, (uint32_t)((j / kStages) & 1), p.status, p.abort_word);
                if (ok && more) ok = wait_warp(sh, K_FULL + s1, (uint32_t)(((j + 1) / kStages) & 1), p.status, p.abort_word);
                if (ok) ok = wait_warp(sh, P_PART + 0, (uint32_t)(j & 1), p.status, p.abort_word);
                if (!ok) break;
                fence_after();
                issue_pv(0, s, j > 0, 0, kPartSteps);  // keys 0..95 while the softmax warps finish the rest
                ok = wait_warp(sh, P_READY + 0, (uint32_t)(j & 1), p.status, p.abort_word);
                if (!ok) break;
                fence_after();
                issue_pv(0, s, true, kPartSteps, kBN / 16);
                if (more) issue_qk(0, s1);
                mma_commit(sh.bar(S_READY + 0));
                ok = wait_warp(sh, P_PART + 1, (uint32_t)(j & 1), p.status, p.abort_word);
                if (!ok) break;
                fence_after();
                issue_pv(1, s, j > 0, 0, kPartSteps);
                ok = wait_warp(sh, P_READY + 1, (uint32_t)(j & 1), p.status, p.abort_word);
                if (!ok) break;
                fence_after();
                issue_pv(1, s, true, kPartSteps, kBN / 16);
                mma_commit(sh.bar(V_EMPTY + s));
                if (more) {
                    issue_qk(1, s1);
                    mma_commit(sh.bar(K_EMPTY + s1));
                }
                mma_commit(sh.bar(S_READY + 1));
            }
        }
        // every MMA this thread issued must be finished before TMEM is released
        mma_commit(sh.bar(DRAIN));
        (void)wait_warp(sh, DRAIN, 0, p.status, p.abort_word);
    }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
        // =========================== softmax + epilogue ===========================
        const int x = (warp - 4) >> 2;                  // 0 = head A, 1 = head B
        const int row = ((warp & 3) << 5) | lane;        // query row in the tile = TMEM lane
        const int head = head0 + x;
        const uint32_t lane_base = (uint32_t)((warp & 3) << 5) << 16;
        const uint32_t t_s = tmem + lane_base + col_s(x);
        const uint32_t t_o = tmem + lane_base + col_o(x);

        // ---- stage this head's Q tile (128-byte swizzle).  Each warp brings in the 32 rows it will own, two rows per
        // instruction: 16 lanes cover the 256 contiguous bytes of a row, so global loads are fully coalesced
        // (one row per lane would touch 32 cache lines per instruction and cost microseconds per CTA).
        const int wrow0 = (warp & 3) << 5;
        {
            uint8_t *qdst = sh.ptr + kOffQ + x * kTileBytes;
            const int c16 = lane & 15;
            const __nv_bfloat16 *src = p.q + ((size_t)(q0 + row0)) * row_stride + (size_t)head * kD + c16 * 8;
            uint4 v[16];
#pragma unroll
            for (int it = 0; it < 16; ++it) {
                const int rr = wrow0 + 2 * it + (lane >> 4);
                v[it] = rr < rows_here ? *reinterpret_cast<const uint4 *>(src + (size_t)rr * row_stride) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int it = 0; it < 16; ++it) {
                const int rr = wrow0 + 2 * it + (lane >> 4);
                *reinterpret_cast<uint4 *>(qdst + (c16 >> 3) * kHalfBytes + rr * 128 + (((c16 & 7) ^ (rr & 7)) << 4)) = v[it];
            }
            fence_proxy_async_smem();
            mbar_arrive(sh.bar(Q_READY));
        }

        const int lim = prefix + row0 + min(row, rows_here - 1);  // last key this row may see
        float m_run = -INFINITY, l_run = 0.f;
        bool ok = true;
        for (int j = 0; j < n_tiles; ++j) {
            const int s = j % kStages;
            ok = wait_warp(sh, S_READY + x, (uint32_t)(j & 1), p.status, p.abort_word);
            if (!ok) break;
            fence_after();
            const int key0 = j * kBN;
            const int bad = *sh.bad_mask(j);
            const bool need_mask = (key0 + kBN - 1 > prefix + row0) || bad != 0;
            // keys of this tile that lie past the sequence end, or in a skipped block, may hold anything
            // (unwritten slots): their V rows must not reach the tensor pipe, because 0 * NaN = NaN
            const bool dirty_v = (key0 + kBN > L) || bad != 0;
            if (dirty_v && x == 0) {
                ok = wait_warp(sh, V_FULL + s, (uint32_t)((j / kStages) & 1), p.status, p.abort_word);
                if (!ok) break;
                uint8_t *vdst = sh.ptr + kOffV + s * kTileBytes;
                if ((key0 + row >= L) || ((bad >> (row >> 4)) & 1)) {  // thread `row` owns key row `row` of the tile
#pragma unroll
                    for (int h2 = 0; h2 < 2; ++h2)
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
            const bool raise = m_tile > m_run + kRescaleThreshold;  // also true for the first finite tile
            if (__any_sync(0xffffffffu, raise)) {
                const float m_new = raise ? m_tile : m_run;
                const float alpha = (raise && m_run > -INFINITY) ? fast_exp2(m_run - m_new) : (raise ? 0.f : 1.f);
                m_run = m_new;
                l_run *= alpha;
                if (j > 0) {  // O holds the sum over earlier tiles and no MMA touches it right now
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        float ov[32];
                        tmem_ld32(ov, t_o + 32 * cc);
#pragma unroll
                        for (int i = 0; i < 32; ++i) ov[i] *= alpha;
                        tmem_st32(t_o + 32 * cc, ov);
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
                if (cc == kPartSteps / 2 - 1) {  // 96 keys stored
                    cp::tcgen05_wait_st();
                    fence_before();
                    mbar_arrive(sh.bar(P_PART + x));
                }
            }
            l_run += (acc_a.x + acc_a.y) + (acc_b.x + acc_b.y);
            cp::tcgen05_wait_st();
            fence_before();
            mbar_arrive(sh.bar(P_READY + x));
        }

        // ---- epilogue: O / l -> bf16 -> this head's (now idle) Q tile in shared memory -> global.  A thread holds a
        // whole row; writing it out directly would again touch 32 cache lines per instruction.  Each warp stages its
        // 32 rows (16-byte pieces XOR-swizzled by row: no bank conflicts either way) and writes them back two rows
        // per instruction, 256 contiguous bytes each.  Only the warp that wrote a row reads it: __syncwarp suffices.
        if (ok) ok = wait_warp(sh, S_READY + x, (uint32_t)(n_tiles & 1), p.status, p.abort_word);
        if (ok) {
            fence_after();  // every MMA that read this Q tile has completed (the commit covers all earlier ones)
            const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
            uint8_t *stage = sh.ptr + kOffQ + x * kTileBytes;
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                float ov[32];
                tmem_ld32(ov, t_o + 32 * cc);
#pragma unroll
                for (int i = 0; i < 32; i += 8) {
                    uint4 v;
                    v.x = pack_bf16x2(ov[i] * inv, ov[i + 1] * inv);
                    v.y = pack_bf16x2(ov[i + 2] * inv, ov[i + 3] * inv);
                    v.z = pack_bf16x2(ov[i + 4] * inv, ov[i + 5] * inv);
                    v.w = pack_bf16x2(ov[i + 6] * inv, ov[i + 7] * inv);
                    const int piece = cc * 4 + (i >> 3);
                    *reinterpret_cast<uint4 *>(stage + row * 256 + ((piece ^ (row & 15)) << 4)) = v;
                }
            }
            __syncwarp();
            const int piece = lane & 15;
            __nv_bfloat16 *dst = p.out + ((size_t)(q0 + row0)) * row_stride + (size_t)head * kD + piece * 8;
#pragma unroll
            for (int it = 0; it < 16; ++it) {
                const int rr = wrow0 + 2 * it + (lane >> 4);
                const uint4 v = *reinterpret_cast<const uint4 *>(stage + rr * 256 + ((piece ^ (rr & 15)) << 4));
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
            (void)mbar_wait(sh.bar(K_FULL + j % kStages), (uint32_t)((j / kStages) & 1), 100000000ull);
            (void)mbar_wait(sh.bar(V_FULL + j % kStages), (uint32_t)((j / kStages) & 1), 100000000ull);
        }
    }
    __syncthreads();
    if (warp == 2) cp::tcgen05_dealloc(cp::cta_group_1, tmem, 512);
}

static ekv_status_t launch_prefill_tc(ekv_pool *pool, int layer, const PrefillParams &p, int q_tiles, cudaStream_t stream) {
    static bool attr_set[64] = {false};
    const int dev = pool->desc.device;
    if (dev >= 64 || !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(prefill_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return cuda_fail(e, "ekv_attn_prefill_chunk: shared-memory attribute");
        if (dev < 64) attr_set[dev] = true;
    }
    dim3 grid(q_tiles, pool->desc.num_q_heads / 2);
    cudaError_t e0 = cudaMemsetAsync(p.abort_word, 0, sizeof(int), stream);
    if (e0 != cudaSuccess) return cuda_fail(e0, "ekv_attn_prefill_chunk: clear abort word");
    prefill_tc_kernel<<<grid, kThreads, kSmemBytes, stream>>>(pool->kv_map[layer], p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "ekv_attn_prefill_chunk: launch");
    return EKV_OK;
}

}  // namespace tc
}  // namespace ekv
