// Chunked-prefill attention on the 5th-generation tensor cores (tcgen05.mma, accumulators in TMEM),
// head_dim 128, query groups of two or more heads.  PERSISTENT: one CTA per SM walks a list of work
// items.
//
// Work item = 128 query positions of one request x TWO query heads (A, B) that share a kv-head, so
// every K/V tile staged in shared memory feeds two 128x128 score tiles (ping-pong: while the
// softmax warps work on one head's scores the tensor pipe runs the other head's MMAs).  A kv group
// with an odd number of query heads (7 for a 28 / 4 model) is cut into pairs and ONE item of a single
// head, which head B's warps sit out; the barriers of a head then count that head's own tiles and
// items, and where a head's last PV and its next first QK^T are no longer one commit the roles take
// care not to wait on a phase parity from two completions away (notes at those places).  Items are
// ordered head pair by head pair and, inside a pair, from the heaviest (latest) query tile to the
// lightest, and are handed out dynamically: warp 3 draws item numbers from a counter in device
// memory and posts them in a small ring in shared memory, from which every role of the CTA reads
// its next item (longest-first greedy scheduling; a static round-robin would give CTA c the same
// position of every request whenever the request length divides the grid).  All roles walk that
// list independently and are only coupled through mbarriers, so the end of one item overlaps the
// start of the next:
// the Q tiles and first K/V tiles of item i+1 are in flight during the last tiles of item i, the
// first QK^T of item i+1 is issued right behind the last PV of item i, and the write-out of item i
// runs while the tensor pipe already works on item i+1.  TMEM and the barriers are set up once.
//
//   warp 0        TMA producer of K tiles: 16-token x 64-channel boxes (128-byte swizzle) of the
//                 blocks the table names, gathered into 128-key tiles, 2 stages
//   warp 1        MMA issuer (whole warp converged, one elected lane issues): S = Q K^T (A, B from
//                 shared memory, K-major) and O += P V (A = P read from TMEM, B = V from shared
//                 memory, MN-major)
//   warp 2        TMA producer of V tiles, 2 stages; TMEM allocation / release (512 columns:
//                 S_A S_B O_A O_B, P aliases S)
//   warp 3        item scheduler; TMA producer of the two Q tiles of an item (one tensor map over
//                 the query tensor)
//   warps 4-7     softmax of head A: one thread per query row (= TMEM lane)
//   warps 8-11    softmax of head B
//   warps 12-15   write-out of both heads (O / l -> bf16 -> global, TMA stores), one warp per quarter
//                 of the TMEM lanes: the softmax warps go from an item's last key tile straight to
//                 the next item's first
//
// The code is kept SMALL on purpose.  Each quarter of the SM has an instruction cache of about 32 KB
// for its four warps (measured: straight-line code runs at 1.0-1.2 cycles per instruction up to that
// footprint and at 2.7 beyond it).  An item of a short request is a few key tiles long, so every role
// walks through all of its code every few thousand cycles; what does not fit is fetched again for
// every item.  Hence one copy of the MMA issuing loop, waits whose slow path is one out-of-line
// function, rare paths as small loops, and one copy of the softmax code (a tile cut by the causal
// boundary has its hidden scores set to -inf in TMEM first).
//
// Softmax is online in the exp2 domain with LAZY rescaling: the running reference max of a row is
// only raised (and O, l rescaled in TMEM) when a tile's max exceeds it by more than 2^8, so P stays
// below 256 and most tiles need no pass over O.  All mbarrier waits are bounded; a wait that runs
// out latches EKV_ERR_TIMEOUT, makes every role leave its loops, and the CTA still drains its
// copies, releases TMEM and exits.
#pragma once
#include <cuda/ptx>
#include <cuda_bf16.h>
#include <math.h>

#include <type_traits>

#include "ekv_internal.h"
#include "ekv_prefill_mma.cuh"  // PrefillParams
#include "ptx.cuh"

#ifndef EKV_TC_PAIR_GROUP
#define EKV_TC_PAIR_GROUP 0
#endif
#ifndef EKV_TC_ITEM_AHEAD
#define EKV_TC_ITEM_AHEAD 1
#endif

namespace ekv {
namespace tc {

namespace cp = cuda::ptx;

static constexpr int kBM = 128;          // query rows per head tile
static constexpr int kBN = 128;          // keys per KV tile
static constexpr int kD = 128;           // head_dim
static constexpr int kHalfBytes = 128 * 128;           // [128 rows][64 bf16]: one swizzled half tile
static constexpr int kTileBytes = 2 * kHalfBytes;       // 32 KiB: a Q, K or V tile
static constexpr int kStages = 2;
static constexpr int kThreads = 512;
static constexpr float kRescaleThreshold = 8.f;        // log2 units
// Register re-partition (setmaxnreg): the CTA owns kLaunchRegs x kThreads registers.  Warps 0-3 (utility) and 12-15
// (write-out) drop to kRegsUtil / kRegsOut, warps 4-11 (softmax) rise to kRegsSoftmax.  The raise BLOCKS until the pool
// has the registers, so the split must fit the CTA's own allocation exactly -- nothing else bounds that wait -- and
// every warpgroup (four consecutive warps from a multiple of four) must ask for the same thing.
static constexpr int kLaunchRegs = 128, kRegsUtil = 72, kRegsSoftmax = 184, kRegsOut = 72;
static_assert(128 * (kRegsUtil + kRegsOut) + 256 * kRegsSoftmax <= kLaunchRegs * kThreads, "setmaxnreg split exceeds the CTA's registers");
static_assert(kLaunchRegs * kThreads <= 65536 && kRegsUtil % 8 == 0 && kRegsSoftmax % 8 == 0 && kRegsOut % 8 == 0, "register split");
static_assert(kRegsUtil == 72 && kRegsSoftmax == 184 && kRegsOut == 72, "the setmaxnreg instructions in the kernel carry these numbers as literals");

// shared-memory map (offsets from the 1024-byte aligned base)
static constexpr int kOffQ = 0;                                   // Q_A, Q_B
static constexpr int kOffK = kOffQ + 2 * kTileBytes;              // K stages
static constexpr int kOffV = kOffK + kStages * kTileBytes;        // V stages
static constexpr int kOffStage = kOffV + kStages * kTileBytes;    // write-out staging: 4 write-out warps x 2 x [32 rows][128 B]
static constexpr int kStageBytes = 32 * 128;
static constexpr int kOffBar = kOffStage + 8 * kStageBytes;       // mbarriers
static constexpr int kOffInvL = kOffBar + 512;                     // 1 / row sum of the finished item: [2 heads][128 rows] floats
static constexpr int kSmemBytes = kOffInvL + 1024 + 64 + 1024;         // barriers, flags, item ring; row sums; + alignment slack
static_assert(kSmemBytes <= 232448, "shared memory of one CTA");

// barrier slots (8 bytes each)
static constexpr int kItemRing = 4;   // item numbers posted ahead of the slowest role
static constexpr int kItemAhead = EKV_TC_ITEM_AHEAD;  // the scheduler keeps this many items posted beyond the one whose Q it loads
enum Bar { Q_FULL = 0, Q_EMPTY = 2, K_FULL = 4, K_EMPTY = 6, V_FULL = 8, V_EMPTY = 10, S_READY = 12, P_READY = 14, P_PART = 16,
           O_FREE = 18, DRAIN = 20, L_READY = 21, ITEM_READY = 23, NBAR = ITEM_READY + kItemRing };
static_assert(8 * NBAR + 32 <= 256, "barrier area");

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
// One lane of the (converged) issuing warp, picked by elect.sync, issues a whole run of MMAs from inside a branch.
// In that form the descriptors are 64-bit values that step by a compile-time constant and the compiler keeps them in
// uniform registers: about three instructions per MMA.  (One elect per MMA with the operands put together inside the
// asm block costs twice that, a plain `if (lane == 0)` nearly three times.  The issuing thread sets the pace of the CTA,
// a 128x128x16 MMA occupies the tensor pipe for only 64 cycles, and the code has to stay small: see below.)
__device__ __forceinline__ bool elect_one() {
    uint32_t e;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(e));
    return e != 0;
}
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
// Older form, one elect per MMA (the one-head kernels still use it).
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
// the same from inside a branch that one elected lane has taken
__device__ __forceinline__ void mma_commit_one(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
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
    // Per-tile mask of key blocks whose shared-memory rows hold stand-in data.  Ring of 4, indexed by the CTA's running
    // key-tile count: the K producer may run two tiles ahead of the softmax warps (it only waits for the QK MMAs), so a
    // slot per STAGE would be overwritten before the softmax of the older tile has read it.
    __device__ __forceinline__ volatile int *bad_mask(int tile) const { return (volatile int *)(ptr + kOffBar + 8 * NBAR + 16 + 4 * (tile & 3)); }
    // Every softmax and write-out warp (12 of them) keeps, in a word of its own, the number of items it is through with, and
    // the scheduler gives a ring slot to a new item once ALL twelve are past the old one.  Not an mbarrier: the scheduler
    // looks only when it needs a slot back, possibly a few items later, and a phase parity cannot tell "not yet" from "two
    // phases ago".  Not one shared count either: the warps of head B skip the items that have one head, and a sum would
    // let their lead pay for a warp that lags.
    __device__ __forceinline__ volatile int *items_done(int w12) const { return (volatile int *)(ptr + kOffInvL + 1024) + w12; }
    __device__ __forceinline__ float *inv_l(int x) const { return (float *)(ptr + kOffInvL) + 128 * x; }
    // items posted by the scheduler: slot k % kItemRing holds the CTA's k-th item
    __device__ __forceinline__ uint4 *item_slot(int k) const { return (uint4 *)(ptr + kOffBar + 256 + 64 * (k % kItemRing)); }
};

// Bounded wait of a whole warp (every lane polls, all lanes agree on the outcome: the roles use warp-collective
// instructions afterwards, so a warp must leave its loop as a whole).  Nearly every wait is over within its first poll
// (a poll sleeps in hardware until the phase completes or a time limit passes), so that case is one poll and a vote.
// Otherwise the warp goes on polling in a loop of a dozen instructions, written in PTX so that it stays that small:
// there are dozens of waits, and the kernel's code has to fit the instruction caches (with the loop, a clock and the
// give-up path written out in C++ at each, the waits were the largest part of the issuing warp's code; as a call to one
// out-of-line copy they cost register spills around every call).  The loop gives up as soon as another role of the CTA
// has given up.  Its bound is a number of polls: a failed mbarrier.try_wait sleeps about 1.5 us on this part (measured:
// 2900 cycles a poll, whatever the number of polling warps), so kPollLimit polls are about three seconds.  A wait that
// runs out leaves 2 in the CTA's abort flag; the teardown turns that into EKV_ERR_TIMEOUT.
static constexpr uint32_t kPollLimit = 1u << 21;
__device__ __forceinline__ bool wait_warp(const Shared &sh, int bar, uint32_t parity) {
    if (__all_sync(0xffffffffu, mbar_try_wait(sh.bar(bar), parity))) return true;  // the usual case: over within the first poll
    return __all_sync(0xffffffffu, mbar_wait_polls(sh.bar(bar), parity, sh.base + kOffBar + 8 * NBAR, kPollLimit));
}

// One work item.  The scheduler decodes it (that takes dependent reads of device memory) and posts it in the ring;
// every role then reads the same 48 bytes from shared memory.
struct Item {
    int req;        // request
    int qrow;       // row of the query / output tensor where the tile starts
    int prow;       // absolute position (prefix + row inside the chunk) of the tile's first row
    int rows_here;  // rows of the tile that belong to the request (1..128)
    int L, n_tiles, n_blocks;  // keys of the request; key tiles / blocks any row of this tile may see
    int head0, g;   // first of the two query heads; their kv-head
    int nh;         // query heads of the item: 2, or 1 for the odd head of a kv group with an odd number of query heads
    int malformed;  // seq_len shorter than the chunk: the scheduler zero-fills the rows itself and never posts the item
    int state;      // kItemWork, or kItemEnd: the list of this CTA ends here
};
static constexpr int kItemWork = 1, kItemEnd = 2;
static_assert(sizeof(Item) == 48, "item slot");
// Item order: head pairs are taken in groups of kPairGroup (0 = all pairs in one group); inside a group the query tiles
// go from the heaviest (latest) to the lightest and every tile is listed for all pairs of the group before the next
// tile.  One group per launch makes the list globally longest-first (the end of the launch is made of one-tile items,
// so the CTAs finish together); smaller groups keep fewer kv-heads' K/V streaming through L2 at a time.
static constexpr int kPairGroup = EKV_TC_PAIR_GROUP;
__host__ __device__ __forceinline__ int head_pairs(const PrefillParams &p) { return p.num_kv_heads * ((p.group + 1) / 2); }
__device__ __forceinline__ bool decode_item(const PrefillParams &p, int m, Item &it) {
    it.state = kItemWork;
    const int npairs = head_pairs(p);
    const int gp = kPairGroup > 0 ? kPairGroup : npairs;
    const int per_group = p.q_tiles * gp;
    const int grp = m / per_group, r = m - grp * per_group;
    const int in_group = min(gp, npairs - grp * gp);       // the last group may be smaller
    const int rank = r / in_group;
    const int pair = grp * gp + (r - rank * in_group);
    const int tile_idx = p.q_tiles - 1 - rank;              // heaviest (latest) tiles first
    int acc_tiles = 0, c_r = 0, q0 = 0;
    if (!find_request(p, tile_idx, kBM, it.req, acc_tiles, q0, c_r)) return false;
    const int per_kv = (p.group + 1) / 2;  // a kv group of g query heads is g / 2 pairs, plus a single head if g is odd
    it.g = pair / per_kv;
    it.head0 = it.g * p.group + 2 * (pair - it.g * per_kv);
    it.nh = min(2, (it.g + 1) * p.group - it.head0);
    const int row0 = (tile_idx - acc_tiles) * kBM;
    it.L = min(p.seq_lens[it.req], p.max_blocks * 16);
    const int prefix = it.L - c_r;
    it.qrow = q0 + row0;
    it.prow = prefix + row0;
    it.rows_here = min(kBM, c_r - row0);
    it.malformed = prefix < 0 ? 1 : 0;
    const int kv_end = min(it.L, it.prow + it.rows_here);  // keys any row of this tile may see
    it.n_tiles = (kv_end + kBN - 1) / kBN;
    it.n_blocks = (kv_end + 15) >> 4;
    return true;
}

// The CTA's k-th item as posted by the scheduler.  Returns 1 for an item to work on, 0 at the end of the list (or for
// an item that names no request), -1 if the wait was given up.
__device__ __forceinline__ int fetch_item(const Shared &sh, int k, Item &it) {
    const bool got = wait_warp(sh, ITEM_READY + k % kItemRing, (uint32_t)((k / kItemRing) & 1));
    if (!got) return -1;
    const uint4 *src = sh.item_slot(k);
    const uint4 a = src[0], b = src[1], c = src[2];  // field by field: the struct stays in registers
    it.req = (int)a.x, it.qrow = (int)a.y, it.prow = (int)a.z, it.rows_here = (int)a.w;
    it.L = (int)b.x, it.nh = (int)b.y, it.n_tiles = (int)b.z, it.n_blocks = (int)b.w;
    it.head0 = (int)c.x, it.g = (int)c.y, it.malformed = (int)c.z, it.state = (int)c.w;
    return it.state == kItemWork ? 1 : 0;
}

// kSingles: the call has items of ONE head (a kv group with an odd number of query heads); the instantiation for even
// groups carries none of the bookkeeping for a head that sits items out.
template <bool kSingles>
__global__ void __launch_bounds__(kThreads, 1) prefill_tc_kernel(const __grid_constant__ CUtensorMap kvmap,
                                                                 const __grid_constant__ CUtensorMap qmap,
                                                                 const __grid_constant__ CUtensorMap omap,
                                                                 const PrefillParams p) {
    // a CTA of this launch already timed out: do not start more work (the flag lives in device memory and is
    // cleared by the launcher; the host-mapped status word is never polled here)
    if (*(volatile int *)p.abort_word) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const size_t row_stride = (size_t)p.num_q_heads * kD;
    const int n_items = p.q_tiles * head_pairs(p);

    extern __shared__ uint8_t smem_raw[];
    Shared sh;
    {
        const uint32_t raw = smem_u32(smem_raw);
        sh.base = (raw + 1023u) & ~1023u;
        sh.ptr = smem_raw + (sh.base - raw);
    }

    if (threadIdx.x == 0) {
        prefetch_tensormap(&kvmap);
        prefetch_tensormap(&qmap);
        prefetch_tensormap(&omap);
        for (int x = 0; x < 2; ++x) {
            mbar_init(sh.bar(Q_FULL + x), 1);
            mbar_init(sh.bar(Q_EMPTY + x), 1);
            mbar_init(sh.bar(S_READY + x), 1);
            mbar_init(sh.bar(P_READY + x), 128);
            mbar_init(sh.bar(P_PART + x), 128);
            mbar_init(sh.bar(O_FREE + x), 4);
            mbar_init(sh.bar(L_READY + x), 128);
        }
        for (int s = 0; s < kStages; ++s) {
            mbar_init(sh.bar(K_FULL + s), 1);
            mbar_init(sh.bar(K_EMPTY + s), 1);
            mbar_init(sh.bar(V_FULL + s), 1);
            mbar_init(sh.bar(V_EMPTY + s), 1);
        }
        mbar_init(sh.bar(DRAIN), 1);
        for (int i = 0; i < kItemRing; ++i) mbar_init(sh.bar(ITEM_READY + i), 1);
        for (int w = 0; w < 12; ++w) *sh.items_done(w) = 0;
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
    // what this warp has put in flight (producers only): the teardown of an aborted CTA waits for the last of it
    int tiles_issued = 0;

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
        int t = 0;  // tiles issued so far (all items): stage t % kStages, use number t / kStages of that stage
        bool ok = true;
        for (int k = 0; ok; ++k) {
            Item it;
            if (fetch_item(sh, k, it) <= 0) break;
            const int *bt = p.block_tables + (size_t)it.req * p.max_blocks;
            auto load_id = [&](int j) {  // lane l: id of block 8j + l%8 (-1 past the end, -2 invalid)
                int id = -1;
                const int bi = 8 * j + (lane & 7);
                if (bi < it.n_blocks) {
                    id = bt[bi];
                    if (id < 0 || (long long)id >= live) id = -2;
                }
                return id;
            };
            int id_next = load_id(0);
            for (int j = 0; j < it.n_tiles; ++j, ++t) {
                const int s = t % kStages;
                const int id_raw = id_next;
                if (j + 1 < it.n_tiles) id_next = load_id(j + 1);
                const unsigned oob = __ballot_sync(0xffffffffu, id_raw == -2) & 0xffu;
                // blocks whose smem rows will hold stand-in data: invalid ids and blocks past the last visible key
                const unsigned bad = __ballot_sync(0xffffffffu, id_raw < 0) & 0xffu;
                const int id = id_raw < 0 ? 0 : id_raw;  // masked later; block 0 is always mapped
                // box b of a tile: block b/2, channel half b%2  ->  [half][block][16 rows][128 B]
                const int b = lane & 15, blk = b >> 1, half = b & 1;
                const int my_id = __shfl_sync(0xffffffffu, id, blk);
                const int row = it.g * 16 + kv_row_off;  // row inside the block: (K|V, kv-head, token)
                if (t >= kStages && !wait_warp(sh, EMPTY + s, (uint32_t)(((t / kStages) - 1) & 1))) {
                    ok = false;
                    break;
                }
                if (lane == 0) {
                    if (!is_v) {
                        if (oob) atomicOr(p.status, EKV_DEV_FLAG_OOB);
                        *sh.bad_mask(t) = (int)bad;
                    }
                    mbar_expect_tx(sh.bar(FULL + s), kTileBytes);
                }
                __syncwarp();
                if (lane < 16)
                    tma_load_3d(tile_base + s * kTileBytes + half * kHalfBytes + blk * 2048, &kvmap, 64 * half, row, my_id, sh.bar(FULL + s));
            }
        }
        tiles_issued = t;
    } else if (warp == 3) {
        // =========================== item scheduler + TMA producer of the Q tiles ===========================
        int nq[2] = {0, 0};  // Q tiles of head A / B requested so far (an item with one head has no tile for B)
        int posted = 0;  // item numbers posted so far
        bool ok = true, drained = false;
        int *counter = p.abort_word + 1;  // next item number of the launch (cleared by the launcher with the abort word)
        // Post item numbers up to the CTA's `upto`-th.  Slot k % kItemRing is free again once the CTA's item
        // k - kItemRing is written out: every role has long read it by then.
        auto post_until = [&](int upto) -> bool {
            while (posted <= upto && !drained) {
                if (posted >= kItemRing) {  // the ring slot is free once the 8 softmax and 4 write-out warps are through with item posted - kItemRing
                    const int need = posted - kItemRing + 1;
                    const uint64_t t0 = global_timer_ns();
                    bool got = false;
                    for (uint32_t i = 0; !got; ++i) {
                        got = __all_sync(0xffffffffu, lane >= 12 || *sh.items_done(lane) >= need);
                        if (!got) __nanosleep(100);  // nothing urgent: leave the issue slots to the softmax warp next door
                        if (!got && (i & 31u) == 31u) {
                            if (*sh.abort_flag()) return false;
                            if (global_timer_ns() - t0 > 2000000000ull) {
                                *sh.abort_flag() = 2;
                                return false;
                            }
                        }
                    }
                }
                int m = 0;
                if (lane == 0) m = atomicAdd(counter, 1);
                m = __shfl_sync(0xffffffffu, m, 0);
                Item it;
                it.req = it.qrow = it.prow = it.rows_here = it.L = it.nh = it.n_tiles = it.n_blocks = it.head0 = it.g = it.malformed = 0;
                if (m >= n_items || !decode_item(p, m, it)) it.state = kItemEnd;  // the end marker is posted once; nobody reads past it
                drained = it.state == kItemEnd;
                if (!drained && it.malformed) {
                    // A request with fewer keys than query rows: its rows are zero-filled here and the item is not posted.
                    // (Posted and skipped by every role it tied the ring in a knot: "O of item i is complete" comes with the
                    // first QK^T of the next item that has work, whose Q tile this warp loads only after it has posted one
                    // item more, for which it needs the slot of an item three back -- item i again, if two such items lie in
                    // between.)
                    if (lane == 0) atomicOr(p.status, EKV_DEV_FLAG_OOB);
                    for (int r = 0; r < it.rows_here; ++r)
                        if (lane < 16 * it.nh)  // 256 bytes per head and row; the item's heads are adjacent in a row
                            reinterpret_cast<uint4 *>(p.out + (size_t)(it.qrow + r) * row_stride + (size_t)it.head0 * kD)[lane] = make_uint4(0u, 0u, 0u, 0u);
                    continue;
                }
                if (lane == 0) {
                    uint4 *dst = sh.item_slot(posted);
                    dst[0] = make_uint4((unsigned)it.req, (unsigned)it.qrow, (unsigned)it.prow, (unsigned)it.rows_here);
                    dst[1] = make_uint4((unsigned)it.L, (unsigned)it.nh, (unsigned)it.n_tiles, (unsigned)it.n_blocks);
                    dst[2] = make_uint4((unsigned)it.head0, (unsigned)it.g, (unsigned)it.malformed, (unsigned)it.state);
                    __threadfence_block();
                    mbar_arrive(sh.bar(ITEM_READY + posted % kItemRing));
                }
                ++posted;
            }
            return true;
        };
        for (int k = 0; ok; ++k) {
            ok = post_until(k + kItemAhead);
            if (!ok || k >= posted) break;
            Item it;
            if (fetch_item(sh, k, it) <= 0) break;  // posted by this warp: the wait passes at once
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                if (kSingles && x >= it.nh) break;
                // the last QK^T of this head's previous item has read the tile
                if (nq[x] > 0 && !wait_warp(sh, Q_EMPTY + x, (uint32_t)((nq[x] - 1) & 1))) {
                    ok = false;
                    break;
                }
                if (lane == 0) mbar_expect_tx(sh.bar(Q_FULL + x), kTileBytes);
                __syncwarp();
                if (lane < 2)  // rows past the end of the query tensor read as zero; rows past the request's chunk are never written out
                    tma_load_3d(sh.base + kOffQ + x * kTileBytes + lane * kHalfBytes, &qmap, 64 * lane, it.head0 + x, it.qrow,
                                sh.bar(Q_FULL + x));
                ++nq[x];
            }
        }
        tiles_issued = (nq[0] << 16) | nq[1];
    } else {
        // =========================== MMA issuer ===========================
        // descriptor low words of the tile origins; stepping inside a tile adds a compile-time constant
        const uint32_t q_lo0 = desc_lo(sh.base + kOffQ, 16);
        const uint32_t k_lo0 = desc_lo(sh.base + kOffK, 16), v_lo0 = desc_lo(sh.base + kOffV, kHalfBytes);
        auto issue_pv = [&](int x, int s, bool acc, int k0, int k1) {  // O_x (+)= P_x[:, 16k0:16k1] V(s)[16k0:16k1, :]
            if (elect_one()) {
                const uint64_t v_desc = ((uint64_t)kDescHi << 32) | (v_lo0 + (uint32_t)s * (kTileBytes >> 4));
                const uint32_t d = tmem + col_o(x), a = tmem + col_s(x);
#pragma unroll
                for (int k = k0; k < k1; ++k) mma_ts(d, a + 8 * k, v_desc + ((k * 2048) >> 4), kIdescPV, (acc || k > 0) ? 1u : 0u);
            }
            __syncwarp();
        };
        // The item list of this CTA, one item ahead: the first QK^T of the next item is issued inside the last key tile of
        // the current one.  The loop below is ONE copy of "PV of this key tile, then QK^T of the next key tile" for both
        // heads, every kind of item boundary and the start of the list (an empty item with one tile that has no PV): this
        // warp sets the pace of the CTA and shares an instruction cache with two softmax warps, so its code has to be
        // small.  (Left to itself the compiler unrolls over the heads and clones the loop for each condition that does
        // not change inside it; the values it would do that for pass through an empty asm statement.)
        int k_item = 0;
        bool list_ok = true, list_end = false;
        int cur_tiles = 1, nxt_tiles = 0;  // all this warp needs of an item: its number of key tiles ...
        int cur_heads = 0, nxt_heads = 0;  // ... and of query heads (2, or 1 for the odd head of an odd kv group)
        bool have_nxt = false;
        int t = 0;   // key tiles whose QK^T (both heads) has been issued: the next QK^T reads K stage t % kStages
        int tv = 0;  // key tiles whose PV has been issued
        // Head B sits out the items that have one head, so the barriers of a head count that head's own tiles and items:
        int tvh[2] = {0, 0};  // key tiles of head x whose PV has been issued (P_PART, P_READY)
        int nit[2] = {0, 0};  // items of head x whose first QK^T has been issued (Q_FULL, O_FREE)
        int primed = 0;  // 0 while the "current item" is the empty one in front of the list
        bool ok = true;
        while (ok) {
            have_nxt = false;  // next well-formed item of this CTA, if any
            while (list_ok && !list_end && !have_nxt) {
                Item it;
                const int st = fetch_item(sh, k_item++, it);
                if (st < 0) list_ok = false;
                else if (st == 0) list_end = true;
                else have_nxt = true;
                nxt_tiles = it.n_tiles;
                nxt_heads = it.nh;
            }
            if (!list_ok || (!primed && !have_nxt)) break;
            int have_next = have_nxt ? 1 : 0, pv = primed, heads_now = kSingles ? cur_heads : 2, heads_next = kSingles ? nxt_heads : 2;
            asm volatile("" : "+r"(have_next), "+r"(pv));
            if (kSingles) asm volatile("" : "+r"(heads_now), "+r"(heads_next));
#pragma unroll 1
            for (int j = 0; j < cur_tiles && ok; ++j) {
                const int s = tv % kStages;
                const bool last = j + 1 == cur_tiles;
                const bool new_item = last && have_next;          // the next key tile opens the next item
                const bool more = !last || have_next;             // another key tile follows (this item's or the next one's)
                const int s1 = t % kStages;                       // its stage
                // that tile is the last one of its item: its QK^T is the last reader of the item's Q tile
                const bool next_closes = new_item ? nxt_tiles == 1 : j + 2 == cur_tiles;
                if (pv) ok = wait_warp(sh, V_FULL + s, (uint32_t)((tv / kStages) & 1));
                const int heads_of_next_tile = last ? heads_next : heads_now;  // heads that take part in the QK^T of the next tile
                const int tv_pre = tvh[0], nit_pre = nit[0];  // (without single-head items both heads count alike: one set of counters)
#pragma unroll
                for (int x = 0; x < 2 && ok; ++x) {
                    const bool pv_x = pv && x < heads_now;                 // head x has a PV on this tile
                    const bool more_x = more && x < heads_of_next_tile;    // ... and a QK^T on the next one
                    const bool new_x = new_item && more_x;                 // which opens an item of head x
                    if (!pv_x && !more_x) continue;
                    const int tvx = kSingles ? tvh[x] : tv_pre, nix = kSingles ? nit[x] : nit_pre;
                    if (pv_x) {
                        // O_x still holds the result of head x's previous item until the write-out warps have read it
                        if (j == 0 && nix > 1) ok = wait_warp(sh, O_FREE + x, (uint32_t)((nix - 2) & 1));
                        if (ok) ok = wait_warp(sh, P_PART + x, (uint32_t)(tvx & 1));
                        if (!ok) break;
                        fence_after();
                        issue_pv(x, s, j > 0, 0, kPartSteps);  // keys 0..95 while the softmax warps finish the rest
                        ok = wait_warp(sh, P_READY + x, (uint32_t)(tvx & 1));
                        if (!ok) break;
                    }
                    if (more_x) {
                        // Head x comes back after sitting out an item: the commit below will be a completion of S_READY_x
                        // of its own, right behind the one that said "O_x complete".  The write-out warps must have seen
                        // that one first (a phase parity cannot tell "not yet" from "two completions ago"), and they have
                        // once they have handed O_x back.  (Without a gap the two are one completion, and the next one
                        // needs a PV that waits for O_FREE anyway.)
                        if (kSingles && new_x && !pv_x && nix > 0) ok = wait_warp(sh, O_FREE + x, (uint32_t)((nix - 1) & 1));
                        // a new item: its Q tile of head x must have landed; head A also checks the K tile
                        if (ok && new_x) ok = wait_warp(sh, Q_FULL + x, (uint32_t)(nix & 1));
                        if (ok && x == 0) ok = wait_warp(sh, K_FULL + s1, (uint32_t)((t / kStages) & 1));
                        if (!ok) break;
                    }
                    fence_after();
                    // The rest of the step in one go, by one elected lane: the last quarter of PV, QK^T of the next tile, and
                    // the commits (this is the stretch between "P is there" and "the next scores are there" on every
                    // head's critical chain, so it is as few instructions as it can be).  A K/V stage goes back to its
                    // producer with the commit of the last head that uses it.
                    if (elect_one()) {
                        const uint64_t hi = (uint64_t)kDescHi << 32;
                        if (pv_x) {
                            const uint64_t v_desc = hi | (v_lo0 + (uint32_t)s * (kTileBytes >> 4));
                            const uint32_t d = tmem + col_o(x), a = tmem + col_s(x);
#pragma unroll
                            for (int k = kPartSteps; k < kBN / 16; ++k) mma_ts(d, a + 8 * k, v_desc + ((k * 2048) >> 4), kIdescPV, 1u);
                            if (x == heads_now - 1) mma_commit_one(sh.bar(V_EMPTY + s));
                        }
                        if (more_x) {
                            const uint64_t k_desc = hi | (k_lo0 + (uint32_t)s1 * (kTileBytes >> 4)), q_desc = hi | (q_lo0 + (uint32_t)x * (kTileBytes >> 4));
                            const uint32_t d = tmem + col_s(x);
#pragma unroll
                            for (int k = 0; k < kD / 16; ++k) {
                                const uint32_t off = ((k >> 2) * kHalfBytes + (k & 3) * 32) >> 4;
                                mma_ss(d, q_desc + off, k_desc + off, kIdescQK, k > 0 ? 1u : 0u);
                            }
                            if (next_closes) mma_commit_one(sh.bar(Q_EMPTY + x));
                            if (x == heads_of_next_tile - 1) mma_commit_one(sh.bar(K_EMPTY + s1));
                        }
                        // scores of head x's next tile and / or (after the last tile of an item of head x) O_x complete: when
                        // head x sits out the next item these are two commits, one here and one when it comes back
                        mma_commit_one(sh.bar(S_READY + x));
                    }
                    __syncwarp();
                    if (pv_x && (kSingles || x == 0)) ++tvh[x];
                    if (new_x && (kSingles || x == 0)) ++nit[x];
                }
                if (!ok) break;
                if (pv) ++tv;
                if (more) ++t;
            }
            if (!ok || !have_nxt) break;
            cur_tiles = nxt_tiles;
            cur_heads = nxt_heads;
            primed = 1;
        }
        // every MMA this thread issued must be finished before TMEM is released
        mma_commit(sh.bar(DRAIN));
        (void)wait_warp(sh, DRAIN, 0);
    }
    } else if (warp < 12) {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 184;");
        // =========================== softmax ===========================
        const int x = (warp - 4) >> 2;                  // 0 = head A, 1 = head B
        const int wrow0 = (warp & 3) << 5;               // this warp's 32 rows of the tile = its TMEM lanes
        const int row = wrow0 | lane;                    // query row in the tile = TMEM lane
        const uint32_t lane_base = (uint32_t)wrow0 << 16;
        const uint32_t t_s = tmem + lane_base + col_s(x);
        const uint32_t t_o = tmem + lane_base + col_o(x);

        // S_READY_x completes once per key tile of the CTA (all items), plus once after the very last PV: completion
        // number t carries the scores of key tile t, and for the first tile of an item also "the previous item's O_x is
        // complete", which is what the write-out warps wait for.
        int t = 0;       // key tiles of the CTA so far (all well-formed items: K/V stages and the mask ring count these)
        int c = 0;       // completions of S_READY_x so far: one per key tile of this head, one more each time the head
                         // sat out an item (its last PV and its next first QK^T are then committed separately)
        bool in_run = false;  // the previous well-formed item had this head
        bool came_back = false;  // ... and it sat out at least one item since
        int n_done = 0;  // items of this head finished so far
        bool ok = true;
        int k = 0;
        auto item_done = [&]() {  // this warp is through with the CTA's k-th item: it will not read its ring slot again
            __syncwarp();
            if (lane == 0) {
                __threadfence_block();
                *sh.items_done(warp - 4) = k + 1;
            }
        };
        for (; ok; ++k) {
            Item it;
            if (fetch_item(sh, k, it) <= 0) break;
            if (kSingles && x >= it.nh) {  // the odd head of an odd kv group: head B sits this item out
                t += it.n_tiles;
                // The head's last PV is committed on its own now ("O_x complete"), and its next first QK^T will be another
                // completion of S_READY_x: count both.
                if (in_run) ++c;
                in_run = false;
                came_back = true;
                item_done();
                continue;
            }
            if (kSingles && came_back && n_done > 0) {
                // Back after sitting out: the wait for the scores below must not be two completions EARLY (a parity wait
                // passes then as well, and these warps published their last P only a moment ago).  Once the write-out warps
                // have handed back O_x of this head's previous item, "O_x complete" is through.  That wait cannot be late:
                // the next hand-back needs the row sums of the item that starts here.
                ok = wait_warp(sh, O_FREE + x, (uint32_t)((n_done - 1) & 1));
                if (!ok) break;
            }
            came_back = false;
            in_run = true;
            const int lim = it.prow + min(row, it.rows_here - 1);  // last key this row may see
            const int prow = it.prow, L = it.L, n_tiles = it.n_tiles;
            float m_run = -INFINITY, l_run = 0.f;
            for (int j = 0; j < n_tiles; ++j, ++t, ++c) {
                const int s = t % kStages;
                ok = wait_warp(sh, S_READY + x, (uint32_t)(c & 1));
                if (!ok) break;
                fence_after();
                const int key0 = j * kBN;
                const int bad = *sh.bad_mask(t);
                const bool need_mask = (key0 + kBN - 1 > prow) || bad != 0;
                // keys of this tile that lie past the sequence end, or in a skipped block, may hold anything
                // (unwritten slots): their V rows must not reach the tensor pipe, because 0 * NaN = NaN
                const bool dirty_v = (key0 + kBN > L) || bad != 0;
                if (dirty_v && x == 0) {
                    ok = wait_warp(sh, V_FULL + s, (uint32_t)((t / kStages) & 1));
                    if (!ok) break;
                    uint8_t *vdst = sh.ptr + kOffV + s * kTileBytes;
                    if ((key0 + row >= L) || ((bad >> (row >> 4)) & 1)) {  // thread `row` owns key row `row` of the tile
#pragma unroll 1
                        for (int c = 0; c < 16; ++c)  // rare: kept small
                            *reinterpret_cast<uint4 *>(vdst + (c >> 3) * kHalfBytes + row * 128 + (c & 7) * 16) = make_uint4(0u, 0u, 0u, 0u);
                    }
                    fence_proxy_async_smem();
                }

                // Lazy rescale, shared by the two forms of a tile below: the reference max of a row is raised only when the
                // tile's max is far above it (also for the row's first finite tile); O, if it holds anything yet, is then
                // scaled in TMEM, 32 columns at a time (rare, so kept small rather than fast).
                auto new_reference = [&](float m_tile) {
                    const bool raise = m_tile > m_run + kRescaleThreshold;
                    if (__any_sync(0xffffffffu, raise)) {
                        const float m_new = raise ? m_tile : m_run;
                        const float alpha = (raise && m_run > -INFINITY) ? fast_exp2(m_run - m_new) : (raise ? 0.f : 1.f);
                        m_run = m_new;
                        l_run *= alpha;
                        if (j > 0) {  // no MMA touches O_x right now
#pragma unroll 1
                            for (int cc = 0; cc < 4; ++cc) {
                                float ov[32];
                                tmem_ld32(ov, t_o + 32 * cc);
#pragma unroll
                                for (int i = 0; i < 32; ++i) ov[i] *= alpha;
                                tmem_st32(t_o + 32 * cc, ov);
                            }
                        }
                    }
                    return m_run > -INFINITY ? m_run : 0.f;
                };
                // A tile that the causal boundary cuts (or that holds a block the table does not really name) first gets
                // its hidden scores overwritten with -inf IN TMEM, by a small loop over 32-column pieces, and then goes
                // through the same code as every other tile.  This row sees columns 0..rel of the tile and rel grows with
                // the row, so a piece is left alone if the warp's first row sees all of it, and is -inf for every row of
                // the warp if the last row sees none of it.  (Such a tile comes once per item: for a long request its speed
                // does not matter, and for a batch of short ones the SIZE of the code does -- their items walk through all
                // of the softmax code every few thousand cycles, and what does not fit the instruction cache of the SM's
                // quarter is fetched again for every item.)
                if (need_mask) {
                    const int rel = lim - key0;
                    const int rel_min = __reduce_min_sync(0xffffffffu, rel), rel_max = __reduce_max_sync(0xffffffffu, rel);
#pragma unroll 1
                    for (int cc = 0; cc < 4; ++cc) {
                        const unsigned b2 = ((unsigned)bad >> (2 * cc)) & 3u;
                        if (32 * cc + 31 <= rel_min && b2 == 0u) continue;
                        const int r = rel - 32 * cc;
                        const unsigned past = r >= 31 ? 0u : (r < 0 ? 0xffffffffu : 0xfffffffeu << r);
                        const unsigned hid = past | ((b2 & 1u) ? 0x0000ffffu : 0u) | ((b2 & 2u) ? 0xffff0000u : 0u);
                        float v[32];
                        if (32 * cc > rel_max) {
#pragma unroll
                            for (int i = 0; i < 32; ++i) v[i] = -INFINITY;
                        } else {
                            tmem_ld32(v, t_s + 32 * cc);
#pragma unroll
                            for (int i = 0; i < 32; ++i) v[i] = ((hid >> i) & 1u) ? -INFINITY : v[i];
                        }
                        tmem_st32(t_s + 32 * cc, v);
                    }
                    cp::tcgen05_wait_st();
                }
                float sv[128];
                {
                    uint32_t(&r)[128] = reinterpret_cast<uint32_t(&)[128]>(sv);
                    cp::tcgen05_ld_32x32b(reinterpret_cast<uint32_t(&)[32]>(r[0]), t_s);
                    cp::tcgen05_ld_32x32b(reinterpret_cast<uint32_t(&)[32]>(r[32]), t_s + 32);
                    cp::tcgen05_ld_32x32b(reinterpret_cast<uint32_t(&)[32]>(r[64]), t_s + 64);
                    cp::tcgen05_ld_32x32b(reinterpret_cast<uint32_t(&)[32]>(r[96]), t_s + 96);
                    cp::tcgen05_wait_ld();
                }
                float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
                for (int i = 0; i < 128; i += 4) {
                    mx0 = fmaxf(mx0, sv[i]);
                    mx1 = fmaxf(mx1, sv[i + 1]);
                    mx2 = fmaxf(mx2, sv[i + 2]);
                    mx3 = fmaxf(mx3, sv[i + 3]);
                }
                const float m_use = new_reference(fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * p.scale_log2);  // scale > 0 on this path
                // ---- P = exp2(S*scale - m) (a hidden -inf gives 0), row sum, bf16 pairs into the S columns.  P of the
                // first 96 keys is published early so the PV MMA overlaps the last quarter of this loop.
                float2 acc_a = make_float2(0.f, 0.f), acc_b = make_float2(0.f, 0.f);
                const float2 sc2 = make_float2(p.scale_log2, p.scale_log2), nm2 = make_float2(-m_use, -m_use);
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    uint32_t pk[16];
                    {
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
            if (!ok) break;

            // ---- the rows' normalisers go to the write-out warps, and this warp is through with the item: the wait for the
            // next item's first scores is the next thing it does
            // (the write-out warps have read the previous item's normalisers once they have handed its O_x back: an item of
            // one key tile can be through here before they have even started on the one before it)
            if (n_done > 0) ok = wait_warp(sh, O_FREE + x, (uint32_t)((n_done - 1) & 1));
            if (!ok) break;
            sh.inv_l(x)[row] = l_run > 0.f ? 1.f / l_run : 0.f;
            mbar_arrive(sh.bar(L_READY + x));
            ++n_done;
            item_done();
        }
    } else {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
        // =========================== write-out: O / l -> bf16 -> global ===========================
        // Four warps, one per quarter of the TMEM lanes, take both heads of every item in turn.  With the write-out here
        // the softmax warps go from an item's last tile straight to the next item's first, and their code is smaller by
        // what this role holds (both matter for batches of short chunks, where an item is only a few key tiles long).
        // The accumulator of a head is complete with the completion of S_READY that follows the item's last key tile; it is
        // read 64 columns at a time and handed back to the MMA warp as soon as the second half is in registers.  A thread
        // holds a whole row, so the rows go through a staging buffer (16-byte pieces XOR-swizzled by row) and leave as
        // 128 contiguous bytes per row: a warp whose 32 rows all belong to the request hands each staged half to the
        // TMA unit (one instruction, the rows leave asynchronously); a warp at the ragged end of a chunk writes its
        // valid rows itself.  Each warp has two staging buffers and alternates between them.
        const int wrow0 = (warp & 3) << 5;               // this warp's 32 rows of the tile = its TMEM lanes
        const int row = wrow0 | lane;
        const uint32_t lane_base = (uint32_t)wrow0 << 16;
        uint8_t *stage0 = sh.ptr + kOffStage + (warp & 3) * 2 * kStageBytes;
        const int piece = lane & 7, sub = lane >> 3;
        int cA = 0, cB = 0;  // completions of S_READY_x up to "O_x of this item is complete": the head's key tiles so far, plus
                             // one for every time it sat out an item (see the softmax role)
        int nA = 0, nB = 0;  // items of head x so far
        bool in_run = false; // the previous well-formed item had head B
        int buf = 0;     // staging buffer of the next half
        int tma_buf = -1;  // buffer that the most recent store handed to the TMA unit reads from
        bool ok = true;
        for (int k = 0; ok; ++k) {
            Item it;
            if (fetch_item(sh, k, it) <= 0) break;
            {
                const bool by_tma = wrow0 + 32 <= it.rows_here;
                if (kSingles && it.nh < 2) {
                    if (in_run) ++cB;
                    in_run = false;
                } else {
                    in_run = true;
                }
#pragma unroll 1
                for (int x = 0; x < (kSingles ? it.nh : 2) && ok; ++x) {
                    if (x == 0) cA += it.n_tiles;
                    else cB += it.n_tiles;
                    ok = wait_warp(sh, L_READY + x, (uint32_t)((x == 0 ? nA : nB) & 1));
                    if (ok) ok = wait_warp(sh, S_READY + x, (uint32_t)((x == 0 ? cA : cB) & 1));
                    if (!ok) break;
                    if (x == 0) ++nA;
                    else ++nB;
                    fence_after();
                    const float inv = sh.inv_l(x)[row];  // read before O_x is handed back: the softmax warps write the next item's late
                    const uint32_t t_o = tmem + lane_base + col_o(x);
                    __nv_bfloat16 *dst = p.out + (size_t)it.qrow * row_stride + (size_t)(it.head0 + x) * kD + piece * 8;
#pragma unroll 1
                    for (int h2 = 0; h2 < 2; ++h2) {
                        // the buffer must no longer be read by an earlier store: the most recent one may still be if it
                        // reads the other buffer
                        if (lane == 0) {
                            if (tma_buf == buf || !by_tma) bulk_wait_group_read_0();
                            else bulk_wait_group_read_1();
                        }
                        __syncwarp();
                        uint8_t *stage = stage0 + buf * kStageBytes;
#pragma unroll 1
                        for (int c2 = 0; c2 < 2; ++c2) {  // 32 columns at a time: this role lives on few registers
                            float ov[32];
                            tmem_ld32(ov, t_o + 64 * h2 + 32 * c2);
                            if (h2 == 1 && c2 == 1) {  // all of O_x is in registers or staged: the next item's first PV may overwrite it
                                fence_before();
                                __syncwarp();
                                if (lane == 0) mbar_arrive(sh.bar(O_FREE + x));
                            }
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                uint4 v;
                                v.x = pack_bf16x2(ov[8 * i] * inv, ov[8 * i + 1] * inv);
                                v.y = pack_bf16x2(ov[8 * i + 2] * inv, ov[8 * i + 3] * inv);
                                v.z = pack_bf16x2(ov[8 * i + 4] * inv, ov[8 * i + 5] * inv);
                                v.w = pack_bf16x2(ov[8 * i + 6] * inv, ov[8 * i + 7] * inv);
                                *reinterpret_cast<uint4 *>(stage + lane * 128 + (((4 * c2 + i) ^ (lane & 7)) << 4)) = v;  // = the 128-byte swizzle
                            }
                        }
                        if (by_tma) {
                            fence_proxy_async_smem();
                            __syncwarp();
                            if (lane == 0) {
                                tma_store_3d(&omap, smem_u32(stage), 64 * h2, it.head0 + x, it.qrow + wrow0);
                                bulk_commit_group();
                            }
                            tma_buf = buf;
                        } else {
                            __syncwarp();
#pragma unroll 1
                            for (int r4 = 0; r4 < 8; ++r4) {
                                const int lr = 4 * r4 + sub;  // row inside this warp's 32
                                const uint4 w = *reinterpret_cast<const uint4 *>(stage + lr * 128 + ((piece ^ (lr & 7)) << 4));
                                if (wrow0 + lr < it.rows_here) *reinterpret_cast<uint4 *>(dst + (size_t)(wrow0 + lr) * row_stride + 64 * h2) = w;
                            }
                            __syncwarp();
                        }
                        buf ^= 1;
                    }
                }
            }
            __syncwarp();  // this warp is through with the CTA's k-th item: it will not read its ring slot again
            if (lane == 0) {
                __threadfence_block();
                *sh.items_done(warp - 4) = k + 1;
            }
        }
        if (lane == 0) bulk_wait_group_0();  // every row this warp handed to the TMA unit has been written
    }

    // ---- teardown: everybody meets, copies in flight get a bounded chance to land, TMEM goes back
    fence_before();
    __syncthreads();
    fence_after();
    if (*sh.abort_flag()) {
        if (threadIdx.x == 0) {  // a wait of this CTA ran out: latch it, and tell the launch's other CTAs
            *(volatile int *)p.abort_word = 1;
            atomicOr(p.status, EKV_DEV_FLAG_TIMEOUT);
        }
        if (warp == 0 || warp == 2) {
            const int FULL = warp == 2 ? V_FULL : K_FULL;
            for (int j = max(0, tiles_issued - kStages); j < tiles_issued; ++j)
                (void)mbar_wait(sh.bar(FULL + j % kStages), (uint32_t)((j / kStages) & 1), 100000000ull);
        } else if (warp == 3) {
            for (int x = 0; x < 2; ++x) {
                const int nqx = x == 0 ? tiles_issued >> 16 : tiles_issued & 0xffff;  // (only the parity of the last load matters)
                if (nqx > 0) (void)mbar_wait(sh.bar(Q_FULL + x), (uint32_t)((nqx - 1) & 1), 100000000ull);
            }
        }
    }
    __syncthreads();
    if (warp == 2) cp::tcgen05_dealloc(cp::cta_group_1, tmem, 512);
}

static ekv_status_t launch_prefill_tc(ekv_pool *pool, int layer, const PrefillParams &p, const void *q, void *out, long long total_rows,
                                      cudaStream_t stream) {
    static bool attr_set[64] = {false};
    const int dev = pool->desc.device;
    if (dev >= 64 || !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(prefill_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(prefill_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return cuda_fail(e, "ekv_attn_prefill_chunk: shared-memory attribute");
        if (dev < 64) attr_set[dev] = true;
    }
    CUtensorMap qmap, omap;
    ekv_status_t st = encode_q_map(q, (uint64_t)total_rows, pool->desc.num_q_heads, kD, kBM, &qmap);
    if (st == EKV_OK) st = encode_q_map(out, (uint64_t)total_rows, pool->desc.num_q_heads, kD, 32, &omap);  // same geometry, 32-row boxes
    if (st != EKV_OK) return st;
    const long long items = (long long)p.q_tiles * head_pairs(p);
    const int grid = (int)(items < pool->sm_count ? items : pool->sm_count);
    cudaError_t e0 = cudaMemsetAsync(p.abort_word, 0, 2 * sizeof(int), stream);  // abort word + item counter
    if (e0 != cudaSuccess) return cuda_fail(e0, "ekv_attn_prefill_chunk: clear abort word and item counter");
    if (p.group % 2 == 0) prefill_tc_kernel<false><<<grid, kThreads, kSmemBytes, stream>>>(pool->kv_map[layer], qmap, omap, p);
    else prefill_tc_kernel<true><<<grid, kThreads, kSmemBytes, stream>>>(pool->kv_map[layer], qmap, omap, p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "ekv_attn_prefill_chunk: launch");
    return EKV_OK;
}

}  // namespace tc
}  // namespace ekv
