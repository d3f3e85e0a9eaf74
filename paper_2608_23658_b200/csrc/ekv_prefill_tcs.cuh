// Chunked-prefill attention on the 5th-generation tensor cores for batches of SHORT chunks (and for odd query
// groups at head_dim 128): the persistent CTA of ekv_prefill_tc.cuh with its two TMEM slots DECOUPLED.
//
// In the two-head kernel slots A and B hold two heads of the same work item: they share every K/V tile (half the
// traffic of a long prompt) but move in lockstep -- both softmax at the same moment, both write out at the same
// moment -- and when an item has one to four key tiles nothing of a head overlaps anything, so most of an item's life
// is set-up, write-out and barrier hops.  Here a work item is 128 query positions of ONE head, slot x (S_x, O_x in
// TMEM, its own Q tile, one K and one V tile in shared memory) takes the CTA's items x, x+2, x+4, ..., and the two
// slots run on their own clocks: one slot's write-out and item switch sit under the other's softmax, and the single
// MMA-issuing warp serves whichever slot has its operands ready (it polls both instead of waiting for one).
// Every K/V tile is staged once per head instead of once per head pair, which a short chunk does not notice.
//
//   warp 0 / warp 2   TMA producer of slot A's / slot B's K and V tiles (one stage each: K(j+1) is loaded while
//                     softmax(j) and PV(j) run, V(j+1) while QK(j+1) and softmax(j+1) run); warp 2 owns TMEM
//   warp 1            MMA issuer: a small state machine per slot, advanced by non-blocking barrier tests
//   warp 3            item scheduler (longest-first list over (query tile, head), drawn from a device counter,
//                     decoded and posted in a ring in shared memory) and TMA producer of both slots' Q tiles
//   warps 4-7         softmax and write-out of slot A: one thread per query row (= TMEM lane)
//   warps 8-11        softmax and write-out of slot B
//
// Softmax, masking, lazy rescaling, write-out and the bounded waits are those of the two-head kernel.
#pragma once
#include "ekv_prefill_tc.cuh"

namespace ekv {
namespace tcs {

namespace cp = cuda::ptx;
using namespace ekv::tc;  // tile geometry, descriptors, MMA / fence / TMEM helpers, Shared, Item, wait_warp

// barrier slots: as in the two-head kernel, but K / V barriers are per SLOT (one stage each) and every slot reports
// its finished items on a barrier of its own
// Item ring of 8: a slot's next item (two indices ahead) must be postable while the slot's previous items are still
// being written out, so that its Q tile and first K/V tile are in flight early.
static constexpr int kSRing = 8;
enum SBar { SQ_FULL = 0, SQ_EMPTY = 2, SK_FULL = 4, SK_EMPTY = 6, SV_FULL = 8, SV_EMPTY = 10, SS_READY = 12, SP_READY = 14,
            SP_PART = 16, SO_FREE = 18, SDRAIN = 20, SITEM_READY = 21, SNBAR = SITEM_READY + kSRing };
static constexpr int kSOffFlags = 8 * SNBAR;            // abort flag, TMEM base, per slot the number of softmax warps that finished an item
static constexpr int kSOffMask = kSOffFlags + 16;       // 2 slots x 4 masks
static constexpr int kSOffItems = 320;                  // kSRing item slots of 64 bytes
static_assert(kSOffMask + 32 <= kSOffItems, "barrier area");
// This kernel's own thread count and register split (setmaxnreg: warps 0-3 drop to 72, warps 4-11 rise to 216; the raise
// blocks until the registers are there, so the split has to fit the CTA's own allocation and the role code must match
// the number of warps launched).
static constexpr int kSThreads = 384, kSLaunchRegs = 168;
static_assert(128 * 72 + 256 * 216 <= kSLaunchRegs * kSThreads && kSLaunchRegs * kSThreads <= 65536, "register split of the two-slot kernel");
static constexpr int kSSmemBytes = kOffBar + kSOffItems + 64 * kSRing + 32 + 1024;  // + per-warp progress, + alignment slack
static_assert(kSSmemBytes <= 232448, "shared memory of one CTA");

struct SShared {
    uint32_t base;
    uint8_t *ptr;
    __device__ __forceinline__ uint32_t bar(int i) const { return base + kOffBar + 8 * i; }
    __device__ __forceinline__ volatile int *abort_flag() const { return (volatile int *)(ptr + kOffBar + kSOffFlags); }
    __device__ __forceinline__ uint32_t *tmem_slot() const { return (uint32_t *)(ptr + kOffBar + kSOffFlags + 4); }
    // Finished items are COUNTED, not signalled on an mbarrier: the scheduler looks only when it needs a ring slot back,
    // possibly several items later, and a phase parity cannot tell "not yet" from "two phases ago".  Every softmax warp
    // keeps its own count (items of its slot it is through with) and the scheduler takes the minimum of a slot's four: in
    // a sum the lead of three warps could pay for the one that lags (they are not tied to each other on items that have
    // no tiles).
    __device__ __forceinline__ volatile int *items_done(int x) const { return (volatile int *)(ptr + kOffBar + kSOffItems + 64 * kSRing) + 4 * x; }
    // per slot a ring of 4 masks of key blocks whose shared-memory rows hold stand-in data
    __device__ __forceinline__ volatile int *bad_mask(int x, int tile) const {
        return (volatile int *)(ptr + kOffBar + kSOffMask + 16 * x + 4 * (tile & 3));
    }
    __device__ __forceinline__ uint4 *item_slot(int k) const { return (uint4 *)(ptr + kOffBar + kSOffItems + 64 * (k % kSRing)); }
};

__device__ __forceinline__ bool s_wait_or_abort(const SShared &sh, int bar, uint32_t parity, unsigned *status, int *abort_word) {
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
__device__ __forceinline__ bool s_wait_warp(const SShared &sh, int bar, uint32_t parity, unsigned *status, int *abort_word) {
    return __all_sync(0xffffffffu, s_wait_or_abort(sh, bar, parity, status, abort_word));
}

// Item m of the call: query tiles from the latest to the earliest, every tile listed for all heads before the next.
__device__ __forceinline__ bool s_decode_item(const PrefillParams &p, int m, Item &it) {
    it.state = kItemWork;
    const int rank = m / p.num_q_heads;
    const int head = m - rank * p.num_q_heads;
    const int tile_idx = p.q_tiles - 1 - rank;
    int acc_tiles = 0, c_r = 0, q0 = 0;
    if (!find_request(p, tile_idx, kBM, it.req, acc_tiles, q0, c_r)) return false;
    it.head0 = head;
    it.g = head / p.group;
    const int row0 = (tile_idx - acc_tiles) * kBM;
    it.L = min(p.seq_lens[it.req], p.max_blocks * 16);
    const int prefix = it.L - c_r;
    it.qrow = q0 + row0;
    it.prow = prefix + row0;
    it.rows_here = min(kBM, c_r - row0);
    it.malformed = prefix < 0 ? 1 : 0;
    it.nh = 0;
    const int kv_end = min(it.L, it.prow + it.rows_here);
    it.n_tiles = (kv_end + kBN - 1) / kBN;
    it.n_blocks = (kv_end + 15) >> 4;
    return true;
}
__device__ __forceinline__ void s_read_item(const SShared &sh, int k, Item &it) {
    const uint4 *src = sh.item_slot(k);
    const uint4 a = src[0], b = src[1], c = src[2];
    it.req = (int)a.x, it.qrow = (int)a.y, it.prow = (int)a.z, it.rows_here = (int)a.w;
    it.L = (int)b.x, it.nh = (int)b.y, it.n_tiles = (int)b.z, it.n_blocks = (int)b.w;
    it.head0 = (int)c.x, it.g = (int)c.y, it.malformed = (int)c.z, it.state = (int)c.w;
}
// 1 = an item to work on (possibly malformed), 0 = end of the list, -1 = the wait was given up
__device__ __forceinline__ int s_fetch_item(const SShared &sh, int k, Item &it, unsigned *status, int *abort_word) {
    if (!s_wait_warp(sh, SITEM_READY + k % kSRing, (uint32_t)((k / kSRing) & 1), status, abort_word)) return -1;
    s_read_item(sh, k, it);
    return it.state == kItemWork ? 1 : 0;
}

__global__ void __launch_bounds__(kSThreads, 1) prefill_tcs_kernel(const __grid_constant__ CUtensorMap kvmap,
                                                                  const __grid_constant__ CUtensorMap qmap,
                                                                  const __grid_constant__ CUtensorMap omap,
                                                                  const PrefillParams p) {
    if (*(volatile int *)p.abort_word) return;  // a CTA of this launch already timed out
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const size_t row_stride = (size_t)p.num_q_heads * kD;
    const int n_items = p.q_tiles * p.num_q_heads;

    extern __shared__ uint8_t smem_raw[];
    SShared sh;
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
            mbar_init(sh.bar(SQ_FULL + x), 1);
            mbar_init(sh.bar(SQ_EMPTY + x), 1);
            mbar_init(sh.bar(SK_FULL + x), 1);
            mbar_init(sh.bar(SK_EMPTY + x), 1);
            mbar_init(sh.bar(SV_FULL + x), 1);
            mbar_init(sh.bar(SV_EMPTY + x), 1);
            mbar_init(sh.bar(SS_READY + x), 1);
            mbar_init(sh.bar(SP_READY + x), 128);
            mbar_init(sh.bar(SP_PART + x), 128);
            mbar_init(sh.bar(SO_FREE + x), 4);
            for (int w = 0; w < 4; ++w) sh.items_done(x)[w] = 0;
        }
        mbar_init(sh.bar(SDRAIN), 1);
        for (int i = 0; i < kSRing; ++i) mbar_init(sh.bar(SITEM_READY + i), 1);
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
    int tiles_issued = 0;  // producers: what this warp has put in flight (the teardown of an aborted CTA waits for the last of it)

    if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
    if (warp == 0 || warp == 2) {
        // =========================== TMA producer of one slot's K and V tiles ===========================
        const int x = warp >> 1;
        const long long live = *p.live;
        int t = 0;  // key tiles of this slot issued so far
        bool ok = true;
        for (int k = x; ok; k += 2) {
            Item it;
            if (s_fetch_item(sh, k, it, p.status, p.abort_word) <= 0) break;
            if (it.malformed) continue;
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
            for (int j = 0; j < it.n_tiles && ok; ++j, ++t) {
                const int id_raw = id_next;
                if (j + 1 < it.n_tiles) id_next = load_id(j + 1);
                const unsigned oob = __ballot_sync(0xffffffffu, id_raw == -2) & 0xffu;
                const unsigned bad = __ballot_sync(0xffffffffu, id_raw < 0) & 0xffu;
                const int id = id_raw < 0 ? 0 : id_raw;  // masked later; block 0 is always mapped
                const int b = lane & 15, blk = b >> 1, half = b & 1;
                const int my_id = __shfl_sync(0xffffffffu, id, blk);
#pragma unroll
                for (int kv = 0; kv < 2; ++kv) {
                    const int FULL = (kv ? SV_FULL : SK_FULL) + x, EMPTY = (kv ? SV_EMPTY : SK_EMPTY) + x;
                    const uint32_t tile_base = sh.base + (kv ? kOffV : kOffK) + x * kTileBytes;
                    const int row = it.g * 16 + (kv ? p.num_kv_heads * 16 : 0);  // row inside the block: (K|V, kv-head, token)
                    if (t > 0 && !s_wait_warp(sh, EMPTY, (uint32_t)((t - 1) & 1), p.status, p.abort_word)) {
                        ok = false;
                        break;
                    }
                    if (lane == 0) {
                        if (!kv) {
                            if (oob) atomicOr(p.status, EKV_DEV_FLAG_OOB);
                            *sh.bad_mask(x, t) = (int)bad;
                        }
                        mbar_expect_tx(sh.bar(FULL), kTileBytes);
                    }
                    __syncwarp();
                    if (lane < 16) tma_load_3d(tile_base + half * kHalfBytes + blk * 2048, &kvmap, 64 * half, row, my_id, sh.bar(FULL));
                    if (kv) tiles_issued = t + 1;
                }
            }
        }
    } else if (warp == 3) {
        // =========================== item scheduler + TMA producer of both slots' Q tiles ===========================
        // One loop serves three things without ever blocking on one of them: posting items a few indices ahead of the
        // slots, and loading the next Q tile of slot A and of slot B as soon as that slot's previous item has issued its
        // last QK^T.  (Walking the items in index order and waiting for each one's Q tile in turn ties the two slots
        // together: a slot that is ahead cannot get its next Q tile before the other slot has caught up.)
        int nq[2] = {0, 0};   // well-formed items of each slot whose Q tile was requested
        int qk[2] = {0, 1};   // next item index of each slot whose Q tile is to be loaded
        bool qdone[2] = {false, false};
        int posted = 0, ends = 0;  // items posted; end markers among them (two in a row: each slot meets one at its own next index)
        int *counter = p.abort_word + 1;  // next item number of the launch (cleared by the launcher with the abort word)
        auto ready = [&](int bar, int count) { return mbar_test_wait(sh.bar(bar), (uint32_t)(count & 1)); };
        uint64_t t_progress = global_timer_ns();
        uint32_t spins = 0;
        bool ok = true;
        while (ok && !(qdone[0] && qdone[1])) {
            bool progressed = false;
            // ---- post items, up to four per pass (decoding one takes two dependent reads of device memory; four lanes do
            // it side by side): up to kSRing - 2 indices ahead of the slower slot, and ring slot idx % kSRing only once the
            // item that used it before (index idx - kSRing, same TMEM slot) is written out
            if (ends < 2) {
                const int idx = posted + lane;
                const bool can = lane < 4 && idx < min(qk[0], qk[1]) + kSRing - 2 &&
                                 (idx < kSRing || min(min(sh.items_done(idx & 1)[0], sh.items_done(idx & 1)[1]),
                                                      min(sh.items_done(idx & 1)[2], sh.items_done(idx & 1)[3])) >= ((idx - kSRing) >> 1) + 1);
                const int n_post = __ffs((int)~__ballot_sync(0xffffffffu, can)) - 1;  // leading lanes that can
                if (n_post > 0) {
                    int base = 0;
                    if (lane == 0) base = atomicAdd(counter, n_post);
                    base = __shfl_sync(0xffffffffu, base, 0);
                    bool is_end = false;
                    if (lane < n_post) {
                        Item it;
                        it.req = it.qrow = it.prow = it.rows_here = it.L = it.nh = it.n_tiles = it.n_blocks = it.head0 = it.g = it.malformed = 0;
                        it.state = kItemEnd;
                        const int m = base + lane;
                        if (m >= n_items || !s_decode_item(p, m, it)) it.state = kItemEnd;
                        is_end = it.state == kItemEnd;
                        uint4 *dst = sh.item_slot(idx);
                        dst[0] = make_uint4((unsigned)it.req, (unsigned)it.qrow, (unsigned)it.prow, (unsigned)it.rows_here);
                        dst[1] = make_uint4((unsigned)it.L, (unsigned)it.nh, (unsigned)it.n_tiles, (unsigned)it.n_blocks);
                        dst[2] = make_uint4((unsigned)it.head0, (unsigned)it.g, (unsigned)it.malformed, (unsigned)it.state);
                        __threadfence_block();
                        mbar_arrive(sh.bar(SITEM_READY + idx % kSRing));
                    }
                    ends += __popc(__ballot_sync(0xffffffffu, is_end));  // once the list has ended every further item is an end marker
                    posted += n_post;
                    progressed = true;
                }
            }
            // ---- Q tiles
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                if (qdone[x] || qk[x] >= posted) continue;
                Item it;
                s_read_item(sh, qk[x], it);
                if (it.state != kItemWork) {
                    qdone[x] = true;
                    progressed = true;
                } else if (it.malformed) {
                    qk[x] += 2;
                    progressed = true;
                } else if (nq[x] == 0 || ready(SQ_EMPTY + x, nq[x] - 1)) {  // the slot's previous item has issued its last QK^T
                    if (lane == 0) mbar_expect_tx(sh.bar(SQ_FULL + x), kTileBytes);
                    __syncwarp();
                    if (lane < 2)
                        tma_load_3d(sh.base + kOffQ + x * kTileBytes + lane * kHalfBytes, &qmap, 64 * lane, it.head0, it.qrow, sh.bar(SQ_FULL + x));
                    ++nq[x];
                    qk[x] += 2;
                    progressed = true;
                }
            }
            if (progressed) {
                t_progress = global_timer_ns();
                spins = 0;
            } else if ((++spins & 63u) == 0u) {
                if (*sh.abort_flag()) ok = false;
                else if (global_timer_ns() - t_progress > 2000000000ull) {
                    *sh.abort_flag() = 1;
                    *(volatile int *)p.abort_word = 1;
                    atomicOr(p.status, EKV_DEV_FLAG_TIMEOUT);
                    ok = false;
                }
            }
        }
        tiles_issued = (nq[0] << 16) | nq[1];
    } else {
        // =========================== MMA issuer: one state machine per slot ===========================
        const uint32_t q_lo[2] = {desc_lo(sh.base + kOffQ, 16), desc_lo(sh.base + kOffQ + kTileBytes, 16)};
        const uint32_t k_lo[2] = {desc_lo(sh.base + kOffK, 16), desc_lo(sh.base + kOffK + kTileBytes, 16)};
        const uint32_t v_lo[2] = {desc_lo(sh.base + kOffV, kHalfBytes), desc_lo(sh.base + kOffV + kTileBytes, kHalfBytes)};
        auto issue_qk = [&](int x) {
#pragma unroll
            for (int k = 0; k < kD / 16; ++k) {
                const uint32_t off = ((k >> 2) * kHalfBytes + (k & 3) * 32) >> 4;
                if (k == 0) mma_ss_lo<false>(tmem + col_s(x), q_lo[x] + off, k_lo[x] + off, kIdescQK);
                else mma_ss_lo<true>(tmem + col_s(x), q_lo[x] + off, k_lo[x] + off, kIdescQK);
            }
        };
        auto issue_pv = [&](int x, bool acc, int k0, int k1) {
#pragma unroll
            for (int k = k0; k < k1; ++k)
                mma_ts_lo_dyn(tmem + col_o(x), tmem + col_s(x) + 8 * k, v_lo[x] + ((k * 2048) >> 4), kIdescPV, (acc || k > 0) ? 1u : 0u);
        };
        auto ready = [&](int bar, int count) { return mbar_test_wait(sh.bar(bar), (uint32_t)(count & 1)); };
        enum { ST_FETCH, ST_QK, ST_PV1, ST_PV2, ST_DONE };
        int st[2] = {ST_FETCH, ST_FETCH};
        int kk[2] = {0, 1};      // next item index of the slot
        int nt[2] = {0, 0};      // key tiles of the current item
        int jj[2] = {0, 0};      // current key tile
        int tq[2] = {0, 0};      // key tiles whose QK^T was issued (K barrier uses)
        int tv[2] = {0, 0};      // key tiles whose PV was issued (V and P barrier uses)
        int ni[2] = {0, 0};      // items whose first QK^T was issued (Q and O barrier uses)
        uint64_t t_progress = global_timer_ns();
        bool ok = true;
        uint32_t spins = 0;
        while (ok && (st[0] != ST_DONE || st[1] != ST_DONE)) {
            bool progressed = false;
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                if (st[x] == ST_FETCH) {
                    if (ready(SITEM_READY + kk[x] % kSRing, kk[x] / kSRing)) {
                        Item it;
                        s_read_item(sh, kk[x], it);
                        if (it.state != kItemWork) {
                            st[x] = ST_DONE;
                        } else if (it.malformed) {
                            kk[x] += 2;
                        } else {
                            nt[x] = it.n_tiles;
                            jj[x] = 0;
                            st[x] = ST_QK;
                        }
                        progressed = true;
                    }
                } else if (st[x] == ST_QK) {
                    if ((jj[x] > 0 || ready(SQ_FULL + x, ni[x])) && ready(SK_FULL + x, tq[x])) {
                        fence_after();
                        issue_qk(x);
                        mma_commit(sh.bar(SK_EMPTY + x));
                        if (jj[x] + 1 == nt[x]) mma_commit(sh.bar(SQ_EMPTY + x));  // the item's last QK^T
                        mma_commit(sh.bar(SS_READY + x));
                        ++tq[x];
                        if (jj[x] == 0) ++ni[x];
                        st[x] = ST_PV1;
                        progressed = true;
                    }
                } else if (st[x] == ST_PV1) {
                    // O_x still holds the previous item's result until its write-out has read it
                    if (ready(SV_FULL + x, tv[x]) && (jj[x] > 0 || ni[x] < 2 || ready(SO_FREE + x, ni[x] - 2)) && ready(SP_PART + x, tv[x])) {
                        fence_after();
                        issue_pv(x, jj[x] > 0, 0, kPartSteps);
                        st[x] = ST_PV2;
                        progressed = true;
                    }
                } else if (st[x] == ST_PV2) {
                    if (ready(SP_READY + x, tv[x])) {
                        fence_after();
                        issue_pv(x, true, kPartSteps, kBN / 16);
                        mma_commit(sh.bar(SV_EMPTY + x));
                        ++tv[x];
                        if (++jj[x] < nt[x]) {
                            st[x] = ST_QK;
                        } else {
                            mma_commit(sh.bar(SS_READY + x));  // O_x of the item is complete
                            kk[x] += 2;
                            st[x] = ST_FETCH;
                        }
                        progressed = true;
                    }
                }
            }
            if (progressed) {
                t_progress = global_timer_ns();
                spins = 0;
            } else if ((++spins & 63u) == 0u) {  // nothing to do for a while: bounded like every other wait
                if (*sh.abort_flag()) ok = false;
                else if (global_timer_ns() - t_progress > 2000000000ull) {
                    *sh.abort_flag() = 1;
                    *(volatile int *)p.abort_word = 1;
                    atomicOr(p.status, EKV_DEV_FLAG_TIMEOUT);
                    ok = false;
                }
            }
        }
        mma_commit(sh.bar(SDRAIN));
        (void)s_wait_warp(sh, SDRAIN, 0, p.status, p.abort_word);
    }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
        // =========================== softmax + write-out of one slot ===========================
        const int x = (warp - 4) >> 2;
        const int wrow0 = (warp & 3) << 5;
        const int row = wrow0 | lane;
        const uint32_t lane_base = (uint32_t)wrow0 << 16;
        const uint32_t t_s = tmem + lane_base + col_s(x);
        const uint32_t t_o = tmem + lane_base + col_o(x);
        uint8_t *stage = sh.ptr + kOffStage + (warp - 4) * kStageBytes;

        // SS_READY_x completes once per key tile (its scores) and once more per item (its last PV): completion number
        // t + n belongs to key tile t of the slot when n items were finished before it.
        int t = 0, n = 0;
        bool ok = true;
        int k = x;
        auto item_done = [&]() {  // this warp will not read the ring slot of the CTA's k-th item again
            __syncwarp();
            if (lane == 0) {
                __threadfence_block();
                sh.items_done(x)[warp & 3] = (k >> 1) + 1;
            }
        };
        for (; ok; k += 2) {
            Item it;
            if (s_fetch_item(sh, k, it, p.status, p.abort_word) <= 0) break;
            if (it.malformed) {  // zero rows, latch
                if ((threadIdx.x & 127) == 0) atomicOr(p.status, EKV_DEV_FLAG_OOB);
                for (int e = (int)(threadIdx.x & 127); e < it.rows_here * kD; e += 128)
                    p.out[((size_t)(it.qrow + e / kD)) * row_stride + (size_t)it.head0 * kD + e % kD] = __float2bfloat16_rn(0.f);
                item_done();
                continue;
            }
            const int lim = it.prow + min(row, it.rows_here - 1);  // last key this row may see
            const int prow = it.prow, L = it.L, n_tiles = it.n_tiles;
            float m_run = -INFINITY, l_run = 0.f;
            for (int j = 0; j < n_tiles; ++j, ++t) {
                ok = s_wait_warp(sh, SS_READY + x, (uint32_t)((t + n) & 1), p.status, p.abort_word);
                if (!ok) break;
                fence_after();
                const int key0 = j * kBN;
                const int bad = *sh.bad_mask(x, t);
                const bool need_mask = (key0 + kBN - 1 > prow) || bad != 0;
                // keys past the sequence end or in a skipped block may hold anything: their V rows must not reach the tensor pipe
                const bool dirty_v = (key0 + kBN > L) || bad != 0;
                if (dirty_v) {
                    ok = s_wait_warp(sh, SV_FULL + x, (uint32_t)(t & 1), p.status, p.abort_word);
                    if (!ok) break;
                    uint8_t *vdst = sh.ptr + kOffV + x * kTileBytes;
                    if ((key0 + row >= L) || ((bad >> (row >> 4)) & 1)) {  // thread `row` owns key row `row` of the tile
#pragma unroll
                        for (int h2 = 0; h2 < 2; ++h2)
#pragma unroll
                            for (int c16 = 0; c16 < 8; ++c16)
                                *reinterpret_cast<uint4 *>(vdst + h2 * kHalfBytes + row * 128 + c16 * 16) = make_uint4(0u, 0u, 0u, 0u);
                    }
                    fence_proxy_async_smem();
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
                const bool raise = m_tile > m_run + kRescaleThreshold;  // lazy rescale; also true for the first finite tile
                if (__any_sync(0xffffffffu, raise)) {
                    const float m_new = raise ? m_tile : m_run;
                    const float alpha = (raise && m_run > -INFINITY) ? fast_exp2(m_run - m_new) : (raise ? 0.f : 1.f);
                    m_run = m_new;
                    l_run *= alpha;
                    if (j > 0) {  // O holds the sum over earlier tiles of this item and no MMA touches it right now
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
                        mbar_arrive(sh.bar(SP_PART + x));
                    }
                }
                l_run += (acc_a.x + acc_a.y) + (acc_b.x + acc_b.y);
                cp::tcgen05_wait_st();
                fence_before();
                mbar_arrive(sh.bar(SP_READY + x));
            }
            if (!ok) break;

            // ---- write-out (as in the two-head kernel): accumulator into registers, handed back at once, rows through
            // the swizzled staging area, TMA store for a warp whose 32 rows all belong to the request
            ok = s_wait_warp(sh, SS_READY + x, (uint32_t)((t + n) & 1), p.status, p.abort_word);
            if (!ok) break;
            ++n;
            fence_after();
            float ov[128];
            {
                uint32_t(&r)[128] = reinterpret_cast<uint32_t(&)[128]>(ov);
                cp::tcgen05_ld_32x32b(reinterpret_cast<uint32_t(&)[32]>(r[0]), t_o);
                cp::tcgen05_ld_32x32b(reinterpret_cast<uint32_t(&)[32]>(r[32]), t_o + 32);
                cp::tcgen05_ld_32x32b(reinterpret_cast<uint32_t(&)[32]>(r[64]), t_o + 64);
                cp::tcgen05_ld_32x32b(reinterpret_cast<uint32_t(&)[32]>(r[96]), t_o + 96);
                cp::tcgen05_wait_ld();
            }
            fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(sh.bar(SO_FREE + x));
            const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
            const int piece = lane & 7, sub = lane >> 3;
            const uint4 slot0 = sh.item_slot(k)[0], slot2 = sh.item_slot(k)[2];  // the slot is this item's until item_done()
            const int qrow = (int)slot0.y, rows_here = (int)slot0.w, head = (int)slot2.x;
            const bool by_tma = wrow0 + 32 <= rows_here;
            __nv_bfloat16 *dst = p.out + (size_t)qrow * row_stride + (size_t)head * kD + piece * 8;
#pragma unroll
            for (int h2 = 0; h2 < 2; ++h2) {
                uint4 v[8];
#pragma unroll
                for (int i = 0; i < 64; i += 8) {
                    v[i >> 3].x = pack_bf16x2(ov[64 * h2 + i] * inv, ov[64 * h2 + i + 1] * inv);
                    v[i >> 3].y = pack_bf16x2(ov[64 * h2 + i + 2] * inv, ov[64 * h2 + i + 3] * inv);
                    v[i >> 3].z = pack_bf16x2(ov[64 * h2 + i + 4] * inv, ov[64 * h2 + i + 5] * inv);
                    v[i >> 3].w = pack_bf16x2(ov[64 * h2 + i + 6] * inv, ov[64 * h2 + i + 7] * inv);
                }
                if (lane == 0) bulk_wait_group_read_0();  // the staging area is no longer being read by an earlier store
                __syncwarp();
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    *reinterpret_cast<uint4 *>(stage + lane * 128 + ((i ^ (lane & 7)) << 4)) = v[i];  // = the 128-byte swizzle
                if (by_tma) {
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_3d(&omap, smem_u32(stage), 64 * h2, head, qrow + wrow0);
                        bulk_commit_group();
                    }
                } else {
                    __syncwarp();
#pragma unroll
                    for (int r4 = 0; r4 < 8; ++r4) {
                        const int lr = 4 * r4 + sub;
                        const uint4 w = *reinterpret_cast<const uint4 *>(stage + lr * 128 + ((piece ^ (lr & 7)) << 4));
                        if (wrow0 + lr < rows_here) *reinterpret_cast<uint4 *>(dst + (size_t)(wrow0 + lr) * row_stride + 64 * h2) = w;
                    }
                    __syncwarp();
                }
            }
            item_done();
        }
        if (lane == 0) bulk_wait_group_0();  // every row this warp handed to the TMA unit has been written
    }

    // ---- teardown: everybody meets, copies in flight get a bounded chance to land, TMEM goes back
    fence_before();
    __syncthreads();
    fence_after();
    if (*sh.abort_flag()) {
        if ((warp == 0 || warp == 2) && tiles_issued > 0) {
            const int x = warp >> 1;
            (void)mbar_wait(sh.bar(SK_FULL + x), (uint32_t)((tiles_issued - 1) & 1), 100000000ull);
            (void)mbar_wait(sh.bar(SV_FULL + x), (uint32_t)((tiles_issued - 1) & 1), 100000000ull);
        } else if (warp == 3) {
            const int nq0 = tiles_issued >> 16, nq1 = tiles_issued & 0xffff;
            if (nq0 > 0) (void)mbar_wait(sh.bar(SQ_FULL + 0), (uint32_t)((nq0 - 1) & 1), 100000000ull);
            if (nq1 > 0) (void)mbar_wait(sh.bar(SQ_FULL + 1), (uint32_t)((nq1 - 1) & 1), 100000000ull);
        }
    }
    __syncthreads();
    if (warp == 2) cp::tcgen05_dealloc(cp::cta_group_1, tmem, 512);
}

static ekv_status_t launch_prefill_tcs(ekv_pool *pool, int layer, const PrefillParams &p, const void *q, void *out, long long total_rows,
                                       cudaStream_t stream) {
    static bool attr_set[64] = {false};
    const int dev = pool->desc.device;
    if (dev >= 64 || !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(prefill_tcs_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSSmemBytes);
        if (e != cudaSuccess) return cuda_fail(e, "ekv_attn_prefill_chunk: shared-memory attribute");
        if (dev < 64) attr_set[dev] = true;
    }
    CUtensorMap qmap, omap;
    ekv_status_t st = encode_q_map(q, (uint64_t)total_rows, pool->desc.num_q_heads, kD, kBM, &qmap);
    if (st == EKV_OK) st = encode_q_map(out, (uint64_t)total_rows, pool->desc.num_q_heads, kD, 32, &omap);
    if (st != EKV_OK) return st;
    const long long items = (long long)p.q_tiles * pool->desc.num_q_heads;
    const long long want = (items + 1) / 2;  // two slots per CTA
    const int grid = (int)(want < pool->sm_count ? want : pool->sm_count);
    cudaError_t e0 = cudaMemsetAsync(p.abort_word, 0, 2 * sizeof(int), stream);  // abort word + item counter
    if (e0 != cudaSuccess) return cuda_fail(e0, "ekv_attn_prefill_chunk: clear abort word and item counter");
    prefill_tcs_kernel<<<grid, kSThreads, kSSmemBytes, stream>>>(pool->kv_map[layer], qmap, omap, p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "ekv_attn_prefill_chunk: launch");
    return EKV_OK;
}

}  // namespace tcs
}  // namespace ekv
