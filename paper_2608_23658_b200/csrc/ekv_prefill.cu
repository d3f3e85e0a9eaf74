// ekv_attn_prefill_chunk: host entry point.  Validates, sizes the launch from the host copy of
// cu_q_lens (no device synchronisation) and dispatches the kernel for the pool's head_dim.
#include "ekv_internal.h"
#include "ekv_prefill_mma.cuh"
#include "ekv_prefill_tc.cuh"
#include "ekv_prefill_tc1.cuh"
#include "ekv_prefill_tcs.cuh"

using namespace ekv;

extern "C" ekv_status_t ekv_attn_prefill_chunk(ekv_pool_t *pool, int32_t layer, const void *q, void *out,
                                               const int32_t *block_tables, int32_t max_blocks_per_seq,
                                               const int32_t *cu_q_lens, const int32_t *cu_q_lens_host,
                                               const int32_t *seq_lens, int32_t R, float scale, void *stream) {
    ekv_status_t st = check_compute(pool, layer, "ekv_attn_prefill_chunk");
    if (st != EKV_OK) return st;
    if (R < 0 || max_blocks_per_seq < 1 || max_blocks_per_seq > (1 << 26) ||
        (R > 0 && (!q || !out || !block_tables || !cu_q_lens || !cu_q_lens_host || !seq_lens)) || ((uintptr_t)q & 15) ||
        ((uintptr_t)out & 15)) {
        set_error("ekv_attn_prefill_chunk: bad argument (R=%d, max_blocks_per_seq=%d)", R, max_blocks_per_seq);
        return EKV_ERR_INVALID;
    }
    if (R == 0) return EKV_OK;
    if (cu_q_lens_host[0] != 0) {
        set_error("ekv_attn_prefill_chunk: cu_q_lens[0] must be 0");
        return EKV_ERR_INVALID;
    }
    // Kernels (scale > 0 unless stated):
    //   two-head tcgen05 kernel   head_dim 128, query groups of 2 or more: a persistent CTA per SM, every K/V tile feeds two
    //                             heads (an odd group is cut into pairs and one single-head item per kv-head).
    //                             Measured, 32768 query tokens in one call, 32q/8kv: 256 x 128 fresh prompts 130 us against
    //                             161 us for the two-slot kernel; 64 x 512: 198 against 335-364; 16 x 2048: 508 against
    //                             769.  28q/4kv (groups of 7): a 16384-token prompt 1.63 against 2.11 ms, 64 x 512 215
    //                             against 299 us
    //   two-slot tcgen05 kernel   head_dim 128, one head per work item, the CTA's two TMEM slots on their own clocks: query
    //                             groups of one (no two heads share a K/V tile)
    //   one-head tcgen05 kernel   head_dim 64 (one CTA per tile and head, two CTAs per SM)
    //   warp-level MMA kernel     non-positive scales, and every call on a pool created with EKV_PREFILL_WARP_MMA (which
    //                             the tests use to check the kernel families against each other)
    // EKV_PREFILL_ONE_HEAD forces the one-head family on any group; EKV_PREFILL_TWO_HEAD is what a group of two or more at
    // head_dim 128 gets anyway (kept so that a caller can say so).
    const int group = pool->desc.num_q_heads / pool->desc.num_kv_heads;
    const uint32_t pf = pool->desc.flags;
    enum { K_TWO_HEAD, K_ONE_HEAD, K_WARP_MMA } kernel;
    if ((pf & EKV_PREFILL_WARP_MMA) || !(scale > 0.f)) {
        kernel = K_WARP_MMA;
    } else if ((pf & EKV_PREFILL_ONE_HEAD) || pool->desc.head_dim != 128 || group == 1) {
        kernel = K_ONE_HEAD;
    } else {
        kernel = K_TWO_HEAD;
    }
    const int bm = kernel == K_WARP_MMA ? kPmBM : tc::kBM;
    PrefillParams p;
    p.n_prefix = R <= kPrefixMax ? 1 : 0;
    long long q_tiles = 0;
    for (int r = 0; r < R; ++r) {
        const int c = cu_q_lens_host[r + 1] - cu_q_lens_host[r];
        if (c < 0) {
            set_error("ekv_attn_prefill_chunk: cu_q_lens decreases at request %d", r);
            return EKV_ERR_INVALID;
        }
        if (p.n_prefix) p.tile_prefix[r] = (int)q_tiles;
        q_tiles += (c + bm - 1) / bm;
        if (q_tiles > 0x7fffffffLL) break;
    }
    if (p.n_prefix && q_tiles <= 0x7fffffffLL) p.tile_prefix[R] = (int)q_tiles;
    if (q_tiles == 0) return EKV_OK;
    if (q_tiles > 0x7fffffffLL) {
        set_error("ekv_attn_prefill_chunk: too many query tiles");
        return EKV_ERR_INVALID;
    }
    p.q = (const __nv_bfloat16 *)q;
    p.out = (__nv_bfloat16 *)out;
    p.block_tables = block_tables;
    p.cu_q_lens = cu_q_lens;
    p.seq_lens = seq_lens;
    p.live = pool->d_live;
    p.status = pool->d_status;
    // every launch gets a device word of its own (abort flag + item counter), so that launches of one pool on different
    // streams do not share them; the launcher clears the word on the stream before the kernel
    p.abort_word = reinterpret_cast<int *>(pool->d_live + 1 + __atomic_fetch_add(&pool->launch_seq, 1u, __ATOMIC_RELAXED) % EKV_LAUNCH_SLOTS);
    p.max_blocks = max_blocks_per_seq;
    p.num_q_heads = pool->desc.num_q_heads;
    p.num_kv_heads = pool->desc.num_kv_heads;
    p.group = pool->desc.num_q_heads / pool->desc.num_kv_heads;
    p.R = R;
    p.q_tiles = (int)q_tiles;
    p.scale_log2 = scale * 1.4426950408889634f;
    const bool d128 = pool->desc.head_dim == 128;
    if (kernel == K_TWO_HEAD) return tc::launch_prefill_tc(pool, layer, p, q, out, cu_q_lens_host[R], (cudaStream_t)stream);
    if (kernel == K_ONE_HEAD)
        return d128 ? tcs::launch_prefill_tcs(pool, layer, p, q, out, cu_q_lens_host[R], (cudaStream_t)stream)
                    : tc1::launch_prefill_tc1<64>(pool, layer, p, (int)q_tiles, (cudaStream_t)stream);
    return d128 ? launch_prefill_mma<128>(pool, layer, p, (int)q_tiles, (cudaStream_t)stream)
                : launch_prefill_mma<64>(pool, layer, p, (int)q_tiles, (cudaStream_t)stream);
}
