// ekv_write_kv: slot-mapped KV write = exact scatter of bf16 bit patterns into the paged pool.
// HBM-bound copy: every thread moves one 16-byte piece; a token's K (and V) row of one kv-head is
// head_dim*2 contiguous bytes on both sides, so loads and stores are fully coalesced.
#include "ekv_internal.h"

namespace ekv {

// One token's K and V rows are 2 * Hkv * (head_dim*2/16) pieces of 16 bytes.  A CTA walks over tokens; its
// threads cover a contiguous chunk of pieces at a time, issuing all loads of the chunk before its stores so
// that several 16-byte requests per thread are in flight.
static constexpr int kWriteThreads = 256;
static constexpr int kWriteUnroll = 4;

__global__ void __launch_bounds__(kWriteThreads) write_kv_kernel(uint4 *__restrict__ cache, const uint4 *__restrict__ k,
                                                                 const uint4 *__restrict__ v,
                                                                 const long long *__restrict__ slot_mapping, int T,
                                                                 int num_kv_heads, int block_size, int block_shift, int pieces_per_row, int row_shift, int token_shift,
                                                                 long long block_stride_pieces,
                                                                 const long long *__restrict__ live_ptr, unsigned *status) {
    const long long live = *live_ptr;
    const int row_pieces = num_kv_heads * pieces_per_row;  // one token's K (or V) over all heads
    const int token_pieces = 2 * row_pieces;
    const long long total = (long long)T * token_pieces;
    // a CTA takes contiguous chunks of kWriteThreads * kWriteUnroll pieces (16 KiB of source rows)
    const long long chunk = (long long)kWriteThreads * kWriteUnroll;
    for (long long base = (long long)blockIdx.x * chunk + threadIdx.x; base < total + threadIdx.x; base += (long long)gridDim.x * chunk) {
        uint4 val[kWriteUnroll];
        long long dst[kWriteUnroll];
        // one 64-bit division per trip; the pieces of the trip are then located with 32-bit arithmetic
        const long long i0 = base / token_pieces;
        const int rem0 = (int)(base - i0 * token_pieces);
#pragma unroll
        for (int u = 0; u < kWriteUnroll; ++u) {
            dst[u] = -1;
            if (base + (long long)u * kWriteThreads >= total) continue;
            const int r = rem0 + u * kWriteThreads;
            int di, rem;
            if (token_shift >= 0) {  // pieces per token a power of two (kv-head count is): no division
                di = r >> token_shift;
                rem = r & (token_pieces - 1);
            } else {
                di = r / token_pieces;
                rem = r - di * token_pieces;
            }
            const long long i = i0 + di;
            const int kv = rem >= row_pieces;
            const int hp = rem - kv * row_pieces;  // head * pieces_per_row + piece
            const int h = hp >> row_shift, c = hp & (pieces_per_row - 1);  // pieces_per_row is 8 or 16
            const long long s = slot_mapping[i];
            if (s < 0) continue;
            const long long n = s >> block_shift;  // block_size is a power of two (checked at pool creation)
            const int t = (int)(s & (block_size - 1));
            if (n >= live) {
                if (rem == 0) atomicOr(status, EKV_DEV_FLAG_OOB);
                continue;
            }
            val[u] = (kv ? v : k)[i * row_pieces + hp];
            dst[u] = n * block_stride_pieces + (((long long)(kv * num_kv_heads + h) * block_size + t) * pieces_per_row) + c;
        }
#pragma unroll
        for (int u = 0; u < kWriteUnroll; ++u)
            if (dst[u] >= 0) cache[dst[u]] = val[u];
    }
}

}  // namespace ekv

using namespace ekv;

extern "C" ekv_status_t ekv_write_kv(ekv_pool_t *pool, int32_t layer, const void *k, const void *v,
                                     const int64_t *slot_mapping, int32_t T, void *stream) {
    ekv_status_t st = check_compute(pool, layer, "ekv_write_kv");
    if (st != EKV_OK) return st;
    if (T < 0 || (T > 0 && (!k || !v || !slot_mapping)) || ((uintptr_t)k & 15) || ((uintptr_t)v & 15)) {
        set_error("ekv_write_kv: bad argument (T=%d, k=%p, v=%p, slot_mapping=%p)", T, k, v, (const void *)slot_mapping);
        return EKV_ERR_INVALID;
    }
    if (T == 0) return EKV_OK;
    const int pieces_per_row = pool->desc.head_dim * 2 / 16;
    int block_shift = 0, row_shift = 0, token_shift = -1;
    while ((1 << block_shift) < pool->desc.block_size) ++block_shift;
    while ((1 << row_shift) < pieces_per_row) ++row_shift;
    const int token_pieces = 2 * pool->desc.num_kv_heads * pieces_per_row;
    if ((token_pieces & (token_pieces - 1)) == 0)
        for (token_shift = 0; (1 << token_shift) < token_pieces;) ++token_shift;
    const long long total = (long long)T * 2 * pool->desc.num_kv_heads * pieces_per_row;
    long long blocks = (total + kWriteThreads * kWriteUnroll - 1) / (kWriteThreads * kWriteUnroll);
    const long long cap = (long long)pool->sm_count * 64;
    if (blocks > cap) blocks = cap;
    write_kv_kernel<<<(unsigned)blocks, kWriteThreads, 0, (cudaStream_t)stream>>>(
        (uint4 *)pool->layer_base(layer), (const uint4 *)k, (const uint4 *)v, (const long long *)slot_mapping, T,
        pool->desc.num_kv_heads, pool->desc.block_size, block_shift, pieces_per_row, row_shift, token_shift, (long long)(pool->block_stride / 16), pool->d_live,
        pool->d_status);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "ekv_write_kv launch");
    return EKV_OK;
}
