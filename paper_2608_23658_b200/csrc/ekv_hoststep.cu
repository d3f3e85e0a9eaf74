// ekv_hoststep_*: one decode step of a layer driven from HOST buffers.
//
// A serving engine's scheduler lives on the host: every step it has new query rows, new K/V rows, slot
// mappings, block tables and lengths in host memory, and it wants the attention output back in host
// memory.  This object owns what such a step needs besides the pool -- `depth` sets of device staging
// buffers, the decode workspace, two copy streams and the events that order them -- so that one call does
//     host -> device copies | ekv_write_kv | ekv_attn_decode | device -> host copy
// and consecutive calls overlap: the inputs of step i+1 are copied in and the result of step i-1 is
// copied out while the kernels of step i run.  Everything is allocated in ekv_hoststep_create; a step
// allocates nothing.
#include <new>
#include <vector>

#include "ekv_internal.h"

struct ekv_hoststep {
    ekv_pool *pool;
    int max_batch, max_blocks, depth;
    size_t q_bytes, kv_bytes, slots_bytes, tables_bytes, lens_bytes;  // capacities of one set
    struct Set {
        uint8_t *dev;          // one allocation: q | k | v | out | slots | tables | lens
        cudaEvent_t in_done;   // inputs of the step using this set have arrived
        cudaEvent_t comp_done; // kernels of that step are done (the set's inputs may be overwritten)
        cudaEvent_t out_done;  // its result has left the device (the set's out rows may be overwritten)
    };
    std::vector<Set> sets;
    void *workspace;
    size_t workspace_bytes;
    cudaStream_t s_in, s_out;
    unsigned long long step;
};

namespace {

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

void destroy(ekv_hoststep *h) {
    if (!h) return;
    for (auto &s : h->sets) {
        if (s.dev) cudaFree(s.dev);
        if (s.in_done) cudaEventDestroy(s.in_done);
        if (s.comp_done) cudaEventDestroy(s.comp_done);
        if (s.out_done) cudaEventDestroy(s.out_done);
    }
    if (h->workspace) cudaFree(h->workspace);
    if (h->s_in) cudaStreamDestroy(h->s_in);
    if (h->s_out) cudaStreamDestroy(h->s_out);
    delete h;
}

}  // namespace

using namespace ekv;

extern "C" ekv_status_t ekv_hoststep_create(ekv_pool_t *pool, int32_t max_batch, int32_t max_blocks_per_seq, int32_t depth,
                                            ekv_hoststep_t **out) {
    if (!out) {
        set_error("ekv_hoststep_create: NULL argument");
        return EKV_ERR_INVALID;
    }
    *out = nullptr;
    ekv_status_t st = check_compute(pool, 0, "ekv_hoststep_create");
    if (st != EKV_OK) return st;
    if (max_batch < 1 || max_batch > 65535 || max_blocks_per_seq < 1 || max_blocks_per_seq > (1 << 26) || depth < 1 || depth > 8) {
        set_error("ekv_hoststep_create: bad argument (max_batch=%d, max_blocks_per_seq=%d, depth=%d)", max_batch, max_blocks_per_seq,
                  depth);
        return EKV_ERR_INVALID;
    }
    ekv_hoststep *h = new (std::nothrow) ekv_hoststep();
    if (!h) {
        set_error("ekv_hoststep_create: host allocation failed");
        return EKV_ERR_OOM;
    }
    h->pool = pool;
    h->max_batch = max_batch;
    h->max_blocks = max_blocks_per_seq;
    h->depth = depth;
    h->step = 0;
    h->workspace = nullptr;
    h->s_in = h->s_out = nullptr;
    const size_t d = pool->desc.head_dim;
    h->q_bytes = align256((size_t)max_batch * pool->desc.num_q_heads * d * 2);
    h->kv_bytes = align256((size_t)max_batch * pool->desc.num_kv_heads * d * 2);
    h->slots_bytes = align256((size_t)max_batch * sizeof(int64_t));
    h->tables_bytes = align256((size_t)max_batch * max_blocks_per_seq * sizeof(int32_t));
    h->lens_bytes = align256((size_t)max_batch * sizeof(int32_t));
    const size_t set_bytes = 2 * h->q_bytes + 2 * h->kv_bytes + h->slots_bytes + h->tables_bytes + h->lens_bytes;
    h->sets.assign(depth, ekv_hoststep::Set{nullptr, nullptr, nullptr, nullptr});
    cudaError_t e = cudaSuccess;
    for (int i = 0; i < depth && e == cudaSuccess; ++i) {
        auto &s = h->sets[i];
        e = cudaMalloc((void **)&s.dev, set_bytes);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&s.in_done, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&s.comp_done, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&s.out_done, cudaEventDisableTiming);
    }
    h->workspace_bytes = ekv_attn_workspace_bytes(pool, max_batch, max_blocks_per_seq * pool->desc.block_size);
    if (e == cudaSuccess) e = cudaMalloc(&h->workspace, h->workspace_bytes ? h->workspace_bytes : 256);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&h->s_in, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&h->s_out, cudaStreamNonBlocking);
    if (e != cudaSuccess) {
        st = cuda_fail(e, "ekv_hoststep_create");
        destroy(h);
        return st;
    }
    *out = h;
    return EKV_OK;
}

extern "C" ekv_status_t ekv_hoststep_destroy(ekv_hoststep_t *h) {
    if (!h) return EKV_OK;
    cudaSetDevice(h->pool->desc.device);
    cudaDeviceSynchronize();
    destroy(h);
    return EKV_OK;
}

extern "C" ekv_status_t ekv_hoststep_decode(ekv_hoststep_t *h, int32_t layer, const void *h_q, const void *h_k, const void *h_v,
                                            const int64_t *h_slot_mapping, const int32_t *h_block_tables,
                                            int32_t max_blocks_per_seq, const int32_t *h_seq_lens, int32_t B, float scale,
                                            void *h_out, void *stream) {
    if (!h) {
        set_error("ekv_hoststep_decode: NULL step object");
        return EKV_ERR_INVALID;
    }
    ekv_pool *pool = h->pool;
    ekv_status_t st = check_compute(pool, layer, "ekv_hoststep_decode");
    if (st != EKV_OK) return st;
    const bool with_write = h_k || h_v || h_slot_mapping;
    if (B < 0 || B > h->max_batch || max_blocks_per_seq < 1 || max_blocks_per_seq > h->max_blocks ||
        (B > 0 && (!h_q || !h_block_tables || !h_seq_lens || !h_out)) || (with_write && (!h_k || !h_v || !h_slot_mapping))) {
        set_error("ekv_hoststep_decode: bad argument (B=%d of at most %d, max_blocks_per_seq=%d of at most %d)", B, h->max_batch,
                  max_blocks_per_seq, h->max_blocks);
        return EKV_ERR_INVALID;
    }
    if (B == 0) return EKV_OK;
    cudaStream_t main = (cudaStream_t)stream;
    auto &s = h->sets[h->step % h->depth];
    uint8_t *d_q = s.dev, *d_k = d_q + h->q_bytes, *d_v = d_k + h->kv_bytes, *d_out = d_v + h->kv_bytes;
    uint8_t *d_slots = d_out + h->q_bytes, *d_tables = d_slots + h->slots_bytes, *d_lens = d_tables + h->tables_bytes;
    const size_t dd = pool->desc.head_dim;
    const size_t q_n = (size_t)B * pool->desc.num_q_heads * dd * 2, kv_n = (size_t)B * pool->desc.num_kv_heads * dd * 2;

    cudaError_t e = cudaSuccess;
    // copy-in stream: the kernels that last read this set must be done before its inputs are overwritten
    if (h->step >= (unsigned long long)h->depth) e = cudaStreamWaitEvent(h->s_in, s.comp_done, 0);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d_q, h_q, q_n, cudaMemcpyHostToDevice, h->s_in);
    if (with_write) {
        if (e == cudaSuccess) e = cudaMemcpyAsync(d_k, h_k, kv_n, cudaMemcpyHostToDevice, h->s_in);
        if (e == cudaSuccess) e = cudaMemcpyAsync(d_v, h_v, kv_n, cudaMemcpyHostToDevice, h->s_in);
        if (e == cudaSuccess) e = cudaMemcpyAsync(d_slots, h_slot_mapping, (size_t)B * sizeof(int64_t), cudaMemcpyHostToDevice, h->s_in);
    }
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(d_tables, h_block_tables, (size_t)B * max_blocks_per_seq * sizeof(int32_t), cudaMemcpyHostToDevice, h->s_in);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d_lens, h_seq_lens, (size_t)B * sizeof(int32_t), cudaMemcpyHostToDevice, h->s_in);
    if (e == cudaSuccess) e = cudaEventRecord(s.in_done, h->s_in);
    // caller's stream: inputs have arrived, and the result that last sat in this set's out rows has left
    if (e == cudaSuccess) e = cudaStreamWaitEvent(main, s.in_done, 0);
    if (e == cudaSuccess && h->step >= (unsigned long long)h->depth) e = cudaStreamWaitEvent(main, s.out_done, 0);
    if (e != cudaSuccess) return cuda_fail(e, "ekv_hoststep_decode: copy in");
    if (with_write) {
        st = ekv_write_kv(pool, layer, d_k, d_v, (const int64_t *)d_slots, B, main);
        if (st != EKV_OK) return st;
    }
    st = ekv_attn_decode(pool, layer, d_q, d_out, (const int32_t *)d_tables, max_blocks_per_seq, (const int32_t *)d_lens, B, scale,
                         h->workspace, h->workspace_bytes, main);
    if (st != EKV_OK) return st;
    e = cudaEventRecord(s.comp_done, main);
    // copy-out stream
    if (e == cudaSuccess) e = cudaStreamWaitEvent(h->s_out, s.comp_done, 0);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h_out, d_out, q_n, cudaMemcpyDeviceToHost, h->s_out);
    if (e == cudaSuccess) e = cudaEventRecord(s.out_done, h->s_out);
    if (e != cudaSuccess) return cuda_fail(e, "ekv_hoststep_decode: copy out");
    ++h->step;
    return EKV_OK;
}

extern "C" ekv_status_t ekv_hoststep_flush(ekv_hoststep_t *h, void *stream) {
    if (!h) {
        set_error("ekv_hoststep_flush: NULL step object");
        return EKV_ERR_INVALID;
    }
    cudaError_t e = cudaSetDevice(h->pool->desc.device);
    const unsigned long long n = h->step < (unsigned long long)h->depth ? h->step : (unsigned long long)h->depth;
    for (unsigned long long i = 0; i < n && e == cudaSuccess; ++i) e = cudaStreamWaitEvent((cudaStream_t)stream, h->sets[i].out_done, 0);
    if (e != cudaSuccess) return cuda_fail(e, "ekv_hoststep_flush");
    return EKV_OK;
}
