/*
 * ekv.h -- C ABI of libekv: attention over a block-indexed KV cache that lives in ONE
 * contiguous virtual address range per layer, backed by a base handle plus an elastic handle.
 *
 * The calls follow the paper's statement of the problem (section "An Elastic KV Mechanism"):
 *   - "Two handles, one virtual range": reserve one range per layer sized base + elastic, keep
 *     the base handle always mapped, map / unmap the elastic handle at the TOP of the range,
 *     aligned to the VMM granularity                        -> ekv_pool_create, ekv_grow, ekv_shrink
 *   - "The contiguity constraint": the attention kernel indexes the layer's tensor by block id
 *     through one base pointer, so the kernels never change when the elastic slice comes or
 *     goes                                                  -> ekv_write_kv, ekv_attn_decode,
 *                                                              ekv_attn_prefill_chunk
 *   - "Controller": committing admits the top block ids, decommitting drains, syncs, unmaps
 *                                                           -> the live-block limit and ordering
 *                                                              rules of ekv_grow / ekv_shrink
 *
 * General rules
 *   - Every call returns an ekv_status_t and never throws.  Argument errors are detected on the
 *     host before any state changes.  ekv_last_error() gives a one-line detail for the calling
 *     thread's most recent failure.
 *   - Pointers marked DEVICE are device addresses owned by the caller (any allocator); pointers
 *     marked HOST are ordinary host memory.  The pool owns the KV ranges and physical handles.
 *   - ekv_write_kv / ekv_attn_* are asynchronous: they enqueue work on `stream` (a cudaStream_t /
 *     CUstream passed as void*, NULL = legacy default stream) and return without synchronising.
 *   - ekv_grow / ekv_shrink are host-synchronous and must not run concurrently with any other
 *     call on the same pool (the caller serialises them at a step boundary).
 *   - There is no CPU fallback: without a CUDA device every compute call fails with EKV_ERR_CUDA.
 *
 * KV layout (part of the boundary).  All layers share one geometry.  From ekv_layer_ptr(layer),
 * channel x of token-in-block t of kv-head h of the K (kv=0) or V (kv=1) half of physical block n
 * is the bf16 at byte offset
 *       n*block_stride_bytes + ((((kv*num_kv_heads + h)*block_size + t)*head_dim + x) * 2 ,
 * with block_stride_bytes = block_bytes = 2*num_kv_heads*block_size*head_dim*2 by default: block n of
 * a layer occupies bytes [n*block_bytes, (n+1)*block_bytes) of that layer's own range.  Blocks
 * 0..base_blocks-1 are backed by the base handle, blocks base_blocks..base_blocks+elastic_blocks-1
 * by the elastic handle.  A slot is block*block_size + t.
 *
 * EKV_FUSED_RANGE (this build's variation on the paper's arrangement, for a cheaper toggle): the
 * driver's map / unmap / set-access cost is per call, not per byte, and one call per layer is what
 * makes a toggle take milliseconds.  With this flag the pool reserves ONE range for the whole model
 * and interleaves the layers inside every block id: block n of layer l lives at
 * (n*num_layers + l)*block_bytes, i.e. ekv_layer_ptr(l) = range + l*block_bytes and
 * block_stride_bytes = num_layers*block_bytes.  Every layer is still ONE pointer indexed by block
 * id (a strided tensor instead of a dense one), the elastic block ids are still the top of the
 * range, and grow / shrink are one map / unmap for all layers.  The kernels are the same code.
 */
#ifndef EKV_H_
#define EKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define EKV_API __attribute__((visibility("default")))
#else
#define EKV_API
#endif

typedef struct ekv_pool ekv_pool_t; /* opaque */

typedef enum ekv_status {
    EKV_OK = 0,
    EKV_ERR_INVALID = 1,   /* bad argument; nothing changed */
    EKV_ERR_CUDA = 2,      /* a CUDA runtime / driver call failed, or no device / driver */
    EKV_ERR_OOM = 3,       /* physical memory could not be created; pool left in its prior state */
    EKV_ERR_STATE = 4,     /* e.g. grow when grown, shrink when shrunk, compute on a host-only pool */
    EKV_ERR_BLOCK_OOB = 5, /* latched by a kernel: a block id or slot was outside [0, live_blocks) */
    EKV_ERR_TIMEOUT = 6,   /* latched by a kernel: a bounded wait on a copy barrier ran out */
    EKV_ERR_WORKSPACE = 7  /* workspace missing, misaligned (256 B) or too small */
} ekv_status_t;

enum { EKV_BF16 = 0 };

/* flag bits */
enum {
    EKV_START_GROWN = 1u << 0,   /* ekv_pool_create: map the elastic slice right away */
    EKV_KEEP_PHYSICAL = 1u << 1, /* ekv_shrink: unmap only, keep the elastic handle (bytes survive
                                    until the next ekv_grow maps it again) */
    EKV_FUSED_RANGE = 1u << 2,   /* ekv_pool_create: ONE virtual range and two handles for all layers
                                    instead of one range and two handles per layer (see above) */
    EKV_PREFILL_ONE_HEAD = 1u << 4, /* ekv_pool_create: ekv_attn_prefill_chunk on this pool always runs a
                                    tcgen05 kernel whose work item is ONE query head (normally chosen for
                                    head_dim 64 and for query groups of one), so that it can be tested and
                                    timed on any shape. */
    EKV_PREFILL_TWO_HEAD = 1u << 5, /* ekv_pool_create: ekv_attn_prefill_chunk on this pool runs the two-head
                                    tcgen05 kernel whenever the shape allows it (head_dim 128, query groups
                                    of two or more heads, scale > 0).  That is also the default choice for
                                    such a shape; the flag states it. */
    EKV_PREFILL_WARP_MMA = 1u << 3 /* ekv_pool_create: ekv_attn_prefill_chunk on this pool always runs the
                                    warp-level (mma.sync) kernel, never a tcgen05 one.  Same results within
                                    the stated tolerance; exists so the two kernel families can be checked
                                    against each other in one process. */
};

typedef struct ekv_pool_desc {
    int32_t device;         /* CUDA device ordinal */
    int32_t num_layers;     /* >= 1 */
    int32_t num_q_heads;    /* multiple of num_kv_heads; group = num_q_heads/num_kv_heads in 1..8 */
    int32_t num_kv_heads;
    int32_t head_dim;       /* 64 or 128 */
    int32_t block_size;     /* 16 */
    int32_t dtype;          /* EKV_BF16 */
    uint32_t flags;         /* EKV_START_GROWN | EKV_FUSED_RANGE | EKV_PREFILL_* */
    int64_t base_blocks;    /* per layer, >= 1; rounded UP to whole granules */
    int64_t elastic_blocks; /* per layer, >= 0; rounded UP to whole granules */
} ekv_pool_desc_t;

typedef struct ekv_pool_info {
    uint64_t granularity;    /* VMM minimum allocation granularity in bytes (2 MiB in the paper) */
    uint64_t block_bytes;    /* 2*num_kv_heads*block_size*head_dim*2 */
    uint64_t base_bytes;     /* per layer, after rounding */
    uint64_t elastic_bytes;  /* per layer, after rounding */
    int64_t base_blocks;     /* after rounding */
    int64_t elastic_blocks;  /* after rounding */
    int64_t live_blocks;     /* the limit last published to the kernels: base_blocks, or base_blocks +
                                elastic_blocks while grown */
    int32_t grown;           /* elastic slice mapped (in every range, or -- only after an ekv_shrink that
                                failed half way -- still in some of them) */
    int32_t physical_held;   /* elastic handles exist (mapped, or kept by EKV_KEEP_PHYSICAL) */
    int32_t num_layers;
    int32_t num_ranges;          /* virtual ranges the pool holds: num_layers, or 1 with EKV_FUSED_RANGE */
    uint64_t block_stride_bytes; /* distance between consecutive block ids of one layer: block_bytes, or
                                    num_layers*block_bytes with EKV_FUSED_RANGE */
} ekv_pool_info_t;

/*
 * ekv_pool_create -- "Two handles, one virtual range".  Per layer: reserve a virtual range of
 * (base+elastic) bytes, create + map + grant the base handle; the elastic sub-range stays unmapped
 * unless EKV_START_GROWN.  Sizes are rounded up to the allocation granularity, which must be a
 * multiple of block_bytes.  desc, out: HOST.  On failure nothing is left allocated.
 */
EKV_API ekv_status_t ekv_pool_create(const ekv_pool_desc_t *desc, ekv_pool_t **out);

/* Unmaps and releases everything the pool owns.  The caller must have synchronised all streams
 * that used the pool.  NULL is accepted. */
EKV_API ekv_status_t ekv_pool_destroy(ekv_pool_t *pool);

/* Geometry and state after rounding.  info: HOST. */
EKV_API ekv_status_t ekv_pool_info(const ekv_pool_t *pool, ekv_pool_info_t *info);

/* Device address of the layer's range; constant for the pool's life whether the elastic slice is
 * mapped or not (the paper's point: a layer's range stays where it is).  dptr: HOST, receives a DEVICE
 * address.  Touching bytes of the elastic sub-range while it is unmapped faults the context. */
EKV_API ekv_status_t ekv_layer_ptr(const ekv_pool_t *pool, int32_t layer, void **dptr);

/*
 * ekv_grow -- commit ("Toggle cost", "Controller"): for every layer create the elastic handle if
 * it is not held, map it at the top of the range, grant access; then raise the device-side live
 * limit to base+elastic on `stream`.  Elastic bytes are undefined after a grow that had to create
 * the handle.  If creation or mapping fails at any layer, everything this call mapped or created
 * is undone, the pool stays shrunk and EKV_ERR_OOM / EKV_ERR_CUDA is returned.
 * ms_out (HOST, may be NULL) receives ms_out[0] = host time of the driver calls alone and
 * ms_out[1] = host time of the whole call including stream synchronisation.
 */
EKV_API ekv_status_t ekv_grow(ekv_pool_t *pool, void *stream, uint32_t flags, double *ms_out);

/*
 * ekv_shrink -- decommit ("Controller": drain, sync, unmap).  Lowers the live limit to base_blocks
 * on `stream`, synchronises the whole device (every stream that may still read elastic blocks),
 * unmaps the elastic sub-range of every layer and, unless EKV_KEEP_PHYSICAL, releases the
 * handles (the memory returns to the driver).  Precondition the library cannot check: the caller
 * no longer uses block ids >= base_blocks (the drain step of "Controller").  A kernel launched afterwards
 * with such an id skips it and latches EKV_ERR_BLOCK_OOB instead of faulting.  ms_out as above.
 * If the driver refuses to unmap some range, the call stops there and returns EKV_ERR_CUDA: ranges
 * already unmapped stay unmapped, the others stay mapped, the pool still counts as grown
 * (ekv_pool_info: grown = 1) while the live limit is already base_blocks, so no kernel reaches the
 * elastic ids; calling ekv_shrink again retries the ranges that are left.
 */
EKV_API ekv_status_t ekv_shrink(ekv_pool_t *pool, void *stream, uint32_t flags, double *ms_out);

/*
 * ekv_write_kv -- slot-mapped KV write into the paged pool (section "Background and Motivation",
 * "KV allocation in vLLM": fixed-size blocks handed to requests).  An exact scatter of bit
 * patterns: token i's k[i,h,:] and v[i,h,:] go to slot slot_mapping[i] of `layer`.
 * k, v: DEVICE, bf16 [T, num_kv_heads, head_dim], contiguous, 16-byte aligned.
 * slot_mapping: DEVICE int64 [T]; negative = skip the token; a slot whose block is >= the live
 * limit is skipped and latches EKV_ERR_BLOCK_OOB.  Duplicate slots in one call: unspecified
 * winner.  T == 0 is a no-op.
 */
EKV_API ekv_status_t ekv_write_kv(ekv_pool_t *pool, int32_t layer, const void *k, const void *v,
                          const int64_t *slot_mapping, int32_t T, void *stream);

/* Bytes of scratch that cover EVERY ekv_attn_decode call with 1 <= B <= max_batch and
 * max_blocks_per_seq*block_size <= max_seq_len (rounded up to a block) -- an upper bound over all
 * those shapes, not the need of the largest one alone (a shorter table can be cut into more key
 * ranges than a longer one).  ekv_attn_prefill_chunk needs none.  Returns 0 for a NULL pool. */
EKV_API size_t ekv_attn_workspace_bytes(const ekv_pool_t *pool, int32_t max_batch, int32_t max_seq_len);

/* The split plan ekv_attn_decode will use for a call of exactly this shape (ours; the paper has no
 * counterpart): keys per range, ranges per sequence at the maximum length, and the scratch that one
 * call needs.  Any of the three HOST out-pointers may be NULL.  Depends only on the pool's geometry,
 * the device's SM count, B and max_blocks_per_seq. */
EKV_API ekv_status_t ekv_attn_decode_plan(const ekv_pool_t *pool, int32_t B, int32_t max_blocks_per_seq,
                                          int32_t *chunk_tokens, int32_t *nsplit, size_t *workspace_bytes);

/*
 * ekv_attn_decode -- grouped-query attention of ONE query token per sequence over that sequence's
 * cached keys/values (the kernel "The contiguity constraint" is about; decode contributes
 * one token per sequence per step, "Why the penalty is small").
 *   out[b,h,:] = sum_j softmax_j(scale * q[b,h,:].K_j) V_j ,  j = 0 .. seq_lens[b]-1,
 * where key j of sequence b is token j%block_size of block block_tables[b][j/block_size] and query
 * head h reads kv-head h/(num_q_heads/num_kv_heads).  seq_lens[b] includes the query token (its
 * K/V were written first).  bf16 in, fp32 accumulate, bf16 out (round to nearest even).
 * q, out: DEVICE bf16 [B, num_q_heads, head_dim], 16-byte aligned.
 * block_tables: DEVICE int32 [B, max_blocks_per_seq]; entries at or past ceil(seq_len/block_size)
 * are never read.  seq_lens: DEVICE int32 [B]; 0 gives a zero row; values above
 * max_blocks_per_seq*block_size are clamped to it.
 * workspace: DEVICE, 256-byte aligned, >= ekv_attn_workspace_bytes(pool, B, max_blocks_per_seq*
 * block_size); contents need no initialisation; calls that share it must be stream-ordered.
 * Two passes: a split pass over fixed-size key ranges writing fp32 partials, and a combine pass.
 * The split plan depends only on (B, max_blocks_per_seq), so results are bitwise reproducible and
 * independent of which physical blocks hold the data.
 */
EKV_API ekv_status_t ekv_attn_decode(ekv_pool_t *pool, int32_t layer, const void *q, void *out,
                             const int32_t *block_tables, int32_t max_blocks_per_seq,
                             const int32_t *seq_lens, int32_t B, float scale, void *workspace,
                             size_t workspace_bytes, void *stream);

/*
 * ekv_attn_decode_static_scratch -- the paper has no counterpart to this call; it exists for users of
 * this library who cannot allocate device memory at the moment they need decode attention: an engine
 * that has already given all free device memory to the KV pool (so that a fresh allocation would
 * fail, or would take the very reserve ekv_shrink hands back), a C host without any tensor library
 * or allocator of its own, or code on a path where entering the CUDA allocator is forbidden.
 * It computes exactly what ekv_attn_decode computes, with the same arguments minus the workspace:
 * the split pass's fp32 partials go to a fixed array of EKV_STATIC_SCRATCH_BYTES that is part of
 * the library image (each GPU that loads the library holds it until the process ends).  The call
 * itself allocates and frees nothing.
 *   - A call whose split plan needs more than EKV_STATIC_SCRATCH_BYTES is refused with
 *     EKV_ERR_WORKSPACE and launches nothing (ekv_last_error() states the need); such shapes must use
 *     ekv_attn_decode.  ekv_attn_workspace_bytes() gives the need of a shape in advance.
 *   - The first call on a device looks up the array's device address (one cudaGetSymbolAddress with
 *     that device current) and remembers it; make that first call outside any stream capture.
 *   - All calls on a device share the one array and find in it whatever the previous call left.
 *     Nothing in it has to start at zero (every partial that is read was written by the same call),
 *     so nothing is cleared.  Two calls whose kernels may overlap on the GPU (different streams
 *     without an ordering between them) race on it: keep them stream-ordered.
 */
#define EKV_STATIC_SCRATCH_BYTES (64u << 20)
EKV_API ekv_status_t ekv_attn_decode_static_scratch(ekv_pool_t *pool, int32_t layer, const void *q, void *out,
                                                    const int32_t *block_tables, int32_t max_blocks_per_seq,
                                                    const int32_t *seq_lens, int32_t B, float scale, void *stream);

/*
 * ekv_attn_decode_two_tensor -- the alternative the paper weighs and rejects in "The contiguity
 * constraint": keep base and elastic blocks in two separate tensors and teach the attention kernel
 * to choose between them.  Same computation
 * and arguments as ekv_attn_decode, except that block ids 0..base_blocks-1 address the pool's base
 * range of `layer` and ids base_blocks..base_blocks+second_blocks-1 address `second_tensor`, a
 * separately allocated DEVICE buffer of second_blocks*block_bytes with the same block layout (16-byte
 * aligned; the pool's elastic range plays no part and may be unmapped).  Ids at or beyond
 * base_blocks+second_blocks are skipped and latch EKV_ERR_BLOCK_OOB.  It exists to measure what the
 * single-range design saves (a second tensor map and a choice per block inside the kernel); results
 * are bitwise identical to ekv_attn_decode on the same logical data.
 */
EKV_API ekv_status_t ekv_attn_decode_two_tensor(ekv_pool_t *pool, int32_t layer, const void *second_tensor,
                                                int64_t second_blocks, const void *q, void *out, const int32_t *block_tables,
                                                int32_t max_blocks_per_seq, const int32_t *seq_lens, int32_t B, float scale,
                                                void *workspace, size_t workspace_bytes, void *stream);

/*
 * ekv_hoststep_* -- one decode step of a layer driven from HOST buffers (the scheduler of the paper's
 * engine lives on the host: "Controller" acts between scheduler steps, and every step hands the
 * attention kernel new rows, slot mappings, block tables and lengths).  The object owns `depth` sets of
 * device staging buffers, the decode workspace, two copy streams and their events; all of it is
 * allocated by ekv_hoststep_create, a step allocates nothing.
 *
 * ekv_hoststep_decode enqueues, for one step,
 *     host -> device copies of the inputs | ekv_write_kv (unless h_k, h_v, h_slot_mapping are all NULL)
 *     | ekv_attn_decode | device -> host copy of the result
 * with the kernels on `stream` and the copies on the object's own streams, so that with depth >= 2 the
 * copy-in of step i+1 and the copy-out of step i-1 overlap the kernels of step i.  It returns without
 * synchronising.  Results are exactly those of ekv_write_kv + ekv_attn_decode on the same data.
 *   h_q, h_out: HOST bf16 [B, num_q_heads, head_dim].  h_k, h_v: HOST bf16 [B, num_kv_heads, head_dim].
 *   h_slot_mapping: HOST int64 [B].  h_block_tables: HOST int32 [B, max_blocks_per_seq].
 *   h_seq_lens: HOST int32 [B].  Use pinned (page-locked) memory: copies from pageable memory are
 *   staged by the driver and do not overlap.  Every host buffer must stay valid and unmodified until
 *   the step has finished; h_out holds the result once the work enqueued by ekv_hoststep_flush (or a
 *   later step on the same set) has completed.
 *   B <= max_batch and max_blocks_per_seq <= the value given at creation, else EKV_ERR_INVALID.
 * ekv_hoststep_flush makes `stream` wait for every copy-out still in flight; synchronise `stream`
 * afterwards to read the results on the host.
 * The object refers to the pool: destroy it before the pool.  Calls on one object must not run
 * concurrently.  ekv_hoststep_destroy synchronises the device.
 */
typedef struct ekv_hoststep ekv_hoststep_t;
EKV_API ekv_status_t ekv_hoststep_create(ekv_pool_t *pool, int32_t max_batch, int32_t max_blocks_per_seq, int32_t depth,
                                         ekv_hoststep_t **out);
EKV_API ekv_status_t ekv_hoststep_destroy(ekv_hoststep_t *step);
EKV_API ekv_status_t ekv_hoststep_decode(ekv_hoststep_t *step, int32_t layer, const void *h_q, const void *h_k, const void *h_v,
                                         const int64_t *h_slot_mapping, const int32_t *h_block_tables,
                                         int32_t max_blocks_per_seq, const int32_t *h_seq_lens, int32_t B, float scale,
                                         void *h_out, void *stream);
EKV_API ekv_status_t ekv_hoststep_flush(ekv_hoststep_t *step, void *stream);

/*
 * ekv_attn_prefill_chunk -- causal attention of a prompt chunk over its cached prefix plus itself
 * (chunked prefill: "The Decisive Test", "Why the penalty is small": chunking splits the same
 * work across steps).  Request r owns query rows cu_q_lens[r] .. cu_q_lens[r+1]-1 (c_r rows) and
 * seq_lens[r] = prefix_r + c_r keys; row i of the chunk sits at absolute position prefix_r + i and
 * attends to keys 0 .. prefix_r + i.  All keys/values, the chunk's own included, are read from
 * the cache (run ekv_write_kv for the chunk first).
 * q, out: DEVICE bf16 [T, num_q_heads, head_dim], 16-byte aligned, T = cu_q_lens[R].
 * block_tables: DEVICE int32 [R, max_blocks_per_seq].  seq_lens: DEVICE int32 [R].
 * cu_q_lens: DEVICE int32 [R+1], non-decreasing, cu_q_lens[0] = 0.
 * cu_q_lens_host: HOST copy of the same R+1 values (used to size the launch without a sync).
 * Requests with seq_lens[r] < c_r are invalid (rows produce zeros, EKV_ERR_BLOCK_OOB is latched).
 * Needs no workspace.  Calls on one pool may run at the same time on different streams; each call in flight
 * holds one of 64 per-pool launch words (work counter of the persistent kernel), so more than 64 calls of one
 * pool in flight at once are not supported.
 */
EKV_API ekv_status_t ekv_attn_prefill_chunk(ekv_pool_t *pool, int32_t layer, const void *q, void *out,
                                    const int32_t *block_tables, int32_t max_blocks_per_seq,
                                    const int32_t *cu_q_lens, const int32_t *cu_q_lens_host,
                                    const int32_t *seq_lens, int32_t R, float scale, void *stream);

/*
 * ---- Block pool with a gated elastic id range, drain, and the one-step-ahead controller ----------
 * Paper, section "An Elastic KV Mechanism".  Paragraph "Two handles, one virtual range": the block
 * ids at the top of the range are gated inside the block pool, which hands them out only while the
 * elastic slice is committed.  Section "Background and Motivation": the block pool is nothing but a
 * free list of integers.  Paragraph "Controller": the slice is lent to the pool while the engine
 * only decodes and taken back at the step boundary before a prefill, with hysteresis; a commit
 * raises the number of usable blocks and admits the top ids; a decommit moves live data out of
 * those ids, waits for the device, and only then unmaps.
 *
 * All of this is host-side bookkeeping (no CUDA call) except ekv_move_blocks.  Intended order of a
 * decommit:  ekv_blockpool_gate_elastic -> ekv_blockpool_drain_plan -> ekv_move_blocks (+ the caller
 * rewrites its block tables) -> ekv_blockpool_drain_commit -> ekv_shrink.   Of a commit:
 * ekv_grow -> ekv_blockpool_admit_elastic.
 */
typedef struct ekv_blockpool ekv_blockpool_t;   /* opaque */
typedef struct ekv_controller ekv_controller_t; /* opaque */

typedef struct ekv_blockpool_stats {
    int64_t base_blocks, elastic_blocks;
    int64_t free_base, free_elastic;
    int64_t elastic_in_use;   /* elastic ids currently handed out (what a drain must move) */
    int64_t num_gpu_blocks;   /* base_blocks, or base_blocks + elastic_blocks while admitted */
    int32_t admitted;         /* elastic ids may be handed out */
    int32_t draining;         /* a drain plan is outstanding */
} ekv_blockpool_stats_t;

/* Ids 0..base_blocks-1 are base blocks, base_blocks..base_blocks+elastic_blocks-1 elastic blocks
 * (gated until ekv_blockpool_admit_elastic).  out: HOST. */
EKV_API ekv_status_t ekv_blockpool_create(int64_t base_blocks, int64_t elastic_blocks, ekv_blockpool_t **out);
EKV_API ekv_status_t ekv_blockpool_destroy(ekv_blockpool_t *bp);
/* Hands out n ids (HOST array ids_out), all or nothing: EKV_ERR_OOM and nothing allocated if fewer
 * are available.  Base ids go first (never-freed ones in ascending order, then most recently freed);
 * elastic ids only while admitted and only once no base id is free. */
EKV_API ekv_status_t ekv_blockpool_alloc(ekv_blockpool_t *bp, int64_t n, int32_t *ids_out);
/* Returns ids to the free list.  Any id that is not currently allocated (or appears twice) fails the
 * whole call with EKV_ERR_INVALID and frees nothing; so does, with EKV_ERR_STATE, an id on either
 * side of an outstanding drain plan. */
EKV_API ekv_status_t ekv_blockpool_free(ekv_blockpool_t *bp, const int32_t *ids, int64_t n);
/* After ekv_grow: elastic ids may be handed out; num_gpu_blocks grows. */
EKV_API ekv_status_t ekv_blockpool_admit_elastic(ekv_blockpool_t *bp);
/* Before ekv_shrink: stop handing out elastic ids; *elastic_in_use (HOST, may be NULL) = how many
 * are still held by requests. */
EKV_API ekv_status_t ekv_blockpool_gate_elastic(ekv_blockpool_t *bp, int64_t *elastic_in_use);
/* Drain plan: for every elastic id in use (ascending) a free base id is reserved; pair i says "move
 * block from_ids[i] to to_ids[i]".  *n_out = number of pairs.  EKV_ERR_OOM (nothing reserved) if the
 * base range has too few free blocks -- the caller must preempt requests first; EKV_ERR_INVALID if
 * capacity < *n_out; EKV_ERR_STATE unless gated and no other drain is outstanding.  HOST arrays.
 * Until ekv_blockpool_drain_commit the ids of the plan (both sides) must not be freed. */
EKV_API ekv_status_t ekv_blockpool_drain_plan(ekv_blockpool_t *bp, int32_t *from_ids, int32_t *to_ids, int64_t capacity,
                                              int64_t *n_out);
/* After the data was moved and the block tables rewritten: the elastic ids of the plan become free. */
EKV_API ekv_status_t ekv_blockpool_drain_commit(ekv_blockpool_t *bp);
EKV_API ekv_status_t ekv_blockpool_stats(const ekv_blockpool_t *bp, ekv_blockpool_stats_t *out);

/* Copies whole blocks src_ids[i] -> dst_ids[i] in EVERY layer of the pool (the data movement of a
 * drain), asynchronously on `stream`.  src_ids, dst_ids: DEVICE int32 [n]; the two sets must be
 * disjoint.  Ids outside the live range are skipped and latch EKV_ERR_BLOCK_OOB.  Bit-exact copy. */
EKV_API ekv_status_t ekv_move_blocks(ekv_pool_t *pool, const int32_t *src_ids, const int32_t *dst_ids, int32_t n, void *stream);

typedef struct ekv_controller_desc {
    int32_t commit_after_decode_steps; /* hysteresis: commit only after this many consecutive steps without a large prefill (>= 1) */
    int32_t reserve_prefill_tokens;    /* a step with at least this many prefill tokens needs the activation reserve (>= 1) */
} ekv_controller_desc_t;

typedef enum ekv_action { EKV_ACT_NONE = 0, EKV_ACT_COMMIT = 1, EKV_ACT_DECOMMIT = 2 } ekv_action_t;

typedef struct ekv_controller_stats {
    int64_t steps, commits, decommits;
    int32_t committed, decode_streak;
} ekv_controller_stats_t;

EKV_API ekv_status_t ekv_controller_create(const ekv_controller_desc_t *desc, int32_t initially_committed, ekv_controller_t **out);
EKV_API ekv_status_t ekv_controller_destroy(ekv_controller_t *ctrl);
/* Called at the scheduler boundary with what the scheduler already knows about the NEXT step: its
 * number of prefill tokens (0 = decode-only).  EKV_ACT_DECOMMIT: the next step needs the reserve, give
 * it back before running it.  EKV_ACT_COMMIT: the hysteresis window of quiet steps has passed, lend the
 * reserve to the KV pool.  The controller assumes the caller carries the action out. */
EKV_API ekv_action_t ekv_controller_decide(ekv_controller_t *ctrl, int32_t next_prefill_tokens);
EKV_API ekv_status_t ekv_controller_stats(const ekv_controller_t *ctrl, ekv_controller_stats_t *out);

/*
 * ekv_selftest_bounded_wait -- ours (error handling; the paper has no counterpart).  Every wait inside
 * the kernels is bounded: when it runs out, the kernel latches EKV_ERR_TIMEOUT, finishes, and the
 * context stays usable.  This call runs that path on purpose and harmlessly: it enqueues on `stream`
 * one small kernel that waits, with the kernels' own wait routines (the one bounded by a clock, then the
 * one bounded by a number of polls) and a limit of limit_us microseconds each (1 .. 100000), on a barrier
 * that nothing arrives on.  After the stream has been synchronised
 * ekv_poll_status returns EKV_ERR_TIMEOUT once, and every other call keeps working.
 * waited_ns_device: DEVICE uint64, or NULL; receives how long the wait lasted.
 */
EKV_API ekv_status_t ekv_selftest_bounded_wait(ekv_pool_t *pool, int32_t limit_us, uint64_t *waited_ns_device, void *stream);

/* Non-blocking read-and-clear of the status latched by kernels (EKV_OK, EKV_ERR_BLOCK_OOB or
 * EKV_ERR_TIMEOUT; the latter wins).  Meaningful after the launching stream was synchronised. */
EKV_API ekv_status_t ekv_poll_status(ekv_pool_t *pool);

EKV_API const char *ekv_status_string(ekv_status_t status);

/* One-line description of the calling thread's most recent failing call ("" if none). */
EKV_API const char *ekv_last_error(void);

/*
 * Virtual-memory backend.  The pool's state machine (rounding, create / grow / shrink / destroy,
 * unwinding after a failure) talks to the driver only through this table.  The default table
 * calls the CUDA driver VMM API (cuMemAddressReserve, cuMemCreate, cuMemMap, cuMemSetAccess,
 * cuMemUnmap, cuMemRelease, cuMemAddressFree, cuMemGetAllocationGranularity).  Installing another
 * table lets the state machine be exercised on a host without a GPU; pools created while a
 * replacement table is installed are host-only: they hold no device state and every compute call
 * on them returns EKV_ERR_STATE.  Each function returns 0 on success, 2 for out-of-memory, any
 * other value for failure.  ekv_set_vmm_backend(NULL) restores the default; it must not be
 * called while pools exist.
 */
typedef struct ekv_vmm_backend {
    void *user;
    int (*granularity)(void *user, int device, uint64_t *bytes);
    int (*reserve)(void *user, uint64_t size, uint64_t alignment, uint64_t *va);
    int (*unreserve)(void *user, uint64_t va, uint64_t size);
    int (*create)(void *user, uint64_t size, int device, uint64_t *handle);
    int (*release)(void *user, uint64_t handle);
    int (*map)(void *user, uint64_t va, uint64_t size, uint64_t handle);
    int (*unmap)(void *user, uint64_t va, uint64_t size);
    int (*set_access)(void *user, uint64_t va, uint64_t size, int device);
} ekv_vmm_backend_t;

EKV_API ekv_status_t ekv_set_vmm_backend(const ekv_vmm_backend_t *backend);

#ifdef __cplusplus
}
#endif
#endif /* EKV_H_ */
