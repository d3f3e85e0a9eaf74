/*
 * ekv_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, obviously-correct CPU statement of what the elastic-KV hot path
 * computes.  Only tests, the smoke check and the benchmark's cpu_baseline /
 * reference legs may build or call this file.  It shares no code, header, table
 * or constant with the CUDA library and neither includes the other.
 *
 * What it states, and where the paper fixes it:
 *
 *  - Addressing.  The paper's section "An Elastic KV Mechanism", paragraph "The
 *    contiguity constraint": the KV cache is one contiguous tensor per layer and
 *    the attention kernel indexes it by block id through one base pointer.
 *    Paragraph "Two handles, one virtual range": the elastic slice is a sub-range
 *    at the TOP of that range, so the outermost index must be the block id.
 *    Section "Background and Motivation", paragraph "KV allocation in vLLM": the
 *    cache is a pool of fixed-size blocks handed to requests.
 *    The element order INSIDE a block is not given by the paper; the reading
 *    used by this build is (K|V, kv-head, token-in-block, channel), restated
 *    here independently in ekv_oracle_elem_index().
 *
 *  - Attention.  The paper only says "the attention kernel" (same section); the
 *    operation is ordinary scaled-dot-product attention with grouped query
 *    heads, written below as its textbook definition: scores, max, exp, sum,
 *    weighted mean of V rows.  Two passes, ascending key order, no tiling, no
 *    running rescale, no split over keys.  Arithmetic is IEEE double on the
 *    exact values of the bf16 inputs; the paper fixes no precision.
 *
 *  - Chunked prefill.  Section "The Decisive Test", paragraph "Why the penalty is
 *    small": a prompt processed in chunks does the same total work as one
 *    step, i.e. a chunk row at absolute position pos attends to keys 0..pos.
 *
 * Parity pins (tests/test_oracle_*.py): brute-force float64 NumPy restatement,
 * torch scaled_dot_product_attention on contiguous KV, closed forms (single key,
 * identical keys, zero query, dominant key), permutation / chunking / GQA
 * invariants, exact-scatter round trip.  Nothing here is "parity unpinned".
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* bf16 -> double, exact: a bf16 is the top 16 bits of an IEEE binary32. */
static double bf16_to_double(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Element index (in bf16 elements) of channel x of token-in-block t of kv-head h
 * of the K (kv=0) or V (kv=1) part of physical block n, from the layer base. */
int64_t ekv_oracle_elem_index(int64_t n, int kv, int h, int t, int x,
                              int num_kv_heads, int block_size, int head_dim) {
    int64_t i = n;
    i = i * 2 + kv;
    i = i * num_kv_heads + h;
    i = i * block_size + t;
    i = i * head_dim + x;
    return i;
}

int ekv_oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Slot-mapped KV write: an exact scatter of bit patterns.
 * For i = 0..T-1 in order: s = slot_mapping[i]; s < 0 -> skip;
 * block n = s / block_size, t = s % block_size; n >= live_blocks -> count it in
 * *oob and skip; else copy K[i,h,:] and V[i,h,:] for every kv-head h.
 * Later tokens overwrite earlier ones that name the same slot.
 */
void ekv_oracle_write_kv(uint16_t *cache, int64_t live_blocks, int num_kv_heads,
                         int block_size, int head_dim, const uint16_t *k,
                         const uint16_t *v, const int64_t *slot_mapping, int T,
                         int64_t *oob) {
    int64_t bad = 0;
    for (int i = 0; i < T; ++i) {
        int64_t s = slot_mapping[i];
        if (s < 0) continue;
        int64_t n = s / block_size;
        int t = (int)(s % block_size);
        if (n >= live_blocks) { ++bad; continue; }
        for (int h = 0; h < num_kv_heads; ++h) {
            for (int x = 0; x < head_dim; ++x) {
                int64_t src = ((int64_t)i * num_kv_heads + h) * head_dim + x;
                cache[ekv_oracle_elem_index(n, 0, h, t, x, num_kv_heads, block_size, head_dim)] = k[src];
                cache[ekv_oracle_elem_index(n, 1, h, t, x, num_kv_heads, block_size, head_dim)] = v[src];
            }
        }
    }
    if (oob) *oob = bad;
}

/*
 * One attention row: query vector qrow (head_dim bf16) of a query head whose
 * kv-head is g, over keys 0..nkeys-1 of the sequence whose physical blocks are
 * table[0], table[1], ...   out[x] = sum_j softmax_j(scale * q.K_j) * V_j[x].
 * nkeys == 0 gives zeros.
 */
static void attend_row(const uint16_t *cache, const int32_t *table, int64_t nkeys,
                       const uint16_t *qrow, int g, int num_kv_heads, int block_size,
                       int head_dim, double scale, double *score, double *out) {
    for (int x = 0; x < head_dim; ++x) out[x] = 0.0;
    if (nkeys <= 0) return;
    /* pass 1: scores and their maximum */
    double m = -INFINITY;
    for (int64_t j = 0; j < nkeys; ++j) {
        int64_t n = table[j / block_size];
        int t = (int)(j % block_size);
        const uint16_t *krow = cache + ekv_oracle_elem_index(n, 0, g, t, 0, num_kv_heads, block_size, head_dim);
        double dot = 0.0;
        for (int x = 0; x < head_dim; ++x) dot += bf16_to_double(qrow[x]) * bf16_to_double(krow[x]);
        score[j] = scale * dot;
        if (score[j] > m) m = score[j];
    }
    /* pass 2: weights, their sum, weighted sum of V rows */
    double l = 0.0;
    for (int64_t j = 0; j < nkeys; ++j) {
        int64_t n = table[j / block_size];
        int t = (int)(j % block_size);
        const uint16_t *vrow = cache + ekv_oracle_elem_index(n, 1, g, t, 0, num_kv_heads, block_size, head_dim);
        double p = exp(score[j] - m);
        l += p;
        for (int x = 0; x < head_dim; ++x) out[x] += p * bf16_to_double(vrow[x]);
    }
    for (int x = 0; x < head_dim; ++x) out[x] /= l;
}

/*
 * Decode attention: one query token per sequence.  seq_lens[b] counts the query
 * token itself (its K/V are already in the cache), so sequence b attends to keys
 * 0..seq_lens[b]-1.  q, out: [B, Hq, d]; block_tables: [B, max_blocks_per_seq].
 * Query head h reads kv-head h / (Hq / Hkv).
 */
void ekv_oracle_attn_decode(const uint16_t *cache, int num_q_heads, int num_kv_heads,
                            int block_size, int head_dim, const uint16_t *q, double *out,
                            const int32_t *block_tables, int max_blocks_per_seq,
                            const int32_t *seq_lens, int B, double scale) {
    int group = num_q_heads / num_kv_heads;
    int64_t work = (int64_t)B * num_q_heads;
#pragma omp parallel
    {
        double *score = NULL;
        int64_t cap = 0;
#pragma omp for schedule(dynamic, 1)
        for (int64_t w = 0; w < work; ++w) {
            int b = (int)(w / num_q_heads), h = (int)(w % num_q_heads);
            int64_t L = seq_lens[b];
            if (L > cap) { free(score); score = (double *)malloc(sizeof(double) * (size_t)L); cap = L; }
            attend_row(cache, block_tables + (int64_t)b * max_blocks_per_seq, L,
                       q + ((int64_t)b * num_q_heads + h) * head_dim, h / group, num_kv_heads,
                       block_size, head_dim, scale, score,
                       out + ((int64_t)b * num_q_heads + h) * head_dim);
        }
        free(score);
    }
}

/*
 * Chunked-prefill attention.  Request r owns query rows cu_q_lens[r] ..
 * cu_q_lens[r+1]-1 (c_r rows); seq_lens[r] = cached prefix p_r + c_r.  Row i of
 * the chunk is the token at absolute position p_r + i and attends to keys
 * 0 .. p_r + i (causal, aligned to the END of the sequence).  All keys and
 * values, the chunk's own included, are read from the cache.
 * q: [T, Hq, d].  If rows == NULL every row is computed and out is [T, Hq, d];
 * otherwise only the nrows global row indices rows[] are computed and out is
 * [nrows, Hq, d] in that order (used to check samples of very large chunks).
 */
void ekv_oracle_attn_prefill_chunk(const uint16_t *cache, int num_q_heads, int num_kv_heads,
                                   int block_size, int head_dim, const uint16_t *q, double *out,
                                   const int32_t *block_tables, int max_blocks_per_seq,
                                   const int32_t *cu_q_lens, const int32_t *seq_lens, int R,
                                   double scale, const int32_t *rows, int nrows) {
    int group = num_q_heads / num_kv_heads;
    int total = rows ? nrows : cu_q_lens[R];
    int64_t work = (int64_t)total * num_q_heads;
#pragma omp parallel
    {
        double *score = NULL;
        int64_t cap = 0;
#pragma omp for schedule(dynamic, 1)
        for (int64_t w = 0; w < work; ++w) {
            int slot = (int)(w / num_q_heads), h = (int)(w % num_q_heads);
            int row = rows ? rows[slot] : slot;
            int r = 0;
            while (r + 1 < R && row >= cu_q_lens[r + 1]) ++r;
            int c = cu_q_lens[r + 1] - cu_q_lens[r];
            int i = row - cu_q_lens[r];
            int64_t prefix = (int64_t)seq_lens[r] - c;
            int64_t nkeys = prefix + i + 1;
            if (nkeys > cap) { free(score); score = (double *)malloc(sizeof(double) * (size_t)nkeys); cap = nkeys; }
            attend_row(cache, block_tables + (int64_t)r * max_blocks_per_seq, nkeys,
                       q + ((int64_t)row * num_q_heads + h) * head_dim, h / group, num_kv_heads,
                       block_size, head_dim, scale, score,
                       out + ((int64_t)slot * num_q_heads + h) * head_dim);
        }
        free(score);
    }
}
