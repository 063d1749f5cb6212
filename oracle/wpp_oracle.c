/*
 * TEST INFRASTRUCTURE — not part of the product path.
 *
 * Plain fp64 CPU oracle for one pipeline stage's chunked-prefill attention over
 * a paged KV cache with a reused prefix.  It is the textbook definition written
 * out row by row; there is no tiling, no online softmax and no reordering.  It
 * shares no code with the CUDA library.
 *
 * What it follows:
 *   - A request with n cached tokens and page size B occupies ceil(n/B) logical
 *     blocks whose physical pages need not be contiguous and may be shared
 *     between requests (paper, Section 3.2 "Reuse").
 *   - Query heads share K/V heads (grouped-query attention; Section 3.1).
 *   - The n-th token attends to all previous tokens and itself (Section 3.1:
 *     O(n) work for the n-th token over a growing KV cache).
 *   - The uncached suffix is processed in contiguous chunks; a chunk is the span
 *     (request, starting token, length) (Section 4 "Waves and lanes", Section 4.6).
 *   - Prefill fills the cache: the chunk's K/V land in the blocks reserved for
 *     the suffix (Section 4.1, steps 3-5).
 *
 * Readings where the paper is silent: bottom-right aligned causal mask (chunk
 * row t, absolute position P+t, sees keys 0..P+t inclusive), scale 1/sqrt(d)
 * unless given, kv_head = q_head / (Hq/Hkv), no bias/window/sinks.
 *
 * Layouts (all bf16 stored as uint16 bit patterns):
 *   q, out      [T][Hq][d]      T = sum of chunk lengths, requests concatenated
 *   k_new,v_new [T][Hkv][d]
 *   pools       [num_pages][Hkv][B][d]
 *   block_tables[R][max_blocks]  int32, entry j = physical page of tokens [jB,(j+1)B)
 *
 * Pins (see tests, "not gpu"): brute-force dense causal attention, chunked ==
 * one-shot, shared == private pages, any chunk split, closed forms, SDPA in fp64.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static inline double bf16_to_f64(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

int wpp_oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* O-append: copy each new token's K/V bit patterns to pool[page][h][slot][:],
 * pos = P_i + t, page = bt[i][pos / B], slot = pos % B.  Returns 0, or -1 on a bad page id. */
int wpp_oracle_append(const uint16_t* k_new, const uint16_t* v_new, uint16_t* k_pool, uint16_t* v_pool,
                      const int32_t* block_tables, const int32_t* prefix_lens, const int32_t* chunk_lens,
                      int32_t R, int32_t Hkv, int32_t d, int32_t B, int32_t max_blocks, int32_t num_pages) {
    int64_t off = 0;
    for (int32_t i = 0; i < R; ++i) {
        for (int32_t t = 0; t < chunk_lens[i]; ++t) {
            int64_t pos = (int64_t)prefix_lens[i] + t;
            int64_t blk = pos / B;
            if (blk >= max_blocks) return -1;
            int32_t page = block_tables[(int64_t)i * max_blocks + blk];
            if (page < 0 || page >= num_pages) return -1;
            int64_t slot = pos % B;
            for (int32_t h = 0; h < Hkv; ++h) {
                const uint16_t* ks = k_new + ((off + t) * Hkv + h) * (int64_t)d;
                const uint16_t* vs = v_new + ((off + t) * Hkv + h) * (int64_t)d;
                int64_t dst = (((int64_t)page * Hkv + h) * B + slot) * (int64_t)d;
                for (int32_t e = 0; e < d; ++e) {
                    k_pool[dst + e] = ks[e];
                    v_pool[dst + e] = vs[e];
                }
            }
        }
        off += chunk_lens[i];
    }
    return 0;
}

/* One (request i, chunk row t, query head h): n = P_i + t + 1 visible keys.
 * s_j = scale * <q, K_j>; m = max s_j; w_j = exp(s_j - m); O = sum w_j V_j / sum w_j; lse = m + log sum w_j.
 * Sums run in increasing j (and increasing e inside the dot product). */
static void attention_row(const uint16_t* q_row, const uint16_t* k_pool, const uint16_t* v_pool,
                          const int32_t* bt_row, int64_t n, int32_t g, int32_t Hkv, int32_t d, int32_t B,
                          double scale, double* scores, double* out_row, double* lse_out, double* top2_out) {
    double qd[1024];
    for (int32_t e = 0; e < d; ++e) qd[e] = bf16_to_f64(q_row[e]);
    double m = -INFINITY, second = -INFINITY;
    for (int64_t j = 0; j < n; ++j) {
        int64_t page = bt_row[j / B];
        const uint16_t* kr = k_pool + ((page * Hkv + g) * B + (j % B)) * (int64_t)d;
        double acc = 0.0;
        for (int32_t e = 0; e < d; ++e) acc += qd[e] * bf16_to_f64(kr[e]);
        double s = scale * acc;
        scores[j] = s;
        if (s > m) { second = m; m = s; }
        else if (s > second) second = s;
    }
    if (top2_out) { top2_out[0] = m; top2_out[1] = second; }
    double denom = 0.0;
    for (int32_t e = 0; e < d; ++e) out_row[e] = 0.0;
    for (int64_t j = 0; j < n; ++j) {
        int64_t page = bt_row[j / B];
        const uint16_t* vr = v_pool + ((page * Hkv + g) * B + (j % B)) * (int64_t)d;
        double w = exp(scores[j] - m);
        denom += w;
        for (int32_t e = 0; e < d; ++e) out_row[e] += w * bf16_to_f64(vr[e]);
    }
    for (int32_t e = 0; e < d; ++e) out_row[e] /= denom;
    if (lse_out) *lse_out = m + log(denom);
}

/* O-attn on a list of (request, row, head) units; out [n_units][d], lse [n_units] (may be NULL), top2 [n_units][2]
 * (may be NULL): the largest and second largest score of the row, which tell how well conditioned the softmax is.
 * Reads the pools only (after O-append), never k_new/v_new, never a slot >= P_i + t + 1. */
int wpp_oracle_attention_units(const uint16_t* q, const uint16_t* k_pool, const uint16_t* v_pool,
                               const int32_t* block_tables, const int32_t* prefix_lens,
                               const int32_t* chunk_lens, int32_t R, int32_t Hq, int32_t Hkv, int32_t d,
                               int32_t B, int32_t max_blocks, double scale, const int32_t* units /* [n][3] */,
                               int64_t n_units, double* out, double* lse, double* top2 /* [n][2] or NULL */) {
    if (d > 1024 || Hq % Hkv != 0) return -2;
    int32_t G = Hq / Hkv;
    int64_t* off = (int64_t*)malloc(sizeof(int64_t) * (size_t)(R + 1));
    off[0] = 0;
    int64_t max_n = 1;
    for (int32_t i = 0; i < R; ++i) {
        off[i + 1] = off[i] + chunk_lens[i];
        int64_t n = (int64_t)prefix_lens[i] + chunk_lens[i];
        if (n > max_n) max_n = n;
    }
    int bad = 0;
#pragma omp parallel
    {
        double* scores = (double*)malloc(sizeof(double) * (size_t)max_n);
#pragma omp for schedule(dynamic, 4)
        for (int64_t u = 0; u < n_units; ++u) {
            int32_t i = units[3 * u], t = units[3 * u + 1], h = units[3 * u + 2];
            if (i < 0 || i >= R || t < 0 || t >= chunk_lens[i] || h < 0 || h >= Hq) { bad = 1; continue; }
            int64_t n = (int64_t)prefix_lens[i] + t + 1;
            const uint16_t* q_row = q + ((off[i] + t) * Hq + h) * (int64_t)d;
            attention_row(q_row, k_pool, v_pool, block_tables + (int64_t)i * max_blocks, n, h / G, Hkv, d, B,
                          scale, scores, out + u * (int64_t)d, lse ? lse + u : NULL, top2 ? top2 + 2 * u : NULL);
        }
        free(scores);
    }
    free(off);
    return bad ? -1 : 0;
}

/* O-attn on every (request, row, head): out [T][Hq][d] fp64, lse [T][Hq] (may be NULL). */
int wpp_oracle_attention(const uint16_t* q, const uint16_t* k_pool, const uint16_t* v_pool,
                         const int32_t* block_tables, const int32_t* prefix_lens, const int32_t* chunk_lens,
                         int32_t R, int32_t Hq, int32_t Hkv, int32_t d, int32_t B, int32_t max_blocks,
                         double scale, double* out, double* lse) {
    int64_t T = 0;
    for (int32_t i = 0; i < R; ++i) T += chunk_lens[i];
    int64_t n_units = T * Hq;
    int32_t* units = (int32_t*)malloc(sizeof(int32_t) * 3 * (size_t)(n_units > 0 ? n_units : 1));
    int64_t u = 0;
    for (int32_t i = 0; i < R; ++i)
        for (int32_t t = 0; t < chunk_lens[i]; ++t)
            for (int32_t h = 0; h < Hq; ++h) {
                units[3 * u] = i; units[3 * u + 1] = t; units[3 * u + 2] = h;
                ++u;
            }
    int rc = wpp_oracle_attention_units(q, k_pool, v_pool, block_tables, prefix_lens, chunk_lens, R, Hq, Hkv, d,
                                        B, max_blocks, scale, units, n_units, out, lse, NULL);
    free(units);
    return rc;
}
