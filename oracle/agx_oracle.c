/*
 * CPU oracle for prefix-cached block attention and greedy speculative acceptance.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the CUDA library is
 * checked against.  Only tests, the smoke check and the benchmark's CPU-baseline leg may call
 * it; the product path never does, and it shares no code with the CUDA sources.
 *
 * Everything is computed in double precision.  Inputs arrive in their storage type (bfloat16
 * bit patterns as uint16, or float32) and are widened exactly, so the oracle consumes exactly
 * the values the GPU sees.  There is no blocking, tiling, online softmax or reordering: each
 * output row is the textbook three-pass softmax written out.
 *
 * What the paper fixes for this path:
 *   - Sec. 2.3 "Prefix caching": a token attends only to the tokens before it (and itself), so
 *     the KV of a shared prefix is reused verbatim and prefill computes only the uncached
 *     suffix, each suffix row attending over the cached prefix plus the suffix rows up to it.
 *   - Sec. 2.3 "Speculative decoding": the target model processes the most recent token
 *     followed by the N drafts in one pass; the first mismatching draft and every draft after
 *     it are discarded; the accepted drafts plus the target's own next token seed the next
 *     round.
 * Readings where the paper is silent (GQA map g = h / G, scale 1/sqrt(d), lowest index wins
 * argmax ties, NaN never beats a number, page size 16) are listed in the design notes.
 *
 * Parity pins: every function here is pinned by CPU tests (closed forms, invariants, a
 * library attention routine, numpy.argmax and brute force on tiny inputs); none is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_PAGE 16

enum { ORACLE_BF16 = 0, ORACLE_F32 = 1 };

/* exact widening of one stored element to double */
static inline double widen(const void* base, int64_t idx, int dtype) {
    if (dtype == ORACLE_BF16) {
        uint32_t bits = ((uint32_t)((const uint16_t*)base)[idx]) << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    return (double)((const float*)base)[idx];
}

/* A key/value store for ONE sequence: either contiguous [L, Hkv, d] or paged
 * [num_pages, Hkv, 16, d] reached through that sequence's page-table row. */
typedef struct {
    const void* k;
    const void* v;
    const int32_t* page_row; /* NULL => contiguous */
    int hkv, d, dtype;
} kv_store;

static inline int64_t kv_index(const kv_store* st, int64_t j, int g) {
    if (st->page_row == NULL) return (j * st->hkv + g) * (int64_t)st->d;
    int64_t page = st->page_row[j / ORACLE_PAGE];
    return ((page * st->hkv + g) * ORACLE_PAGE + (j % ORACLE_PAGE)) * (int64_t)st->d;
}

/* One output row: query vector qv[d] (already widened) against keys 0..n-1 of kv head g.
 * s_j = scale * <q, K_j>;  m = max_j s_j;  p_j = exp(s_j - m);  l = sum_j p_j;
 * out = (sum_j p_j V_j) / l;  lse = m + log(l);  psum = (sum_j p_j / l)  (should be 1).
 * scratch must hold n doubles. */
static void attend_row(const double* qv, const kv_store* st, int g, int64_t n, double scale,
                       double* scratch, double* out, double* lse, double* psum) {
    const int d = st->d;
    double m = -INFINITY;
    for (int64_t j = 0; j < n; ++j) {
        const int64_t base = kv_index(st, j, g);
        double acc = 0.0;
        for (int c = 0; c < d; ++c) acc += qv[c] * widen(st->k, base + c, st->dtype);
        scratch[j] = scale * acc;
        if (scratch[j] > m) m = scratch[j];
    }
    double l = 0.0;
    for (int64_t j = 0; j < n; ++j) {
        scratch[j] = exp(scratch[j] - m);
        l += scratch[j];
    }
    for (int c = 0; c < d; ++c) out[c] = 0.0;
    double ps = 0.0;
    for (int64_t j = 0; j < n; ++j) {
        const int64_t base = kv_index(st, j, g);
        const double w = scratch[j];
        ps += w / l;
        for (int c = 0; c < d; ++c) out[c] += w * widen(st->v, base + c, st->dtype);
    }
    for (int c = 0; c < d; ++c) out[c] /= l;
    if (lse) *lse = m + log(l);
    if (psum) *psum = ps;
}

/* Block attention for one sequence.  Row i of the block (absolute position P + i) sees keys
 * 0 .. P + i inclusive: the whole cached prefix plus the block rows up to and including itself
 * (Sec. 2.3, prefix caching; the verify block of Sec. 2.3 is the same shape with q = N + 1).
 * q_block: [q, Hq, d] storage.  out: [q, Hq, d] double.  lse, psum: [q, Hq] double or NULL.
 * If n_sel > 0 only the (sel_i[t], sel_h[t]) rows are computed and written densely to
 * out[t, :], lse[t], psum[t]. */
static void attend_block(const void* q_block, const kv_store* st, int hq, int64_t P, int64_t q,
                         double scale, int64_t n_sel, const int32_t* sel_i, const int32_t* sel_h,
                         double* out, double* lse, double* psum) {
    const int d = st->d;
    const int G = hq / st->hkv;
    const int64_t n_rows = n_sel > 0 ? n_sel : q * hq;
#pragma omp parallel
    {
        double* scratch = (double*)malloc(sizeof(double) * (size_t)(P + q + 1));
        double* qv = (double*)malloc(sizeof(double) * (size_t)d);
#pragma omp for schedule(dynamic, 1)
        for (int64_t t = 0; t < n_rows; ++t) {
            const int64_t i = n_sel > 0 ? sel_i[t] : t / hq;
            const int h = n_sel > 0 ? sel_h[t] : (int)(t % hq);
            const int g = h / G;
            for (int c = 0; c < d; ++c) qv[c] = widen(q_block, (i * hq + h) * (int64_t)d + c, st->dtype);
            attend_row(qv, st, g, P + i + 1, scale, scratch, out + t * d, lse ? lse + t : NULL,
                       psum ? psum + t : NULL);
        }
        free(scratch);
        free(qv);
    }
}

/* ---- exported: contiguous form.  K, V: [P + q, Hkv, d] storage. */
void oracle_attn_contiguous(const void* q_block, const void* K, const void* V, int dtype, int hq,
                            int hkv, int d, int64_t P, int64_t q, double scale, int64_t n_sel,
                            const int32_t* sel_i, const int32_t* sel_h, double* out, double* lse,
                            double* psum) {
    kv_store st = {K, V, NULL, hkv, d, dtype};
    attend_block(q_block, &st, hq, P, q, scale, n_sel, sel_i, sel_h, out, lse, psum);
}

/* ---- exported: paged form for one sequence.  Pools: [num_pages, Hkv, 16, d] storage;
 * page_row: that sequence's page-table row. */
void oracle_attn_paged(const void* q_block, const void* k_pool, const void* v_pool,
                       const int32_t* page_row, int dtype, int hq, int hkv, int d, int64_t P,
                       int64_t q, double scale, int64_t n_sel, const int32_t* sel_i,
                       const int32_t* sel_h, double* out, double* lse, double* psum) {
    kv_store st = {k_pool, v_pool, page_row, hkv, d, dtype};
    attend_block(q_block, &st, hq, P, q, scale, n_sel, sel_i, sel_h, out, lse, psum);
}

/* ---- exported: ragged batch, paged.  Calls the single-sequence form per sequence.
 * q_block/out rows are sequence-major via cu_q.  out: [total_q, Hq, d]; lse: [total_q, Hq]. */
void oracle_attn_paged_batch(const void* q_block, const void* k_pool, const void* v_pool,
                             const int32_t* page_table, int64_t page_table_stride, int dtype,
                             int hq, int hkv, int d, int B, const int32_t* prefix_len,
                             const int32_t* q_len, const int32_t* cu_q, double scale, double* out,
                             double* lse) {
    const int64_t esz = dtype == ORACLE_BF16 ? 2 : 4;
    for (int s = 0; s < B; ++s) {
        const int64_t row0 = cu_q[s];
        oracle_attn_paged((const char*)q_block + row0 * hq * d * esz, k_pool, v_pool,
                          page_table + s * page_table_stride, dtype, hq, hkv, d, prefix_len[s],
                          q_len[s], scale, 0, NULL, NULL, out + row0 * hq * d,
                          lse ? lse + row0 * hq : NULL, NULL);
    }
}

/* ---- exported: plain single-token decode attention, written independently of the block
 * code above (no mask logic, weights normalised before the value sum).  One query token with
 * Hq heads against all L keys.  qv: [Hq, d]; K, V: [L, Hkv, d]; out: [Hq, d] double. */
void oracle_decode_plain(const void* qv, const void* K, const void* V, int dtype, int hq, int hkv,
                         int d, int64_t L, double scale, double* out) {
    const int G = hq / hkv;
    double* w = (double*)malloc(sizeof(double) * (size_t)L);
    for (int h = 0; h < hq; ++h) {
        const int g = h / G;
        double top = -INFINITY;
        for (int64_t j = 0; j < L; ++j) {
            double dot = 0.0;
            for (int c = 0; c < d; ++c)
                dot += widen(qv, (int64_t)h * d + c, dtype) * widen(K, (j * hkv + g) * (int64_t)d + c, dtype);
            w[j] = dot * scale;
            top = fmax(top, w[j]);
        }
        double z = 0.0;
        for (int64_t j = 0; j < L; ++j) z += exp(w[j] - top);
        for (int64_t j = 0; j < L; ++j) w[j] = exp(w[j] - top) / z;
        for (int c = 0; c < d; ++c) {
            double acc = 0.0;
            for (int64_t j = 0; j < L; ++j) acc += w[j] * widen(V, (j * hkv + g) * (int64_t)d + c, dtype);
            out[(int64_t)h * d + c] = acc;
        }
    }
    free(w);
}

/* ---- exported: KV append.  Writes the block's K/V rows of every sequence into that
 * sequence's pages at token slots P .. P + q - 1 (storage bits copied unchanged).  In a verify
 * step these entries are speculative; acceptance later commits a length, it moves no data. */
void oracle_kv_append(void* k_pool, void* v_pool, const void* k_new, const void* v_new, int dtype,
                      int hkv, int d, const int32_t* page_table, int64_t page_table_stride, int B,
                      const int32_t* prefix_len, const int32_t* cu_q) {
    const size_t esz = dtype == ORACLE_BF16 ? 2 : 4;
    const size_t row_bytes = (size_t)d * esz;
    for (int s = 0; s < B; ++s) {
        for (int64_t r = cu_q[s]; r < cu_q[s + 1]; ++r) {
            const int64_t tok = prefix_len[s] + (r - cu_q[s]);
            const int64_t page = page_table[s * page_table_stride + tok / ORACLE_PAGE];
            for (int g = 0; g < hkv; ++g) {
                const size_t dst = (size_t)(((page * hkv + g) * ORACLE_PAGE + tok % ORACLE_PAGE)) * row_bytes;
                const size_t src = (size_t)(r * hkv + g) * row_bytes;
                memcpy((char*)k_pool + dst, (const char*)k_new + src, row_bytes);
                memcpy((char*)v_pool + dst, (const char*)v_new + src, row_bytes);
            }
        }
    }
}

/* ---- exported: greedy acceptance (Sec. 2.3, speculative decoding, steps 2 and 3).
 * Per logits row r: t_r = lowest index attaining the row maximum; NaN never beats a number; a
 * row of only NaN yields 0.  Per sequence s with k = q_s - 1 drafts d_1..d_k: row 0 belongs to
 * the most recent token, row i to draft d_i.  a = number of leading drafts with d_i == t_{i-1};
 * counting stops at the first mismatch, so later coincidental matches are discarded with it.
 * next = t_a (the target's own token after the accepted drafts); committed length = P + a + 1.
 * logits: [rows, row_stride] storage, only the first `vocab` columns of a row are logits. */
void oracle_accept_greedy(const void* logits, int dtype, int64_t row_stride, int vocab,
                          const int32_t* drafts, const int32_t* cu_q, int B,
                          const int32_t* prefix_len, int32_t* argmax_out, int32_t* accept_len,
                          int32_t* next_token, int32_t* seq_len_out) {
    const int64_t rows = cu_q[B];
    int32_t* t = (int32_t*)malloc(sizeof(int32_t) * (size_t)(rows > 0 ? rows : 1));
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        int64_t best = -1;
        double best_val = 0.0;
        for (int64_t v = 0; v < vocab; ++v) {
            const double x = widen(logits, r * row_stride + v, dtype);
            if (isnan(x)) continue;
            if (best < 0 || x > best_val) {
                best = v;
                best_val = x;
            }
        }
        t[r] = (int32_t)(best < 0 ? 0 : best);
    }
    for (int s = 0; s < B; ++s) {
        const int64_t r0 = cu_q[s];
        const int k = (int)(cu_q[s + 1] - r0) - 1;
        const int32_t* dr = drafts + (r0 - s);
        int a = 0;
        while (a < k && dr[a] == t[r0 + a]) ++a;
        accept_len[s] = a;
        next_token[s] = t[r0 + a];
        if (seq_len_out) seq_len_out[s] = prefix_len[s] + a + 1;
    }
    if (argmax_out) memcpy(argmax_out, t, sizeof(int32_t) * (size_t)rows);
    free(t);
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
