/*
 * TEST INFRASTRUCTURE -- NOT PART OF THE PRODUCT PATH.
 *
 * Plain, slow, fp64 CPU statement of what the decode-attention hot path computes,
 * written from the paper's definitions ("Fast Transformer Decoding: One Write-Head
 * is All You Need", arXiv 1911.02150).  Only the tests, the smoke check and the
 * bench's cpu_baseline / reference legs may call this.  It shares no code, header,
 * table or constant with the CUDA path.
 *
 * What each function follows:
 *   oracle_dot_product_attention  Section 2.1 (dot-product attention on one query):
 *                                 logits = K q, weights = softmax(logits), y = weights V.
 *   oracle_mha_decode_step        Section 2.4, the three attention lines of the
 *                                 incremental multi-head step: every head hh of every
 *                                 sequence attends over its own K[b,hh,:,:], V[b,hh,:,:].
 *   oracle_mqa_decode_step        Section 3, the same three lines of the incremental
 *                                 multi-query step: all h heads of a sequence attend
 *                                 over the one shared K[b,:,:], V[b,:,:].
 *   oracle_mqa_batched_attention  Section 3, the three attention lines of the batched multi-query
 *                                 function (logits = einsum(bhnk,bmk->bhnm), weights =
 *                                 softmax(logits + mask), O = einsum(bhnm,bmv->bhnv)) with the
 *                                 mask of Section 2.3 for an autoregressive model: -inf where
 *                                 a query would look at a later position, 0 elsewhere.
 *   oracle_kv_cache_append        Sections 2.4 / 3, the concatenation of the new
 *                                 token's key and value row on the m axis, done in
 *                                 place in a cache padded to m_max rows.
 *
 * Readings of the paper used here:
 *   - no 1/sqrt(k) factor on the logits (the note that closes Section 2.2);
 *   - softmax is over the memory axis m, written in its shift-by-max form, which
 *     equals the plain exp/sum form in exact arithmetic;
 *   - the additive -inf mask of Section 2.3 restricted to "positions >= lens[b] are
 *     illegal" is the same as summing over the first lens[b] rows only, so rows at
 *     or beyond lens[b] are never read;
 *   - an empty prefix (lens[b] == 0) cannot arise in the paper's flow (the append
 *     comes before the attention); it is defined here as an all-zero output.
 *
 * There is no blocking, no running max, no fusion: logits for the whole prefix, then
 * the max, then the exponentials and their sum, then the weighted sum of V rows.
 * bf16 inputs are widened exactly (bits << 16 is the fp32 with the same value).
 * OpenMP only spreads independent (sequence, head) pairs over threads.
 *
 * Parity pins: every function here is pinned by tests/test_oracle_pins.py (closed
 * forms, brute-force einsum, reductions to the single-query function, invariants).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double widen_bf16(uint16_t bits) {
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_num_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* Section 2.1.  q[k], K[m,k], V[m,v] -> y[v], all fp64, row-major.  m >= 1.
 * Returns 0, or 1 if scratch could not be allocated. */
int oracle_dot_product_attention(const double* q, const double* K, const double* V,
                                 double* y, int m, int k, int v) {
    double* logits = (double*)malloc((size_t)(m > 0 ? m : 1) * sizeof(double));
    if (!logits) return 1;
    for (int j = 0; j < m; ++j) {
        double s = 0.0;
        for (int c = 0; c < k; ++c) s += q[c] * K[(size_t)j * k + c];
        logits[j] = s;
    }
    double top = -INFINITY;
    for (int j = 0; j < m; ++j)
        if (logits[j] > top) top = logits[j];
    double Z = 0.0;
    for (int j = 0; j < m; ++j) {
        logits[j] = exp(logits[j] - top); /* now the unnormalised weight */
        Z += logits[j];
    }
    for (int c = 0; c < v; ++c) {
        double s = 0.0;
        for (int j = 0; j < m; ++j) s += logits[j] * V[(size_t)j * v + c];
        y[c] = s / Z;
    }
    free(logits);
    return 0;
}

/* One head of one sequence on bf16 storage: q_row[k], Kseq[L..,k], Vseq[L..,v] (only the
 * first L rows are read) -> out[v] fp64.  scratch holds L doubles. */
static void attend_prefix_bf16(const uint16_t* q_row, const uint16_t* Kseq, const uint16_t* Vseq,
                               int L, int k, int v, double* scratch, double* out) {
    if (L <= 0) {
        for (int c = 0; c < v; ++c) out[c] = 0.0;
        return;
    }
    for (int j = 0; j < L; ++j) {
        double s = 0.0;
        for (int c = 0; c < k; ++c)
            s += widen_bf16(q_row[c]) * widen_bf16(Kseq[(size_t)j * k + c]);
        scratch[j] = s;
    }
    double top = -INFINITY;
    for (int j = 0; j < L; ++j)
        if (scratch[j] > top) top = scratch[j];
    double Z = 0.0;
    for (int j = 0; j < L; ++j) {
        scratch[j] = exp(scratch[j] - top);
        Z += scratch[j];
    }
    for (int c = 0; c < v; ++c) {
        double s = 0.0;
        for (int j = 0; j < L; ++j) s += scratch[j] * widen_bf16(Vseq[(size_t)j * v + c]);
        out[c] = s / Z;
    }
}

static int clamp_len(int L, int m_max) {
    if (L < 0) return 0;
    if (L > m_max) return m_max;
    return L;
}

/* Section 3 (multi-query, incremental): q[b,h,k], K[b,m_max,k], V[b,m_max,v] as bf16 bit
 * patterns, lens[b] rows valid -> o[b,h,v] fp64.  Returns 0, or 1 on allocation failure. */
int oracle_mqa_decode_step(const uint16_t* q, const uint16_t* K, const uint16_t* V,
                           const int32_t* lens, double* o,
                           int b, int h, int m_max, int k, int v) {
    int failed = 0;
    long units = (long)b * h;
#pragma omp parallel
    {
        double* scratch = (double*)malloc((size_t)(m_max > 0 ? m_max : 1) * sizeof(double));
        if (!scratch) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for schedule(dynamic, 1)
        for (long u = 0; u < units; ++u) {
            if (!scratch) continue;
            long bi = u / h, hh = u % h;
            int L = clamp_len(lens[bi], m_max);
            attend_prefix_bf16(q + ((size_t)bi * h + hh) * k,
                               K + (size_t)bi * m_max * k,  /* shared by all heads */
                               V + (size_t)bi * m_max * v,
                               L, k, v, scratch, o + ((size_t)bi * h + hh) * v);
        }
        free(scratch);
    }
    return failed;
}

/* Section 2.4 (multi-head, incremental): q[b,h,k], K[b,h,m_max,k], V[b,h,m_max,v] bf16,
 * lens[b] shared by the heads of a sequence -> o[b,h,v] fp64. */
int oracle_mha_decode_step(const uint16_t* q, const uint16_t* K, const uint16_t* V,
                           const int32_t* lens, double* o,
                           int b, int h, int m_max, int k, int v) {
    int failed = 0;
    long units = (long)b * h;
#pragma omp parallel
    {
        double* scratch = (double*)malloc((size_t)(m_max > 0 ? m_max : 1) * sizeof(double));
        if (!scratch) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for schedule(dynamic, 1)
        for (long u = 0; u < units; ++u) {
            if (!scratch) continue;
            long bi = u / h, hh = u % h;
            int L = clamp_len(lens[bi], m_max);
            attend_prefix_bf16(q + ((size_t)bi * h + hh) * k,
                               K + ((size_t)bi * h + hh) * m_max * k,  /* this head's own cache */
                               V + ((size_t)bi * h + hh) * m_max * v,
                               L, k, v, scratch, o + ((size_t)bi * h + hh) * v);
        }
        free(scratch);
    }
    return failed;
}

/* Section 3 (multi-query, batched), the attention lines only: Q[b,h,n,k], K[b,m_max,k], V[b,m_max,v] as bf16
 * bit patterns -> O[b,h,n,v] fp64.  Sequence bi has start[bi] + n memory positions (the n query positions are its
 * last n: position t of the queries is memory position start[bi] + t; start may be NULL = all zero, i.e. m = n,
 * memory and queries from the same positions).  The mask of Section 2.3 is written out as the paper states it: an
 * additive term, -inf where memory position j lies after the query's own position, 0 where it does not; the softmax
 * then runs over all start[bi] + n positions.  Rows beyond that are never read.  Returns 0, 1 on allocation
 * failure, 2 if some sequence does not fit m_max. */
int oracle_mqa_batched_attention(const uint16_t* Q, const uint16_t* K, const uint16_t* V, const int32_t* start,
                                 double* O, int b, int h, int n, int m_max, int k, int v) {
    for (int bi = 0; bi < b; ++bi) {
        int st = start ? start[bi] : 0;
        if (st < 0 || st + n > m_max) return 2;
    }
    int failed = 0;
    long units = (long)b * h * n;
#pragma omp parallel
    {
        double* logits = (double*)malloc((size_t)(m_max > 0 ? m_max : 1) * sizeof(double));
        if (!logits) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for schedule(dynamic, 16)
        for (long u = 0; u < units; ++u) {
            if (!logits) continue;
            long bi = u / ((long)h * n), hh = (u / n) % h, t = u % n;
            int st = start ? start[bi] : 0;
            int m = st + n;                                    /* memory positions of this sequence */
            const uint16_t* q_row = Q + (((size_t)bi * h + hh) * n + t) * k;
            const uint16_t* Kseq = K + (size_t)bi * m_max * k;
            const uint16_t* Vseq = V + (size_t)bi * m_max * v;
            for (int j = 0; j < m; ++j) {
                double s = 0.0;
                for (int c = 0; c < k; ++c) s += widen_bf16(q_row[c]) * widen_bf16(Kseq[(size_t)j * k + c]);
                double mask = (j > st + t) ? -INFINITY : 0.0;  /* a later position is illegal */
                logits[j] = s + mask;
            }
            double top = -INFINITY;
            for (int j = 0; j < m; ++j)
                if (logits[j] > top) top = logits[j];
            double Z = 0.0;
            for (int j = 0; j < m; ++j) {
                logits[j] = exp(logits[j] - top);              /* exp(-inf) = 0 for the masked positions */
                Z += logits[j];
            }
            double* out = O + (((size_t)bi * h + hh) * n + t) * v;
            for (int c = 0; c < v; ++c) {
                double s = 0.0;
                for (int j = 0; j < m; ++j) s += logits[j] * widen_bf16(Vseq[(size_t)j * v + c]);
                out[c] = s / Z;
            }
        }
        free(logits);
    }
    return failed;
}

/* Sections 2.4 / 3: append the new token's rows.  K[b,kv_heads,m_max,k], V[b,kv_heads,m_max,v],
 * k_new[b,kv_heads,k], v_new[b,kv_heads,v] as 16-bit words (never interpreted as numbers);
 * row written = lens[b]; a sequence whose lens[b] is outside [0, m_max) is left untouched and
 * counted.  If advance != 0, lens[b] += 1 for every sequence that was written.
 * Returns the number of sequences skipped. */
int oracle_kv_cache_append(uint16_t* K, uint16_t* V, const uint16_t* k_new, const uint16_t* v_new,
                           int32_t* lens, int advance,
                           int b, int kv_heads, int m_max, int k, int v) {
    int skipped = 0;
    for (int bi = 0; bi < b; ++bi) {
        int row = lens[bi];
        if (row < 0 || row >= m_max) {
            ++skipped;
            continue;
        }
        for (int g = 0; g < kv_heads; ++g) {
            size_t cache_row = ((size_t)bi * kv_heads + g) * m_max + row;
            size_t new_row = (size_t)bi * kv_heads + g;
            for (int c = 0; c < k; ++c) K[cache_row * k + c] = k_new[new_row * k + c];
            for (int c = 0; c < v; ++c) V[cache_row * v + c] = v_new[new_row * v + c];
        }
        if (advance) lens[bi] = row + 1;
    }
    return skipped;
}
