/*
 * TEST INFRASTRUCTURE -- fp64 CPU oracle for P-EAGLE's masked parallel-drafting attention.
 *
 * This file is the slow, plain statement of what the hot path computes.  It is used only by
 * the tests, the smoke check and the benchmark's CPU-baseline leg.  It shares no code with
 * the CUDA library and the CUDA library never calls it.
 *
 * What it follows (paper sections):
 *   - Section 3, first paragraph: every length-n sequence is expanded to K prediction depths;
 *     a token is (anchor a, depth d) and sits at sequence position p = a + d.
 *   - Section 3, COD paragraph: a depth-d token may look at earlier depths only, never d+1...
 *   - Section 3.2, "Challenge 2": position p at depth d depends on position p-1 at depth d-1
 *     (same anchor, one depth down; transitively the whole chain back to depth 0).
 *   - Figure 1 (architecture) caption / Section 2: the depth-0 (NTP) position behaves like
 *     ordinary autoregressive prediction over the real context.
 *   - Section 3.2 + Algorithm 1, phase 3: a segment sees depth-0 tokens cumulatively up to its
 *     boundary; gradients are summed over the segments of one sequence.
 *
 * Readings taken where the paper is silent: a token sees itself; a depth>=1 token sees the
 * depth-0 token at its own anchor; scale and natural-log LSE are the caller's / usual ones.
 *
 * All functions work on ONE sequence given as arrays over its T expanded tokens.  Inputs that
 * are bf16 on the GPU arrive here as fp32 arrays holding exactly those bf16 values; all
 * arithmetic is fp64.  Pins: tests/test_oracle_pins.py (brute-force pair sets, closed-form
 * pair counts, library causal attention, finite differences, partition invariance).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* Section 3 / 3.2: may query (a_q, d_q) look at key (a_k, d_k) of the same sequence? */
int peagle_oracle_allowed(int a_q, int d_q, int a_k, int d_k)
{
    if (d_k == 0)
        return a_k <= a_q; /* real context token, known to a chain anchored at a_q iff not after it */
    return (a_k == a_q) && (d_k <= d_q); /* own chain, same or earlier depth */
}

int peagle_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* The mask the paper pre-computes, materialised: M[q*T + k] in {0,1}.
 * seq_id[t] tells which sequence token t belongs to (tokens of different sequences never mix). */
void peagle_oracle_mask_dense(int T, const int32_t *seq_id, const int32_t *anchor,
                              const int32_t *depth, uint8_t *M)
{
    for (int q = 0; q < T; ++q)
        for (int k = 0; k < T; ++k)
            M[(size_t)q * T + k] =
                (uint8_t)(seq_id[q] == seq_id[k] &&
                          peagle_oracle_allowed(anchor[q], depth[q], anchor[k], depth[k]));
}

static int visible(int k, const int32_t *kranges, int nk)
{
    if (nk == 0)
        return 1;
    for (int i = 0; i < nk; ++i)
        if (k >= kranges[2 * i] && k < kranges[2 * i + 1])
            return 1;
    return 0;
}

/* Row q of the mask restricted to the visible keys. */
static void mask_row(int T, const int32_t *anchor, const int32_t *depth, const int32_t *kranges,
                     int nk, int q, uint8_t *m)
{
    for (int k = 0; k < T; ++k)
        m[k] = (uint8_t)(peagle_oracle_allowed(anchor[q], depth[q], anchor[k], depth[k]) &&
                         visible(k, kranges, nk));
}

/* Number of allowed, visible (q,k) pairs over the given rows. */
int64_t peagle_oracle_count_pairs(int T, const int32_t *anchor, const int32_t *depth,
                                  const int32_t *kranges, int nk, const int32_t *rows, int nrows)
{
    int64_t total = 0;
#pragma omp parallel for schedule(dynamic, 16) reduction(+ : total)
    for (int r = 0; r < nrows; ++r) {
        int q = rows[r];
        for (int k = 0; k < T; ++k)
            total += peagle_oracle_allowed(anchor[q], depth[q], anchor[k], depth[k]) &&
                     visible(k, kranges, nk);
    }
    return total;
}

/*
 * Tile classes for one call, from the dense definition.
 * Query tiles: BM consecutive rows starting at q_begin (last one ragged).
 * Key tiles: for every visible range, BN consecutive tokens from the range's begin (last ragged).
 *   0 SKIP    : no allowed pair between an in-range row and an in-range column
 *   2 FULL    : the key tile has all BN columns and every in-range row allows every column
 *   1 PARTIAL : anything else
 * out[qt * n_ktiles + kt].  Returns n_ktiles; n_qtiles = ceil((q_end-q_begin)/BM).
 */
int peagle_oracle_classify_tiles(int T, const int32_t *anchor, const int32_t *depth,
                                 int q_begin, int q_end, const int32_t *kranges, int nk, int BM,
                                 int BN, uint8_t *out, int32_t *ktile_start, int32_t *ktile_len)
{
    int32_t whole[2] = {0, T};
    if (nk == 0) {
        kranges = whole;
        nk = 1;
    }
    int n_kt = 0;
    for (int i = 0; i < nk; ++i)
        for (int b = kranges[2 * i]; b < kranges[2 * i + 1]; b += BN) {
            int len = kranges[2 * i + 1] - b < BN ? kranges[2 * i + 1] - b : BN;
            if (ktile_start) {
                ktile_start[n_kt] = b;
                ktile_len[n_kt] = len;
            }
            ++n_kt;
        }
    if (!out)
        return n_kt;
    int n_qt = (q_end - q_begin + BM - 1) / BM;
#pragma omp parallel for schedule(dynamic, 1)
    for (int qt = 0; qt < n_qt; ++qt) {
        int r0 = q_begin + qt * BM, r1 = r0 + BM < q_end ? r0 + BM : q_end;
        int kt = 0;
        for (int i = 0; i < nk; ++i)
            for (int b = kranges[2 * i]; b < kranges[2 * i + 1]; b += BN, ++kt) {
                int e = b + BN < kranges[2 * i + 1] ? b + BN : kranges[2 * i + 1];
                int64_t n_allowed = 0;
                for (int q = r0; q < r1; ++q)
                    for (int k = b; k < e; ++k)
                        n_allowed += peagle_oracle_allowed(anchor[q], depth[q], anchor[k], depth[k]);
                uint8_t c;
                if (n_allowed == 0)
                    c = 0;
                else if (e - b == BN && n_allowed == (int64_t)(r1 - r0) * BN)
                    c = 2;
                else
                    c = 1;
                out[(size_t)qt * n_kt + kt] = c;
            }
    }
    return n_kt;
}

/*
 * Forward.  For each listed row q and head h in [h_begin,h_end), g = h / (Hq/Hkv):
 *   A_q  = { k : allowed(q,k) and visible(k) }
 *   s_k  = scale * <Q[q,h,:], K[k,g,:]>,  LSE = log sum_{k in A_q} exp(s_k),
 *   O    = sum_k exp(s_k - LSE) V[k,g,:]
 * Empty A_q gives O = 0, LSE = -inf.
 * Layouts: Q [T][Hq][D], K,V [T][Hkv][D]; O [nrows][h_end-h_begin][D]; LSE [nrows][h_end-h_begin].
 */
int peagle_oracle_attn_fwd(int T, const int32_t *anchor, const int32_t *depth, int Hq, int Hkv,
                           int D, double scale, const int32_t *kranges, int nk,
                           const int32_t *rows, int nrows, int h_begin, int h_end, const float *Q,
                           const float *K, const float *V, double *O, double *LSE)
{
    if (Hq % Hkv != 0 || h_begin < 0 || h_end > Hq || h_begin > h_end)
        return -1;
    const int G = Hq / Hkv, HS = h_end - h_begin;
#pragma omp parallel
    {
        uint8_t *m = (uint8_t *)malloc((size_t)T);
        double *s = (double *)malloc(sizeof(double) * (size_t)T);
#pragma omp for schedule(dynamic, 4)
        for (int r = 0; r < nrows; ++r) {
            const int q = rows[r];
            mask_row(T, anchor, depth, kranges, nk, q, m);
            for (int h = h_begin; h < h_end; ++h) {
                const int g = h / G;
                const float *qv = Q + ((size_t)q * Hq + h) * D;
                double *o = O + ((size_t)r * HS + (h - h_begin)) * D;
                double smax = -INFINITY;
                for (int k = 0; k < T; ++k) {
                    if (!m[k])
                        continue;
                    const float *kv = K + ((size_t)k * Hkv + g) * D;
                    double acc = 0.0;
                    for (int d = 0; d < D; ++d)
                        acc += (double)qv[d] * (double)kv[d];
                    s[k] = scale * acc;
                    if (s[k] > smax)
                        smax = s[k];
                }
                for (int d = 0; d < D; ++d)
                    o[d] = 0.0;
                if (smax == -INFINITY) {
                    LSE[(size_t)r * HS + (h - h_begin)] = -INFINITY;
                    continue;
                }
                double denom = 0.0;
                for (int k = 0; k < T; ++k)
                    if (m[k])
                        denom += exp(s[k] - smax);
                const double lse = smax + log(denom);
                for (int k = 0; k < T; ++k) {
                    if (!m[k])
                        continue;
                    const double p = exp(s[k] - lse);
                    const float *vv = V + ((size_t)k * Hkv + g) * D;
                    for (int d = 0; d < D; ++d)
                        o[d] += p * (double)vv[d];
                }
                LSE[(size_t)r * HS + (h - h_begin)] = lse;
            }
        }
        free(m);
        free(s);
    }
    return 0;
}

/*
 * Backward of the function above with respect to Q, K, V, for upstream gradient dO [T][Hq][D].
 * Per row q and head h (probabilities P_k recomputed in fp64 from Q,K):
 *   Delta = <dO, O>,  dP_k = <dO, V[k]>,  dS_k = P_k (dP_k - Delta)
 *   dQ[q,h,:]  = scale * sum_k dS_k K[k,g,:]
 *   dK[k,g,:] += scale * dS_k Q[q,h,:]        dV[k,g,:] += P_k dO[q,h,:]
 * dQ is [nrows][h_end-h_begin][D] (overwritten).  dK, dV are [T][Hkv][D] and are ADDED to, so a
 * caller can sum the contributions of several query partitions (within-sequence gradient
 * accumulation, Section 3.2).
 *
 * Two sweeps: the first goes row by row (LSE, Delta and dQ of each row); the second goes key by
 * key and sums that key's dK, dV over the listed rows, so no two threads write the same place.
 */
int peagle_oracle_attn_bwd(int T, const int32_t *anchor, const int32_t *depth, int Hq, int Hkv,
                           int D, double scale, const int32_t *kranges, int nk,
                           const int32_t *rows, int nrows, int h_begin, int h_end, const float *Q,
                           const float *K, const float *V, const float *dO, double *dQ, double *dK,
                           double *dV)
{
    if (Hq % Hkv != 0 || h_begin < 0 || h_end > Hq || h_begin > h_end)
        return -1;
    const int G = Hq / Hkv, HS = h_end - h_begin;
    double *LSE = (double *)malloc(sizeof(double) * (size_t)(nrows > 0 ? nrows : 1) * (HS > 0 ? HS : 1));
    double *DEL = (double *)malloc(sizeof(double) * (size_t)(nrows > 0 ? nrows : 1) * (HS > 0 ? HS : 1));
    /* ---- sweep 1: per row: LSE, O, Delta, dQ */
#pragma omp parallel
    {
        uint8_t *m = (uint8_t *)malloc((size_t)T);
        double *s = (double *)malloc(sizeof(double) * (size_t)T);
        double *o = (double *)malloc(sizeof(double) * (size_t)D);
#pragma omp for schedule(dynamic, 4)
        for (int r = 0; r < nrows; ++r) {
            const int q = rows[r];
            mask_row(T, anchor, depth, kranges, nk, q, m);
            for (int h = h_begin; h < h_end; ++h) {
                const int g = h / G;
                const float *qv = Q + ((size_t)q * Hq + h) * D;
                const float *gov = dO + ((size_t)q * Hq + h) * D;
                double *dq = dQ + ((size_t)r * HS + (h - h_begin)) * D;
                for (int d = 0; d < D; ++d)
                    dq[d] = 0.0;
                double smax = -INFINITY;
                for (int k = 0; k < T; ++k) {
                    if (!m[k])
                        continue;
                    const float *kv = K + ((size_t)k * Hkv + g) * D;
                    double acc = 0.0;
                    for (int d = 0; d < D; ++d)
                        acc += (double)qv[d] * (double)kv[d];
                    s[k] = scale * acc;
                    if (s[k] > smax)
                        smax = s[k];
                }
                LSE[(size_t)r * HS + (h - h_begin)] = -INFINITY;
                DEL[(size_t)r * HS + (h - h_begin)] = 0.0;
                if (smax == -INFINITY)
                    continue;
                double denom = 0.0;
                for (int k = 0; k < T; ++k)
                    if (m[k])
                        denom += exp(s[k] - smax);
                const double lse = smax + log(denom);
                for (int d = 0; d < D; ++d)
                    o[d] = 0.0;
                for (int k = 0; k < T; ++k) {
                    if (!m[k])
                        continue;
                    const double p = exp(s[k] - lse);
                    const float *vv = V + ((size_t)k * Hkv + g) * D;
                    for (int d = 0; d < D; ++d)
                        o[d] += p * (double)vv[d];
                }
                double delta = 0.0;
                for (int d = 0; d < D; ++d)
                    delta += (double)gov[d] * o[d];
                for (int k = 0; k < T; ++k) {
                    if (!m[k])
                        continue;
                    const double p = exp(s[k] - lse);
                    const float *kv = K + ((size_t)k * Hkv + g) * D;
                    const float *vv = V + ((size_t)k * Hkv + g) * D;
                    double dp = 0.0;
                    for (int d = 0; d < D; ++d)
                        dp += (double)gov[d] * (double)vv[d];
                    const double ds = p * (dp - delta);
                    for (int d = 0; d < D; ++d)
                        dq[d] += scale * ds * (double)kv[d];
                }
                LSE[(size_t)r * HS + (h - h_begin)] = lse;
                DEL[(size_t)r * HS + (h - h_begin)] = delta;
            }
        }
        free(m);
        free(s);
        free(o);
    }
    /* ---- sweep 2: per key: dK, dV summed over the listed rows and the heads of its group */
#pragma omp parallel for schedule(dynamic, 8)
    for (int k = 0; k < T; ++k) {
        if (!visible(k, kranges, nk))
            continue;
        for (int r = 0; r < nrows; ++r) {
            const int q = rows[r];
            if (!peagle_oracle_allowed(anchor[q], depth[q], anchor[k], depth[k]))
                continue;
            for (int h = h_begin; h < h_end; ++h) {
                const double lse = LSE[(size_t)r * HS + (h - h_begin)];
                if (lse == -INFINITY)
                    continue;
                const int g = h / G;
                const float *qv = Q + ((size_t)q * Hq + h) * D;
                const float *gov = dO + ((size_t)q * Hq + h) * D;
                const float *kv = K + ((size_t)k * Hkv + g) * D;
                const float *vv = V + ((size_t)k * Hkv + g) * D;
                double acc = 0.0, dp = 0.0;
                for (int d = 0; d < D; ++d) {
                    acc += (double)qv[d] * (double)kv[d];
                    dp += (double)gov[d] * (double)vv[d];
                }
                const double p = exp(scale * acc - lse);
                const double ds = p * (dp - DEL[(size_t)r * HS + (h - h_begin)]);
                double *dk = dK + ((size_t)k * Hkv + g) * D;
                double *dv = dV + ((size_t)k * Hkv + g) * D;
                for (int d = 0; d < D; ++d) {
                    dk[d] += scale * ds * (double)qv[d];
                    dv[d] += p * (double)gov[d];
                }
            }
        }
    }
    free(LSE);
    free(DEL);
    return 0;
}
