/*
 * enl_oracle.c -- float64 CPU oracle for selective-KV attention with per-group mass.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing on the product path may call this file; it exists so
 * that the CUDA path can be compared against a plain statement of what the paper defines.
 * It shares no code, header, table or helper with the CUDA library.
 *
 * What it computes (paper, App. A "LLM inference and KV Cache"; Sec. 3.2 "Discrete Memory
 * Caching"; App. C "Detailed Planning Example"; Sec. 3.3 "Attention-based Memory Clustering"):
 *
 *   - The prompt of a planning step is the selected groups' cached K/V, in the order the
 *     caller lists them, followed by the step's new tokens (App. C: groups first, then
 *     instruction + trajectory).  Each group's K/V was produced independently and is used
 *     verbatim (Sec. 3.2); this code applies no position encoding.
 *   - Every new token attends over all cached keys of all selected groups and over the new
 *     keys up to and including itself (App. A: Attn = softmax(Q K^T / sqrt(D)) V, the V
 *     factor is implied by "attention output"; decode concatenates K_new / V_new, so a call
 *     with n_q < n_new aligns the queries with the LAST n_q new keys).
 *   - mass[row, head, slot] is the post-softmax probability summed over the keys of one
 *     slot; slot s < n_sel is the s-th selected group, slot n_sel is the visible new tokens
 *     (Sec. 3.3: the attention between new tokens and an existing group).
 *   - sel_off is the exclusive prefix sum of the selected groups' lengths.
 *   - GQA: q head h reads kv head h / (Hq / Hkv).
 *
 * All inputs are bf16 bit patterns, widened exactly to double; every intermediate is double.
 * Loops follow the definition: scores, max, exp, sum, weighted sum.  No tiling, no fusion.
 *
 * Pins (tests/test_oracle_pins.py): dense masked attention through an independent library
 * routine, an exp/sum brute force without max subtraction in extended precision, closed
 * forms (uniform, two-way softmax, one-hot), invariants (mass rows sum to 1, select-order
 * permutation, group splitting), the O<->mass tie with indicator V, prefill-row == decode
 * call, and prefix sums written by hand.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* bf16 -> double: a bf16 is the upper 16 bits of an IEEE-754 binary32. */
static double bf16_to_f64(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int enl_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Exclusive prefix sum of selected lengths: sel_off[0] = 0, sel_off[s+1] = sel_off[s] + len[s]. */
void enl_oracle_sel_off(int n_sel, const int32_t *sel_len, int64_t *sel_off)
{
    sel_off[0] = 0;
    for (int s = 0; s < n_sel; ++s)
        sel_off[s + 1] = sel_off[s] + (int64_t)sel_len[s];
}

/*
 * One episode, one layer.
 *
 *   sel_k[s], sel_v[s] : slot s's cached rows, [sel_len[s]][Hkv][D] bf16 bits
 *   q                  : [n_q][Hq][D];  k_new, v_new : [n_new][Hkv][D]
 *   rows               : n_rows query-row indices in [0, n_q) to evaluate (NULL = 0..n_rows-1)
 *   out                : [n_rows][Hq][D] double
 *   mass               : [n_rows][Hq][n_sel + 1] double (may be NULL)
 *
 * Query row r sees new keys j <= c, c = (n_new - n_q) + r.
 * Returns 0, or -1 on a malformed argument.
 */
int enl_oracle_attend(int Hq, int Hkv, int D,
                      int n_sel, const int32_t *sel_len,
                      const uint16_t *const *sel_k, const uint16_t *const *sel_v,
                      int n_q, int n_new,
                      const uint16_t *q, const uint16_t *k_new, const uint16_t *v_new,
                      int n_rows, const int32_t *rows,
                      double *out, double *mass)
{
    if (Hq <= 0 || Hkv <= 0 || D <= 0 || Hq % Hkv != 0) return -1;
    if (n_sel < 0 || n_q < 0 || n_new < n_q || n_rows < 0) return -1;
    const int rep = Hq / Hkv;
    int64_t S = 0;
    for (int s = 0; s < n_sel; ++s) {
        if (sel_len[s] < 0) return -1;
        S += sel_len[s];
    }
    const double inv_sqrt_d = 1.0 / sqrt((double)D);
    int bad = 0;

#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int ir = 0; ir < n_rows; ++ir) {
        for (int h = 0; h < Hq; ++h) {
            const int r = rows ? rows[ir] : ir;
            if (r < 0 || r >= n_q) {
#pragma omp atomic write
                bad = 1;
                continue;
            }
            const int kvh = h / rep;
            const int c = (n_new - n_q) + r;           /* last visible new key */
            const int64_t n_keys = S + (int64_t)c + 1;
            double *score = (double *)malloc((size_t)n_keys * sizeof(double));
            double *qd = (double *)malloc((size_t)D * sizeof(double));
            if (!score || !qd) {
#pragma omp atomic write
                bad = 1;
                free(score);
                free(qd);
                continue;
            }
            for (int d = 0; d < D; ++d)
                qd[d] = bf16_to_f64(q[((size_t)r * Hq + h) * D + d]);

            /* scores over the concatenation: slot 0 rows, slot 1 rows, ..., new keys 0..c */
            int64_t j = 0;
            for (int s = 0; s < n_sel; ++s) {
                for (int t = 0; t < sel_len[s]; ++t, ++j) {
                    const uint16_t *krow = sel_k[s] + ((size_t)t * Hkv + kvh) * D;
                    double dot = 0.0;
                    for (int d = 0; d < D; ++d) dot += qd[d] * bf16_to_f64(krow[d]);
                    score[j] = dot * inv_sqrt_d;
                }
            }
            for (int t = 0; t <= c; ++t, ++j) {
                const uint16_t *krow = k_new + ((size_t)t * Hkv + kvh) * D;
                double dot = 0.0;
                for (int d = 0; d < D; ++d) dot += qd[d] * bf16_to_f64(krow[d]);
                score[j] = dot * inv_sqrt_d;
            }

            /* softmax with the maximum subtracted */
            double mx = score[0];
            for (int64_t i = 1; i < n_keys; ++i) if (score[i] > mx) mx = score[i];
            double denom = 0.0;
            for (int64_t i = 0; i < n_keys; ++i) { score[i] = exp(score[i] - mx); denom += score[i]; }
            for (int64_t i = 0; i < n_keys; ++i) score[i] /= denom;     /* score now holds p */

            /* O = sum_j p_j v_j ; mass[slot] = sum of p over the slot's keys */
            double *o = out + ((size_t)ir * Hq + h) * D;
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            double *m = mass ? mass + ((size_t)ir * Hq + h) * (size_t)(n_sel + 1) : NULL;
            j = 0;
            for (int s = 0; s < n_sel; ++s) {
                double ms = 0.0;
                for (int t = 0; t < sel_len[s]; ++t, ++j) {
                    const uint16_t *vrow = sel_v[s] + ((size_t)t * Hkv + kvh) * D;
                    const double p = score[j];
                    ms += p;
                    for (int d = 0; d < D; ++d) o[d] += p * bf16_to_f64(vrow[d]);
                }
                if (m) m[s] = ms;
            }
            double mn = 0.0;
            for (int t = 0; t <= c; ++t, ++j) {
                const uint16_t *vrow = v_new + ((size_t)t * Hkv + kvh) * D;
                const double p = score[j];
                mn += p;
                for (int d = 0; d < D; ++d) o[d] += p * bf16_to_f64(vrow[d]);
            }
            if (m) m[n_sel] = mn;
            free(score);
            free(qd);
        }
    }
    return bad ? -1 : 0;
}
