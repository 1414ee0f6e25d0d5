/*
 * fp64 CPU oracle for SEKA / AdaSEKA steered causal attention.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the GPU
 * library is checked against.  It shares no code with the CUDA path and the
 * product never calls it.  Every function works on ONE sequence, takes and
 * returns fp64, and follows the paper's definitions step by step with no
 * blocking, fusion or reordering.  OpenMP is used only across units that the
 * definition makes independent (tokens, heads, query rows).
 *
 * Layouts (row-major, one sequence):
 *   Q [L, Hq, d]   K, V [L, Hkv, d]   mask [L]   U [M, Hkv, d, r]
 *   sigma [M, Hkv, r]   alpha [Hkv, M]   head_enable [Hkv]
 * Query head hq reads KV head hq / (Hq / Hkv)  (grouped-query attention with
 * consecutive query heads sharing one KV head; Appendix I's "interleaved
 * repetition" of KV-head selections).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------
 * AdaSEKA routing coefficients, Eq. 6 (Section 3.3) / Algorithm 2.
 *   s_m     = sum_{k<k_route} (q . u_m^(k)) * sigma_m^(k)
 *   alpha_m = s_m / max_m' |s_m'|
 * q is the query of the prompt's last token.  The paper indexes q by the same
 * head as the projector, which is a KV head; under GQA several query heads
 * share it, and the reading taken here is their SUM (alpha is invariant to a
 * positive scale of q, so sum and mean agree).  PARITY UNPINNED for that
 * choice: nothing in the paper fixes it.  If every s_m is zero, alpha = 0.
 *   q_last [Hq, d]  ->  alpha_out [Hkv, M]
 * ---------------------------------------------------------------------- */
void seka_oracle_route(int Hq, int Hkv, int d, int r, int M, int k_route,
                       const double* q_last, const double* U, const double* sigma,
                       double* alpha_out)
{
    const int G = Hq / Hkv;
    for (int h = 0; h < Hkv; ++h) {
        double* qbar = (double*)calloc((size_t)d, sizeof(double));
        for (int g = 0; g < G; ++g)
            for (int i = 0; i < d; ++i)
                qbar[i] += q_last[(size_t)(h * G + g) * d + i];
        double smax = 0.0;
        for (int m = 0; m < M; ++m) {
            const double* Um = U + ((size_t)m * Hkv + h) * d * r;
            const double* sg = sigma + ((size_t)m * Hkv + h) * r;
            double s = 0.0;
            for (int k = 0; k < k_route; ++k) {
                double dot = 0.0;
                for (int i = 0; i < d; ++i) dot += qbar[i] * Um[(size_t)i * r + k];
                s += dot * sg[k];
            }
            alpha_out[(size_t)h * M + m] = s;
            if (fabs(s) > smax) smax = fabs(s);
        }
        for (int m = 0; m < M; ++m)
            alpha_out[(size_t)h * M + m] = (smax > 0.0) ? alpha_out[(size_t)h * M + m] / smax : 0.0;
        free(qbar);
    }
}

/* ------------------------------------------------------------------------
 * Key edit: the hook of Algorithm 1 / Algorithm 2 with the single-projector
 * form of the edit (Section 2: k' = k + g P k; Eq. 7 with P = U U^T) and the
 * AdaSEKA blend P = sum_m alpha_m U_m U_m^T (Section 3.3).
 * For every token t with mask[t] != 0 and every enabled KV head h:
 *   c_m = U_m^T k            (r numbers per expert)
 *   k'  = k + g * sum_m alpha[h,m] * U_m c_m
 * Every other key is copied unchanged.  alpha may be NULL (all ones);
 * head_enable may be NULL (all heads steered, Section 3.4 otherwise).
 * ---------------------------------------------------------------------- */
void seka_oracle_edit_keys(int L, int Hkv, int d, int r, int M,
                           const double* K, const uint8_t* mask, const double* U,
                           const double* alpha, double g, const uint8_t* head_enable,
                           double* K_out)
{
    memcpy(K_out, K, (size_t)L * Hkv * d * sizeof(double));
#pragma omp parallel for schedule(static)
    for (int t = 0; t < L; ++t) {
        if (!mask[t]) continue;
        double* c = (double*)malloc((size_t)r * sizeof(double));
        for (int h = 0; h < Hkv; ++h) {
            if (head_enable && !head_enable[h]) continue;
            const double* k = K + ((size_t)t * Hkv + h) * d;
            double* ko = K_out + ((size_t)t * Hkv + h) * d;
            for (int m = 0; m < M; ++m) {
                const double* Um = U + ((size_t)m * Hkv + h) * d * r;
                const double a = alpha ? alpha[(size_t)h * M + m] : 1.0;
                for (int j = 0; j < r; ++j) {
                    double s = 0.0;
                    for (int i = 0; i < d; ++i) s += Um[(size_t)i * r + j] * k[i];
                    c[j] = s;
                }
                for (int i = 0; i < d; ++i) {
                    double s = 0.0;
                    for (int j = 0; j < r; ++j) s += Um[(size_t)i * r + j] * c[j];
                    ko[i] += g * a * s;
                }
            }
        }
        free(c);
    }
}

/* ------------------------------------------------------------------------
 * Causal softmax attention over already-edited keys, for a list of query rows.
 * Score definition of Section 2: s_ij = q_i . k'_j * scale (scale = 1/sqrt(d)
 * unless the caller overrides it), keys j <= i only (decoder-only models),
 *   p_ij = exp(s_ij - max_j s_ij) / sum_j exp(s_ij - max_j s_ij)
 *   o_i  = sum_j p_ij v_j              lse_i = max_j s_ij + log sum_j exp(...)
 * V is never edited (Appendix C: only the routing side, Q/K, is touched).
 *   rows [n_rows] (query positions)  ->  O [n_rows, Hq, d],  LSE [n_rows, Hq]
 * ---------------------------------------------------------------------- */
void seka_oracle_attention_rows(int L, int Hq, int Hkv, int d,
                                const double* Q, const double* Kp, const double* V,
                                double scale, int n_rows, const int32_t* rows,
                                double* O, double* LSE)
{
    const int G = Hq / Hkv;
    (void)L;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int a = 0; a < n_rows; ++a) {
        for (int hq = 0; hq < Hq; ++hq) {
            const int i = rows[a];
            const int h = hq / G;
            const double* q = Q + ((size_t)i * Hq + hq) * d;
            double* s = (double*)malloc((size_t)(i + 1) * sizeof(double));
            double smax = -INFINITY;
            for (int j = 0; j <= i; ++j) {
                const double* k = Kp + ((size_t)j * Hkv + h) * d;
                double dot = 0.0;
                for (int c = 0; c < d; ++c) dot += q[c] * k[c];
                s[j] = dot * scale;
                if (s[j] > smax) smax = s[j];
            }
            double denom = 0.0;
            for (int j = 0; j <= i; ++j) {
                s[j] = exp(s[j] - smax);
                denom += s[j];
            }
            double* o = O + ((size_t)a * Hq + hq) * d;
            for (int c = 0; c < d; ++c) o[c] = 0.0;
            for (int j = 0; j <= i; ++j) {
                const double p = s[j] / denom;
                const double* v = V + ((size_t)j * Hkv + h) * d;
                for (int c = 0; c < d; ++c) o[c] += p * v[c];
            }
            if (LSE) LSE[(size_t)a * Hq + hq] = smax + log(denom);
            free(s);
        }
    }
}

/* Number of OpenMP threads the attention loop will use (reported by the bench). */
#ifdef _OPENMP
#include <omp.h>
int seka_oracle_threads(void) { return omp_get_max_threads(); }
#else
int seka_oracle_threads(void) { return 1; }
#endif
