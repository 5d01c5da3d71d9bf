/*
 * CPU oracle for the FDA monitoring pass, the variance estimate and the model average.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, obviously-correct statement
 * of what the method computes, written from the paper's equations.  It shares no code,
 * header, table or constant with the CUDA library, and nothing on the product path may
 * call it.  Everything is accumulated in fp64; the fp32 inputs are widened exactly.
 *
 * Notation follows the paper (Table 1):
 *   w^(k)      model of worker k (row k of the K x d tensor w)
 *   w_t0       model after the most recent synchronisation
 *   u^(k)      local drift  w^(k) - w_t0
 *   S^(k)      local state  (||u^(k)||^2 , <xi,u^(k)> , sk(u^(k)))
 *   sk(.)      AMS sketch operator R^d -> R^{l x m}               (Section 3.1)
 *   M2(.)      median over the l rows of the squared row norm     (Section 3.1)
 *   H(.)       variance over-estimate of SketchFDA / LinearFDA    (Theorems 1 and 2)
 *
 * The paper cites the sketch literature for sk(.) and prints no hash family.  The family
 * used here is the classical one for AMS / Count-Sketch F2 estimation: per row a 2-wise
 * independent bucket hash and a 4-wise independent sign hash over the prime field
 * p = 2^61 - 1, with explicit coefficients supplied by the caller:
 *   bucket_i(j) = ((a_i*j + b_i) mod p) mod m
 *   g_i(j)      = (((c3_i*j + c2_i)*j + c1_i)*j + c0_i) mod p        (Horner)
 *   sign_i(j)   = +1 if g_i(j) is even, -1 if odd
 * with every residue taken in canonical form [0, p-1].  Coefficient layout per row:
 * {a, b, c3, c2, c1, c0}.
 *
 * Parity pins (tests marked "not gpu"): hash against arbitrary-precision integer
 * arithmetic; basis-vector probing; exact linearity on integer inputs; exact norm
 * recovery under injective bucketing; AMS estimator moments; the variance identity
 * (Eq. 4) by brute force; Cauchy-Schwarz bound of LinearFDA with its equality case;
 * zero state after synchronisation; exact averages on integer inputs.
 */
#include <stdint.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

typedef unsigned __int128 u128;

static const uint64_t FDA_P = ((uint64_t)1 << 61) - 1;

/* (a*x + b) mod p with a, x, b in [0, p-1]; the 128-bit product is reduced by the
 * remainder operator, i.e. the plain definition. */
static uint64_t mul_add_mod_p(uint64_t a, uint64_t x, uint64_t b)
{
    u128 t = (u128)a * (u128)x + (u128)b;
    return (uint64_t)(t % (u128)FDA_P);
}

/* Bucket of index j in sketch row with coefficients c[0..5] = {a,b,c3,c2,c1,c0}. */
static uint32_t bucket_of(const uint64_t *c, uint64_t j, uint32_t m)
{
    uint64_t y = mul_add_mod_p(c[0], j % FDA_P, c[1]);
    return (uint32_t)(y % (uint64_t)m);
}

/* Sign (+1 / -1) of index j: parity of the cubic polynomial evaluated mod p. */
static int sign_of(const uint64_t *c, uint64_t j)
{
    uint64_t x = j % FDA_P;
    uint64_t g = mul_add_mod_p(c[2], x, c[3]);
    g = mul_add_mod_p(g, x, c[4]);
    g = mul_add_mod_p(g, x, c[5]);
    return (g & 1u) ? -1 : +1;
}

/* Hash dump: buckets[i*n + t], signs[i*n + t] for j = j0 + t, t < n, rows i < l. */
int fda_oracle_hash(const uint64_t *coeffs, int l, int m, int64_t j0, int64_t n,
                    int32_t *buckets, int8_t *signs)
{
    if (!coeffs || l < 1 || m < 1 || j0 < 0 || n < 0) return 1;
    for (int i = 0; i < l; ++i)
        for (int64_t t = 0; t < n; ++t) {
            buckets[(size_t)i * n + t] = (int32_t)bucket_of(coeffs + 6 * i, (uint64_t)(j0 + t), (uint32_t)m);
            signs[(size_t)i * n + t] = (int8_t)sign_of(coeffs + 6 * i, (uint64_t)(j0 + t));
        }
    return 0;
}

/*
 * Local states S^(k) for workers k in [k_begin, k_end)  (Section 3, "Efficiently
 * monitoring the RI"; Theorem 1 for the sketch part, Theorem 2 for the projection).
 *   states[k*(2+l*m) + 0]           = ||u^(k)||^2
 *   states[k*(2+l*m) + 1]           = <xi, u^(k)>           (0 when xi == NULL)
 *   states[k*(2+l*m) + 2 + i*m + c] = sk(u^(k))[i][c]       (skipped when l == 0)
 * Only the rows of `states` in the worker range are written.
 */
int fda_oracle_local_state(const float *w, int64_t row_stride, int K, int64_t d,
                           const float *w_t0, const float *xi,
                           const uint64_t *coeffs, int l, int m,
                           int k_begin, int k_end, double *states)
{
    if (!w || !w_t0 || !states || K < 1 || d < 1 || row_stride < d) return 1;
    if (l < 0 || (l > 0 && (!coeffs || m < 1))) return 1;
    if (k_begin < 0 || k_end > K || k_begin > k_end) return 1;
    size_t slen = 2 + (size_t)l * (size_t)m;
    for (int k = k_begin; k < k_end; ++k) {
        const float *wk = w + (size_t)k * (size_t)row_stride;
        double *S = states + (size_t)k * slen;
        memset(S, 0, slen * sizeof(double));
        double sq = 0.0, pr = 0.0;
        for (int64_t j = 0; j < d; ++j) {
            double u = (double)wk[j] - (double)w_t0[j];      /* drift, Table 1 */
            sq += u * u;                                     /* ||u||^2        */
            if (xi) pr += (double)xi[j] * u;                 /* <xi,u>         */
            for (int i = 0; i < l; ++i) {                    /* sk(u), row i   */
                uint32_t c = bucket_of(coeffs + 6 * i, (uint64_t)j, (uint32_t)m);
                int s = sign_of(coeffs + 6 * i, (uint64_t)j);
                S[2 + (size_t)i * m + c] += (double)s * u;
            }
        }
        S[0] = sq;
        S[1] = pr;
    }
    return 0;
}

static int cmp_double(const void *a, const void *b)
{
    double x = *(const double *)a, y = *(const double *)b;
    return (x > y) - (x < y);
}

/*
 * Average state, M2, H and the trigger (Algorithm 1 "AllReduce(S)" and the test
 * H(S-bar) > Theta; Theorem 1: H = S-bar[0] - M2(S-bar sketch)/(1+eps); Theorem 2:
 * H = S-bar[0] - S-bar[1]^2).
 *   variant 0 = LinearFDA, 1 = SketchFDA.
 *   out[0] = mean_k ||u^(k)||^2      out[1] = estimate of ||u-bar||^2 that is subtracted
 *   out[2] = H                       out[3] = 1.0 if H > theta else 0.0
 *   out[4 + i] = ||row i of the averaged sketch||^2,  i < l
 * The median of an even number of rows is the mean of the two middle values.
 */
int fda_oracle_combine(const double *states, int K, int l, int m, int variant,
                       double epsilon, double theta, double *out)
{
    if (!states || !out || K < 1 || l < 0 || (l > 0 && m < 1)) return 1;
    if (variant != 0 && variant != 1) return 1;
    if (variant == 1 && l < 1) return 1;
    size_t slen = 2 + (size_t)l * (size_t)m;
    double *Sbar = (double *)calloc(slen, sizeof(double));
    if (!Sbar) return 2;
    for (size_t e = 0; e < slen; ++e) {
        double acc = 0.0;
        for (int k = 0; k < K; ++k) acc += states[(size_t)k * slen + e];
        Sbar[e] = acc / (double)K;
    }
    double rows[64];
    if (l > 64) { free(Sbar); return 1; }
    for (int i = 0; i < l; ++i) {
        double r = 0.0;
        for (int c = 0; c < m; ++c) {
            double v = Sbar[2 + (size_t)i * m + c];
            r += v * v;
        }
        rows[i] = r;
        out[4 + i] = r;
    }
    double est;
    if (variant == 1) {
        double sorted[64];
        memcpy(sorted, rows, (size_t)l * sizeof(double));
        qsort(sorted, (size_t)l, sizeof(double), cmp_double);
        double med = (l & 1) ? sorted[l / 2] : 0.5 * (sorted[l / 2 - 1] + sorted[l / 2]);
        est = med / (1.0 + epsilon);
    } else {
        est = Sbar[1] * Sbar[1];
    }
    out[0] = Sbar[0];
    out[1] = est;
    out[2] = Sbar[0] - est;
    out[3] = (out[2] > theta) ? 1.0 : 0.0;
    free(Sbar);
    return 0;
}

/* Average model w-bar[j] = (1/K) sum_k w^(k)[j]  (Notation; "AllReduce") for j in
 * [j_begin, j_end); writes avg[j - j_begin]. */
int fda_oracle_average(const float *w, int64_t row_stride, int K, int64_t d,
                       int64_t j_begin, int64_t j_end, double *avg)
{
    if (!w || !avg || K < 1 || d < 1 || row_stride < d) return 1;
    if (j_begin < 0 || j_end > d || j_begin > j_end) return 1;
    for (int64_t j = j_begin; j < j_end; ++j) {
        double acc = 0.0;
        for (int k = 0; k < K; ++k) acc += (double)w[(size_t)k * (size_t)row_stride + (size_t)j];
        avg[j - j_begin] = acc / (double)K;
    }
    return 0;
}

/* Model variance by its definition, Eq. (2): (1/K) sum_k ||w^(k) - w-bar||^2, and the
 * two terms of Eq. (4).  out = { Var (Eq. 2), mean_k ||u^(k)||^2, ||u-bar||^2 }. */
int fda_oracle_variance(const float *w, int64_t row_stride, int K, int64_t d,
                        const float *w_t0, double *out)
{
    if (!w || !w_t0 || !out || K < 1 || d < 1 || row_stride < d) return 1;
    double var = 0.0, msq = 0.0, ubar2 = 0.0;
    for (int64_t j = 0; j < d; ++j) {
        double wbar = 0.0;
        for (int k = 0; k < K; ++k) wbar += (double)w[(size_t)k * (size_t)row_stride + (size_t)j];
        wbar /= (double)K;
        for (int k = 0; k < K; ++k) {
            double wk = (double)w[(size_t)k * (size_t)row_stride + (size_t)j];
            double dv = wk - wbar;
            double u = wk - (double)w_t0[j];
            var += dv * dv;
            msq += u * u;
        }
        double ub = wbar - (double)w_t0[j];
        ubar2 += ub * ub;
    }
    out[0] = var / (double)K;
    out[1] = msq / (double)K;
    out[2] = ubar2;
    return 0;
}

/* LinearFDA direction heuristic (Section 3.2, Table 1): xi = (w_new - w_old) / ||w_new - w_old||,
 * the normalised step of the global model between two synchronisations.  w_new is the fp64
 * average model, w_old the fp32 model it replaces.  A zero step gives xi = 0. */
int fda_oracle_direction(const double *w_new, const float *w_old, int64_t d, double *xi)
{
    if (!w_new || !w_old || !xi || d < 1) return 1;
    double sq = 0.0;
    for (int64_t j = 0; j < d; ++j) {
        double dl = w_new[j] - (double)w_old[j];
        sq += dl * dl;
    }
    double norm = sqrt(sq);
    for (int64_t j = 0; j < d; ++j)
        xi[j] = norm > 0.0 ? (w_new[j] - (double)w_old[j]) / norm : 0.0;
    return 0;
}
