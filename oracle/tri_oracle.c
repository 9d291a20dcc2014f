/*
 * tri_oracle.c -- float64 CPU oracle for the TriAttention KV-compression round.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, literal statement of what the
 * compression round computes, written from the paper's formulas.  It shares no code,
 * header, table or constant with the CUDA library and is only ever called from the
 * tests, the smoke check and the benchmark's CPU-baseline leg.
 *
 * Everything is evaluated term by term, in double precision, in the paper's notation:
 *   d        head dimension, F = d/2 frequency bands
 *   omega_f  = theta^(-2f/d)                                   (Section 2.1)
 *   k_f      complex pre-RoPE component of a key in band f     (Section 4.1)
 *   Delta    = p_q - p_k                                       (Section 4.1)
 *   phi_f    = arg(E[q_f]) - arg(k_f)                          (Section 4.1)
 *   S_trig, S_norm, S~, z-score, S_final                       (Sections 4.1-4.3)
 * No term is folded, reordered or cached beyond what those formulas state.
 *
 * Band layout: layout 0 pairs components (x[2f], x[2f+1]) exactly as the rotation
 * matrix of Section 2.1 is printed; layout 1 pairs (x[f], x[f+F]).
 *
 * Every routine is pinned by tests that do not reuse its formula (explicit 2x2
 * rotations + dot products, closed forms, invariants, exhaustive subsets), so no
 * function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ---- band helpers ---------------------------------------------------------------- */

static inline int re_index(int f, int F, int layout) { return layout == 0 ? 2 * f : f; }
static inline int im_index(int f, int F, int layout) { return layout == 0 ? 2 * f + 1 : f + F; }

/* omega_f = theta^(-2f/d), f = 0..d/2-1 (Section 2.1). */
void tri_oracle_omega(double theta, int d, double *omega)
{
    for (int f = 0; f < d / 2; ++f)
        omega[f] = pow(theta, -2.0 * (double)f / (double)d);
}

/* bf16 -> double, exact: a bf16 is the upper half of an IEEE binary32. */
void tri_oracle_bf16_to_f64(const uint16_t *in, int64_t n, double *out)
{
    for (int64_t i = 0; i < n; ++i) {
        uint32_t bits = (uint32_t)in[i] << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        out[i] = (double)f;
    }
}

/*
 * Inverse of RoPE (Appendix B.1: k~_f(p) = k_f * e^{i omega_f p}):
 * k_f = k~_f * e^{-i omega_f p}, applied row by row with each row's own position.
 */
void tri_oracle_unrotate(const double *k_post, const int64_t *pos, int64_t N, int d,
                         double theta, int layout, double *k_pre)
{
    const int F = d / 2;
    for (int64_t n = 0; n < N; ++n) {
        const double *x = k_post + n * d;
        double *y = k_pre + n * d;
        for (int f = 0; f < F; ++f) {
            double w = pow(theta, -2.0 * (double)f / (double)d);
            double a = w * (double)pos[n];
            double c = cos(a), s = sin(a);
            double xr = x[re_index(f, F, layout)], xi = x[im_index(f, F, layout)];
            /* (xr + i xi) * (c - i s) */
            y[re_index(f, F, layout)] = xr * c + xi * s;
            y[im_index(f, F, layout)] = xi * c - xr * s;
        }
    }
}

/* ---- scoring (Sections 4.1, 4.2) ------------------------------------------------- */

/*
 * S_trig(k, Delta) = sum_f |E[q_f]| * |k_f| * cos(omega_f * Delta + phi_f),
 * phi_f = arg(E[q_f]) - arg(k_f)                                     (Section 4.1)
 */
double tri_oracle_s_trig(const double *k_pre, const double *q_center, int d, double theta,
                         int layout, double Delta)
{
    const int F = d / 2;
    double acc = 0.0;
    for (int f = 0; f < F; ++f) {
        double w = pow(theta, -2.0 * (double)f / (double)d);
        double qr = q_center[re_index(f, F, layout)], qi = q_center[im_index(f, F, layout)];
        double kr = k_pre[re_index(f, F, layout)], ki = k_pre[im_index(f, F, layout)];
        double qn = hypot(qr, qi), kn = hypot(kr, ki);
        double phi = atan2(qi, qr) - atan2(ki, kr);
        acc += qn * kn * cos(w * Delta + phi);
    }
    return acc;
}

/*
 * Norm term.  variant 0: sum_f (E|q_f| - |E q_f|) |k_f|   (Section 4.2, rewritten form)
 *             variant 1: sum_f  E|q_f| |k_f|              (Section 4.1, S_norm^(0))
 *             variant 2: 0                                (ablation without the norm term)
 *             variant 3: sum_f (1 - R_f) E|q_f| |k_f|, R_f = |E q_f| / E|q_f|
 *                        (Section 4.2, first form; equals variant 0 algebraically)
 */
double tri_oracle_s_norm(const double *k_pre, const double *q_center, const double *q_mean_norm,
                         int d, int layout, int variant)
{
    const int F = d / 2;
    double acc = 0.0;
    if (variant == 2) return 0.0;
    for (int f = 0; f < F; ++f) {
        double qr = q_center[re_index(f, F, layout)], qi = q_center[im_index(f, F, layout)];
        double kr = k_pre[re_index(f, F, layout)], ki = k_pre[im_index(f, F, layout)];
        double kn = hypot(kr, ki);
        double cn = hypot(qr, qi);
        double en = q_mean_norm[f];
        double wgt;
        if (variant == 0) wgt = en - cn;
        else if (variant == 1) wgt = en;
        else { double R = (en != 0.0) ? cn / en : 0.0; wgt = (1.0 - R) * en; }
        acc += wgt * kn;
    }
    return acc;
}

/*
 * S~(k) = (1/|D|) sum_{delta in D} [ S_trig(k, Delta + delta) + S_norm(k) ]  (Section 4.2)
 * for every key of one unit and every query head g of its group.
 *   k_pre        [N][d]   pre-RoPE keys
 *   pos          [N]      original position of each key
 *   p_q                   position of the query (Delta = p_q - pos[n])
 *   q_center     [G][d]   E[q_f] per query head, same band layout as the keys
 *   q_mean_norm  [G][F]   E|q_f|
 *   raw          [G][N]   output
 */
void tri_oracle_score_raw(const double *k_pre, const int64_t *pos, int64_t N, int d, int64_t p_q,
                          const double *q_center, const double *q_mean_norm, int G,
                          const int64_t *offsets, int n_off, double theta, int layout,
                          int norm_variant, double *raw)
{
    const int F = d / 2;
    for (int g = 0; g < G; ++g) {
        const double *qc = q_center + (int64_t)g * d;
        const double *qn = q_mean_norm + (int64_t)g * F;
#pragma omp parallel for schedule(static)
        for (int64_t n = 0; n < N; ++n) {
            const double *k = k_pre + n * d;
            double Delta = (double)(p_q - pos[n]);
            double acc = 0.0;
            for (int j = 0; j < n_off; ++j) {
                double S = tri_oracle_s_trig(k, qc, d, theta, layout, Delta + (double)offsets[j])
                         + tri_oracle_s_norm(k, qc, qn, d, layout, norm_variant);
                acc += S;
            }
            raw[(int64_t)g * N + n] = acc / (double)n_off;
        }
    }
}

/* ---- GQA normalise-then-aggregate (Section 4.3) ---------------------------------- */

/*
 * z^(g)(k) = (S~^(g)(k) - mu_g) / sigma_g with mu_g, sigma_g the mean and (population)
 * standard deviation over the N keys; S_final(k) = max_g z^(g)(k).
 * A head whose scores are all equal has sigma_g = 0 and gets z^(g) == 0 (tested on the
 * values themselves, so that summation rounding cannot turn "constant" into sigma ~ 1e-16).
 *   raw [G][N] in, zscore [G][N] out (may be NULL), s_final [N] out.
 */
void tri_oracle_normalize(const double *raw, int G, int64_t N, double *zscore, double *s_final)
{
    for (int64_t n = 0; n < N; ++n) s_final[n] = -INFINITY;
    for (int g = 0; g < G; ++g) {
        const double *x = raw + (int64_t)g * N;
        double mu = 0.0;
        for (int64_t n = 0; n < N; ++n) mu += x[n];
        mu /= (double)N;
        double var = 0.0;
        for (int64_t n = 0; n < N; ++n) var += (x[n] - mu) * (x[n] - mu);
        var /= (double)N;
        double sigma = sqrt(var);
        double lo = x[0], hi = x[0];
        for (int64_t n = 1; n < N; ++n) { if (x[n] < lo) lo = x[n]; if (x[n] > hi) hi = x[n]; }
        if (lo == hi) sigma = 0.0;
        for (int64_t n = 0; n < N; ++n) {
            double z = (sigma > 0.0) ? (x[n] - mu) / sigma : 0.0;
            if (zscore) zscore[(int64_t)g * N + n] = z;
            if (z > s_final[n]) s_final[n] = z;
        }
    }
}

/* ---- top-B retention (Section 4.3) ------------------------------------------------ */

typedef struct { double s; int32_t i; } scored_t;

static int by_score_desc_then_index(const void *a, const void *b)
{
    const scored_t *x = (const scored_t *)a, *y = (const scored_t *)b;
    if (x->s > y->s) return -1;
    if (x->s < y->s) return 1;
    return (x->i > y->i) - (x->i < y->i);
}

static int by_index(const void *a, const void *b)
{
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

/*
 * Keep the B keys with the highest S_final; equal scores: the lower slot wins.
 * N <= B keeps everything.  Kept slot indices are returned in ascending order.
 * Returns the number kept (min(B, N)).
 */
int64_t tri_oracle_select(const double *s_final, int64_t N, int64_t B, int32_t *kept_idx)
{
    int64_t cnt = N < B ? N : B;
    if (cnt <= 0) return 0;
    scored_t *a = (scored_t *)malloc((size_t)N * sizeof *a);
    for (int64_t n = 0; n < N; ++n) { a[n].s = s_final[n]; a[n].i = (int32_t)n; }
    qsort(a, (size_t)N, sizeof *a, by_score_desc_then_index);
    for (int64_t j = 0; j < cnt; ++j) kept_idx[j] = a[j].i;
    free(a);
    qsort(kept_idx, (size_t)cnt, sizeof *kept_idx, by_index);
    return cnt;
}

/* ---- eviction = order-preserving gather (Section 4.3) ----------------------------- */

/* out[j] = rows[kept_idx[j]], rows being opaque records of row_bytes bytes. */
void tri_oracle_compact(const void *rows, int64_t row_bytes, const int32_t *kept_idx, int64_t cnt,
                        void *out)
{
    for (int64_t j = 0; j < cnt; ++j)
        memcpy((char *)out + j * row_bytes, (const char *)rows + (int64_t)kept_idx[j] * row_bytes,
               (size_t)row_bytes);
}

/* ---- one whole unit from a bf16 post-RoPE cache ----------------------------------- */

/*
 * The round for one (sequence, layer, KV head) unit whose keys are cached post-RoPE in
 * bf16: widen, undo the rotation with each slot's position, score, normalise, select.
 *   k_post_bf16 [N][d]; pos [N]; raw [G][N] (may be NULL); s_final [N]; kept_idx [min(B,N)].
 * Returns the number kept.
 */
int64_t tri_oracle_unit_bf16(const uint16_t *k_post_bf16, const int64_t *pos, int64_t N, int d,
                             int64_t p_q, const double *q_center, const double *q_mean_norm,
                             int G, const int64_t *offsets, int n_off, double theta, int layout,
                             int norm_variant, int64_t B, double *raw, double *s_final,
                             int32_t *kept_idx)
{
    double *k_post = (double *)malloc((size_t)N * d * sizeof(double));
    double *k_pre = (double *)malloc((size_t)N * d * sizeof(double));
    double *raw_l = raw ? raw : (double *)malloc((size_t)G * N * sizeof(double));
    tri_oracle_bf16_to_f64(k_post_bf16, N * d, k_post);
    tri_oracle_unrotate(k_post, pos, N, d, theta, layout, k_pre);
    tri_oracle_score_raw(k_pre, pos, N, d, p_q, q_center, q_mean_norm, G, offsets, n_off, theta,
                         layout, norm_variant, raw_l);
    tri_oracle_normalize(raw_l, G, N, NULL, s_final);
    int64_t cnt = tri_oracle_select(s_final, N, B, kept_idx);
    if (!raw) free(raw_l);
    free(k_post);
    free(k_pre);
    return cnt;
}

/* ---- 8-bit caches ------------------------------------------------------------------ */

/*
 * The paper does not speak of 8-bit key caches; the reading taken here: a key stored as e4m3 stands for the value
 * its eight bits encode, and everything of Sections 4.1-4.3 applies to that value unchanged (a positive scale shared
 * by a unit's keys multiplies every raw score of the unit and drops out of the z-score).
 * e4m3 (the 8-bit floating-point format with 4 exponent and 3 mantissa bits, bias 7, no infinities): bits s eeee mmm.
 *   eeee = 0          : (-1)^s * 2^-6 * (mmm / 8)                (subnormal; +0 and -0)
 *   eeee = 15, mmm = 7: not a number
 *   otherwise         : (-1)^s * 2^(eeee - 7) * (1 + mmm / 8)    (largest finite value 448)
 */
void tri_oracle_e4m3_to_f64(const uint8_t *in, int64_t n, double *out)
{
    for (int64_t i = 0; i < n; ++i) {
        const int b = in[i], e = (b >> 3) & 15, m = b & 7;
        double v;
        if (e == 15 && m == 7) v = NAN;
        else if (e == 0) v = ldexp((double)m / 8.0, -6);
        else v = ldexp(1.0 + (double)m / 8.0, e - 7);
        out[i] = (b & 128) ? -v : v;
    }
}

/* tri_oracle_unit_bf16 for a unit cached post-RoPE in e4m3: k_post_e4m3 [N][d] bytes. */
int64_t tri_oracle_unit_e4m3(const uint8_t *k_post_e4m3, const int64_t *pos, int64_t N, int d,
                             int64_t p_q, const double *q_center, const double *q_mean_norm,
                             int G, const int64_t *offsets, int n_off, double theta, int layout,
                             int norm_variant, int64_t B, double *raw, double *s_final,
                             int32_t *kept_idx)
{
    double *k_post = (double *)malloc((size_t)N * d * sizeof(double));
    double *k_pre = (double *)malloc((size_t)N * d * sizeof(double));
    double *raw_l = raw ? raw : (double *)malloc((size_t)G * N * sizeof(double));
    tri_oracle_e4m3_to_f64(k_post_e4m3, N * d, k_post);
    tri_oracle_unrotate(k_post, pos, N, d, theta, layout, k_pre);
    tri_oracle_score_raw(k_pre, pos, N, d, p_q, q_center, q_mean_norm, G, offsets, n_off, theta,
                         layout, norm_variant, raw_l);
    tri_oracle_normalize(raw_l, G, N, NULL, s_final);
    int64_t cnt = tri_oracle_select(s_final, N, B, kept_idx);
    if (!raw) free(raw_l);
    free(k_post);
    free(k_pre);
    return cnt;
}

int tri_oracle_num_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---- calibration statistics (Sections 3.3, 4.1, Appendix B.5) ----------------------- */

/*
 * Per band f over T pre-RoPE query vectors q[t]:
 *   center      E[q_f]   complex mean, stored in the input's own component layout   [d]
 *   mean_norm   E|q_f|   mean of the band magnitudes                                 [d/2]
 *   mrl         R_f = |E[q_f]| / E|q_f|  (mean resultant length; 0 where E|q_f| = 0) [d/2]
 * Plain sums in double, token by token.
 */
void tri_oracle_calibrate(const double *q, int64_t T, int d, int layout, double *center,
                          double *mean_norm, double *mrl)
{
    const int F = d / 2;
    for (int i = 0; i < d; ++i) center[i] = 0.0;
    for (int f = 0; f < F; ++f) mean_norm[f] = 0.0;
    for (int64_t t = 0; t < T; ++t) {
        const double *x = q + t * d;
        for (int i = 0; i < d; ++i) center[i] += x[i];
        for (int f = 0; f < F; ++f)
            mean_norm[f] += hypot(x[re_index(f, F, layout)], x[im_index(f, F, layout)]);
    }
    for (int i = 0; i < d; ++i) center[i] /= (double)T;
    for (int f = 0; f < F; ++f) {
        mean_norm[f] /= (double)T;
        double cn = hypot(center[re_index(f, F, layout)], center[im_index(f, F, layout)]);
        mrl[f] = mean_norm[f] > 0.0 ? cn / mean_norm[f] : 0.0;
    }
}
