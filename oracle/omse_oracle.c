/*
 * CPU oracle for the constrained-MMSE quantization path of "Low-bit Quantization of
 * Neural Networks for Efficient Inference" (Choukroun et al., arXiv:1902.06822).
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is a plain, slow, one-element-at-a-time
 * restatement of what the method computes, written so that it can be checked against
 * the paper by eye.  The CUDA library shares no code with it and never calls it; only
 * the tests, the smoke check and the benchmark's CPU-baseline leg may load it.
 *
 * Everything is evaluated in the order the paper states it, with no blocking, fusion
 * or reordering.  Decisions that produce an integer (the codes) are taken in IEEE
 * binary32 exactly as Section 3.1 writes them (divide, round to nearest, saturate);
 * every sum is accumulated in binary64.
 *
 * Parity pins (tests marked "not gpu"): exact piecewise-quadratic optimum by breakpoint
 * enumeration on tiny tensors, hand-worked examples, on-grid inputs, the no-offset
 * uniform quantizer of Section 3.1, invariants of Sections 3.4/3.5, pack round trip.
 * No function in this file is "parity unpinned".
 *
 * The optional OpenMP pragmas only distribute independent kernels (rows) or independent
 * candidates over threads; each row / candidate is still computed serially.
 */
#include <float.h>
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* status bits reported per call (data-dependent conditions, never an error) */
#define ORACLE_STATUS_NONFINITE 1u /* a NaN or Inf was seen in the input            */
#define ORACLE_STATUS_DEGENERATE 2u /* a segment had no usable scale (all zero/tiny) */

int omse_oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Section 3.1: the quantization range Z_p.  Unsigned {0..2^p-1}; signed {-2^(p-1)..2^(p-1)-1}. */
void omse_oracle_grid_bounds(int bits, int is_signed, int *lo, int *hi)
{
    if (is_signed) {
        *lo = -(1 << (bits - 1));
        *hi = (1 << (bits - 1)) - 1;
    } else {
        *lo = 0;
        *hi = (1 << bits) - 1;
    }
}

/* Section 3.1, operator [.]_Zp applied to T_i/alpha (Section 3.4, optimal codes given alpha):
 * binary32 division, round to nearest (ties to even: the default IEEE mode), then saturate. */
static int code_of(float x, float alpha, int lo, int hi)
{
    float r = rintf(x / alpha);
    if (r < (float)lo) r = (float)lo;
    if (r > (float)hi) r = (float)hi;
    if (r != r) r = 0.0f; /* NaN input: any in-range code */
    return (int)r;
}

/* Section 3.4, objective ||T - alpha*T~||_F^2 for the codes that alpha implies. */
static double sse_of(const float *x, int64_t k, float alpha, int lo, int hi)
{
    double s = 0.0;
    for (int64_t i = 0; i < k; ++i) {
        double d = (double)x[i] - (double)alpha * (double)code_of(x[i], alpha, lo, hi);
        s += d * d;
    }
    return s;
}

double omse_oracle_sse_at(const float *x, int64_t k, float alpha, int bits, int is_signed)
{
    int lo, hi;
    omse_oracle_grid_bounds(bits, is_signed, &lo, &hi);
    return sse_of(x, k, alpha, lo, hi);
}

void omse_oracle_codes(const float *x, int64_t n, float alpha, int bits, int is_signed, int8_t *codes)
{
    int lo, hi;
    omse_oracle_grid_bounds(bits, is_signed, &lo, &hi);
    for (int64_t i = 0; i < n; ++i)
        codes[i] = (alpha > 0.0f) ? (int8_t)code_of(x[i], alpha, lo, hi) : (int8_t)0;
}

/* The candidate scales of the line search (Section 3.4 names a grid and leaves its points open): C points spaced
 * linearly in (0, hi_frac*max|x|], every operation in binary32. */
float omse_oracle_candidate(float max_abs, float hi_frac, int n_cand, int c)
{
    float a_hi = hi_frac * max_abs;
    float step = a_hi / (float)n_cand;
    return (float)(c + 1) * step;
}

static float max_abs_of(const float *x, int64_t k, uint32_t *status)
{
    float m = 0.0f;
    for (int64_t i = 0; i < k; ++i) {
        float a = fabsf(x[i]);
        if (!(a <= FLT_MAX)) *status |= ORACLE_STATUS_NONFINITE;
        if (a > m) m = a;
    }
    return m;
}

/* Closed-form scale for fixed codes (least squares of the Section 3.4 objective in alpha),
 * alternated with re-quantization as in the alternating scheme the paper cites; applied
 * `iters` times starting from `alpha`. */
static float refine_from(const float *x, int64_t k, float alpha, int lo, int hi, int iters)
{
    for (int it = 0; it < iters; ++it) {
        int64_t sqq = 0;
        double sxq = 0.0;
        for (int64_t i = 0; i < k; ++i) {
            int q = code_of(x[i], alpha, lo, hi);
            sqq += (int64_t)q * q;
            sxq += (double)x[i] * (double)q;
        }
        if (sqq == 0) break;
        float a_new = (float)(sxq / (double)sqq);
        if (!(a_new >= FLT_MIN) || !(a_new <= FLT_MAX)) break;
        alpha = a_new;
    }
    return alpha;
}

/*
 * The quantization mapping phi(T, p) of Section 3.4 on one segment x[0..k):
 *   grid line search over n_cand scales, lowest index on ties, then `refine_iters`
 *   closed-form polish steps, then the final codes and squared error.
 * start_idx < 0: run the search.  start_idx >= 0: skip the search and start the polish
 *   from that candidate (used by the harness when two candidates tie).
 * Outputs: *alpha, *sse (binary64), *best_idx (-1 for a degenerate segment),
 *   codes[k] (nullable), sse_curve[n_cand] (nullable; +inf for unusable candidates).
 * Degenerate segment (max|x| == 0, or every candidate below FLT_MIN): alpha = 0,
 *   all codes 0, sse = sum x^2, best_idx = -1.
 */
void omse_oracle_phi(const float *x, int64_t k, int bits, int is_signed, int n_cand, float hi_frac,
                     int refine_iters, int start_idx, float *alpha, double *sse, int32_t *best_idx,
                     int8_t *codes, double *sse_curve, uint32_t *status)
{
    int lo, hi;
    uint32_t st = 0;
    omse_oracle_grid_bounds(bits, is_signed, &lo, &hi);
    float m = max_abs_of(x, k, &st);

    int best = -1;
    double best_sse = INFINITY;
    if (start_idx >= 0) {
        best = start_idx;
        best_sse = 0.0;
        if (!(omse_oracle_candidate(m, hi_frac, n_cand, best) >= FLT_MIN)) best = -1;
    } else {
        for (int c = 0; c < n_cand; ++c) {
            float a = omse_oracle_candidate(m, hi_frac, n_cand, c);
            double s = INFINITY;
            if (a >= FLT_MIN && a <= FLT_MAX) s = sse_of(x, k, a, lo, hi);
            if (sse_curve) sse_curve[c] = s;
            if (s < best_sse) {
                best_sse = s;
                best = c;
            }
        }
    }

    if (best < 0) {
        double s = 0.0;
        for (int64_t i = 0; i < k; ++i) s += (double)x[i] * (double)x[i];
        *alpha = 0.0f;
        *sse = s;
        *best_idx = -1;
        if (codes) memset(codes, 0, (size_t)k);
        *status |= st | ORACLE_STATUS_DEGENERATE;
        return;
    }

    float a = omse_oracle_candidate(m, hi_frac, n_cand, best);
    a = refine_from(x, k, a, lo, hi, refine_iters);
    *alpha = a;
    *sse = sse_of(x, k, a, lo, hi);
    *best_idx = best;
    if (codes)
        for (int64_t i = 0; i < k; ++i) codes[i] = (int8_t)code_of(x[i], a, lo, hi);
    *status |= st;
}

/* Kernel-wise quantization (Section 3.3): phi applied independently to each of the
 * n_kernels contiguous segments of kernel_len elements.  start_idx is nullable. */
void omse_oracle_quantize_rows(const float *w, int64_t n_kernels, int64_t kernel_len, int bits,
                               int is_signed, int n_cand, float hi_frac, int refine_iters,
                               const int32_t *start_idx, float *alpha, double *sse,
                               int32_t *best_idx, int8_t *codes, uint32_t *status)
{
    uint32_t st_all = 0;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) reduction(| : st_all)
#endif
    for (int64_t s = 0; s < n_kernels; ++s) {
        uint32_t st = 0;
        omse_oracle_phi(w + s * kernel_len, kernel_len, bits, is_signed, n_cand, hi_frac,
                        refine_iters, start_idx ? start_idx[s] : -1, &alpha[s], &sse[s],
                        &best_idx[s], codes ? codes + s * kernel_len : NULL, NULL, &st);
        st_all |= st;
    }
    *status |= st_all;
}

/* Per-tensor search (Section 3.7, one beta for a whole activation tensor): the same phi on
 * one segment of n elements, with the independent candidates spread over threads. */
void omse_oracle_activation_scale(const float *x, int64_t n, int bits, int is_signed, int n_cand,
                                  float hi_frac, int refine_iters, float *alpha, double *sse,
                                  int32_t *best_idx, double *sse_curve, uint32_t *status)
{
    int lo, hi;
    uint32_t st = 0;
    omse_oracle_grid_bounds(bits, is_signed, &lo, &hi);
    float m = max_abs_of(x, n, &st);
    double *curve = sse_curve ? sse_curve : (double *)malloc(sizeof(double) * (size_t)n_cand);
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1)
#endif
    for (int c = 0; c < n_cand; ++c) {
        float a = omse_oracle_candidate(m, hi_frac, n_cand, c);
        curve[c] = (a >= FLT_MIN && a <= FLT_MAX) ? sse_of(x, n, a, lo, hi) : INFINITY;
    }
    int best = -1;
    double best_sse = INFINITY;
    for (int c = 0; c < n_cand; ++c)
        if (curve[c] < best_sse) {
            best_sse = curve[c];
            best = c;
        }
    if (!sse_curve) free(curve);
    /* polish and final error from the chosen candidate (serial, as in phi) */
    omse_oracle_phi(x, n, bits, is_signed, n_cand, hi_frac, refine_iters, best >= 0 ? best : 0,
                    alpha, sse, best_idx, NULL, NULL, &st);
    if (best < 0) *best_idx = -1;
    *status |= st;
}

/*
 * Algorithm 1 (alternating optimisation for multiple quantization) on one segment:
 * for each sweep, for j = 1..n: r = T - sum_{i != j} alpha_i T~^i, (alpha_j, T~^j) = phi(r, p_j).
 * All alpha_i and T~^i start at zero, so the first sweep quantizes the residual of the
 * previous approximation (Section 3.7 runs a single sweep).  The residual is formed in
 * binary32 by successive fused multiply-adds in increasing i.
 * Outputs (last sweep): alpha[n], sse[n] (error after tensors 1..j were updated),
 * best_idx[n], codes[n][k]; r_scratch[k] is caller-provided scratch.
 */
static void alg1_segment(const float *x, int64_t k, const int *bits, const int *is_signed, int n_cand,
                         float hi_frac, int refine_iters, int n_tensors, int n_sweeps,
                         int64_t out_stride, float *alpha, double *sse, int32_t *best_idx,
                         int8_t *codes, int64_t code_stride, float *r, double *sse_sweeps,
                         double eps, int32_t *sweeps_done, uint32_t *status)
{   /* is_signed: one flag per quantized tensor; sse_sweeps (nullable): [n_sweeps][n_tensors] with stride
     * out_stride, the error after every update, i.e. the convergence history of the while-loop.
     * eps >= 0: the while-condition of Algorithm 1.  The paper does not define the rate its condition tests;
     * here it is the relative decrease of the squared error over one sweep, (E_prev - E_cur)/E_prev
     * with E the error after the last tensor's update and E_0 = ||T||^2 (all tensors zero); the loop
     * ends after the first sweep whose rate is not above eps (tested as E_prev - E_cur > eps*E_prev),
     * or after n_sweeps sweeps.  History entries of sweeps that did not run repeat the last error.
     * eps < 0: exactly n_sweeps sweeps.  sweeps_done (nullable): sweeps that ran. */
    double e_prev = 0.0;
    for (int64_t e = 0; e < k; ++e) e_prev += (double)x[e] * (double)x[e];
    int ran = 0;
    for (int j = 0; j < n_tensors; ++j) {
        alpha[j * out_stride] = 0.0f;
        memset(codes + j * code_stride, 0, (size_t)k);
    }
    for (int sweep = 0; sweep < n_sweeps; ++sweep) {
        for (int j = 0; j < n_tensors; ++j) {
            for (int64_t e = 0; e < k; ++e) {
                float v = x[e];
                for (int i = 0; i < n_tensors; ++i)
                    if (i != j)
                        v = fmaf(-alpha[i * out_stride], (float)codes[i * code_stride + e], v);
                r[e] = v;
            }
            double s_j;
            omse_oracle_phi(r, k, bits[j], is_signed[j], n_cand, hi_frac, refine_iters, -1,
                            &alpha[j * out_stride], &s_j, &best_idx[j * out_stride],
                            codes + j * code_stride, NULL, status);
            sse[j * out_stride] = s_j;
            if (sse_sweeps) sse_sweeps[((int64_t)sweep * n_tensors + j) * out_stride] = s_j;
        }
        ran = sweep + 1;
        if (eps >= 0.0) {
            double e_cur = sse[(n_tensors - 1) * out_stride];
            int go_on = (e_prev - e_cur) > eps * e_prev;
            e_prev = e_cur;
            if (!go_on) break;
        }
    }
    if (sse_sweeps)
        for (int sweep = ran; sweep < n_sweeps; ++sweep)
            for (int j = 0; j < n_tensors; ++j)
                sse_sweeps[((int64_t)sweep * n_tensors + j) * out_stride] = sse[j * out_stride];
    if (sweeps_done) *sweeps_done = ran;
}

/* Algorithm 1 kernel-wise with one signedness flag per quantized tensor and the error after every
 * update: sse_sweeps (nullable) is [n_sweeps][n_tensors][n_kernels]. */
void omse_oracle_alg1_rows_eps(const float *t, int64_t n_kernels, int64_t kernel_len, const int *bits,
                               const int *is_signed, int n_cand, float hi_frac, int refine_iters,
                               int n_tensors, int max_sweeps, double eps, float *alpha, double *sse,
                               int32_t *best_idx, int8_t *codes, double *sse_sweeps, int32_t *sweeps_done,
                               uint32_t *status)
{
    /* layouts as omse_oracle_alg1_rows; sweeps_done [n_kernels] (nullable) */
    int64_t n = n_kernels * kernel_len;
    uint32_t st_all = 0;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) reduction(| : st_all)
#endif
    for (int64_t s = 0; s < n_kernels; ++s) {
        uint32_t st = 0;
        float *r = (float *)malloc(sizeof(float) * (size_t)kernel_len);
        alg1_segment(t + s * kernel_len, kernel_len, bits, is_signed, n_cand, hi_frac, refine_iters,
                     n_tensors, max_sweeps, n_kernels, alpha + s, sse + s, best_idx + s,
                     codes + s * kernel_len, n, r, sse_sweeps ? sse_sweeps + s : NULL, eps,
                     sweeps_done ? sweeps_done + s : NULL, &st);
        free(r);
        st_all |= st;
    }
    *status |= st_all;
}

void omse_oracle_alg1_rows(const float *t, int64_t n_kernels, int64_t kernel_len, const int *bits,
                           const int *is_signed, int n_cand, float hi_frac, int refine_iters,
                           int n_tensors, int n_sweeps, float *alpha, double *sse, int32_t *best_idx,
                           int8_t *codes, double *sse_sweeps, uint32_t *status)
{
    /* layouts: alpha/sse/best_idx [n_tensors][n_kernels]; codes [n_tensors][n_kernels*kernel_len] */
    int64_t n = n_kernels * kernel_len;
    uint32_t st_all = 0;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) reduction(| : st_all)
#endif
    for (int64_t s = 0; s < n_kernels; ++s) {
        uint32_t st = 0;
        float *r = (float *)malloc(sizeof(float) * (size_t)kernel_len);
        alg1_segment(t + s * kernel_len, kernel_len, bits, is_signed, n_cand, hi_frac, refine_iters,
                     n_tensors, n_sweeps, n_kernels, alpha + s, sse + s, best_idx + s,
                     codes + s * kernel_len, n, r, sse_sweeps ? sse_sweeps + s : NULL, -1.0, NULL, &st);
        free(r);
        st_all |= st;
    }
    *status |= st_all;
}

void omse_oracle_residual_rows(const float *t, int64_t n_kernels, int64_t kernel_len,
                               const int *bits, int is_signed, int n_cand, float hi_frac,
                               int refine_iters, int n_tensors, int n_sweeps, float *alpha,
                               double *sse, int32_t *best_idx, int8_t *codes, uint32_t *status)
{
    int flags[16];
    for (int j = 0; j < n_tensors && j < 16; ++j) flags[j] = is_signed;
    omse_oracle_alg1_rows(t, n_kernels, kernel_len, bits, flags, n_cand, hi_frac, refine_iters, n_tensors,
                          n_sweeps, alpha, sse, best_idx, codes, NULL, status);
}

/*
 * Dual line search (Section 3.5, the n = 2 case, third displayed equation of that section): for a
 * pair of scales (alpha1, alpha2) every element picks the first code t in Z_p1 by enumeration, the
 * second code being the rounding of what is left:
 *     min over t in Z_p1 of ( T_j - alpha1*t - alpha2*[ (T_j - alpha1*t)/alpha2 ]_Zp2 )^2 ,
 * and the pair of scales is found on a two-dimensional grid.  The paper gives no grid; here
 * alpha1_c = (c+1)/C1 * hi_frac1 * max|T|  and  alpha2_{c,d} = (d+1)/C2 * hi_frac2 * alpha1_c,
 * every operation in binary32 (same form as the one-dimensional grid).
 * Decisions are taken in binary32: r = fmaf(-alpha1, t, x); q = [r/alpha2]_Zp2;
 * e = fmaf(-alpha2, q, r); the t with the smallest e*e wins, lowest t on ties.  The reported error is
 * the objective itself in binary64 for the chosen codes.
 */
static void dual_codes_of(float x, float a1, float a2, int lo1, int hi1, int lo2, int hi2, int *t_out,
                          int *q_out)
{
    float best = INFINITY;
    int bt = lo1, bq = 0;
    for (int t = lo1; t <= hi1; ++t) {
        float r = fmaf(-a1, (float)t, x);
        int q = code_of(r, a2, lo2, hi2);
        float e = fmaf(-a2, (float)q, r);
        float ee = e * e;
        if (ee < best) {
            best = ee;
            bt = t;
            bq = q;
        }
    }
    *t_out = bt;
    *q_out = bq;
}

static double dual_sse_of(const float *x, int64_t k, float a1, float a2, int lo1, int hi1, int lo2,
                          int hi2)
{
    double s = 0.0;
    for (int64_t i = 0; i < k; ++i) {
        int t, q;
        dual_codes_of(x[i], a1, a2, lo1, hi1, lo2, hi2, &t, &q);
        double d = (double)x[i] - (double)a1 * (double)t - (double)a2 * (double)q;
        s += d * d;
    }
    return s;
}

double omse_oracle_dual_sse_at(const float *x, int64_t k, float a1, float a2, int bits1, int bits2,
                               int is_signed)
{
    int lo1, hi1, lo2, hi2;
    omse_oracle_grid_bounds(bits1, is_signed, &lo1, &hi1);
    omse_oracle_grid_bounds(bits2, is_signed, &lo2, &hi2);
    return dual_sse_of(x, k, a1, a2, lo1, hi1, lo2, hi2);
}

void omse_oracle_dual_scales(float max_abs, float hi_frac1, float hi_frac2, int n_cand1, int n_cand2,
                             int c, int d, float *a1, float *a2)
{
    *a1 = omse_oracle_candidate(max_abs, hi_frac1, n_cand1, c);
    *a2 = omse_oracle_candidate(*a1, hi_frac2, n_cand2, d);
}

/* One segment.  start_idx >= 0 skips the search and takes that flat pair index c*C2+d.
 * Outputs: alpha[2], *sse, *best_idx (-1 degenerate), codes1[k], codes2[k] (nullable),
 * sse_curve[C1*C2] (nullable, +inf for unusable pairs). */
void omse_oracle_dual(const float *x, int64_t k, int bits1, int bits2, int is_signed, int n_cand1,
                      int n_cand2, float hi_frac1, float hi_frac2, int start_idx, float *alpha,
                      double *sse, int32_t *best_idx, int8_t *codes1, int8_t *codes2,
                      double *sse_curve, uint32_t *status)
{
    int lo1, hi1, lo2, hi2;
    uint32_t st = 0;
    omse_oracle_grid_bounds(bits1, is_signed, &lo1, &hi1);
    omse_oracle_grid_bounds(bits2, is_signed, &lo2, &hi2);
    float m = max_abs_of(x, k, &st);
    int best = -1;
    double best_sse = INFINITY;
    float a1, a2;
    if (start_idx >= 0) {
        omse_oracle_dual_scales(m, hi_frac1, hi_frac2, n_cand1, n_cand2, start_idx / n_cand2,
                                start_idx % n_cand2, &a1, &a2);
        if (a1 >= FLT_MIN && a2 >= FLT_MIN && a1 <= FLT_MAX) best = start_idx;
    } else {
        for (int c = 0; c < n_cand1; ++c)
            for (int d = 0; d < n_cand2; ++d) {
                omse_oracle_dual_scales(m, hi_frac1, hi_frac2, n_cand1, n_cand2, c, d, &a1, &a2);
                double s = INFINITY;
                if (a1 >= FLT_MIN && a2 >= FLT_MIN && a1 <= FLT_MAX)
                    s = dual_sse_of(x, k, a1, a2, lo1, hi1, lo2, hi2);
                if (sse_curve) sse_curve[c * n_cand2 + d] = s;
                if (s < best_sse) {
                    best_sse = s;
                    best = c * n_cand2 + d;
                }
            }
    }
    if (best < 0) {
        double s = 0.0;
        for (int64_t i = 0; i < k; ++i) s += (double)x[i] * (double)x[i];
        alpha[0] = alpha[1] = 0.0f;
        *sse = s;
        *best_idx = -1;
        if (codes1) memset(codes1, 0, (size_t)k);
        if (codes2) memset(codes2, 0, (size_t)k);
        *status |= st | ORACLE_STATUS_DEGENERATE;
        return;
    }
    omse_oracle_dual_scales(m, hi_frac1, hi_frac2, n_cand1, n_cand2, best / n_cand2, best % n_cand2,
                            &a1, &a2);
    alpha[0] = a1;
    alpha[1] = a2;
    *best_idx = best;
    double s = 0.0;
    for (int64_t i = 0; i < k; ++i) {
        int t, q;
        dual_codes_of(x[i], a1, a2, lo1, hi1, lo2, hi2, &t, &q);
        if (codes1) codes1[i] = (int8_t)t;
        if (codes2) codes2[i] = (int8_t)q;
        double dd = (double)x[i] - (double)a1 * (double)t - (double)a2 * (double)q;
        s += dd * dd;
    }
    *sse = s;
    *status |= st;
}

/* Kernel-wise dual search; alpha [2][n_kernels], codes [2][n_kernels*kernel_len]. */
void omse_oracle_dual_rows(const float *t, int64_t n_kernels, int64_t kernel_len, int bits1, int bits2,
                           int is_signed, int n_cand1, int n_cand2, float hi_frac1, float hi_frac2,
                           const int32_t *start_idx, float *alpha, double *sse, int32_t *best_idx,
                           int8_t *codes, uint32_t *status)
{
    int64_t n = n_kernels * kernel_len;
    uint32_t st_all = 0;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) reduction(| : st_all)
#endif
    for (int64_t s = 0; s < n_kernels; ++s) {
        uint32_t st = 0;
        float a[2];
        omse_oracle_dual(t + s * kernel_len, kernel_len, bits1, bits2, is_signed, n_cand1, n_cand2,
                         hi_frac1, hi_frac2, start_idx ? start_idx[s] : -1, a, &sse[s], &best_idx[s],
                         codes ? codes + s * kernel_len : NULL,
                         codes ? codes + n + s * kernel_len : NULL, NULL, &st);
        alpha[s] = a[0];
        alpha[n_kernels + s] = a[1];
        st_all |= st;
    }
    *status |= st_all;
}

/*
 * Quantization with offset (Section 3.1, first displayed scheme: T^ = alpha*[(T - delta)/alpha]_Zp + delta with
 * delta = min_i T_i and the unsigned range), with the scale found by the MMSE search instead of the
 * (max - delta)/(2^p - 1) rule: the shifted tensor fl(T_i - delta) (binary32 subtraction) goes through the
 * same phi on the unsigned grid.  The error is that of the shifted tensor.
 */
void omse_oracle_offset_phi(const float *x, int64_t k, int bits, int n_cand, float hi_frac, int refine_iters,
                            int start_idx, float *alpha, float *delta, double *sse, int32_t *best_idx,
                            int8_t *codes, uint32_t *status)
{
    float d = INFINITY;
    for (int64_t i = 0; i < k; ++i)
        if (fabsf(x[i]) <= FLT_MAX && x[i] < d) d = x[i];
    if (!(d < INFINITY)) d = 0.0f;
    float *r = (float *)malloc(sizeof(float) * (size_t)(k > 0 ? k : 1));
    for (int64_t i = 0; i < k; ++i) r[i] = x[i] - d;
    omse_oracle_phi(r, k, bits, 0, n_cand, hi_frac, refine_iters, start_idx, alpha, sse, best_idx, codes, NULL,
                    status);
    *delta = d;
    free(r);
}

void omse_oracle_offset_rows(const float *w, int64_t n_kernels, int64_t kernel_len, int bits, int n_cand,
                             float hi_frac, int refine_iters, const int32_t *start_idx, float *alpha,
                             float *delta, double *sse, int32_t *best_idx, int8_t *codes, uint32_t *status)
{
    uint32_t st_all = 0;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) reduction(| : st_all)
#endif
    for (int64_t s = 0; s < n_kernels; ++s) {
        uint32_t st = 0;
        omse_oracle_offset_phi(w + s * kernel_len, kernel_len, bits, n_cand, hi_frac, refine_iters,
                               start_idx ? start_idx[s] : -1, &alpha[s], &delta[s], &sse[s], &best_idx[s],
                               codes ? codes + s * kernel_len : NULL, &st);
        st_all |= st;
    }
    *status |= st_all;
}

/*
 * Comparison solvers of Section 3.4 (the columns of the paper's table comparing quantization methods):
 * other ways of choosing the scale alpha for the same objective ||T - alpha*[T/alpha]_Zp||^2.
 *   solver 0, "uniform": the no-offset uniform quantizer of Section 3.1, alpha = max|T| / L with
 *       L = 2^(p-1)-1 (signed range) or 2^p-1 (unsigned range); no search.
 *   solver 1, "alternating": alternating optimisation started from the uniform scale: n_iter times
 *       q = [T/alpha]_Zp, alpha = <T,q>/<q,q> (the least-squares scale for fixed codes).
 *   solver 2, "golden": golden-section search for the minimum of the objective on the bracket
 *       [0, hi_frac*max|T|].  The paper gives neither bracket nor stopping rule; here n_iter shrink
 *       steps, all scales in binary32: with rho = 0.618034f the interior points are
 *       x1 = b - rho*(b-a), x2 = a + rho*(b-a) (each operation rounded); if f(x1) <= f(x2) the
 *       bracket becomes [a, x2] (equal values keep the smaller scale) else [x1, b]; one new
 *       evaluation per step; the result is the interior point with the smaller error, x1 on
 *       equal errors.  A scale below FLT_MIN has error +inf.
 * After the solver, refine_iters further least-squares steps (0 for the plain columns), then the
 * final codes and squared error, as in phi.  n_evals (nullable) receives the number of objective
 * evaluations the solver made.
 */
void omse_oracle_solver_phi(const float *x, int64_t k, int bits, int is_signed, int solver, int n_iter,
                            float hi_frac, int refine_iters, float *alpha, double *sse, int8_t *codes,
                            int32_t *n_evals, uint32_t *status)
{
    int lo, hi;
    uint32_t st = 0;
    omse_oracle_grid_bounds(bits, is_signed, &lo, &hi);
    float m = max_abs_of(x, k, &st);
    float a = 0.0f;
    int evals = 0;
    if (solver == 0 || solver == 1) {
        float levels = is_signed ? (float)((1 << (bits - 1)) - 1) : (float)((1 << bits) - 1);
        a = m / levels;
        if (solver == 1 && a >= FLT_MIN && a <= FLT_MAX) a = refine_from(x, k, a, lo, hi, n_iter);
    } else {
        const float rho = 0.618034f;
        float lo_a = 0.0f, hi_a = hi_frac * m;
        float d = hi_a - lo_a;
        float t = rho * d;
        float x1 = hi_a - t;
        float x2 = lo_a + t;
        double f1 = (x1 >= FLT_MIN && x1 <= FLT_MAX) ? sse_of(x, k, x1, lo, hi) : INFINITY;
        double f2 = (x2 >= FLT_MIN && x2 <= FLT_MAX) ? sse_of(x, k, x2, lo, hi) : INFINITY;
        evals = 2;
        for (int it = 0; it < n_iter; ++it) {
            if (f1 <= f2) {
                hi_a = x2;
                x2 = x1;
                f2 = f1;
                d = hi_a - lo_a;
                t = rho * d;
                x1 = hi_a - t;
                f1 = (x1 >= FLT_MIN && x1 <= FLT_MAX) ? sse_of(x, k, x1, lo, hi) : INFINITY;
            } else {
                lo_a = x1;
                x1 = x2;
                f1 = f2;
                d = hi_a - lo_a;
                t = rho * d;
                x2 = lo_a + t;
                f2 = (x2 >= FLT_MIN && x2 <= FLT_MAX) ? sse_of(x, k, x2, lo, hi) : INFINITY;
            }
            ++evals;
        }
        a = (f1 <= f2) ? x1 : x2;
        if (!(((f1 <= f2) ? f1 : f2) < INFINITY)) a = 0.0f;
    }
    if (n_evals) *n_evals = evals;
    if (!(a >= FLT_MIN) || !(a <= FLT_MAX)) { /* no usable scale: same outputs as a degenerate phi */
        double s = 0.0;
        for (int64_t i = 0; i < k; ++i) s += (double)x[i] * (double)x[i];
        *alpha = 0.0f;
        *sse = s;
        if (codes) memset(codes, 0, (size_t)k);
        *status |= st | ORACLE_STATUS_DEGENERATE;
        return;
    }
    a = refine_from(x, k, a, lo, hi, refine_iters);
    *alpha = a;
    *sse = sse_of(x, k, a, lo, hi);
    if (codes)
        for (int64_t i = 0; i < k; ++i) codes[i] = (int8_t)code_of(x[i], a, lo, hi);
    *status |= st;
}

void omse_oracle_solver_rows(const float *w, int64_t n_kernels, int64_t kernel_len, int bits, int is_signed,
                             int solver, int n_iter, float hi_frac, int refine_iters, float *alpha,
                             double *sse, int8_t *codes, uint32_t *status)
{
    uint32_t st_all = 0;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) reduction(| : st_all)
#endif
    for (int64_t s = 0; s < n_kernels; ++s) {
        uint32_t st = 0;
        omse_oracle_solver_phi(w + s * kernel_len, kernel_len, bits, is_signed, solver, n_iter, hi_frac,
                               refine_iters, &alpha[s], &sse[s], codes ? codes + s * kernel_len : NULL, NULL,
                               &st);
        st_all |= st;
    }
    *status |= st_all;
}

/*
 * Quantization with offset (Section 3.1, first displayed scheme) with BOTH parameters searched:
 * T^ = alpha*[(T - delta)/alpha]_Zp + delta on the unsigned range, minimising the squared error over a
 * grid of offsets and, for each offset, the line-search grid of Section 3.4 on the shifted tensor.
 * The paper fixes delta = min T and gives no search; this reading: with lo = min T, R = fl(max T - lo),
 *     delta_d = fl(lo + fl(fl(d) * fl(fl(off_frac*R) / fl(n_delta)))),  d = 0 .. n_delta-1,
 * (d = 0 is the paper's delta = min T), the shifted tensor is r_i = fl(T_i - delta_d) in binary32 and
 * its candidates are phi's: n_cand scales in (0, hi_frac*max|r|].  The pair with the smallest
 * error sum_i (r_i - alpha*[r_i/alpha]_Zp)^2 wins, lowest flat index d*n_cand + c on equal errors;
 * then refine_iters least-squares steps on the scale (offset fixed), final codes and error of the
 * shifted values.  start_flat >= 0 skips the search and starts from that flat index.
 */
void omse_oracle_affine_phi(const float *x, int64_t k, int bits, int n_cand, float hi_frac, int n_delta,
                            float off_frac, int refine_iters, int start_flat, float *alpha, float *delta,
                            double *sse, int32_t *best_idx, int8_t *codes, double *sse_curve, uint32_t *status)
{
    int lo, hi;
    uint32_t st = 0;
    omse_oracle_grid_bounds(bits, 0, &lo, &hi);
    float tmin = INFINITY, tmax = -INFINITY;
    for (int64_t i = 0; i < k; ++i) {
        if (!(fabsf(x[i]) <= FLT_MAX)) {
            st |= ORACLE_STATUS_NONFINITE;
            continue;
        }
        if (x[i] < tmin) tmin = x[i];
        if (x[i] > tmax) tmax = x[i];
    }
    if (!(tmin <= tmax)) tmin = tmax = 0.0f;
    float range = tmax - tmin;
    float dstep = (off_frac * range) / (float)n_delta;
    float *r = (float *)malloc(sizeof(float) * (size_t)(k > 0 ? k : 1));
    int best = -1;
    double best_sse = INFINITY;
    if (start_flat >= 0) {
        best = start_flat;
    } else {
        for (int d = 0; d < n_delta; ++d) {
            float dl = tmin + (float)d * dstep;
            for (int64_t i = 0; i < k; ++i) r[i] = x[i] - dl;
            uint32_t st_d = 0;
            float m = max_abs_of(r, k, &st_d);
            for (int c = 0; c < n_cand; ++c) {
                float a = omse_oracle_candidate(m, hi_frac, n_cand, c);
                double s = INFINITY;
                if (a >= FLT_MIN && a <= FLT_MAX) s = sse_of(r, k, a, lo, hi);
                if (sse_curve) sse_curve[(int64_t)d * n_cand + c] = s;
                if (s < best_sse) {
                    best_sse = s;
                    best = d * n_cand + c;
                }
            }
        }
    }
    int bd = best >= 0 ? best / n_cand : 0;
    float dl = tmin + (float)bd * dstep;
    for (int64_t i = 0; i < k; ++i) r[i] = x[i] - dl;
    /* polish, final codes and error: phi on the shifted tensor started from the winning candidate */
    omse_oracle_phi(r, k, bits, 0, n_cand, hi_frac, refine_iters, best >= 0 ? best % n_cand : 0, alpha, sse,
                    best_idx, codes, NULL, &st);
    if (best < 0 || *best_idx < 0) {
        *best_idx = -1;
        if (best < 0) { /* no usable pair at all: report the error of the tensor shifted by its minimum */
            *alpha = 0.0f;
            double s = 0.0;
            for (int64_t i = 0; i < k; ++i) s += (double)r[i] * (double)r[i];
            *sse = s;
            if (codes) memset(codes, 0, (size_t)k);
            st |= ORACLE_STATUS_DEGENERATE;
        }
    } else {
        *best_idx = best;
    }
    *delta = dl;
    *status |= st;
    free(r);
}

void omse_oracle_affine_rows(const float *w, int64_t n_kernels, int64_t kernel_len, int bits, int n_cand,
                             float hi_frac, int n_delta, float off_frac, int refine_iters,
                             const int32_t *start_flat, float *alpha, float *delta, double *sse,
                             int32_t *best_idx, int8_t *codes, uint32_t *status)
{
    uint32_t st_all = 0;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) reduction(| : st_all)
#endif
    for (int64_t s = 0; s < n_kernels; ++s) {
        uint32_t st = 0;
        omse_oracle_affine_phi(w + s * kernel_len, kernel_len, bits, n_cand, hi_frac, n_delta, off_frac,
                               refine_iters, start_flat ? start_flat[s] : -1, &alpha[s], &delta[s], &sse[s],
                               &best_idx[s], codes ? codes + s * kernel_len : NULL, NULL, &st);
        st_all |= st;
    }
    *status |= st_all;
}

/* Key layers (Section 3.5): a layer is a key layer when its MSE exceeds a threshold tau.  The MSE of a
 * layer is the sum of its kernels' squared errors over its number of elements (Section 3.2 drops the
 * mean factor inside the analysis; the threshold values the paper quotes, e.g. 8e-5, are per element). */
double omse_oracle_layer_mse(const float *sse, int64_t n_kernels, int64_t kernel_len)
{
    double s = 0.0;
    for (int64_t i = 0; i < n_kernels; ++i) s += (double)sse[i];
    return s / ((double)n_kernels * (double)kernel_len);
}

/* Compression ratio (Section 3.5): size of the quantized model (codes and one binary32 scale per
 * kernel and per quantized tensor) over the size of the binary32 model. */
double omse_oracle_compression_ratio(const int64_t *n_kernels, const int64_t *kernel_len, const int *bits,
                                     const int *n_tensors, int n_layers)
{
    double q = 0.0, f = 0.0;
    for (int l = 0; l < n_layers; ++l) {
        double n = (double)n_kernels[l] * (double)kernel_len[l];
        q += (double)n_tensors[l] * (n * bits[l] + 32.0 * (double)n_kernels[l]);
        f += 32.0 * n;
    }
    return q / f;
}

/* INT4 code emission.  The paper fixes no byte layout; this library's layout is: element e
 * (flat, row-major) goes to byte e/2, even e in bits 0-3, odd e in bits 4-7, the nibble being
 * the low four bits of the two's-complement code; a trailing odd element leaves bits 4-7 zero. */
void omse_oracle_pack_int4(const int8_t *codes, int64_t n, uint8_t *packed)
{
    for (int64_t b = 0; b < (n + 1) / 2; ++b) {
        uint8_t lo = (uint8_t)codes[2 * b] & 0xF;
        uint8_t hi = (2 * b + 1 < n) ? ((uint8_t)codes[2 * b + 1] & 0xF) : 0;
        packed[b] = (uint8_t)(lo | (hi << 4));
    }
}

void omse_oracle_unpack_int4(const uint8_t *packed, int64_t n, int is_signed, int8_t *codes)
{
    for (int64_t e = 0; e < n; ++e) {
        int v = (packed[e >> 1] >> ((e & 1) * 4)) & 0xF;
        if (is_signed && v >= 8) v -= 16;
        codes[e] = (int8_t)v;
    }
}
