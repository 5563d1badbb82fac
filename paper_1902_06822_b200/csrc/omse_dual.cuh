// Dual line search (Section 3.5, n = 2): a two-dimensional grid over (alpha1, alpha2); for every pair
// each element picks its first code t in Z_p1 by enumeration, the second code being the rounding of
// the rest:  min_t ( x - alpha1*t - alpha2*[ (x - alpha1*t)/alpha2 ]_Zp2 )^2.
//
// One thread block owns one kernel (row) in shared memory.  Pairs are spread over threads: a thread
// holds one alpha1 and DPT consecutive alpha2 in registers, so x - alpha1*t is formed once per t and
// shared by its alpha2's; elements are broadcast from shared memory.  The enumeration over t is
// restricted, exactly, to a window around round(x/alpha1).  A first code whose rest saturates the second
// code errs by more than alpha2/2, one whose rest does not by at most alpha2/2, and the latter all lie
// within (max|Z_p2| + 1/2)*alpha2/alpha1 of x/alpha1; when every rest saturates, the error grows with
// the distance from x/alpha1 up to the asymmetry of Z_p2, which can only move the winner to the other
// neighbour of x/alpha1.  So the codes within (max|Z_p2| + 1/2)*alpha2/alpha1 + 1/2 of round(x/alpha1),
// and at least the two neighbours, hold the minimum (codes beyond Z_p1 collapse onto its ends).
// Grid values are compared in fp32 (blocks of 64 elements folded
// into fp64); pairs within the fp32 noise band of the minimum are re-scored with the full
// enumeration in the reference arithmetic, and the final codes always use the full enumeration.
#pragma once
#include "omse_device.cuh"

namespace omse {

constexpr int kDualDpt = 8;        // alpha2 candidates per thread
constexpr int kDualThreads = 128;
constexpr int kDualListCap = 256;  // near-minimal pairs listed at a time for re-scoring with the full enumeration

struct DualArgs {
    const float* t;          // [S][K]
    long long S, K;
    int n_cand1, n_cand2;
    float hi_frac1, hi_frac2;
    int lo1, hi1, lo2, hi2;
    float* alpha;            // [2][S]
    float* sse;              // [S]
    int* best_idx;           // [S] flat pair index c*n_cand2+d, nullable
    signed char* codes;      // [2][N], nullable
    unsigned char* packed;   // [2][ceil(N/2)], nullable
    unsigned long long* evals;   // executed (element, pair, first code) evaluations (instrumentation), nullable
    float* curve;            // workspace: [gridDim.x][n_cand1*n_cand2] fp32 grid values of the block's current row
    unsigned int* status;
    int rows_per_unit;       // 2 when nibble packing needs an even element count per unit (odd K)
};

// scales of pair (c, d) for a row with max|x| = m: the same binary32 expressions as the 1-D grid
__device__ __forceinline__ void dual_scales(float m, const DualArgs& a, int c, int d, float& a1, float& a2) {
    const float step1 = __fdiv_rn(__fmul_rn(a.hi_frac1, m), (float)a.n_cand1);
    a1 = __fmul_rn((float)(c + 1), step1);
    const float step2 = __fdiv_rn(__fmul_rn(a.hi_frac2, a1), (float)a.n_cand2);
    a2 = __fmul_rn((float)(d + 1), step2);
}

// Full enumeration for one element in the reference arithmetic: lowest t on equal fp32 errors.
__device__ __forceinline__ void dual_codes_of(float x, float a1, float a2, const DualArgs& a, int& t_out, int& q_out) {
    float best = INFINITY;
    int bt = a.lo1, bq = 0;
    for (int t = a.lo1; t <= a.hi1; ++t) {
        const float r = fmaf(-a1, (float)t, x);
        const int q = code_of(r, a2, (float)a.lo2, (float)a.hi2);
        const float e = fmaf(-a2, (float)q, r);
        const float ee = __fmul_rn(e, e);
        if (ee < best) {
            best = ee;
            bt = t;
            bq = q;
        }
    }
    t_out = bt;
    q_out = bq;
}

__global__ void __launch_bounds__(kDualThreads) dual_kernel(const DualArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* xs = reinterpret_cast<float*>(smem_raw);                  // [k]
    const int k = (int)a.K;
    double* scratch = reinterpret_cast<double*>(xs + ((k + 3) & ~3)); // [64]
    int* list = reinterpret_cast<int*>(scratch + 64);                // [kDualListCap]
    int* misc = list + kDualListCap;                                 // [4]: list count, carried codes
    const int tid = threadIdx.x, nthr = blockDim.x;
    const long long n_total = a.S * a.K;
    const long long packed_stride = (n_total + 1) >> 1;
    const long long n_units = (a.S + a.rows_per_unit - 1) / a.rows_per_unit;
    const int dgroups = (a.n_cand2 + kDualDpt - 1) / kDualDpt;
    const int n_slots = a.n_cand1 * dgroups;                         // thread slots: (c, group of DPT d's)
    const float flo2 = (float)a.lo2, fhi2 = (float)a.hi2;
    const float half_range2 = fmaxf(fhi2, -flo2) + 0.5f;
    const int n_levels = a.hi1 - a.lo1 + 1;
    unsigned int st = 0;
    unsigned long long ev = 0ull;

    for (long long unit = blockIdx.x; unit < n_units; unit += gridDim.x) {
        for (int ru = 0; ru < a.rows_per_unit; ++ru) {
            const long long row = unit * a.rows_per_unit + ru;
            if (row >= a.S) break;
            const bool more = (ru + 1 < a.rows_per_unit) && (row + 1 < a.S);
            const long long row_base = row * a.K;
            __syncthreads();
            // ---- stage the row, maxima
            float mx = 0.f;
            bool bad = false;
            for (int i = tid; i < k; i += nthr) {
                const float v = __ldg(a.t + row_base + i);
                xs[i] = v;
                if (fabsf(v) <= FLT_MAX) mx = fmaxf(mx, fabsf(v));
                else bad = true;
            }
            if (bad) st |= 1u;
            float dummy = 0.f;
            block_max2(mx, dummy, scratch);
            const float m = mx;
            float a1_last, a2_last;
            dual_scales(m, a, a.n_cand1 - 1, a.n_cand2 - 1, a1_last, a2_last);
            bool degenerate = !(m > 0.f) || !(a2_last >= FLT_MIN);

            // ---- grid: every thread slot sweeps the row for its alpha1 and DPT alpha2's; values to the workspace
            const int n_pairs_grid = a.n_cand1 * a.n_cand2;
            float* curve = a.curve + (size_t)blockIdx.x * n_pairs_grid;
            if (!degenerate) {
                for (int slot = tid; slot < n_slots; slot += nthr) {
                    // consecutive threads take consecutive alpha1 of one group of alpha2's: the window of first codes
                    // depends on alpha2/alpha1 = (d+1)*hi_frac2/C2 only, so a warp's lanes run the same number of steps
                    const int dg = slot / a.n_cand1, c = slot - dg * a.n_cand1, d0 = dg * kDualDpt;
                    float a1, a2[kDualDpt], inv2[kDualDpt], acc[kDualDpt];
                    double dacc[kDualDpt];
                    bool ok[kDualDpt];
#pragma unroll
                    for (int j = 0; j < kDualDpt; ++j) {
                        dual_scales(m, a, c, min(d0 + j, a.n_cand2 - 1), a1, a2[j]);
                        ok[j] = (d0 + j < a.n_cand2) && a1 >= FLT_MIN && a2[j] >= FLT_MIN;
                        inv2[j] = ok[j] ? __fdiv_rn(1.0f, a2[j]) : 0.f;
                        acc[j] = 0.f;
                        dacc[j] = 0.0;
                    }
                    const float inv1 = a1 >= FLT_MIN ? __fdiv_rn(1.0f, a1) : 0.f;
                    // window of first codes that can win: |t - round(x/alpha1)| <= half_range2*alpha2/alpha1 + 1/2, at least 1
                    const float ratio = a2[kDualDpt - 1] * inv1;         // largest alpha2 of the group
                    const int w = max(1, (int)(half_range2 * fminf(ratio, 16.f) * 1.0001f + 0.501f));
                    const bool full = !(ratio <= 16.f) || 2 * w + 1 >= n_levels;
                    const int n_t = full ? n_levels : 2 * w + 1;
                    ev += (unsigned long long)k * (unsigned long long)n_t * kDualDpt;
                    const float clo2 = kMagic + flo2, chi2 = kMagic + fhi2, flo1 = (float)a.lo1, fhi1 = (float)a.hi1;
                    for (int i = 0; i < k; ++i) {
                        const float x = xs[i];
                        const float t0 = full ? flo1 : rintf(x * inv1) - (float)w;
                        // smallest |error| over the first codes: squaring is monotone, so the square of the smallest
                        // magnitude is the smallest squared error
                        float best[kDualDpt];
#pragma unroll
                        for (int j = 0; j < kDualDpt; ++j) best[j] = INFINITY;
                        // one first code per step: the thread's alpha2's give independent chains, and a window
                        // always holds an odd number of codes
                        float tcur = t0;
                        for (int s = 0; s < n_t; ++s) {
                            const float ta = fminf(fmaxf(tcur, flo1), fhi1);
                            tcur += 1.0f;
                            const float ra = fmaf(-a1, ta, x);
#pragma unroll
                            for (int j = 0; j < kDualDpt; ++j) {
                                float ua = fmaf(ra, inv2[j], kMagic);
                                ua = fminf(fmaxf(ua, clo2), chi2);
                                const float ea = fmaf(-a2[j], ua - kMagic, ra);
                                best[j] = fminf(best[j], fabsf(ea));
                            }
                        }
#pragma unroll
                        for (int j = 0; j < kDualDpt; ++j) acc[j] = fmaf(best[j], best[j], acc[j]);
                        if ((i & 63) == 63) {
#pragma unroll
                            for (int j = 0; j < kDualDpt; ++j) {
                                dacc[j] += (double)acc[j];
                                acc[j] = 0.f;
                            }
                        }
                    }
#pragma unroll
                    for (int j = 0; j < kDualDpt; ++j)
                        if (d0 + j < a.n_cand2)
                            curve[c * a.n_cand2 + d0 + j] = ok[j] ? (float)(dacc[j] + (double)acc[j]) : INFINITY;
                }
            }
            __syncthreads();                            // the block's grid values are visible to the block
            double bv = INFINITY;
            int bi = 0x7fffffff;
            if (!degenerate) {
                for (int p = tid; p < n_pairs_grid; p += nthr) {
                    const float v = curve[p];
                    if (v < bv) {                       // ascending p within a thread: strict < keeps the lowest index
                        bv = v;
                        bi = p;
                    }
                }
            }
            if (tid == 0) misc[0] = 0;
            block_argmin(bv, bi, scratch);
            if (bi == 0x7fffffff || !(bv < INFINITY)) degenerate = true;

            float alpha1 = 0.f, alpha2 = 0.f;
            int best_pair = -1;
            if (!degenerate) {
                // ---- pairs within the fp32 noise band of the minimum: re-score with the full enumeration.
                // The fp32 value squares e = r - alpha2*q with r = fl(x - alpha1*t) ROUNDED to binary32; the
                // winning t leaves |r| <= (max|Z_p2| + 1/2)*alpha2, so r is off by at most 2^-25 of that and a
                // sum of k terms by at most 2*sqrt(k*SSE) * 2^-25 * (max|Z_p2| + 1/2) * alpha2 (Cauchy-Schwarz).
                float a1_top, a2_top;
                dual_scales(m, a, a.n_cand1 - 1, a.n_cand2 - 1, a1_top, a2_top);     // largest alpha2 on the grid
                const double noise = 2.0 * sqrt((double)k * bv) * 2.98e-8 * (double)half_range2 * (double)a2_top;
                const double band = bv * (1.0 + kRescoreBand) + 2.0 * noise;
                for (int p = tid; p < n_pairs_grid; p += nthr) {
                    if ((double)curve[p] <= band) {
                        const int pos = atomicAdd(&misc[0], 1);
                        if (pos < kDualListCap) list[pos] = p;
                    }
                }
                __syncthreads();
                const int n_list = misc[0];
                best_pair = bi;
                if (n_list > 1) {
                    double best_sse = INFINITY;
                    best_pair = 0x7fffffff;
                    auto rescore = [&](int p) {      // full enumeration in the reference arithmetic, fp64 sum
                        float a1, a2;
                        dual_scales(m, a, p / a.n_cand2, p % a.n_cand2, a1, a2);
                        double ss = 0.0;
                        long long zero = 0;
                        for (int i = tid; i < k; i += nthr) {
                            int t, q;
                            dual_codes_of(xs[i], a1, a2, a, t, q);
                            const double d = (double)xs[i] - (double)a1 * (double)t - (double)a2 * (double)q;
                            ss += d * d;
                        }
                        block_sum2(ss, zero, scratch);
                        if (ss < best_sse || (ss == best_sse && p < best_pair)) {
                            best_sse = ss;
                            best_pair = p;
                        }
                    };
                    if (n_list <= kDualListCap) {
                        for (int l = 0; l < n_list; ++l) rescore(list[l]);
                    } else {
                        // more pairs in the band than the list holds: the same re-scoring, one window of
                        // kDualListCap consecutive pairs at a time
                        for (int base = 0; base < n_pairs_grid; base += kDualListCap) {
                            __syncthreads();
                            if (tid == 0) misc[0] = 0;
                            __syncthreads();
                            const int stop = min(base + kDualListCap, n_pairs_grid);
                            for (int p = base + tid; p < stop; p += nthr)
                                if ((double)curve[p] <= band) list[atomicAdd(&misc[0], 1)] = p;
                            __syncthreads();
                            const int n_win = misc[0];
                            for (int l = 0; l < n_win; ++l) rescore(list[l]);
                        }
                    }
                }
                dual_scales(m, a, best_pair / a.n_cand2, best_pair % a.n_cand2, alpha1, alpha2);
            } else {
                st |= 2u;
            }

            // ---- final codes (full enumeration), squared error, emission: one output byte pair per thread
            double ss = 0.0;
            const int o = (int)(row_base & 1);
            const int n_pairs = (k + o + 1) >> 1;
            for (int p = tid; p < n_pairs; p += nthr) {
                const int e0 = 2 * p - o, e1 = e0 + 1;
                int t0c = 0, q0c = 0, t1c = 0, q1c = 0;
                if (e0 >= 0) {
                    const float x = xs[e0];
                    if (!degenerate) dual_codes_of(x, alpha1, alpha2, a, t0c, q0c);
                    const double d = (double)x - (double)alpha1 * (double)t0c - (double)alpha2 * (double)q0c;
                    ss += d * d;
                    if (a.codes) {
                        a.codes[row_base + e0] = (signed char)t0c;
                        a.codes[n_total + row_base + e0] = (signed char)q0c;
                    }
                } else {
                    t0c = misc[1];
                    q0c = misc[2];
                }
                const bool has1 = e1 < k;
                if (has1) {
                    const float x = xs[e1];
                    if (!degenerate) dual_codes_of(x, alpha1, alpha2, a, t1c, q1c);
                    const double d = (double)x - (double)alpha1 * (double)t1c - (double)alpha2 * (double)q1c;
                    ss += d * d;
                    if (a.codes) {
                        a.codes[row_base + e1] = (signed char)t1c;
                        a.codes[n_total + row_base + e1] = (signed char)q1c;
                    }
                }
                if (a.packed) {
                    if (has1 || !more) {
                        const long long b = (row_base + e0) >> 1;
                        a.packed[b] = (unsigned char)((t0c & 0xf) | ((t1c & 0xf) << 4));
                        a.packed[packed_stride + b] = (unsigned char)((q0c & 0xf) | ((q1c & 0xf) << 4));
                    } else {   // last element of the row: its byte is completed by the next row of the unit
                        misc[1] = t0c;
                        misc[2] = q0c;
                    }
                }
            }
            long long zero = 0;
            block_sum2(ss, zero, scratch);
            if (tid == 0) {
                a.alpha[row] = alpha1;
                a.alpha[a.S + row] = alpha2;
                a.sse[row] = (float)ss;
                if (a.best_idx) a.best_idx[row] = best_pair;
            }
        }
    }
    if (st) atomicOr(a.status, st);
    report_evaluations(a.evals, ev);
}

}  // namespace omse
