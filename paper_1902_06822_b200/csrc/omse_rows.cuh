// Kernel-wise MMSE quantization (Sections 3.3, 3.4) and Algorithm 1 (Section 3.5): one thread block
// owns one kernel (row) at a time, staged once from HBM into shared memory; everything that follows
// (max, candidate sweep, argmin, polish, codes, packing, residual update) reads the on-chip copy.
#pragma once
#include "omse_device.cuh"

#ifndef OMSE_ROWS_MAX_THREADS
#define OMSE_ROWS_MAX_THREADS 512
#endif

namespace omse {

// One weight tensor of a launch (Section 3.1: W_l = {W_lk}, row k is kernel W_lk flattened).
struct RowTensor {
    const float* w;          // [S][K]
    long long S, K;
    float* alpha;            // [n_tensors][S]
    float* sse;              // [n_tensors][S]
    int* best_idx;           // [S] (single quantized tensor only), nullable
    signed char* codes;      // [n_tensors][N], nullable
    unsigned char* packed;   // [n_tensors][ceil(N/2)], nullable
    float* delta;            // [S] offset subtracted from each row (Section 3.1 scheme with offset), nullable = no offset
    const float* prior_alpha;   // [S] nullable: scale of an earlier quantized tensor of this row; the row is replaced by its
                                // residual fl(x - alpha*[x/alpha]_Zp) before the search (second tensor of a key layer, Section 3.5)
    const int* gate;         // nullable: the tensor's units are skipped when *gate == 0 (key-layer flag written by an earlier kernel)
    long long unit_begin;    // index of this tensor's first work unit in the launch-wide numbering
    int rows_per_unit;       // long rows: 2 when nibble packing needs an even element count per unit (odd K), else 1;
                             // short rows: the batch size B (even)
    int small;               // bit 0: short-row path (batch of rows per unit, a warp finishes each row);
                             // bit 1: that path regroups rows by magnitude class;
                             // bit 2: thread-per-row path for very short rows (rows_per_unit = block size)
};

struct RowArgs {
    const RowTensor* tensors;   // device array, ordered by decreasing K (longest rows are handed out first)
    RowTensor one;              // the tensor itself when n_tensors_in_launch == 1 (tensors == nullptr)
    int n_launch_tensors;
    long long n_units;          // work units in the launch
    unsigned long long* ticket; // [2] next unit to hand out, blocks finished; both return to 0 at kernel end
    int n_cand;
    float hi_frac;
    int refine_iters;
    int n_tensors, n_sweeps;    // Algorithm 1: quantized tensors per row, sweeps
    int lo[4], hi[4];           // grid bounds per quantized tensor (Section 3.1)
    float* sse_history;         // [n_sweeps][n_tensors][S] error after every update of Algorithm 1, nullable (single tensor launches)
    unsigned int* status;
    unsigned long long* evals;  // executed (element, candidate) evaluations, summed over the launch (instrumentation), nullable
    int groups;                 // element groups per block
    int tg;                     // threads per group (multiple of 32); candidate c = slot*tg + t
    int keep_x0;                // n_sweeps > 1: keep the original row next to the residual
    int max_k4;                 // float4s of the longest row in the launch (shared-memory carve-up)
    int prune;                  // 1: rows are regrouped by magnitude so that candidates skip elements they code as 0
    int solver;                 // 0: grid line search (Section 3.4); 1: uniform scale max|x|/L; 2: alternating from the
                                // uniform scale; 3: golden-section search (the comparison solvers of Section 3.4)
    int solver_iters;           // alternating: least-squares steps; golden: shrink steps
    int n_delta;                // > 0: offsets searched per row (offset scheme of Section 3.1 with delta on a grid); needs keep_x0
    float off_frac;             // offsets span [min, min + off_frac*(max-min))
    float eps;                  // >= 0: Algorithm 1 stops after the first sweep whose relative error decrease is <= eps
    int* sweeps_done;           // [S] sweeps Algorithm 1 ran per row, nullable
    int ext_tensors;            // a tensor of a batched launch has a gate or an earlier tensor's scale
};

}  // namespace omse

#include "omse_rows_small.cuh"
#include "omse_rows_tiny.cuh"

namespace omse {

constexpr int kScratchDoubles = 64 + 16 * 9;

struct PhiOut {
    float alpha;
    double sse;       // with PhiCtl::want_sse: squared error at the chosen grid candidate (true division, fp64)
    int idx;
    bool degenerate;
};

// What phi_block does on the row in s.xs besides the default "grid search, then refine_iters polish steps".
struct PhiCtl {
    int solver;       // as RowArgs::solver
    int n_iter;       // as RowArgs::solver_iters
    int start_idx;    // >= 0: skip the search and start from this grid candidate
    int n_refine;     // polish steps
    bool want_sse;    // also return the fp64 error at the chosen candidate (before any polish)
};

// Per-row state of the pass loop of rows_kernel (shared memory; thread 0 writes between barriers).
struct RowMode {
    PhiCtl ctl;             // what the next phi_block call does
    double aff_best;        // offset search: smallest error so far, its offset index and scale index
    int aff_d, aff_c;
    float aff_lo, aff_dstep, aff_dl;   // row minimum, offset step, offset of the current pass
    double e_prev;          // Algorithm 1: error after the previous sweep
    int sweeps_ran;
};

// ||x - alpha*[x/alpha]_Zp||^2 of the row in s.xs in fp64 with true division; every thread gets the sum.
__device__ __forceinline__ double exact_sse_block(const float* xs, int k, float alpha, float flo, float fhi,
                                                   double* scratch) {
    double ss = 0.0;
    long long zero = 0;
    const float inv = __fdiv_rn(1.0f, alpha), thr = ambiguity_threshold(flo, fhi);
    const double ad = (double)alpha;
    // four elements per step (the row is zero padded to a multiple of four; a zero has code 0 and error 0)
    const float4* xs4 = reinterpret_cast<const float4*>(xs);
    const int k4 = (k + 3) >> 2;
    for (int i4 = threadIdx.x; i4 < k4; i4 += blockDim.x) {
        const float4 v = xs4[i4];
        const float x[4] = {v.x, v.y, v.z, v.w};
        double d[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) d[e] = fma(-ad, int_double(exact_code(x[e], alpha, inv, flo, fhi, thr)), (double)x[e]);
#pragma unroll
        for (int e = 0; e < 4; ++e) ss = fma(d[e], d[e], ss);
    }
    block_sum2(ss, zero, scratch);
    return ss;
}

// Least-squares polish of Section 3.4's objective: alpha <- <x,q>/<q,q>, q = [x/alpha]_Zp, at most n times.
__device__ __forceinline__ float polish_block(const float* xs, int k, float alpha, float flo, float fhi, int n,
                                              double* scratch) {
    const float4* xs4 = reinterpret_cast<const float4*>(xs);
    const int k4 = (k + 3) >> 2;
    for (int it = 0; it < n; ++it) {
        double sxq = 0.0;
        long long sqq = 0;
        const float inv = __fdiv_rn(1.0f, alpha), thr = ambiguity_threshold(flo, fhi);
        for (int i4 = threadIdx.x; i4 < k4; i4 += blockDim.x) {   // four elements per step; the zero padding adds nothing
            const float4 v = xs4[i4];
            const float x[4] = {v.x, v.y, v.z, v.w};
            int q[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) q[e] = exact_code(x[e], alpha, inv, flo, fhi, thr);
            int qq = 0;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                qq += q[e] * q[e];
                sxq = fma((double)x[e], int_double(q[e]), sxq);
            }
            sqq += qq;
        }
        block_sum2(sxq, sqq, scratch);
        if (sqq == 0) break;
        const float a_new = (float)(sxq / (double)sqq);
        if (!(a_new >= FLT_MIN) || !(a_new <= FLT_MAX)) break;
        if (a_new == alpha) break;   // fixed point: further steps would repeat it exactly
        alpha = a_new;
    }
    return alpha;
}

// shared-memory carve-up for one block
struct RowSmem {
    float* xs;        // [k4*4] current tensor (row or residual), zero padded to a multiple of 4
    float* x0;        // [k4*4] original row (only when keep_x0)
    float* xb;        // [k4*4 + 4*CPT] the row regrouped by magnitude class (only when pruning)
    double* xg;       // [(groups-1)*CPT*tg] partial sums of the other element groups
    double* scratch;  // [kScratchDoubles] reductions
    double* skip;     // [CPT] squared sum of the elements a candidate slot does not evaluate
    int* seg;         // [2*(CPT+1)] first element and padded length of each magnitude class in xb
    int* misc;        // [8]: 1..4 nibble carried to the next row, per tensor
};

// ---------------------------------------------------------------------------------------------
// Magnitude classes.  Candidate slot sl of every thread holds scales >= alpha_{sl*tg} = (sl*tg+1)*step.
// An element with |x| <= 0.4999*alpha gets code 0 from that scale and from every larger one, and
// then contributes exactly x^2 to their errors.  So the row is regrouped (stable counting sort, fixed
// order) into classes nb = number of leading slots that still have to evaluate the element; the
// sweep runs slots 0..nb-1 on class nb, and each slot adds the squared sum of the classes it skipped.
// With the grid reaching up to max|x| most (element, candidate) pairs fall away: the large scales
// only see the few large elements.
// ---------------------------------------------------------------------------------------------
template <int CPT>
__device__ void partition_row(const RowSmem& s, int k, const GridSetup& g, int tg) {
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarp = nthr >> 5;
    const float inv_thr = g.rstep * (1.0f / 0.4999f);
    const float inv_tg = 1.0f / (float)tg;
    // Thread t owns the float4s t, t + nthr, ... of the zero-padded row (conflict-free 128-bit reads, four independent
    // elements per step); within a class the elements keep the order (thread, then index), which is fixed, so the
    // sums that follow do not depend on scheduling.  The padding zeros fall into class 0 and add nothing.
    // ---- pass 1: class counts of this thread's elements (16-bit fields), squared sum of class 0
    const float4* xs4 = reinterpret_cast<const float4*>(s.xs);
    const int k4 = (k + 3) >> 2;
    u64 c0 = 0ull, c1 = 0ull;                  // classes 1..4 and 5..8
    double zero_sq = 0.0;
    for (int i4 = tid; i4 < k4; i4 += nthr) {
        const float4 v = xs4[i4];
        const float x[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int nb = magnitude_class<CPT>(x[e], inv_thr, inv_tg);
            const double xd = (double)x[e];
            zero_sq = fma(nb == 0 ? xd : 0.0, xd, zero_sq);
            const u64 one = nb >= 1 ? 1ull << (16 * ((nb - 1) & 3)) : 0ull;
            c0 += nb < 5 ? one : 0ull;
            c1 += nb >= 5 ? one : 0ull;
        }
    }
    // ---- exclusive scan of the counts over the block (lanes by shuffle, warps in order)
    u64 i0 = c0, i1 = c1;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const u64 u0 = __shfl_up_sync(0xffffffffu, i0, o);
        const u64 u1 = __shfl_up_sync(0xffffffffu, i1, o);
        if (lane >= o) {
            i0 += u0;
            i1 += u1;
        }
    }
    u64* wt = reinterpret_cast<u64*>(s.scratch);          // [nwarp][2]
    __syncthreads();
    if (lane == 31) {
        wt[2 * warp] = i0;
        wt[2 * warp + 1] = i1;
    }
    __syncthreads();
    u64 off0 = i0 - c0, off1 = i1 - c1, tot0 = 0ull, tot1 = 0ull;
    for (int w = 0; w < nwarp; ++w) {
        const u64 a0 = wt[2 * w], a1 = wt[2 * w + 1];
        if (w < warp) {
            off0 += a0;
            off1 += a1;
        }
        tot0 += a0;
        tot1 += a1;
    }
    // ---- class layout in xb: class CPT first, each class padded with zeros to a multiple of 4.  The class starts are
    //      added to the packed offsets, which then hold positions in xb (a regrouped row has fewer than 2^16 elements).
    int base[CPT + 1], cnt[CPT + 1];
    int pos = 0;
    u64 b0 = 0ull, b1 = 0ull;
#pragma unroll
    for (int b = CPT; b >= 1; --b) {
        cnt[b] = (int)(((b >= 5 ? tot1 : tot0) >> (16 * ((b - 1) & 3))) & 0xffffull);
        base[b] = pos;
        if (b >= 5) b1 |= (u64)pos << (16 * ((b - 1) & 3));
        else b0 |= (u64)pos << (16 * ((b - 1) & 3));
        const int padded = (cnt[b] + 3) & ~3;
        if (tid == 0) {
            s.seg[2 * b] = pos;
            s.seg[2 * b + 1] = padded;
        }
        if (tid < padded - cnt[b]) s.xb[pos + cnt[b] + tid] = 0.f;
        pos += padded;
    }
    off0 += b0;
    off1 += b1;
    // ---- pass 2: scatter
    for (int i4 = tid; i4 < k4; i4 += nthr) {
        const float4 v = xs4[i4];
        const float x[4] = {v.x, v.y, v.z, v.w};
        int nb[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) nb[e] = magnitude_class<CPT>(x[e], inv_thr, inv_tg);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (nb[e] >= 1) {
                const int sh = 16 * ((nb[e] - 1) & 3);
                const u64 word = nb[e] >= 5 ? off1 : off0;
                const u64 one = 1ull << sh;
                s.xb[(int)((word >> sh) & 0xffffull)] = x[e];
                off0 += nb[e] >= 5 ? 0ull : one;
                off1 += nb[e] >= 5 ? one : 0ull;
            }
        }
    }
    __syncthreads();
    // ---- squared sums per class from the regrouped row (class 0 was summed on the way; padding zeros add nothing)
    const float4* xb4 = reinterpret_cast<const float4*>(s.xb);
    double d[CPT + 1];
    d[0] = zero_sq;
#pragma unroll
    for (int b = 1; b <= CPT; ++b) {
        double v = 0.0;
        const int first4 = base[b] >> 2, len4 = (cnt[b] + 3) >> 2;
        for (int i4 = tid; i4 < len4; i4 += nthr) {
            const float4 q = xb4[first4 + i4];
            const double q0 = (double)q.x, q1 = (double)q.y, q2 = (double)q.z, q3 = (double)q.w;
            v = fma(q0, q0, v);
            v = fma(q1, q1, v);
            v = fma(q2, q2, v);
            v = fma(q3, q3, v);
        }
        d[b] = v;
    }
    double* ds = s.scratch + 64;                           // [nwarp][CPT+1]
#pragma unroll
    for (int b = 0; b <= CPT; ++b) {
        const double v = warp_sum(d[b]);
        if (lane == 0) ds[warp * (CPT + 1) + b] = v;
    }
    __syncthreads();
    if (tid < CPT) {
        double acc = 0.0;                                  // slot `tid` skips classes 0..tid
        for (int b = 0; b <= tid; ++b)
            for (int w = 0; w < nwarp; ++w) acc += ds[w * (CPT + 1) + b];
        s.skip[tid] = acc;
    }
    __syncthreads();
}

// The quantization mapping phi of Section 3.4 on the row held in s.xs (k elements, k4 float4s).
template <int CPT, bool EXT>
__device__ PhiOut phi_block(const RowArgs& a, const RowSmem& s, int k, int k4, float flo, float fhi,
                             const float (&rcp)[CPT], unsigned long long& ev, const PhiCtl& ctl) {
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int grp = tid / a.tg, t = tid - grp * a.tg;
    const float4* xs4 = reinterpret_cast<const float4*>(s.xs);
    PhiOut out;

    // ---- max of the positive and of the negative part (range of the grid; which candidates saturate)
    float mpos = 0.f, mneg = 0.f;
    for (int i4 = tid; i4 < k4; i4 += nthr) {   // the zero padding leaves both maxima alone
        const float4 v4 = xs4[i4];
        const float x[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (fabsf(x[e]) <= FLT_MAX) {
                mpos = fmaxf(mpos, x[e]);
                mneg = fmaxf(mneg, -x[e]);
            }
        }
    }
    block_max2(mpos, mneg, s.scratch);
    const float m = fmaxf(mpos, mneg);
    const GridSetup g = grid_setup(mpos, mneg, a.hi_frac, a.n_cand, flo, fhi);
    const float a_last = __fmul_rn((float)a.n_cand, g.step);
    out.alpha = 0.f;
    out.sse = 0.0;
    out.idx = -1;
    out.degenerate = true;
    if (EXT && ctl.solver != 0) {
        // ---- comparison solvers of Section 3.4: another way to the starting scale, then the same polish
        float alpha = 0.f;
        if (ctl.solver == 3) {
            // golden-section search on [0, hi_frac*max|x|], scales in binary32, errors in fp64 (uniform over the block)
            const float rho = 0.618034f;
            float lo_a = 0.f, hi_a = __fmul_rn(a.hi_frac, m);
            float t = __fmul_rn(rho, __fsub_rn(hi_a, lo_a));
            float x1 = __fsub_rn(hi_a, t), x2 = __fadd_rn(lo_a, t);
            auto f = [&](float al) -> double {
                return (al >= FLT_MIN && al <= FLT_MAX) ? exact_sse_block(s.xs, k, al, flo, fhi, s.scratch) : (double)INFINITY;
            };
            double f1 = f(x1), f2 = f(x2);
            for (int it = 0; it < ctl.n_iter; ++it) {
                if (f1 <= f2) {          // equal errors keep the smaller scale
                    hi_a = x2;
                    x2 = x1;
                    f2 = f1;
                    t = __fmul_rn(rho, __fsub_rn(hi_a, lo_a));
                    x1 = __fsub_rn(hi_a, t);
                    f1 = f(x1);
                } else {
                    lo_a = x1;
                    x1 = x2;
                    f1 = f2;
                    t = __fmul_rn(rho, __fsub_rn(hi_a, lo_a));
                    x2 = __fadd_rn(lo_a, t);
                    f2 = f(x2);
                }
            }
            alpha = (f1 <= f2) ? x1 : x2;
            if (!(fmin(f1, f2) < (double)INFINITY)) alpha = 0.f;
        } else {
            // no-offset uniform quantizer of Section 3.1: alpha = max|x| / L
            alpha = __fdiv_rn(m, fhi);   // L = 2^(p-1)-1 (signed) or 2^p-1 (unsigned) is the top code of the range
        }
        if (!(alpha >= FLT_MIN) || !(alpha <= FLT_MAX)) return out;
        out.degenerate = false;
        out.idx = 0;
        const int steps = ctl.n_refine + (ctl.solver == 2 ? ctl.n_iter : 0);
        out.alpha = polish_block(s.xs, k, alpha, flo, fhi, steps, s.scratch);
        return out;
    }
    if (!(m > 0.f) || !(a_last >= FLT_MIN)) return out;   // no usable scale: alpha = 0, all codes 0
    if (EXT && ctl.start_idx >= 0) {
        const float ac = __fmul_rn((float)(ctl.start_idx + 1), g.step);
        if (!(ac >= FLT_MIN) || ctl.start_idx >= a.n_cand) return out;
        out.degenerate = false;
        out.idx = ctl.start_idx;
        out.alpha = polish_block(s.xs, k, ac, flo, fhi, ctl.n_refine, s.scratch);
        return out;
    }

    // ---- per-thread candidate constants
    u64 inv2[CPT], na2[CPT];
    double dacc[CPT];
#pragma unroll
    for (int sl = 0; sl < CPT; ++sl) {
        const int c = sl * a.tg + t;
        const float ac = __fmul_rn((float)(c + 1), g.step);
        float inv = g.tiny ? __fdiv_rn(1.0f, ac) : rcp[sl] * g.rstep;
        if (!(ac >= FLT_MIN) || c >= a.n_cand) inv = 0.f;  // unusable: evaluated harmlessly, discarded below
        inv2[sl] = pack2(inv, inv);
        na2[sl] = pack2(-ac, -ac);
        dacc[sl] = 0.0;
    }
    const int warp_t0 = t & ~31;
    int ncl = (g.c_sat - warp_t0 + a.tg - 1) / a.tg;
    ncl = max(0, min(CPT, ncl));

    // ---- sweep: this group's contiguous share of the row (of every magnitude class), all candidates
    if (a.prune && !g.tiny) {
        partition_row<CPT>(s, k, g, a.tg);
        const float4* xb4 = reinterpret_cast<const float4*>(s.xb);
        for (int b = CPT; b >= 1; --b) {
            const int first4 = s.seg[2 * b] >> 2, len4 = s.seg[2 * b + 1] >> 2;
            const int beg4 = first4 + (int)(((long long)len4 * grp) / a.groups);
            const int end4 = first4 + (int)(((long long)len4 * (grp + 1)) / a.groups);
            int ncl_b = (class_sat_count(b, CPT, a.tg, g.c_sat, flo, fhi) - warp_t0 + a.tg - 1) / a.tg;
            ncl_b = max(0, min(CPT, ncl_b));
            sweep_dispatch<CPT>(b, ncl_b, xb4, beg4, end4, inv2, na2, dacc, kMagic + flo, kMagic + fhi);
            ev += (unsigned long long)(end4 - beg4) * 4ull * (unsigned long long)b;
        }
        if (grp == 0) {
#pragma unroll
            for (int sl = 0; sl < CPT; ++sl) dacc[sl] += s.skip[sl];
        }
    } else {
        const int beg4 = (int)(((long long)k4 * grp) / a.groups);
        const int end4 = (int)(((long long)k4 * (grp + 1)) / a.groups);
        sweep_dispatch<CPT>(ncl, xs4, beg4, end4, inv2, na2, dacc, kMagic + flo, kMagic + fhi);        ev += (unsigned long long)(end4 - beg4) * 4ull * CPT;
    }

    if (a.groups > 1) {
        if (grp > 0) {
#pragma unroll
            for (int sl = 0; sl < CPT; ++sl) s.xg[((grp - 1) * CPT + sl) * a.tg + t] = dacc[sl];
        }
        __syncthreads();
        if (grp == 0) {
            for (int gg = 1; gg < a.groups; ++gg)
#pragma unroll
                for (int sl = 0; sl < CPT; ++sl) dacc[sl] += s.xg[((gg - 1) * CPT + sl) * a.tg + t];
        }
    }

    // ---- argmin over candidates (fp32-block / fp64-fold sums), lowest index on ties
    double bv = INFINITY;
    int bi = 0x7fffffff;
#pragma unroll
    for (int sl = 0; sl < CPT; ++sl) {
        const int c = sl * a.tg + t;
        const float ac = __fmul_rn((float)(c + 1), g.step);
        const bool ok = grp == 0 && c < a.n_cand && ac >= FLT_MIN;
        dacc[sl] = ok ? dacc[sl] : INFINITY;
        if (dacc[sl] < bv) {   // slots are in increasing c, strict < keeps the lowest index
            bv = dacc[sl];
            bi = c;
        }
    }
    block_argmin(bv, bi, s.scratch);
    if (bi == 0x7fffffff) return out;  // every error is Inf/NaN (non-finite input): same as no usable scale
    out.degenerate = false;

    // ---- every candidate within the fp32 noise band of the minimum is re-scored in fp64 with true division,
    //      in increasing index order, however many there are (the block agrees on the next one by a reduction)
    const double band = bv * (1.0 + kRescoreBand);
    int mine = 0;
#pragma unroll
    for (int sl = 0; sl < CPT; ++sl) mine += (dacc[sl] <= band) ? 1 : 0;
    const int holders = __syncthreads_count(mine > 0);
    const int multi = __syncthreads_or(mine > 1);
    int best = bi;
    double best_sse = INFINITY;
    if (holders > 1 || multi) {
        best = 0x7fffffff;
        int prev = -1;
        for (;;) {
            int c = 0x7fffffff;
#pragma unroll
            for (int sl = CPT - 1; sl >= 0; --sl) {
                const int cc = sl * a.tg + t;
                if (dacc[sl] <= band && cc > prev) c = cc;   // descending slots: the smallest index above prev stays
            }
            double cv = (double)c;
            block_argmin(cv, c, s.scratch);
            if (c == 0x7fffffff) break;
            prev = c;
            const float ac = __fmul_rn((float)(c + 1), g.step);
            double ss = 0.0;
            long long zero = 0;
            const float inv = __fdiv_rn(1.0f, ac), thr = ambiguity_threshold(flo, fhi);
            const double ad = (double)ac;
            for (int i4 = tid; i4 < k4; i4 += nthr) {
                const float4 v4 = xs4[i4];
                const float x[4] = {v4.x, v4.y, v4.z, v4.w};
                double d[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) d[e] = fma(-ad, int_double(exact_code(x[e], ac, inv, flo, fhi, thr)), (double)x[e]);
#pragma unroll
                for (int e = 0; e < 4; ++e) ss = fma(d[e], d[e], ss);
            }
            block_sum2(ss, zero, s.scratch);
            if (ss < best_sse) {   // increasing index: strict < keeps the lowest among equal errors
                best_sse = ss;
                best = c;
            }
        }
    }

    // ---- polish: alpha <- <x,q>/<q,q>, q = [x/alpha]_Zp
    const float a_grid = __fmul_rn((float)(best + 1), g.step);
    if (EXT && ctl.want_sse)
        out.sse = best_sse < INFINITY ? best_sse : exact_sse_block(s.xs, k, a_grid, flo, fhi, s.scratch);
    out.alpha = polish_block(s.xs, k, a_grid, flo, fhi, EXT ? ctl.n_refine : a.refine_iters, s.scratch);
    out.idx = best;
    return out;
}

// Final codes at `alpha`, their squared error, and emission as int8 and/or nibbles.
// row_base = flat index of the row's first element in the tensor; n_total = S*K.
__device__ double emit_block(const RowSmem& s, int k, float alpha, float flo, float fhi,
                             signed char* codes, unsigned char* packed, long long row_base,
                             int* carry, bool more_rows_in_unit) {
    const int tid = threadIdx.x, nthr = blockDim.x;
    double ss = 0.0;
    const bool zero = !(alpha > 0.f);
    const float inv = zero ? 0.f : __fdiv_rn(1.0f, alpha), thr = ambiguity_threshold(flo, fhi);
    const double ad = (double)alpha;
    const bool aligned = ((reinterpret_cast<unsigned long long>(codes) & 3ull) == 0) &&
                         ((reinterpret_cast<unsigned long long>(packed) & 1ull) == 0);
    if ((k & 3) == 0 && aligned) {
        // aligned fast path: four codes per thread, 32-bit and 16-bit stores
        const float4* xs4 = reinterpret_cast<const float4*>(s.xs);
        for (int i4 = tid; i4 < (k >> 2); i4 += nthr) {
            const float4 v = xs4[i4];
            const float x[4] = {v.x, v.y, v.z, v.w};
            int q[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                q[e] = zero ? 0 : exact_code(x[e], alpha, inv, flo, fhi, thr);
                const double d = fma(-ad, int_double(q[e]), (double)x[e]);
                ss = fma(d, d, ss);
            }
            if (codes) {
                const unsigned int w = (q[0] & 0xff) | ((q[1] & 0xff) << 8) | ((q[2] & 0xff) << 16) | ((unsigned)(q[3] & 0xff) << 24);
                *reinterpret_cast<unsigned int*>(codes + row_base + 4ll * i4) = w;
            }
            if (packed) {
                const unsigned short h = (unsigned short)((q[0] & 0xf) | ((q[1] & 0xf) << 4) | ((q[2] & 0xf) << 8) | ((q[3] & 0xf) << 12));
                *reinterpret_cast<unsigned short*>(packed + ((row_base + 4ll * i4) >> 1)) = h;
            }
        }
    } else {
        // general path: one output byte (two flat-consecutive elements) per thread; a byte that
        // straddles two rows is completed by the second row of the unit from the saved nibble
        const int o = (int)(row_base & 1);
        const int n_pairs = (k + o + 1) >> 1;
        for (int p = tid; p < n_pairs; p += nthr) {
            const int e0 = 2 * p - o, e1 = e0 + 1;
            int q0 = 0, q1 = 0;
            if (e0 >= 0) {
                const float x = s.xs[e0];
                q0 = zero ? 0 : code_of(x, alpha, flo, fhi);
                const double d = (double)x - (double)alpha * (double)q0;
                ss += d * d;
                if (codes) codes[row_base + e0] = (signed char)q0;
            } else {
                q0 = *carry;
            }
            const bool has1 = e1 < k;
            if (has1) {
                const float x = s.xs[e1];
                q1 = zero ? 0 : code_of(x, alpha, flo, fhi);
                const double d = (double)x - (double)alpha * (double)q1;
                ss += d * d;
                if (codes) codes[row_base + e1] = (signed char)q1;
            }
            if (packed) {
                if (has1 || !more_rows_in_unit) {
                    packed[(row_base + e0) >> 1] = (unsigned char)((q0 & 0xf) | ((q1 & 0xf) << 4));
                } else {
                    *carry = q0;   // last element of the row: its byte is written by the next row
                }
            }
        }
    }
    long long zero64 = 0;
    block_sum2(ss, zero64, s.scratch);
    return ss;
}

// EXT = false: the grid search with polish (and Algorithm 1 with a fixed number of sweeps) and nothing else, so that
// the common launches keep their register allocation and code size; EXT = true adds the comparison solvers, the offset
// search, Algorithm 1's loop condition, gated layers and rows that start from an earlier tensor's residual.
// PATH says which of the three row paths the instantiation contains (bit 0: block per row, bit 1: batched short rows,
// bit 2: thread per row).  A launch whose tensors all take one path uses the instantiation with only that path: the
// kernel is sensitive to its own code size (instruction cache), and code of a path no block runs still costs.
template <int CPT, bool EXT, int PATH>
__global__ void __launch_bounds__(OMSE_ROWS_MAX_THREADS) rows_kernel(const RowArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ unsigned long long s_unit;
    __shared__ RowMode s_mode;
    const int tid = threadIdx.x, nthr = blockDim.x;
    RowSmem s;
    s.xs = reinterpret_cast<float*>(smem_raw);
    s.x0 = s.xs + (a.keep_x0 ? 4 * a.max_k4 : 0);
    s.xb = s.x0 + 4 * a.max_k4;
    s.xg = reinterpret_cast<double*>(s.xb + (a.prune ? 4 * a.max_k4 + 4 * CPT : 0));
    s.scratch = s.xg + (size_t)(a.groups - 1) * CPT * a.tg;
    s.skip = s.scratch + kScratchDoubles;
    s.seg = reinterpret_cast<int*>(s.skip + CPT);
    s.misc = s.seg + 2 * (CPT + 1);
    unsigned int st = 0;
    unsigned long long ev = 0ull;      // (element, candidate) evaluations this thread executed

    // 1/(c+1) for this thread's candidates: 1/alpha_c = (1/(c+1)) * (1/step) to within 2 ulp
    float rcp[CPT];
#pragma unroll
    for (int sl = 0; sl < CPT; ++sl) rcp[sl] = __fdiv_rn(1.0f, (float)(sl * a.tg + (tid % a.tg) + 1));

    for (;;) {
        __syncthreads();   // previous unit fully consumed (shared row, s_unit)
        if (tid == 0) s_unit = atomicAdd(a.ticket, 1ull);
        __syncthreads();
        const long long unit = (long long)s_unit;
        if (unit >= a.n_units) break;
        // ---- which tensor this unit belongs to (tensors are few: linear scan from the end)
        const RowTensor* tp = &a.one;
        if (a.tensors) {
            int ti = a.n_launch_tensors - 1;
            while (ti > 0 && a.tensors[ti].unit_begin > unit) --ti;
            tp = a.tensors + ti;
        }
        const RowTensor& T = *tp;
        if (EXT && T.gate && *T.gate == 0) continue;   // not a key layer: nothing to do for this unit
        if constexpr ((PATH & 4) != 0) {
            if (T.small & 4) {
                tiny_dispatch<CPT>(a, T, unit - T.unit_begin, smem_raw, st, ev);
                continue;
            }
        }
        if constexpr ((PATH & 2) != 0) {
            if (T.small) {
                small_unit<CPT, EXT>(a, T, unit - T.unit_begin, smem_raw, rcp, st, ev);
                continue;
            }
        }
        if constexpr ((PATH & 1) == 0) continue;   // (the host never puts a block-per-row tensor into such a launch)
        const int k = (int)T.K;
        const int k4 = (k + 3) >> 2;
        const long long n_total = T.S * T.K;
        const long long packed_stride = (n_total + 1) >> 1;
        const long long unit_local = unit - T.unit_begin;

        for (int ru = 0; ru < T.rows_per_unit; ++ru) {
            const long long row = unit_local * T.rows_per_unit + ru;
            if (row >= T.S) break;
            const bool more = (ru + 1 < T.rows_per_unit) && (row + 1 < T.S);
            const long long row_base = row * T.K;
            const float* src = T.w + row_base;
            if (ru > 0) __syncthreads();   // previous row of the unit fully consumed
            // ---- stage the row once from HBM (128-bit loads when the row start allows it)
            bool bad = false;
            if ((reinterpret_cast<unsigned long long>(src) & 15ull) == 0) {
                const float4* src4 = reinterpret_cast<const float4*>(src);
                for (int i4 = tid; i4 < (k >> 2); i4 += nthr) {
                    const float4 v = __ldg(src4 + i4);
                    reinterpret_cast<float4*>(s.xs)[i4] = v;
                    bad |= !(fabsf(v.x) <= FLT_MAX) || !(fabsf(v.y) <= FLT_MAX) || !(fabsf(v.z) <= FLT_MAX) || !(fabsf(v.w) <= FLT_MAX);
                }
                for (int i = (k & ~3) + tid; i < 4 * k4; i += nthr) {
                    const float v = i < k ? __ldg(src + i) : 0.f;
                    s.xs[i] = v;
                    bad |= !(fabsf(v) <= FLT_MAX);
                }
            } else {
                for (int i = tid; i < 4 * k4; i += nthr) {
                    const float v = i < k ? __ldg(src + i) : 0.f;
                    s.xs[i] = v;
                    bad |= !(fabsf(v) <= FLT_MAX);
                }
            }
            if (bad) st |= 1u;
            if (EXT && T.prior_alpha) {
                // second quantized tensor of a key layer: the row becomes the residual of the first tensor
                __syncthreads();
                const float a1 = T.prior_alpha[row];
                const float flo0 = (float)a.lo[0], fhi0 = (float)a.hi[0];
                if (a1 > 0.f)
                    for (int i = tid; i < k; i += nthr) {
                        const float x = s.xs[i];
                        s.xs[i] = fmaf(-a1, (float)code_of(x, a1, flo0, fhi0), x);
                    }
            }
            if (T.delta && !(EXT && a.n_delta > 0)) {
                // quantization with offset: delta = min of the row, the shifted row fl(x - delta) is what gets searched
                __syncthreads();
                float lo = INFINITY;
                for (int i = tid; i < k; i += nthr) {
                    const float v = s.xs[i];
                    if (fabsf(v) <= FLT_MAX) lo = fminf(lo, v);
                }
                __shared__ float s_min[32];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
                if ((tid & 31) == 0) s_min[tid >> 5] = lo;
                __syncthreads();
                float d = INFINITY;
                for (int w = 0; w < ((nthr + 31) >> 5); ++w) d = fminf(d, s_min[w]);
                if (!(d < INFINITY)) d = 0.f;
                for (int i = tid; i < k; i += nthr) s.xs[i] = s.xs[i] - d;
                if (tid == 0) T.delta[row] = d;
            }
            if (a.keep_x0) {
                __syncthreads();
                for (int i = tid; i < 4 * k4; i += nthr) s.x0[i] = s.xs[i];
            }
            __syncthreads();

            // ---- The row goes through phi one or more times; all modes share the one call below.
            //  * default / Algorithm 1 (Section 3.5): pass = (sweep, tensor j); the residual of the other tensors is
            //    quantized; one tensor and one sweep is plain phi.
            //  * offset searched as well (Section 3.1 scheme, a.n_delta > 0): passes 0..n_delta-1 run the line search
            //    on the row shifted by offset d and keep the pair with the smallest error (lowest offset, then lowest
            //    scale index, on equal errors); the last pass polishes and emits at that pair.
            // Everything that steers the passes lives in shared memory (s_mode), not in registers: the sweep inside
            // phi_block needs the whole register budget.
            const bool affine = EXT && a.n_delta > 0;
            if (affine) {
                float lo = INFINITY, hi = -INFINITY;   // extremes of the finite values of the row
                for (int i = tid; i < k; i += nthr) {
                    const float v = s.x0[i];
                    if (fabsf(v) <= FLT_MAX) {
                        lo = fminf(lo, v);
                        hi = fmaxf(hi, v);
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
                    hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
                }
                __shared__ float s_ext[2][32];
                if ((tid & 31) == 0) {
                    s_ext[0][tid >> 5] = lo;
                    s_ext[1][tid >> 5] = hi;
                }
                __syncthreads();
                if (tid == 0) {
                    lo = INFINITY;
                    hi = -INFINITY;
                    for (int w = 0; w < ((nthr + 31) >> 5); ++w) {
                        lo = fminf(lo, s_ext[0][w]);
                        hi = fmaxf(hi, s_ext[1][w]);
                    }
                    if (!(lo <= hi)) lo = hi = 0.f;
                    s_mode.aff_lo = lo;
                    s_mode.aff_dstep = __fdiv_rn(__fmul_rn(a.off_frac, __fsub_rn(hi, lo)), (float)a.n_delta);
                    s_mode.aff_best = INFINITY;
                    s_mode.aff_d = -1;
                    s_mode.aff_c = -1;
                }
            }
            if (EXT && a.eps >= 0.f) {
                // Algorithm 1: error before the first sweep (all tensors zero) is ||T||^2
                double e0 = 0.0;
                long long zero = 0;
                for (int i = tid; i < k; i += nthr) e0 += (double)s.xs[i] * (double)s.xs[i];
                block_sum2(e0, zero, s.scratch);
                if (tid == 0) s_mode.e_prev = e0;
            }
            if (EXT && tid == 0) s_mode.sweeps_ran = 0;
            const int n_pass = affine ? a.n_delta + 1 : a.n_sweeps * a.n_tensors;
            for (int pass = 0; pass < n_pass; ++pass) {
                const int sweep = affine ? 0 : pass / a.n_tensors;
                const int j = affine ? 0 : pass - sweep * a.n_tensors;
                if (EXT) __syncthreads();   // every thread is done with the previous pass's control block
                if (EXT && tid == 0) {
                    PhiCtl c = {a.solver, a.solver_iters, -1, a.refine_iters, false};
                    if (affine) {
                        const bool last = pass == a.n_delta;
                        if (last) {
                            c.start_idx = s_mode.aff_d >= 0 ? s_mode.aff_c : a.n_cand;   // n_cand: no offset had a usable scale
                        } else {
                            c.n_refine = 0;
                            c.want_sse = true;
                        }
                        s_mode.aff_dl = __fadd_rn(s_mode.aff_lo, __fmul_rn((float)(last ? max(s_mode.aff_d, 0) : pass), s_mode.aff_dstep));
                    }
                    s_mode.ctl = c;
                }
                if (affine) {
                    __syncthreads();
                    const float dl = s_mode.aff_dl;
                    for (int i = tid; i < 4 * k4; i += nthr) s.xs[i] = i < k ? __fsub_rn(s.x0[i], dl) : 0.f;
                    __syncthreads();
                } else if (a.keep_x0 && pass > 0) {
                    // residual T - sum_{i != j} alpha_i q^i from the original row, increasing i
                    for (int i = tid; i < k; i += nthr) {
                        float v = s.x0[i];
                        for (int i2 = 0; i2 < a.n_tensors; ++i2) {
                            if (i2 == j || (sweep == 0 && i2 > j)) continue;
                            const float ai = T.alpha[(long long)i2 * T.S + row];
                            const float qi = (float)T.codes[(long long)i2 * n_total + row_base + i];
                            v = fmaf(-ai, qi, v);
                        }
                        s.xs[i] = v;
                    }
                    __syncthreads();
                }
                const float flo = (float)a.lo[j], fhi = (float)a.hi[j];
                PhiOut r = phi_block<CPT, EXT>(a, s, k, k4, flo, fhi, rcp, ev, s_mode.ctl);
                if (affine && pass < a.n_delta) {
                    if (tid == 0 && !r.degenerate && r.sse < s_mode.aff_best) {   // increasing offset: strict < keeps the lowest flat index
                        s_mode.aff_best = r.sse;
                        s_mode.aff_d = pass;
                        s_mode.aff_c = r.idx;
                    }
                    continue;      // the barriers of the next pass order these writes before their readers
                }
                if (r.degenerate) st |= 2u;
                const double sse = emit_block(s, k, r.alpha, flo, fhi,
                                              T.codes ? T.codes + (long long)j * n_total : nullptr,
                                              T.packed ? T.packed + (long long)j * packed_stride : nullptr,
                                              row_base, &s.misc[1 + j], more);
                if (tid == 0) {
                    T.alpha[(long long)j * T.S + row] = r.alpha;
                    T.sse[(long long)j * T.S + row] = (float)sse;
                    if (a.sse_history) a.sse_history[((long long)sweep * a.n_tensors + j) * T.S + row] = (float)sse;
                    if (affine) {
                        if (T.delta) T.delta[row] = s_mode.aff_dl;
                        if (T.best_idx) T.best_idx[row] = r.degenerate ? -1 : s_mode.aff_d * a.n_cand + s_mode.aff_c;
                    } else if (T.best_idx && j == 0) {
                        T.best_idx[row] = r.idx;
                    }
                }
                if (!a.keep_x0 && j + 1 < a.n_tensors) {
                    // first sweep without a kept copy: the residual is updated in place
                    const float inv = r.alpha > 0.f ? __fdiv_rn(1.0f, r.alpha) : 0.f, thr = ambiguity_threshold(flo, fhi);
                    for (int i = tid; i < k; i += nthr) {
                        const float x = s.xs[i];
                        const int q = r.alpha > 0.f ? exact_code(x, r.alpha, inv, flo, fhi, thr) : 0;
                        s.xs[i] = fmaf(-r.alpha, (float)q, x);
                    }
                }
                bool stop = false;
                if (EXT && j == a.n_tensors - 1) {
                    if (tid == 0) s_mode.sweeps_ran = sweep + 1;
                    if (a.eps >= 0.f) {
                        // loop condition of Algorithm 1: go on while the sweep lowered the error by more than eps (relative);
                        // every thread holds the same sse, so the decision is uniform
                        const double e_prev = s_mode.e_prev;
                        stop = !((e_prev - sse) > (double)a.eps * e_prev);
                    }
                }
                __syncthreads();   // alpha / codes of tensor j visible to the block (global + shared); e_prev read by all
                if (EXT && j == a.n_tensors - 1 && a.eps >= 0.f && tid == 0) s_mode.e_prev = sse;
                if (stop) break;
            }
            const int sweeps_ran = EXT ? s_mode.sweeps_ran : a.n_sweeps;
            if (EXT && tid == 0 && !affine) {
                if (a.sweeps_done) a.sweeps_done[row] = sweeps_ran;
                if (a.sse_history)     // sweeps that did not run repeat the last error
                    for (int sweep = sweeps_ran; sweep < a.n_sweeps; ++sweep)
                        for (int j = 0; j < a.n_tensors; ++j)
                            a.sse_history[((long long)sweep * a.n_tensors + j) * T.S + row] = T.sse[(long long)j * T.S + row];
            }
        }
    }
    if (st) atomicOr(a.status, st);   // any thread that saw a flag reports it
    report_evaluations(a.evals, ev);
    // ---- the last block to leave re-arms the ticket pair for the next launch (no block waits)
    if (tid == 0) {
        __threadfence();
        const unsigned long long done = atomicAdd(a.ticket + 1, 1ull);
        if (done == (unsigned long long)gridDim.x - 1ull) {
            a.ticket[0] = 0ull;
            a.ticket[1] = 0ull;
            __threadfence();
        }
    }
}

}  // namespace omse
