// Device-side building blocks of the MMSE scale search for sm_100a.
//
// Section 3.4 of the paper reduces the constrained MSE problem to a one-dimensional search over the
// scale alpha, the codes being [T_i/alpha]_Zp.  The search evaluates the squared error at every
// point of a grid of scales.  Here the tensor (one kernel, or a tile of an activation tensor) sits
// in shared memory, every thread owns a few candidate scales in registers, and all threads stream
// the same elements (shared-memory broadcast), so the inner loop is pure FP32 arithmetic:
//     t = x*inv_alpha + M       (M = 1.5*2^23: the add rounds to the nearest integer, ties to even)
//     t = min(max(t, M+lo), M+hi)            only for candidates that can saturate on this tensor
//     q = t - M ;  e = x - alpha*q ;  acc += e*e
// written with Blackwell's packed fma.rn.f32x2 / add.rn.f32x2 on two elements at a time.
#pragma once
#include <cfloat>
#include <cstdint>
#include <cuda_runtime.h>

namespace omse {

typedef unsigned long long u64;

constexpr float kMagic = 12582912.0f;   // 1.5 * 2^23
#ifndef OMSE_FLUSH4
#define OMSE_FLUSH4 32
#endif
// float4 loads per unrolled step of the sweep loop, by the number of active candidate slots: few slots mean few
// independent chains per load, so several loads are interleaved; many slots have the parallelism already and are
// kept compact (the kernels are sensitive to instruction-cache pressure)
#ifndef OMSE_UNROLL_1
#define OMSE_UNROLL_1 8
#endif
#ifndef OMSE_UNROLL_2
#define OMSE_UNROLL_2 3
#endif
#ifndef OMSE_UNROLL_3
#define OMSE_UNROLL_3 2
#endif
#ifndef OMSE_UNROLL_N
#define OMSE_UNROLL_N 1
#endif
#ifndef OMSE_ACC_UNROLL_1
#define OMSE_ACC_UNROLL_1 1
#endif
#ifndef OMSE_ACC_UNROLL_2
#define OMSE_ACC_UNROLL_2 1
#endif
template <int NACT>
struct AccumUnroll {      // the same for the short spans of the batched short-row path
    static constexpr int value = NACT == 1 ? OMSE_ACC_UNROLL_1 : NACT == 2 ? OMSE_ACC_UNROLL_2 : 1;
};
template <int NACT>
struct SweepUnroll {
    static constexpr int value = NACT == 1 ? OMSE_UNROLL_1 : NACT == 2 ? OMSE_UNROLL_2 : NACT == 3 ? OMSE_UNROLL_3 : OMSE_UNROLL_N;
};
constexpr int kFlushEvery4 = OMSE_FLUSH4;   // float4 loads between folds of the fp32 partial sums into fp64
constexpr double kRescoreBand = 4e-6;   // candidates within this relative band of the fp32 minimum are re-scored

__device__ __forceinline__ u64 pack2(float a, float b) {
    u64 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void unpack2(u64 v, float& a, float& b) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ u64 fma2(u64 a, u64 b, u64 c) {
    u64 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ u64 add2(u64 a, u64 b) {
    u64 d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// [x/alpha]_Zp exactly as Section 3.1 writes it: IEEE division, round to nearest even, saturate.
__device__ __forceinline__ int code_of(float x, float alpha, float flo, float fhi) {
    float r = rintf(__fdiv_rn(x, alpha));
    r = fminf(fmaxf(r, flo), fhi);
    return (int)r;
}

// [x/alpha]_Zp without a division on the common path.  t = fl(x*inv + M) rounds the exact product to the nearest
// integer (ties to even); with inv = fl(1/alpha) the product is within 2^-24 relative of x/alpha, and so is the IEEE
// quotient, so both round to the same integer unless the product lies within (|integer| + 1) * 2^-21 of a
// half-integer.  Integers beyond the range by more than one saturate either way, so the test only has to hold for
// |integer| <= range + 1: amb_thr = 1/2 - (range + 2) * 2^-21 serves every element; `ambiguous` reports a product
// closer to a half-integer than that (or too large to be rounded by the addition), and the caller then takes the
// division.  Returns M + code (the code sits in the low mantissa bits).
__device__ __forceinline__ float magic_code(float x, float inv, float clo, float chi, float amb_thr, bool& ambiguous) {
    const float t = fmaf(x, inv, kMagic);
    const float rq = t - kMagic;
    const float delta = fmaf(x, inv, -rq);
    ambiguous = !(fabsf(delta) <= amb_thr);
    return fminf(fmaxf(t, clo), chi);
}

// integer held by M + q as an int, and as a double without a conversion instruction
__device__ __forceinline__ int magic_int(float tc) { return __float_as_int(tc) - 0x4B400000; }
__device__ __forceinline__ double int_double(int q) {
    return __hiloint2double(0x43380000 + (q >> 31), q) - 6755399441055744.0;   // (1.5*2^52 + q) - 1.5*2^52, exact
}

// The code of x at scale alpha (inv = fl(1/alpha)) as an int, equal to code_of(x, alpha, flo, fhi) bit for bit.
__device__ __forceinline__ int exact_code(float x, float alpha, float inv, float flo, float fhi, float amb_thr) {
    bool amb;
    const float tc = magic_code(x, inv, kMagic + flo, kMagic + fhi, amb_thr, amb);
    return amb ? code_of(x, alpha, flo, fhi) : magic_int(tc);   // rare: the division decides
}
__device__ __forceinline__ float ambiguity_threshold(float flo, float fhi) {
    return 0.5f - (fmaxf(fhi, -flo) + 2.0f) * 4.76837158203125e-7f;
}

// ---------------------------------------------------------------------------------------------
// Candidate sweep over float4 indices [beg4, end4) of a shared-memory span.  CPT candidates per
// thread, of which only the first NACT are evaluated on this span (the others are known to code
// every element of the span as zero); the first NCL of them are evaluated with saturation.
// acc2 holds two fp32 partial sums per candidate (even / odd element of each pair); every
// kFlushEvery4 loads they are folded into the fp64 accumulators so that the rounding noise of the
// fp32 sums stays near 1e-7 relative whatever the span length.
// ---------------------------------------------------------------------------------------------
template <int CPT, int NACT, int NCL>
__device__ __forceinline__ void sweep_range(const float4* __restrict__ xs4, int beg4, int end4,
                                            const u64 (&inv2)[CPT], const u64 (&na2)[CPT],
                                            double (&dacc)[CPT], float clo, float chi) {
    const u64 M2 = pack2(kMagic, kMagic);
    const u64 NM2 = pack2(-kMagic, -kMagic);
    u64 acc2[NACT];
#pragma unroll
    for (int s = 0; s < NACT; ++s) acc2[s] = 0ull;
    int i = beg4;
    while (i < end4) {
        const int stop = min(end4, i + kFlushEvery4);
#pragma unroll(SweepUnroll<NACT>::value)
        for (; i < stop; ++i) {
            const float4 v = xs4[i];
            const u64 xa = pack2(v.x, v.y), xb = pack2(v.z, v.w);
#pragma unroll
            for (int s = 0; s < NACT; ++s) {
                u64 ta = fma2(xa, inv2[s], M2);
                u64 tb = fma2(xb, inv2[s], M2);
                if (s < NCL) {
                    float a0, a1, b0, b1;
                    unpack2(ta, a0, a1);
                    unpack2(tb, b0, b1);
                    a0 = fminf(fmaxf(a0, clo), chi);
                    a1 = fminf(fmaxf(a1, clo), chi);
                    b0 = fminf(fmaxf(b0, clo), chi);
                    b1 = fminf(fmaxf(b1, clo), chi);
                    ta = pack2(a0, a1);
                    tb = pack2(b0, b1);
                }
                const u64 qa = add2(ta, NM2);
                const u64 qb = add2(tb, NM2);
                const u64 ea = fma2(na2[s], qa, xa);
                const u64 eb = fma2(na2[s], qb, xb);
                acc2[s] = fma2(ea, ea, acc2[s]);
                acc2[s] = fma2(eb, eb, acc2[s]);
            }
        }
#pragma unroll
        for (int s = 0; s < NACT; ++s) {
            float p0, p1;
            unpack2(acc2[s], p0, p1);
            dacc[s] += (double)(p0 + p1);
            acc2[s] = 0ull;
        }
    }
}

// Dispatch on the (warp-uniform) number of leading candidates per thread that need saturation ...
template <int CPT, int NACT>
__device__ __forceinline__ void sweep_ncl(int ncl, const float4* xs4, int beg4, int end4, const u64 (&inv2)[CPT],
                                          const u64 (&na2)[CPT], double (&dacc)[CPT], float clo, float chi) {
    if (ncl <= 0) {
        sweep_range<CPT, NACT, 0>(xs4, beg4, end4, inv2, na2, dacc, clo, chi);
    } else if (ncl == 1) {
        sweep_range<CPT, NACT, 1>(xs4, beg4, end4, inv2, na2, dacc, clo, chi);
    } else if (ncl == 2 && NACT > 2) {
        sweep_range<CPT, NACT, (NACT > 2 ? 2 : NACT)>(xs4, beg4, end4, inv2, na2, dacc, clo, chi);
    } else {
        sweep_range<CPT, NACT, NACT>(xs4, beg4, end4, inv2, na2, dacc, clo, chi);
    }
}

// ... and on the number of candidates per thread that are evaluated at all on this span.
template <int CPT>
__device__ __forceinline__ void sweep_dispatch(int nact, int ncl, const float4* xs4, int beg4, int end4,
                                               const u64 (&inv2)[CPT], const u64 (&na2)[CPT],
                                               double (&dacc)[CPT], float clo, float chi) {
    if (beg4 >= end4 || nact <= 0) return;
    if (ncl > nact) ncl = nact;
    switch (nact) {
        case 1: sweep_ncl<CPT, 1>(ncl, xs4, beg4, end4, inv2, na2, dacc, clo, chi); break;
        case 2: if constexpr (CPT >= 2) sweep_ncl<CPT, 2>(ncl, xs4, beg4, end4, inv2, na2, dacc, clo, chi); break;
        case 3: if constexpr (CPT >= 4) sweep_ncl<CPT, 3>(ncl, xs4, beg4, end4, inv2, na2, dacc, clo, chi); break;
        case 4: if constexpr (CPT >= 4) sweep_ncl<CPT, 4>(ncl, xs4, beg4, end4, inv2, na2, dacc, clo, chi); break;
        case 5: if constexpr (CPT >= 8) sweep_ncl<CPT, 5>(ncl, xs4, beg4, end4, inv2, na2, dacc, clo, chi); break;
        case 6: if constexpr (CPT >= 8) sweep_ncl<CPT, 6>(ncl, xs4, beg4, end4, inv2, na2, dacc, clo, chi); break;
        default: sweep_ncl<CPT, CPT>(ncl, xs4, beg4, end4, inv2, na2, dacc, clo, chi); break;
    }
}

template <int CPT>
__device__ __forceinline__ void sweep_dispatch(int ncl, const float4* xs4, int beg4, int end4,
                                               const u64 (&inv2)[CPT], const u64 (&na2)[CPT],
                                               double (&dacc)[CPT], float clo, float chi) {
    sweep_dispatch<CPT>(CPT, ncl, xs4, beg4, end4, inv2, na2, dacc, clo, chi);
}

// ---------------------------------------------------------------------------------------------
// The same evaluation without the fp64 fold: the caller keeps the fp32 pair sums across several
// spans (at most kFlushEvery4 loads between two folds) and folds them itself.  Used where a row is
// swept as a handful of short spans (magnitude classes of a short row).
// ---------------------------------------------------------------------------------------------
template <int CPT, int NACT, int NCL>
__device__ __forceinline__ void sweep_accum(const float4* __restrict__ xs4, int beg4, int end4,
                                            const u64 (&inv2)[CPT], const u64 (&na2)[CPT], u64 (&acc2)[CPT],
                                            float clo, float chi) {
    const u64 M2 = pack2(kMagic, kMagic);
    const u64 NM2 = pack2(-kMagic, -kMagic);
#pragma unroll(AccumUnroll<NACT>::value)
    for (int i = beg4; i < end4; ++i) {
        const float4 v = xs4[i];
        const u64 xa = pack2(v.x, v.y), xb = pack2(v.z, v.w);
#pragma unroll
        for (int s = 0; s < NACT; ++s) {
            u64 ta = fma2(xa, inv2[s], M2);
            u64 tb = fma2(xb, inv2[s], M2);
            if (s < NCL) {
                float a0, a1, b0, b1;
                unpack2(ta, a0, a1);
                unpack2(tb, b0, b1);
                a0 = fminf(fmaxf(a0, clo), chi);
                a1 = fminf(fmaxf(a1, clo), chi);
                b0 = fminf(fmaxf(b0, clo), chi);
                b1 = fminf(fmaxf(b1, clo), chi);
                ta = pack2(a0, a1);
                tb = pack2(b0, b1);
            }
            const u64 qa = add2(ta, NM2);
            const u64 qb = add2(tb, NM2);
            const u64 ea = fma2(na2[s], qa, xa);
            const u64 eb = fma2(na2[s], qb, xb);
            acc2[s] = fma2(ea, ea, acc2[s]);
            acc2[s] = fma2(eb, eb, acc2[s]);
        }
    }
}

template <int CPT, int NACT>
__device__ __forceinline__ void sweep_accum_ncl(int ncl, const float4* xs4, int beg4, int end4,
                                                const u64 (&inv2)[CPT], const u64 (&na2)[CPT], u64 (&acc2)[CPT],
                                                float clo, float chi) {
    if (ncl <= 0) {
        sweep_accum<CPT, NACT, 0>(xs4, beg4, end4, inv2, na2, acc2, clo, chi);
    } else if (ncl == 1) {
        sweep_accum<CPT, NACT, 1>(xs4, beg4, end4, inv2, na2, acc2, clo, chi);
    } else if (ncl == 2 && NACT > 2) {
        sweep_accum<CPT, NACT, (NACT > 2 ? 2 : NACT)>(xs4, beg4, end4, inv2, na2, acc2, clo, chi);
    } else {
        sweep_accum<CPT, NACT, NACT>(xs4, beg4, end4, inv2, na2, acc2, clo, chi);
    }
}

template <int CPT>
__device__ __forceinline__ void sweep_accum_dispatch(int nact, int ncl, const float4* xs4, int beg4, int end4,
                                                     const u64 (&inv2)[CPT], const u64 (&na2)[CPT],
                                                     u64 (&acc2)[CPT], float clo, float chi) {
    if (beg4 >= end4 || nact <= 0) return;
    if (ncl > nact) ncl = nact;
    switch (nact) {
        case 1: sweep_accum_ncl<CPT, 1>(ncl, xs4, beg4, end4, inv2, na2, acc2, clo, chi); break;
        case 2: if constexpr (CPT >= 2) sweep_accum_ncl<CPT, 2>(ncl, xs4, beg4, end4, inv2, na2, acc2, clo, chi); break;
        case 3: if constexpr (CPT >= 4) sweep_accum_ncl<CPT, 3>(ncl, xs4, beg4, end4, inv2, na2, acc2, clo, chi); break;
        case 4: if constexpr (CPT >= 4) sweep_accum_ncl<CPT, 4>(ncl, xs4, beg4, end4, inv2, na2, acc2, clo, chi); break;
        case 5: if constexpr (CPT >= 8) sweep_accum_ncl<CPT, 5>(ncl, xs4, beg4, end4, inv2, na2, acc2, clo, chi); break;
        case 6: if constexpr (CPT >= 8) sweep_accum_ncl<CPT, 6>(ncl, xs4, beg4, end4, inv2, na2, acc2, clo, chi); break;
        default: sweep_accum_ncl<CPT, CPT>(ncl, xs4, beg4, end4, inv2, na2, acc2, clo, chi); break;
    }
}

// ---------------------------------------------------------------------------------------------
// Block-wide reductions (fixed order: lanes by shuffle tree, warps in index order) so that results
// do not depend on scheduling.  `scratch` holds at least 2*32 doubles.  All threads get the result.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ long long warp_sum(long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    return v;
}

// sums a double and a 64-bit integer over the block
__device__ __forceinline__ void block_sum2(double& d, long long& q, double* scratch) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
    d = warp_sum(d);
    q = warp_sum(q);
    long long* qs = reinterpret_cast<long long*>(scratch + 32);
    __syncthreads();
    if (lane == 0) {
        scratch[warp] = d;
        qs[warp] = q;
    }
    __syncthreads();
    double dt = 0.0;
    long long qt = 0;
    for (int w = 0; w < nwarp; ++w) {
        dt += scratch[w];
        qt += qs[w];
    }
    d = dt;
    q = qt;
}

__device__ __forceinline__ void block_max2(float& a, float& b, double* scratch) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        a = fmaxf(a, __shfl_down_sync(0xffffffffu, a, o));
        b = fmaxf(b, __shfl_down_sync(0xffffffffu, b, o));
    }
    float* fs = reinterpret_cast<float*>(scratch);
    __syncthreads();
    if (lane == 0) {
        fs[warp] = a;
        fs[32 + warp] = b;
    }
    __syncthreads();
    float ta = 0.f, tb = 0.f;
    for (int w = 0; w < nwarp; ++w) {
        ta = fmaxf(ta, fs[w]);
        tb = fmaxf(tb, fs[32 + w]);
    }
    a = ta;
    b = tb;
}

// lexicographic minimum of (value, index) over the block
__device__ __forceinline__ void block_argmin(double& v, int& idx, double* scratch) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const double ov = __shfl_down_sync(0xffffffffu, v, o);
        const int oi = __shfl_down_sync(0xffffffffu, idx, o);
        if (ov < v || (ov == v && oi < idx)) {
            v = ov;
            idx = oi;
        }
    }
    int* is = reinterpret_cast<int*>(scratch + 32);
    __syncthreads();
    if (lane == 0) {
        scratch[warp] = v;
        is[warp] = idx;
    }
    __syncthreads();
    double bv = scratch[0];
    int bi = is[0];
    for (int w = 1; w < nwarp; ++w) {
        const double ov = scratch[w];
        const int oi = is[w];
        if (ov < bv || (ov == bv && oi < bi)) {
            bv = ov;
            bi = oi;
        }
    }
    v = bv;
    idx = bi;
}

// Number of leading candidate slots that must still evaluate x, for a thread group whose slot sl holds the scales
// >= (c_base + sl*tg + 1)*step: the others code it as 0.  inv_thr = 1/(0.4999*step), inv_tg = 1/tg.
template <int CPT>
__device__ __forceinline__ int magnitude_class(float x, float inv_thr, float inv_tg, float c_base = 0.f) {
    const float ax = fabsf(x);
    if (!(ax <= FLT_MAX)) return CPT;          // non-finite: every slot sees it (and reports it)
    const float r = ax * inv_thr - c_base;     // |x| / (0.4999*step), counted from the group's first candidate
    if (r <= 1.0f) return 0;
    const float f = (r - 1.0f) * inv_tg;       // slot sl needs x iff r > sl*tg + 1
    int nb = f >= (float)CPT ? CPT : (int)f + 1;
    if (CPT == 8 && nb == 7) ++nb;   // class 7 is merged upwards: fewer sweep variants (a class 5 of its own pays, a class 7 does not)
    return nb;
}

// Candidates with index below the returned value may saturate on an element of magnitude class nb
// (nb < CPT bounds |x| from above: |x| < 0.4999*(c_base + nb*tg + 1)*step, and candidate c saturates only if
// |x| >= min(hi+1/2, 1/2-lo)*alpha_c); class CPT has no upper bound and keeps the row's own count.
__device__ __forceinline__ int class_sat_count(int nb, int cpt, int tg, int c_sat_row, float flo, float fhi,
                                               int c_base = 0) {
    if (nb >= cpt) return c_sat_row;
    const float den = fminf(fhi + 0.5f, 0.5f - flo);
    const int c = (int)(0.5f * (float)(c_base + nb * tg + 1) / den) + 2;
    return min(c, c_sat_row);
}

// Adds this thread's count of executed (element, candidate) evaluations to a global counter: one atomic per warp.
__device__ __forceinline__ void report_evaluations(unsigned long long* counter, unsigned long long mine) {
    if (!counter) return;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, o);
    if ((threadIdx.x & 31) == 0 && mine) atomicAdd(counter, mine);
}

// Register-only loop of independent packed multiply-adds: measures the FP32 lane-operation rate of the FMA pipe,
// the roof the candidate sweep is compared with.  Every thread runs kPeakChains chains of fma.rn.f32x2.
constexpr int kPeakChains = 8;
__global__ void __launch_bounds__(256) fma_peak_kernel(float* __restrict__ out, int iters, float seed) {
    u64 v[kPeakChains];
#pragma unroll
    for (int s = 0; s < kPeakChains; ++s) v[s] = pack2(seed + 1e-3f * (float)(threadIdx.x + s), seed - 1e-3f * (float)s);
    const u64 m = pack2(0.9999999f, 1.0000001f), c = pack2(1e-7f, -1e-7f);
#pragma unroll 16   // long straight-line stretches: with a short body the loop bookkeeping costs ~8 % of the rate
    for (int i = 0; i < iters; ++i) {
#pragma unroll
        for (int s = 0; s < kPeakChains; ++s) v[s] = fma2(v[s], m, c);
    }
    float r = 0.f;
#pragma unroll
    for (int s = 0; s < kPeakChains; ++s) {
        float a, b;
        unpack2(v[s], a, b);
        r += a + b;
    }
    out[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = r;
}

// Per-candidate constants of one thread for the grid of Section 3.4 on a tensor with max|x| = m.
// Candidate c has alpha_c = fl(fl(c+1)*step), step = fl(fl(hi_frac*m)/fl(C)), all binary32.
// In the sweep x/alpha_c is replaced by x*inv_c with inv_c within 2 ulp of 1/alpha_c: a code can
// differ from the divided one only where both neighbours give the same error to ~1e-7, and the
// winners are re-scored with true division afterwards.
struct GridSetup {
    float step;      // alpha step
    float rstep;     // ~1/step
    bool tiny;       // step so small that 1/step may overflow: use per-candidate division
    int c_sat;       // candidates with index < c_sat may saturate on this tensor
};

__device__ __forceinline__ GridSetup grid_setup(float mpos, float mneg, float hi_frac, int n_cand,
                                                float flo, float fhi) {
    GridSetup g;
    const float m = fmaxf(mpos, mneg);
    const float a_hi = __fmul_rn(hi_frac, m);
    g.step = __fdiv_rn(a_hi, (float)n_cand);
    g.tiny = !(g.step > 1e-30f);
    g.rstep = g.tiny ? 0.f : __fdiv_rn(1.0f, g.step);
    // x*inv_c stays strictly below hi+1/2 (and above lo-1/2) for every x once
    // c+1 > max(mpos/(hi+1/2), mneg/(1/2-lo)) / step; 1e-5 covers the rounding of inv_c and alpha_c.
    const float need = fmaxf(mpos / (fhi + 0.5f), mneg / (0.5f - flo));
    const float cs = g.tiny ? (float)n_cand : need * g.rstep * 1.00001f + 1.0f;
    g.c_sat = cs >= (float)n_cand ? n_cand : (int)cs;
    return g;
}

}  // namespace omse
