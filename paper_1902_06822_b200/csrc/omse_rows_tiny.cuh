// Very short kernels (up to 32 weights, e.g. the 3x3x3 kernels of a first convolution) in large
// numbers: one THREAD owns one row.  The row sits in registers as packed pairs, the thread walks the
// whole grid of candidate scales serially (no reduction across threads at all), re-scores in fp64 the
// candidates within the fp32 noise band of the minimum, polishes and emits.
// A work unit is blockDim.x consecutive rows, staged and written back through shared memory so that
// global accesses stay coalesced.  Same candidate arithmetic and decisions as the other paths.
#pragma once
#include "omse_device.cuh"

namespace omse {

template <int KP>
__device__ void tiny_unit(const RowArgs& a, const RowTensor& T, long long unit_local, unsigned char* smem_raw,
                          unsigned int& st, unsigned long long& ev) {
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int k = (int)T.K;
    const int B = T.rows_per_unit;                       // == blockDim.x
    const long long row0 = unit_local * B;
    const int nrows = (int)min((long long)B, T.S - row0);
    const int n_el = nrows * k;
    float* xs = reinterpret_cast<float*>(smem_raw);      // [B*k] the unit's rows, flat
    float* rcpt = xs + ((B * k + 3) & ~3);               // [n_cand] 1/(c+1)
    signed char* qs = reinterpret_cast<signed char*>(rcpt + ((a.n_cand + 3) & ~3));   // [B*k] codes
    const float flo = (float)a.lo[0], fhi = (float)a.hi[0];
    const float* src = T.w + row0 * T.K;

    // ---- stage (coalesced), table of reciprocals
    bool bad = false;
    for (int i = tid; i < n_el; i += nthr) {
        const float v = __ldg(src + i);
        xs[i] = v;
        bad |= !(fabsf(v) <= FLT_MAX);
    }
    if (bad) st |= 1u;
    for (int c = tid; c < a.n_cand; c += nthr) rcpt[c] = __fdiv_rn(1.0f, (float)(c + 1));
    __syncthreads();

    const bool active = tid < nrows;
    float alpha = 0.f;
    int best = -1;
    float x[2 * KP];
    double sse = 0.0;
    if (active) {
        // ---- the row into registers; offset scheme; maxima
        float lo = INFINITY;
#pragma unroll
        for (int i = 0; i < 2 * KP; ++i) {
            x[i] = i < k ? xs[tid * k + i] : 0.f;        // row stride k: odd strides are conflict free, others mildly
            if (i < k && fabsf(x[i]) <= FLT_MAX) lo = fminf(lo, x[i]);
        }
        if (T.delta) {
            if (!(lo < INFINITY)) lo = 0.f;
#pragma unroll
            for (int i = 0; i < 2 * KP; ++i)
                if (i < k) x[i] -= lo;
            T.delta[row0 + tid] = lo;
        }
        float mpos = 0.f, mneg = 0.f;
#pragma unroll
        for (int i = 0; i < 2 * KP; ++i) {
            if (fabsf(x[i]) <= FLT_MAX) {
                mpos = fmaxf(mpos, x[i]);
                mneg = fmaxf(mneg, -x[i]);
            }
        }
        const GridSetup g = grid_setup(mpos, mneg, a.hi_frac, a.n_cand, flo, fhi);
        const float a_last = __fmul_rn((float)a.n_cand, g.step);
        bool degenerate = !(fmaxf(mpos, mneg) > 0.f) || !(a_last >= FLT_MIN);
        u64 x2[KP];
#pragma unroll
        for (int p = 0; p < KP; ++p) x2[p] = pack2(x[2 * p], x[2 * p + 1]);

        // ---- the whole grid, serially: the three smallest fp32 errors (two with their indices)
        const u64 M2 = pack2(kMagic, kMagic), NM2 = pack2(-kMagic, -kMagic);
        const float clo = kMagic + flo, chi = kMagic + fhi;
        auto sweep_error = [&](int c, float cf) -> float {   // fp32 error of candidate c on this row; cf = c + 1
            const float ac = __fmul_rn(cf, g.step);
            const float inv = g.tiny ? __fdiv_rn(1.0f, ac) : rcpt[c] * g.rstep;
            const u64 inv2 = pack2(inv, inv), na2 = pack2(-ac, -ac);
            u64 acc = 0ull, acc_b = 0ull;             // two accumulators: shorter dependency chain
            if (c < g.c_sat) {      // candidates that may saturate on this row (divergence only near c_sat)
#pragma unroll
                for (int p = 0; p < KP; ++p) {
                    float t0, t1;
                    unpack2(fma2(x2[p], inv2, M2), t0, t1);
                    t0 = fminf(fmaxf(t0, clo), chi);
                    t1 = fminf(fmaxf(t1, clo), chi);
                    const u64 e = fma2(na2, add2(pack2(t0, t1), NM2), x2[p]);
                    if (p & 1) acc_b = fma2(e, e, acc_b);
                    else acc = fma2(e, e, acc);
                }
            } else {
#pragma unroll
                for (int p = 0; p < KP; ++p) {
                    const u64 e = fma2(na2, add2(fma2(x2[p], inv2, M2), NM2), x2[p]);
                    if (p & 1) acc_b = fma2(e, e, acc_b);
                    else acc = fma2(e, e, acc);
                }
            }
            acc = add2(acc, acc_b);
            float p0, p1;
            unpack2(acc, p0, p1);
            return (ac >= FLT_MIN) ? p0 + p1 : INFINITY;
        };
        auto exact_error = [&](int c) -> double {            // fp64 error with true division
            const float ac = __fmul_rn((float)(c + 1), g.step);
            double ss = 0.0;
#pragma unroll
            for (int i = 0; i < 2 * KP; ++i) {
                if (i < k) {
                    const double d = (double)x[i] - (double)ac * (double)code_of(x[i], ac, flo, fhi);
                    ss += d * d;
                }
            }
            return ss;
        };
        // The grid is walked once.  Beside the smallest fp32 error the walk keeps the index window [w_lo, w_hi] outside
        // which no candidate can lie within the noise band of the final minimum: a candidate inside the band of the
        // final minimum is inside the band of the running minimum when it is seen (the running minimum only falls),
        // and when the running minimum falls by more than the band everything seen before drops out.
        float b1v = INFINITY;
        int b1i = 0x7fffffff, w_lo = 0, w_hi = -1;
        const float band_f = 1.0f + 1.25f * (float)kRescoreBand;   // a little wider than the fp64 test below: a superset
        if (!degenerate) {
            float cf = 0.f;                               // c + 1 as a float (exact: n_cand <= 4096)
            for (int c = 0; c < a.n_cand; ++c) {
                cf += 1.0f;
                const float v = sweep_error(c, cf);
                if (v <= b1v * band_f) {
                    w_hi = c;
                    if (v < b1v) {      // ascending c: strict < keeps the lowest index
                        if (v * band_f < b1v) w_lo = c;
                        b1v = v;
                        b1i = c;
                    }
                }
            }
            ev += (unsigned long long)a.n_cand * (2ull * KP);
            if (b1i == 0x7fffffff) degenerate = true;    // every error Inf/NaN
        }
        if (degenerate) {
            st |= 2u;
        } else {
            best = b1i;
            // ---- candidates within the fp32 noise band of the minimum: decide in fp64 with true division
            if (w_hi > w_lo) {
                const double band = (double)b1v * (1.0 + kRescoreBand);
                double best_sse = INFINITY;
                best = 0x7fffffff;
                int n_band = 0;
                for (int c = w_lo; c <= w_hi; ++c) {
                    if ((double)sweep_error(c, (float)(c + 1)) <= band) {
                        const double ss = exact_error(c);
                        ++n_band;
                        if (ss < best_sse) {   // ascending c: strict < keeps the lowest index
                            best_sse = ss;
                            best = c;
                        }
                    }
                }
                ev += (unsigned long long)(w_hi - w_lo + 1) * (2ull * KP);
                if (n_band == 0) best = b1i;
            }
            // ---- polish
            alpha = __fmul_rn((float)(best + 1), g.step);
            for (int it = 0; it < a.refine_iters; ++it) {
                double sxq = 0.0;
                int sqq = 0;
#pragma unroll
                for (int i = 0; i < 2 * KP; ++i) {
                    if (i < k) {
                        const int q = code_of(x[i], alpha, flo, fhi);
                        sqq += q * q;
                        sxq += (double)x[i] * (double)q;
                    }
                }
                if (sqq == 0) break;
                const float a_new = (float)(sxq / (double)sqq);
                if (!(a_new >= FLT_MIN) || !(a_new <= FLT_MAX)) break;
                if (a_new == alpha) break;   // fixed point: further steps would repeat it exactly
                alpha = a_new;
            }
        }
        // ---- final codes and error
#pragma unroll
        for (int i = 0; i < 2 * KP; ++i) {
            if (i < k) {
                const int q = alpha > 0.f ? code_of(x[i], alpha, flo, fhi) : 0;
                const double d = (double)x[i] - (double)alpha * (double)q;
                sse += d * d;
                qs[tid * k + i] = (signed char)q;
            }
        }
        T.alpha[row0 + tid] = alpha;
        T.sse[row0 + tid] = (float)sse;
        if (T.best_idx) T.best_idx[row0 + tid] = best;
    }
    __syncthreads();
    // ---- emission of the unit's codes, coalesced; the unit starts at an even flat index (even B)
    const long long base = row0 * T.K;
    if (T.codes)
        for (int i = tid; i < n_el; i += nthr) T.codes[base + i] = qs[i];
    if (T.packed) {
        const int n_bytes = (n_el + 1) >> 1;
        for (int b = tid; b < n_bytes; b += nthr) {
            const int q0 = qs[2 * b];
            const int q1 = (2 * b + 1 < n_el) ? qs[2 * b + 1] : 0;
            T.packed[(base >> 1) + b] = (unsigned char)((q0 & 0xf) | ((q1 & 0xf) << 4));
        }
    }
}

template <int CPT_UNUSED>
__device__ __forceinline__ void tiny_dispatch(const RowArgs& a, const RowTensor& T, long long unit_local,
                                              unsigned char* smem_raw, unsigned int& st, unsigned long long& ev) {
    const int k = (int)T.K;
    if (k <= 8) tiny_unit<4>(a, T, unit_local, smem_raw, st, ev);
    else if (k <= 16) tiny_unit<8>(a, T, unit_local, smem_raw, st, ev);
    else if (k <= 24) tiny_unit<12>(a, T, unit_local, smem_raw, st, ev);
    else if (k <= 28) tiny_unit<14>(a, T, unit_local, smem_raw, st, ev);
    else tiny_unit<16>(a, T, unit_local, smem_raw, st, ev);
}

}  // namespace omse
