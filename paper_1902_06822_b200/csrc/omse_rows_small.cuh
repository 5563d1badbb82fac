// Short kernels (rows of a few dozen to a few hundred weights): the per-row fixed costs of the
// block-cooperative path (barriers, reductions, global round trips) would dominate, so a work unit
// here is a batch of B consecutive rows: staged together, swept one after the other by the whole
// block (error curve of each row kept in shared memory), then finished by one warp per row with
// shuffle reductions only.  Results are identical in meaning to the long-row path: same candidate
// arithmetic, same fp64 re-scoring of near-minimal candidates, same polish and emission.
#pragma once
#include "omse_device.cuh"

namespace omse {

__device__ __forceinline__ double warp_allsum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;   // a + b == b + a: every lane ends with the same bits
}
__device__ __forceinline__ int warp_allsum(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Per-row quantities every thread needs, computed once by the warp that takes the row's maxima.
struct SmallRowParams {
    float step;     // candidate step
    float rstep;    // ~1/step
    int c_sat;      // candidates below this index may saturate
    int flags;      // bit 0: step so small that reciprocals need a division; bit 1: no usable scale
};

// Candidate sweep of a row of at most 4*kFlushEvery4 elements: one fp32 block, no fp64 fold.
template <int CPT, int NCL>
__device__ __forceinline__ void sweep_short(const float4* __restrict__ xs4, int n4, const u64 (&inv2)[CPT],
                                            const u64 (&na2)[CPT], float (&out)[CPT], float clo, float chi) {
    const u64 M2 = pack2(kMagic, kMagic);
    const u64 NM2 = pack2(-kMagic, -kMagic);
    u64 acc2[CPT];
#pragma unroll
    for (int s = 0; s < CPT; ++s) acc2[s] = 0ull;
#pragma unroll 1
    for (int i = 0; i < n4; ++i) {
        const float4 v = xs4[i];
        const u64 xa = pack2(v.x, v.y), xb = pack2(v.z, v.w);
#pragma unroll
        for (int s = 0; s < CPT; ++s) {
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
    for (int s = 0; s < CPT; ++s) {
        float p0, p1;
        unpack2(acc2[s], p0, p1);
        out[s] = p0 + p1;
    }
}

template <int CPT>
__device__ __forceinline__ void sweep_short_dispatch(int ncl, const float4* xs4, int n4, const u64 (&inv2)[CPT],
                                                     const u64 (&na2)[CPT], float (&out)[CPT], float clo, float chi) {
    if (ncl <= 0) {
        sweep_short<CPT, 0>(xs4, n4, inv2, na2, out, clo, chi);
    } else if (ncl == 1) {
        sweep_short<CPT, 1>(xs4, n4, inv2, na2, out, clo, chi);
    } else if (ncl == 2 && CPT > 2) {
        sweep_short<CPT, (CPT > 2 ? 2 : CPT)>(xs4, n4, inv2, na2, out, clo, chi);
    } else if (ncl <= CPT / 2 && CPT > 4) {
        sweep_short<CPT, CPT / 2>(xs4, n4, inv2, na2, out, clo, chi);
    } else {
        sweep_short<CPT, CPT>(xs4, n4, inv2, na2, out, clo, chi);
    }
}

// One row, one warp: argmin of the stored curve, re-score, polish, final codes, outputs.
// xr: the row in shared memory (k elements), cv: its error curve (n_cand floats).
// prev_x_last / prev_alpha: last element and final scale of the previous row when this row starts
// at an odd flat index (its first nibble shares a byte with that element); more: the next row will
// complete this row's last byte.
__device__ __forceinline__ float small_row_epilogue(const RowArgs& a, const RowTensor& T, const float* xr,
                                                    const float* cv, int k, const SmallRowParams& rp, long long row,
                                                    float prev_x_last, float prev_alpha, bool more,
                                                    unsigned int& st) {
    const int lane = threadIdx.x & 31;
    const float flo = (float)a.lo[0], fhi = (float)a.hi[0];
    const float thr = ambiguity_threshold(flo, fhi);
    struct { float step; } g = {rp.step};
    float alpha = 0.f;
    int best = -1;
    bool degenerate = (rp.flags & 2) != 0;
    const int n4 = (a.n_cand + 3) >> 2;          // the curve is padded with +Inf up to a multiple of 4
    if (!degenerate) {
        float bv = INFINITY;
        int bi = 0x7fffffff;
        const float4* cv4 = reinterpret_cast<const float4*>(cv);
        for (int j = lane; j < n4; j += 32) {    // ascending candidate index within a lane: strict < keeps the lowest
            const float4 v = cv4[j];
            if (v.x < bv) { bv = v.x; bi = 4 * j; }
            if (v.y < bv) { bv = v.y; bi = 4 * j + 1; }
            if (v.z < bv) { bv = v.z; bi = 4 * j + 2; }
            if (v.w < bv) { bv = v.w; bi = 4 * j + 3; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ov < bv || (ov == bv && oi < bi)) {
                bv = ov;
                bi = oi;
            }
        }
        if (bi == 0x7fffffff) {
            degenerate = true;   // every error Inf/NaN: non-finite input
        } else {
            best = bi;
            const float band = (float)((double)bv * (1.0 + kRescoreBand));
            int cnt = 0;
            for (int j = lane; j < n4; j += 32) {
                const float4 v = cv4[j];
                cnt += (v.x <= band) + (v.y <= band) + (v.z <= band) + (v.w <= band);
            }
            cnt = warp_allsum(cnt);
            if (cnt > 1) {   // every candidate in the band is re-scored, however many there are
                double best_sse = INFINITY;
                best = 0x7fffffff;
                for (int c0 = 0; c0 < a.n_cand; c0 += 32) {
                    const float v = (c0 + lane < a.n_cand) ? cv[c0 + lane] : INFINITY;
                    unsigned int mask = __ballot_sync(0xffffffffu, v <= band);
                    while (mask) {
                        const int c = c0 + __ffs(mask) - 1;
                        mask &= mask - 1;
                        const float ac = __fmul_rn((float)(c + 1), g.step);
                        const float inv = __fdiv_rn(1.0f, ac);
                        const double ad = (double)ac;
                        double ss = 0.0;
                        for (int i = lane; i < k; i += 32) {
                            const float x = xr[i];
                            const double d = fma(-ad, int_double(exact_code(x, ac, inv, flo, fhi, thr)), (double)x);
                            ss = fma(d, d, ss);
                        }
                        ss = warp_allsum(ss);
                        if (ss < best_sse || (ss == best_sse && c < best)) {
                            best_sse = ss;
                            best = c;
                        }
                    }
                }
            }
            alpha = __fmul_rn((float)(best + 1), g.step);
            for (int it = 0; it < a.refine_iters; ++it) {
                double sxq = 0.0;
                int sqq = 0;
                const float inv = __fdiv_rn(1.0f, alpha);
                for (int i = lane; i < k; i += 32) {
                    const float x = xr[i];
                    const int q = exact_code(x, alpha, inv, flo, fhi, thr);
                    sqq += q * q;
                    sxq = fma((double)x, int_double(q), sxq);
                }
                sxq = warp_allsum(sxq);
                sqq = warp_allsum(sqq);
                if (sqq == 0) break;
                const float a_new = (float)(sxq / (double)sqq);
                if (!(a_new >= FLT_MIN) || !(a_new <= FLT_MAX)) break;
                if (a_new == alpha) break;   // fixed point: further steps would repeat it exactly
                alpha = a_new;
            }
        }
    }
    if (degenerate) {
        st |= 2u;
        alpha = 0.f;
        best = -1;
    }

    // ---- final codes, squared error, emission
    const long long row_base = row * T.K;
    const bool zero = !(alpha > 0.f);
    const float inv_f = zero ? 0.f : __fdiv_rn(1.0f, alpha);
    const double ad = (double)alpha;
    double ss = 0.0;
    const bool aligned = ((reinterpret_cast<unsigned long long>(T.codes) & 3ull) == 0) &&
                         ((reinterpret_cast<unsigned long long>(T.packed) & 1ull) == 0);
    if ((k & 3) == 0 && aligned) {
        const float4* xr4 = reinterpret_cast<const float4*>(xr);
        for (int i4 = lane; i4 < (k >> 2); i4 += 32) {
            const float4 v = xr4[i4];
            const float x[4] = {v.x, v.y, v.z, v.w};
            int q[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                q[e] = zero ? 0 : exact_code(x[e], alpha, inv_f, flo, fhi, thr);
                const double d = fma(-ad, int_double(q[e]), (double)x[e]);
                ss = fma(d, d, ss);
            }
            if (T.codes) {
                const unsigned int w = (q[0] & 0xff) | ((q[1] & 0xff) << 8) | ((q[2] & 0xff) << 16) | ((unsigned)(q[3] & 0xff) << 24);
                *reinterpret_cast<unsigned int*>(T.codes + row_base + 4ll * i4) = w;
            }
            if (T.packed) {
                const unsigned short h = (unsigned short)((q[0] & 0xf) | ((q[1] & 0xf) << 4) | ((q[2] & 0xf) << 8) | ((q[3] & 0xf) << 12));
                *reinterpret_cast<unsigned short*>(T.packed + ((row_base + 4ll * i4) >> 1)) = h;
            }
        }
    } else {
        const int o = (int)(row_base & 1);
        const int n_pairs = (k + o + 1) >> 1;
        for (int p = lane; p < n_pairs; p += 32) {
            const int e0 = 2 * p - o, e1 = e0 + 1;
            int q0 = 0, q1 = 0;
            if (e0 >= 0) {
                const float x = xr[e0];
                q0 = zero ? 0 : code_of(x, alpha, flo, fhi);
                const double d = (double)x - (double)alpha * (double)q0;
                ss += d * d;
                if (T.codes) T.codes[row_base + e0] = (signed char)q0;
            } else {
                q0 = prev_alpha > 0.f ? code_of(prev_x_last, prev_alpha, flo, fhi) : 0;
            }
            const bool has1 = e1 < k;
            if (has1) {
                const float x = xr[e1];
                q1 = zero ? 0 : code_of(x, alpha, flo, fhi);
                const double d = (double)x - (double)alpha * (double)q1;
                ss += d * d;
                if (T.codes) T.codes[row_base + e1] = (signed char)q1;
            }
            if (T.packed && (has1 || !more))
                T.packed[(row_base + e0) >> 1] = (unsigned char)((q0 & 0xf) | ((q1 & 0xf) << 4));
        }
    }
    ss = warp_allsum(ss);
    if (lane == 0) {
        T.alpha[row] = alpha;
        T.sse[row] = (float)ss;
        if (T.best_idx) T.best_idx[row] = best;
    }
    return alpha;
}

// One work unit of the short-row path: rows [unit_local*B, +B) of tensor T.  Requires a single
// element group (blockDim.x == a.tg) and a single quantized tensor per row.
template <int CPT, bool EXT>
__device__ void small_unit(const RowArgs& a, const RowTensor& T, long long unit_local, unsigned char* smem_raw,
                           const float (&rcp)[CPT], unsigned int& st, unsigned long long& ev) {
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarp = nthr >> 5;
    const int k = (int)T.K, kpad = (k + 3) & ~3, k4 = kpad >> 2;
    const int B = T.rows_per_unit;
    const long long row0 = unit_local * B;
    const int nrows = (int)min((long long)B, T.S - row0);
    const int ncs = CPT * a.tg;
    const bool prune = (T.small & 2) != 0;       // rows regrouped by magnitude class before the sweep
    const int kb = kpad + 4 * CPT;               // floats of a regrouped row (every class padded to 4)
    float* xs = reinterpret_cast<float*>(smem_raw);
    float* curve = xs + B * kpad;
    SmallRowParams* rowp = reinterpret_cast<SmallRowParams*>(curve + B * ncs);
    double* skip = reinterpret_cast<double*>(rowp + B);            // [B][CPT]   (prune only)
    int* seg = reinterpret_cast<int*>(skip + B * CPT);              // [B][2*(CPT+1)]
    float* xb = reinterpret_cast<float*>(seg + B * 2 * (CPT + 1));  // [B][kb]
    const float flo = (float)a.lo[0], fhi = (float)a.hi[0];

    // ---- stage the rows (contiguous in HBM) into rows of kpad floats, zero padded
    const float* src = T.w + row0 * T.K;
    const int n_el = nrows * k;
    bool bad = false;
    if ((k & 3) == 0 && (reinterpret_cast<unsigned long long>(src) & 15ull) == 0) {
        const float4* src4 = reinterpret_cast<const float4*>(src);
        for (int i4 = tid; i4 < (n_el >> 2); i4 += nthr) {
            const float4 v = __ldg(src4 + i4);
            reinterpret_cast<float4*>(xs)[i4] = v;
            bad |= !(fabsf(v.x) <= FLT_MAX) || !(fabsf(v.y) <= FLT_MAX) || !(fabsf(v.z) <= FLT_MAX) || !(fabsf(v.w) <= FLT_MAX);
        }
    } else {
        for (int i = tid; i < n_el; i += nthr) {
            const int r = i / k, c = i - r * k;
            const float v = __ldg(src + i);
            xs[r * kpad + c] = v;
            bad |= !(fabsf(v) <= FLT_MAX);
        }
        const int npad = kpad - k;
        for (int i = tid; i < nrows * npad; i += nthr) {
            const int r = i / npad, c = k + (i - r * npad);
            xs[r * kpad + c] = 0.f;
        }
    }
    if (bad) st |= 1u;
    __syncthreads();
    if (EXT && T.prior_alpha) {
        // second quantized tensor of a key layer: every row becomes the residual of its first tensor
        for (int i = tid; i < nrows * kpad; i += nthr) {
            const int r = i / kpad, c = i - r * kpad;
            const float a1 = T.prior_alpha[row0 + r];
            if (c < k && a1 > 0.f) {
                const float x = xs[i];
                xs[i] = fmaf(-a1, (float)code_of(x, a1, flo, fhi), x);
            }
        }
        __syncthreads();
    }

    // ---- max of the positive and negative part of every row, and the row's grid: a warp per row
    for (int r = warp; r < nrows; r += nwarp) {
        if (T.delta) {   // quantization with offset: subtract the row minimum first
            float lo = INFINITY;
            for (int i = lane; i < k; i += 32) {
                const float v = xs[r * kpad + i];
                if (fabsf(v) <= FLT_MAX) lo = fminf(lo, v);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
            if (!(lo < INFINITY)) lo = 0.f;
            for (int i = lane; i < k; i += 32) xs[r * kpad + i] = xs[r * kpad + i] - lo;
            if (lane == 0) T.delta[row0 + r] = lo;
            __syncwarp();
        }
        float mp = 0.f, mn = 0.f;
        for (int i = lane; i < k; i += 32) {
            const float v = xs[r * kpad + i];
            if (fabsf(v) <= FLT_MAX) {
                mp = fmaxf(mp, v);
                mn = fmaxf(mn, -v);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            mp = fmaxf(mp, __shfl_xor_sync(0xffffffffu, mp, o));
            mn = fmaxf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        }
        if (lane == 0) {
            const GridSetup g = grid_setup(mp, mn, a.hi_frac, a.n_cand, flo, fhi);
            const float a_last = __fmul_rn((float)a.n_cand, g.step);
            SmallRowParams rp;
            rp.step = g.step;
            rp.rstep = g.rstep;
            rp.c_sat = g.c_sat;
            rp.flags = (g.tiny ? 1 : 0) | ((!(fmaxf(mp, mn) > 0.f) || !(a_last >= FLT_MIN)) ? 2 : 0);
            rowp[r] = rp;
        }
        if (prune) {
            // ---- regroup the row by magnitude class: the same counting sort as the long-row path, by one warp
            __syncwarp();
            const SmallRowParams rp = rowp[r];
            const bool plain = (rp.flags & 3) != 0;           // denormal-range or unusable row: one class, all slots
            const float inv_thr = rp.rstep * (1.0f / 0.4999f), inv_tg = 1.0f / (float)a.tg;
            const float* xr = xs + r * kpad;
            // lane l owns the elements l, l + 32, ...; within a class they keep the order (lane, then index)
            u64 c0 = 0ull, c1 = 0ull;
            double d[CPT + 1];
            d[0] = 0.0;
            for (int i = lane; i < k; i += 32) {
                const float x = xr[i];
                const int nb = plain ? CPT : magnitude_class<CPT>(x, inv_thr, inv_tg);
                const double xd = (double)x;
                d[0] = fma(nb == 0 ? xd : 0.0, xd, d[0]);
                if (nb >= 5) c1 += 1ull << (16 * (nb - 5));
                else if (nb >= 1) c0 += 1ull << (16 * (nb - 1));
            }
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
            u64 off0 = i0 - c0, off1 = i1 - c1;
            const u64 tot0 = __shfl_sync(0xffffffffu, i0, 31), tot1 = __shfl_sync(0xffffffffu, i1, 31);
            int base[CPT + 1], cnt[CPT + 1];
            int pos = 0;
            float* xbr = xb + r * kb;
#pragma unroll
            for (int b = CPT; b >= 1; --b) {
                cnt[b] = (int)(((b >= 5 ? tot1 : tot0) >> (16 * ((b - 1) & 3))) & 0xffffull);
                base[b] = pos;
                const int padded = (cnt[b] + 3) & ~3;
                if (lane == 0) {
                    seg[(r * (CPT + 1) + b) * 2] = pos;
                    seg[(r * (CPT + 1) + b) * 2 + 1] = padded;
                }
                if (lane < padded - cnt[b]) xbr[pos + cnt[b] + lane] = 0.f;
                pos += padded;
            }
            for (int i = lane; i < k; i += 32) {
                const float x = xr[i];
                const int nb = plain ? CPT : magnitude_class<CPT>(x, inv_thr, inv_tg);
                if (nb >= 1) {
                    const int sh = 16 * ((nb - 1) & 3);
                    int within;
                    if (nb >= 5) {
                        within = (int)((off1 >> sh) & 0xffffull);
                        off1 += 1ull << sh;
                    } else {
                        within = (int)((off0 >> sh) & 0xffffull);
                        off0 += 1ull << sh;
                    }
                    int bs = 0;
#pragma unroll
                    for (int b = 1; b <= CPT; ++b) bs = (nb == b) ? base[b] : bs;
                    xbr[bs + within] = x;
                }
            }
            __syncwarp();
            // squared sums of classes 1.. from the regrouped row (class 0 was summed on the way)
#pragma unroll
            for (int b = 1; b <= CPT; ++b) {
                double v = 0.0;
                for (int i = lane; i < cnt[b]; i += 32) {
                    const double xd = (double)xbr[base[b] + i];
                    v = fma(xd, xd, v);
                }
                d[b] = v;
            }
            double run = 0.0;                                   // slot sl skips classes 0..sl
#pragma unroll
            for (int b = 0; b < CPT; ++b) {
                run += warp_allsum(d[b]);
                if (lane == 0) skip[r * CPT + b] = run;
            }
        }
    }
    __syncthreads();

    // ---- candidate sweep, row after row, by the whole block; error curves to shared memory
    const bool short_rows = k4 <= kFlushEvery4;       // one fp32 block per candidate: no fp64 fold needed
    bool in_range[CPT];
#pragma unroll
    for (int sl = 0; sl < CPT; ++sl) in_range[sl] = sl * a.tg + tid < a.n_cand;
    for (int r = 0; r < nrows; ++r) {
        const SmallRowParams rp = rowp[r];
        if (rp.flags & 2) continue;   // no usable scale: the epilogue reports it
        u64 inv2[CPT], na2[CPT];
        bool ok[CPT];
#pragma unroll
        for (int sl = 0; sl < CPT; ++sl) {
            const float cf = (float)(sl * a.tg + tid + 1);
            const float ac = __fmul_rn(cf, rp.step);
            float inv = rcp[sl] * rp.rstep;
            ok[sl] = in_range[sl];
            if (rp.flags & 1) {       // denormal-range row: exact reciprocal, per-candidate validity
                inv = __fdiv_rn(1.0f, ac);
                ok[sl] = ok[sl] && (ac >= FLT_MIN);
            }
            if (!ok[sl]) inv = 0.f;
            inv2[sl] = pack2(inv, inv);
            na2[sl] = pack2(-ac, -ac);
        }
        int ncl = (rp.c_sat - (tid & ~31) + a.tg - 1) / a.tg;
        ncl = max(0, min(CPT, ncl));
        const float4* xr4 = reinterpret_cast<const float4*>(xs) + r * k4;
        float* cvr = curve + r * ncs;
        if (prune) {
            // class nb is evaluated by slots 0..nb-1; fp32 pair sums are kept across classes and folded
            // into fp64 every kFlushEvery4 loads
            const float4* xb4 = reinterpret_cast<const float4*>(xb + r * kb);
            u64 acc2[CPT];
            double dacc[CPT];
#pragma unroll
            for (int sl = 0; sl < CPT; ++sl) {
                acc2[sl] = 0ull;
                dacc[sl] = 0.0;
            }
            int pending = 0;
            for (int b = CPT; b >= 1; --b) {
                int i = seg[(r * (CPT + 1) + b) * 2] >> 2;
                const int stop = i + (seg[(r * (CPT + 1) + b) * 2 + 1] >> 2);
                int ncl_b = (class_sat_count(b, CPT, a.tg, rp.c_sat, flo, fhi) - (tid & ~31) + a.tg - 1) / a.tg;
                ncl_b = max(0, min(CPT, ncl_b));
                while (i < stop) {
                    const int n = min(stop - i, kFlushEvery4 - pending);
                    sweep_accum_dispatch<CPT>(b, ncl_b, xb4, i, i + n, inv2, na2, acc2, kMagic + flo, kMagic + fhi);
                    ev += (unsigned long long)n * 4ull * (unsigned long long)b;
                    i += n;
                    pending += n;
                    if (pending == kFlushEvery4) {
#pragma unroll
                        for (int sl = 0; sl < CPT; ++sl) {
                            float p0, p1;
                            unpack2(acc2[sl], p0, p1);
                            dacc[sl] += (double)(p0 + p1);
                            acc2[sl] = 0ull;
                        }
                        pending = 0;
                    }
                }
            }
#pragma unroll
            for (int sl = 0; sl < CPT; ++sl) {
                float p0, p1;
                unpack2(acc2[sl], p0, p1);
                const double v = dacc[sl] + (double)(p0 + p1) + skip[r * CPT + sl];
                cvr[sl * a.tg + tid] = ok[sl] ? (float)v : INFINITY;
            }
        } else if (short_rows) {
            ev += (unsigned long long)k4 * 4ull * CPT;
            float out[CPT];
            sweep_short_dispatch<CPT>(ncl, xr4, k4, inv2, na2, out, kMagic + flo, kMagic + fhi);
#pragma unroll
            for (int sl = 0; sl < CPT; ++sl) cvr[sl * a.tg + tid] = ok[sl] ? out[sl] : INFINITY;
        } else {
            double dacc[CPT];
#pragma unroll
            for (int sl = 0; sl < CPT; ++sl) dacc[sl] = 0.0;
            sweep_dispatch<CPT>(ncl, xr4, 0, k4, inv2, na2, dacc, kMagic + flo, kMagic + fhi);
            ev += (unsigned long long)k4 * 4ull * CPT;
#pragma unroll
            for (int sl = 0; sl < CPT; ++sl) cvr[sl * a.tg + tid] = ok[sl] ? (float)dacc[sl] : INFINITY;
        }
    }
    __syncthreads();

    // ---- a warp finishes each row; two consecutive rows stay in one warp when a packed byte can
    //      straddle them (odd row length)
    const int rpt = (T.packed && (k & 1)) ? 2 : 1;
    for (int task = warp; task * rpt < nrows; task += nwarp) {
        float prev_alpha = 0.f;
        for (int rr = 0; rr < rpt; ++rr) {
            const int r = task * rpt + rr;
            if (r >= nrows) break;
            const bool more = (rr + 1 < rpt) && (r + 1 < nrows);
            const float prev_x_last = r > 0 ? xs[(r - 1) * kpad + k - 1] : 0.f;
            prev_alpha = small_row_epilogue(a, T, xs + r * kpad, curve + r * ncs, k, rowp[r], row0 + r, prev_x_last,
                                            prev_alpha, more, st);
        }
    }
}

}  // namespace omse
