// Per-tensor MMSE scale (Section 3.7, first equation): one scale for a whole activation tensor.
// The tensor does not fit on chip, so the search is a short pipeline of grid-wide kernels ordered
// by the stream (no kernel waits on another block):
//   absmax -> sweep (tiles through shared memory, partial error sums per block) -> finish (sum the
//   partials in fixed order, argmin, near-minimal list) -> rescore (fp64, true division) ->
//   refine x R (<x,q>, <q,q>) -> final (error at the final scale).
// Grid-wide sums use "the last block to arrive reduces" (a ticket from atomicAdd, no waiting).
#pragma once
#include "omse_device.cuh"

namespace omse {

struct TensorState {          // lives in the context workspace
    unsigned int mpos_bits, mneg_bits;   // max of positive / negative part as float bits (atomicMax)
    unsigned int ticket;                 // arrivals for last-block reductions (reset by the last block)
    int best_idx;
    float alpha;
    float step;
    int n_list;                      // candidates to re-score in fp64 (0: the fp32 winner is the only one in the band)
    int list_overflow;               // (unused)
    int polish_done;                 // set when a polish step stops or reaches a fixed point: later steps return at once
    int key_min, key_max;                // offset mode: order-preserving integer keys of min and max of the tensor
    float delta;                         // offset subtracted from every element (0 without offset)
};

constexpr int kTileListCap = 32;   // flagged tiles one block of the second sweep launch lists for itself (static shared
                                   // memory of that kernel must stay below the 1 KB left beside the dynamic maximum)

struct TensorArgs {
    const float* x;
    long long n;
    int n_cand;
    float hi_frac;
    int lo, hi;
    int tg, groups;         // sweep block = groups*tg threads; candidate c = c_base + slot*tg + t
    int c_base, c_count;    // candidates [c_base, c_base + c_count) are swept by this launch
    int tile4;              // float4s per tile
    // Tile flags between the two sweep launches (all nullable / 0): the first launch sets bit t when tile t (of
    // flag_tile4 float4s) holds a value that reaches the second launch's first candidate, and leaves the squared sum
    // of everything each of its blocks staged in block_totals; the second launch then reads only flagged tiles.
    unsigned int* tile_flags;
    int flag_words;         // words of tile_flags (the absmax kernel clears them)
    int flag_tile4;
    int flag_role;          // 1: this launch sets the flags, 2: this launch uses them
    float flag_split;       // role 1: a value with |x|/(0.4999*step) above this reaches the second launch
    double* block_totals;   // role 1: [gridDim.x] written; role 2: n_totals entries read
    int n_totals;
    TensorState* st;
    double* partials;       // sweep: [grid][n_cand]; passes: [blocks][listed candidates] doubles + [blocks] int64
    long long partial_doubles;   // capacity of `partials`
    int* list;              // [n_cand] candidates inside the fp32 noise band of the minimum (workspace)
    double* curve;          // [n_cand] summed error per candidate (workspace)
    double* curve_out;      // user copy, nullable
    float* alpha_out;
    float* sse_out;
    int* idx_out;
    float* delta_out;       // offset mode: receives delta; nullptr = no offset
    unsigned long long* evals;   // executed (element, candidate) evaluations (instrumentation), nullable
    unsigned int* status;
};

__global__ void tensor_init_kernel(TensorState* st) {
    if (threadIdx.x == 0) {
        st->mpos_bits = 0u;
        st->mneg_bits = 0u;
        st->ticket = 0u;
        st->best_idx = -1;
        st->alpha = 0.f;
        st->step = 0.f;
        st->n_list = 0;
        st->list_overflow = 0;
        st->polish_done = 0;
        st->key_min = 0x7fffffff;
        st->key_max = (int)0x80000000;
        st->delta = 0.f;
    }
}

// order-preserving map float -> int (finite values)
__device__ __forceinline__ int float_key(float f) {
    const int i = __float_as_int(f);
    return i >= 0 ? i : i ^ 0x7fffffff;
}
__device__ __forceinline__ float key_float(int k) { return __int_as_float(k >= 0 ? k : k ^ 0x7fffffff); }

// Offset mode (Section 3.1 scheme with offset): delta = min, and the search range is that of the shifted tensor.
__global__ void tensor_offset_kernel(TensorState* st) {
    if (threadIdx.x == 0 && st->key_min <= st->key_max) {
        const float lo = key_float(st->key_min), hi = key_float(st->key_max);
        st->delta = lo;
        st->mpos_bits = __float_as_uint(hi - lo);    // max of fl(x - delta): subtraction is monotone
        st->mneg_bits = 0u;
    }
}

__global__ void __launch_bounds__(256) tensor_absmax_kernel(const float* __restrict__ x, long long n,
                                                             TensorState* st, unsigned int* status,
                                                             unsigned int* tile_flags, int flag_words) {
    __shared__ double scratch[64];
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < flag_words; i += gridDim.x * blockDim.x) tile_flags[i] = 0u;
    float lo = INFINITY, hi = -INFINITY;          // extremes of the finite values this thread saw
    bool bad = false;
    const long long n4 = n >> 2;
    const float4* x4 = reinterpret_cast<const float4*>(x);
    const long long stride = (long long)gridDim.x * blockDim.x;
    auto one = [&](float e) {
        const bool finite = fabsf(e) <= FLT_MAX;
        bad |= !finite;
        lo = fminf(lo, finite ? e : lo);
        hi = fmaxf(hi, finite ? e : hi);
    };
    auto four = [&](const float4& v) {
        one(v.x);
        one(v.y);
        one(v.z);
        one(v.w);
    };
    // four 128-bit loads in flight per thread before any of them is used
    long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    for (; i + 3 * stride < n4; i += 4 * stride) {
        const float4 v0 = __ldg(x4 + i), v1 = __ldg(x4 + i + stride), v2 = __ldg(x4 + i + 2 * stride),
                     v3 = __ldg(x4 + i + 3 * stride);
        four(v0);
        four(v1);
        four(v2);
        four(v3);
    }
    for (; i < n4; i += stride) four(__ldg(x4 + i));
    for (long long e = (n4 << 2) + (long long)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += stride) one(x[e]);
    // maxima of the positive and of the negative part follow from the extremes (both 0 when nothing finite was seen)
    float mpos = fmaxf(hi, 0.f), mneg = fmaxf(-lo, 0.f);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
        hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    if ((threadIdx.x & 31) == 0 && lo <= hi) {   // the warp saw a finite value: integer atomics on order-preserving keys
        atomicMin(&st->key_min, float_key(lo));
        atomicMax(&st->key_max, float_key(hi));
    }
    block_max2(mpos, mneg, scratch);
    if (threadIdx.x == 0) {
        atomicMax(&st->mpos_bits, __float_as_uint(mpos));   // non-negative floats order like their bits
        atomicMax(&st->mneg_bits, __float_as_uint(mneg));
    }
    if (bad) atomicOr(status, 1u);
}

// Candidate sweep over tiles of the tensor; block b handles tiles b, b+grid, ...; one launch covers the candidates
// [c_base, c_base + c_count).  While a tile is staged its elements are regrouped by magnitude class (see
// magnitude_class): class nb is evaluated by candidate slots 0..nb-1 only, class 0 (|x| <= 0.4999*alpha of the
// launch's first candidate; in particular the exact zeros of a post-ReLU tensor) by none; every slot adds the
// squared sum of the classes it skipped.  The regrouping is a deterministic block-wide counting sort, so results do
// not depend on scheduling.  The host covers the grid with two launches when it has more than 256 candidates: the
// first 256 with 32 candidates per slot (most elements of a heavy-tailed tensor are small against max|x| and
// matter only to the smallest scales, so the fine classes there prune the most), the rest with wider slots.
template <int CPT>
__global__ void __launch_bounds__(512) tensor_sweep_kernel(const TensorArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ u64 warp_tot[16][2];
    __shared__ double dscratch[64];
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarp = nthr >> 5;
    // A group of 32 threads is one warp: it then regroups and sweeps its own share of every tile by itself (no block
    // barrier inside the tile loop).  Wider groups share the whole tile and regroup it together.
    const bool solo = false;   // launches with 32-candidate slots use tensor_sweep_fine_kernel
    const int region = solo ? 4 * (a.tile4 / nwarp) + 4 * CPT : 4 * a.tile4 + 4 * CPT;   // floats of a regrouped tile (share)
    float* tile = reinterpret_cast<float*>(smem_raw) + (solo ? warp * region : 0);
    float4* raw4 = reinterpret_cast<float4*>(reinterpret_cast<float*>(smem_raw) + (solo ? nwarp * region : region));   // [tile4] landing zone of the asynchronous copies
    double* xg = reinterpret_cast<double*>(raw4);    // partial sums of the other groups (after the last tile)
    const int grp = tid / a.tg, t = tid - grp * a.tg;
    const float mpos = __uint_as_float(a.st->mpos_bits), mneg = __uint_as_float(a.st->mneg_bits);
    const float m = fmaxf(mpos, mneg);
    const float flo = (float)a.lo, fhi = (float)a.hi;
    const GridSetup g = grid_setup(mpos, mneg, a.hi_frac, a.n_cand, flo, fhi);
    const float a_last = __fmul_rn((float)a.n_cand, g.step);
    if (!(m > 0.f) || !(a_last >= FLT_MIN)) return;   // degenerate tensor: finish kernel reports it
    const float inv_thr = g.rstep * (1.0f / 0.4999f);
    const float inv_tg = 1.0f / (float)a.tg;
    const float cbase_f = (float)a.c_base;
    const float delta = a.st->delta;                  // 0 unless the offset scheme is used

    u64 inv2[CPT], na2[CPT];
    double dacc[CPT];
#pragma unroll
    for (int sl = 0; sl < CPT; ++sl) {
        const int cl = sl * a.tg + t, c = a.c_base + cl;
        const float ac = __fmul_rn((float)(c + 1), g.step);
        float inv = g.tiny ? __fdiv_rn(1.0f, ac) : __fdiv_rn(1.0f, (float)(c + 1)) * g.rstep;
        if (!(ac >= FLT_MIN) || cl >= a.c_count) inv = 0.f;
        inv2[sl] = pack2(inv, inv);
        na2[sl] = pack2(-ac, -ac);
        dacc[sl] = 0.0;
    }
    const int warp_t0 = t & ~31;

    const long long n4_total = (a.n + 3) >> 2;
    const long long n4_full = a.n >> 2;               // float4s that lie completely inside the tensor
    const long long n_tiles = (n4_total + a.tile4 - 1) / a.tile4;
    const float4* x4 = reinterpret_cast<const float4*>(a.x);
    const int per_thread4 = a.tile4 / nthr;          // consecutive float4s staged by one thread (<= 4)
    unsigned long long ev = 0ull;                    // evaluations this thread executed
    double sq[CPT + 1];                              // squared sums per class over this block's tiles (this thread's share)
#pragma unroll
    for (int b = 0; b <= CPT; ++b) sq[b] = 0.0;

    // Asynchronous copy of this thread's float4s of tile tl into their landing slots; a thread only ever reads the
    // slots it filled itself, so the copies need no barrier, and they run while the previous tile is processed.
    auto prefetch = [&](long long tl) {
        const long long base4 = tl * a.tile4;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int i = tid * per_thread4 + j;
            if (j < per_thread4 && base4 + i < n4_full) {
                const unsigned int dst = (unsigned int)__cvta_generic_to_shared(raw4 + i);
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(x4 + base4 + i) : "memory");
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    // With tile flags from the first launch only the tiles that hold a value for this launch are read at all (a flag
    // tile is a tile of this launch).  The flagged tiles are dealt out evenly: the tile of rank r among the set bits
    // goes to block r mod gridDim.x, listed once per block by its first warp (fixed order).  When more than half of
    // the tiles are flagged (the strided sequences are then even enough) or more than the lists hold, every block
    // walks its strided sequence and skips the unflagged tiles instead.
    const bool flagged_only = a.flag_role == 2 && a.tile_flags != nullptr;
    __shared__ int s_tiles[kTileListCap];
    __shared__ int s_n_mine;
    if (flagged_only) {
        if (warp == 0) {
            int total = 0;
            for (int wi = lane; wi < a.flag_words; wi += 32) total += __popc(__ldg(a.tile_flags + wi));
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
            int n_mine = -1;
            if ((long long)total <= (long long)kTileListCap * gridDim.x && 2ll * total <= n_tiles) {
                n_mine = 0;
                int running = 0;                      // set bits in the words before this group of 32
                for (int w0 = 0; w0 < a.flag_words; w0 += 32) {
                    const int wi = w0 + lane;
                    const unsigned int word = wi < a.flag_words ? __ldg(a.tile_flags + wi) : 0u;
                    const int cnt = __popc(word);
                    int incl = cnt;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const int u = __shfl_up_sync(0xffffffffu, incl, o);
                        if (lane >= o) incl += u;
                    }
                    int r = running + incl - cnt;     // rank of this word's first set bit
                    unsigned int mine = 0u;
                    for (unsigned int m2 = word; m2; m2 &= m2 - 1, ++r)
                        if (r % (int)gridDim.x == (int)blockIdx.x) mine |= m2 & (0u - m2);
                    const int mcnt = __popc(mine);
                    int mincl = mcnt;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const int u = __shfl_up_sync(0xffffffffu, mincl, o);
                        if (lane >= o) mincl += u;
                    }
                    int pos = n_mine + mincl - mcnt;
                    for (unsigned int m2 = mine; m2; m2 &= m2 - 1) s_tiles[pos++] = wi * 32 + (__ffs(m2) - 1);
                    n_mine += __shfl_sync(0xffffffffu, mincl, 31);
                    running += __shfl_sync(0xffffffffu, incl, 31);
                }
            }
            if (lane == 0) s_n_mine = n_mine;
        }
        __syncthreads();
    }
    const int n_mine = flagged_only ? s_n_mine : -1;   // >= 0: this block's tiles are s_tiles[0 .. n_mine)
    auto next_tile = [&](long long tl) {             // first tile >= tl of this block's strided sequence that has to be read
        if (!flagged_only) return tl;
        for (; tl < n_tiles; tl += gridDim.x)
            if ((__ldg(a.tile_flags + (tl >> 5)) >> (tl & 31)) & 1u) break;
        return tl;
    };
    int sidx = 0;
    long long tl = n_mine >= 0 ? (n_mine > 0 ? (long long)s_tiles[0] : n_tiles) : next_tile(blockIdx.x);
    if (tl < n_tiles) prefetch(tl);
    while (tl < n_tiles) {
        const long long base4 = tl * a.tile4;
        ++sidx;
        const long long tl_next = n_mine >= 0 ? (sidx < n_mine ? (long long)s_tiles[sidx] : n_tiles) : next_tile(tl + gridDim.x);
        asm volatile("cp.async.wait_all;" ::: "memory");
        // ---- this thread's span into registers (elements past the end count as zeros)
        float vals[16];
        bool big = false;                            // some value reaches this launch's first candidate
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float4 v = make_float4(delta, delta, delta, delta);
            const int i = tid * per_thread4 + j;
            if (j < per_thread4) {
                if (base4 + i < n4_full) {
                    v = raw4[i];
                } else {
                    const long long e = (base4 + i) << 2;
                    if (e < a.n) v.x = a.x[e];
                    if (e + 1 < a.n) v.y = a.x[e + 1];
                    if (e + 2 < a.n) v.z = a.x[e + 2];
                }
            }
            vals[4 * j] = v.x - delta;
            vals[4 * j + 1] = v.y - delta;
            vals[4 * j + 2] = v.z - delta;
            vals[4 * j + 3] = v.w - delta;
        }
        tl = tl_next;
        if (tl < n_tiles) prefetch(tl);              // the slots are free again: next tile on its way
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            const float x = vals[e];
            big |= !(fabsf(x) * inv_thr - cbase_f <= 1.0f) || (g.tiny && x != 0.f);
        }
        // previous tile fully swept (tile and warp_tot free).  If nothing of this tile (share) reaches the first
        // candidate, every slot skips all of it.
        const bool any = solo ? __any_sync(0xffffffffu, big) : (__syncthreads_or(big) != 0);
        if (!any) {
            double z = 0.0;
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                const double xd = (double)vals[e];
                z = fma(xd, xd, z);
            }
            sq[0] += z;
            continue;
        }
        // ---- classify, count
        u64 cls = 0ull, c0 = 0ull, c1 = 0ull;        // 4-bit class per value; counts in 16-bit fields
        double zero_sq = 0.0;
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            const float x = vals[e];
            int nb = magnitude_class<CPT>(x, inv_thr, inv_tg, cbase_f);
            if (g.tiny && x != 0.f) nb = CPT;
            cls |= (u64)nb << (4 * e);
            const double xd = (double)x;
            zero_sq = fma(nb == 0 ? xd : 0.0, xd, zero_sq);
            if (nb >= 5) c1 += 1ull << (16 * (nb - 5));
            else if (nb >= 1) c0 += 1ull << (16 * (nb - 1));
        }
        sq[0] += zero_sq;
        // ---- exclusive scan of the class counts (lanes by shuffle; warps in order when the block shares the tile)
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
        u64 off0 = i0 - c0, off1 = i1 - c1, tot0, tot1;
        if (solo) {
            tot0 = __shfl_sync(0xffffffffu, i0, 31);
            tot1 = __shfl_sync(0xffffffffu, i1, 31);
        } else {
            if (lane == 31) {
                warp_tot[warp][0] = i0;
                warp_tot[warp][1] = i1;
            }
            __syncthreads();
            tot0 = 0ull;
            tot1 = 0ull;
            for (int w = 0; w < nwarp; ++w) {
                const u64 a0 = warp_tot[w][0], a1 = warp_tot[w][1];
                if (w < warp) {
                    off0 += a0;
                    off1 += a1;
                }
                tot0 += a0;
                tot1 += a1;
            }
        }
        // ---- class layout in the tile buffer: class CPT first, each padded with zeros to a multiple of 4
        const int who = solo ? lane : tid;
        int base[CPT + 1], cnt[CPT + 1];
        int pos = 0;
#pragma unroll
        for (int b = CPT; b >= 1; --b) {
            cnt[b] = (int)(((b >= 5 ? tot1 : tot0) >> (16 * ((b - 1) & 3))) & 0xffffull);
            base[b] = pos;
            const int padded = (cnt[b] + 3) & ~3;
            if (who < padded - cnt[b]) tile[pos + cnt[b] + who] = 0.f;
            pos += padded;
        }
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            const int nb = (int)((cls >> (4 * e)) & 0xfull);
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
                tile[bs + within] = vals[e];
            }
        }
        if (solo) __syncwarp();
        else __syncthreads();
        const float4* tile4p = reinterpret_cast<const float4*>(tile);
        const int n_share = solo ? 32 : nthr;
#pragma unroll 1
        for (int b = CPT; b >= 1; --b) {
            if (cnt[b] == 0) continue;
            // squared sum of the class (what the slots that skip it add), from the regrouped tile
            for (int i = who; i < cnt[b]; i += n_share) {
                const double xd = (double)tile[base[b] + i];
                sq[b] = fma(xd, xd, sq[b]);
            }
            const int first4 = base[b] >> 2, len4 = (cnt[b] + 3) >> 2;
            const int beg4 = solo ? first4 : first4 + (int)(((long long)len4 * grp) / a.groups);
            const int end4 = solo ? first4 + len4 : first4 + (int)(((long long)len4 * (grp + 1)) / a.groups);
            int ncl_b = (class_sat_count(b, CPT, a.tg, g.c_sat, flo, fhi, a.c_base) - (a.c_base + warp_t0) + a.tg - 1) / a.tg;
            ncl_b = max(0, min(CPT, ncl_b));
            sweep_dispatch<CPT>(b, ncl_b, tile4p, beg4, end4, inv2, na2, dacc, kMagic + flo, kMagic + fhi);
            ev += (unsigned long long)(end4 - beg4) * 4ull * (unsigned long long)b;
        }
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    if (a.groups > 1) {
        __syncthreads();
        if (grp > 0) {
#pragma unroll
            for (int sl = 0; sl < CPT; ++sl) xg[((grp - 1) * CPT + sl) * a.tg + t] = dacc[sl];
        }
        __syncthreads();
        if (grp == 0) {
            for (int gg = 1; gg < a.groups; ++gg)
#pragma unroll
                for (int sl = 0; sl < CPT; ++sl) dacc[sl] += xg[((gg - 1) * CPT + sl) * a.tg + t];
        }
    }
    report_evaluations(a.evals, ev);
    // ---- what each slot skipped (block sums in fixed order)
    long long zero = 0;
    if (flagged_only) {
        // Not every element passed through this launch, so the skipped sums are taken from the other side: the squared
        // sum of the whole tensor (left by the first launch, added once, by block 0) less the classes a slot did sweep.
        double bs[CPT + 1];
#pragma unroll
        for (int b = 1; b <= CPT; ++b) {
            bs[b] = sq[b];
            block_sum2(bs[b], zero, dscratch);
        }
        double total = 0.0;
        if (blockIdx.x == 0)
            for (int i = 0; i < a.n_totals; ++i) total += __ldcg(a.block_totals + i);
        double above = 0.0;
#pragma unroll
        for (int sl = CPT - 1; sl >= 0; --sl) {
            above += bs[sl + 1];
            dacc[sl] += total - above;   // slot sl sweeps the classes above sl
        }
    } else {
        double run = 0.0;
#pragma unroll
        for (int b = 0; b < CPT; ++b) {
            double v = sq[b];
            block_sum2(v, zero, dscratch);
            run += v;
            dacc[b] += run;          // slot b skips classes 0..b
        }
    }
    if (grp == 0) {
#pragma unroll
        for (int sl = 0; sl < CPT; ++sl) {
            const int cl = sl * a.tg + t;
            if (cl < a.c_count) a.partials[(long long)blockIdx.x * a.n_cand + a.c_base + cl] = dacc[sl];
        }
    }
}

// The same sweep for launches whose slots hold 32 candidates (a warp is an element group of its own): every warp
// keeps its own share of a tile (the float4s its lanes copied) and never waits for the block.  The elements are
// split three ways in a fixed order (a warp scan of the per-lane counts): dropped (coded 0 by every candidate of the launch), "first slot
// only" (by far the most for a tensor with many small values) and the rest, which all slots evaluate; the two lists
// grow from the two ends of the warp's region.  Slot 0 adds the squared sum of the dropped elements, the other slots
// that of the dropped and of the first-slot-only elements.
template <int CPT>
__global__ void __launch_bounds__(256) tensor_sweep_fine_kernel(const TensorArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ double dscratch[64];
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarp = nthr >> 5;
    const int share = 16 * 32;                       // elements of a tile that one warp stages
    const int region = share + 8;                    // + zero padding of the two lists
    float* reg = reinterpret_cast<float*>(smem_raw) + warp * region;
    float4* raw4 = reinterpret_cast<float4*>(reinterpret_cast<float*>(smem_raw) + nwarp * region);   // [tile4] landing zone
    double* xg = reinterpret_cast<double*>(raw4);    // partial sums of the other warps (after the last tile)
    const float mpos = __uint_as_float(a.st->mpos_bits), mneg = __uint_as_float(a.st->mneg_bits);
    const float m = fmaxf(mpos, mneg);
    const float flo = (float)a.lo, fhi = (float)a.hi;
    const GridSetup g = grid_setup(mpos, mneg, a.hi_frac, a.n_cand, flo, fhi);
    const float a_last = __fmul_rn((float)a.n_cand, g.step);
    if (!(m > 0.f) || !(a_last >= FLT_MIN)) return;   // degenerate tensor: finish kernel reports it
    const float inv_thr = g.rstep * (1.0f / 0.4999f);
    const float cbase_f = (float)a.c_base;
    const float delta = a.st->delta;

    u64 inv2[CPT], na2[CPT];
    double dacc[CPT];
#pragma unroll
    for (int sl = 0; sl < CPT; ++sl) {
        const int cl = sl * 32 + lane, c = a.c_base + cl;
        const float ac = __fmul_rn((float)(c + 1), g.step);
        float inv = g.tiny ? __fdiv_rn(1.0f, ac) : __fdiv_rn(1.0f, (float)(c + 1)) * g.rstep;
        if (!(ac >= FLT_MIN) || cl >= a.c_count) inv = 0.f;
        inv2[sl] = pack2(inv, inv);
        na2[sl] = pack2(-ac, -ac);
        dacc[sl] = 0.0;
    }
    // Saturation.  The first-slot-only list holds no value that any candidate of the launch could saturate (such values
    // go to the rest), so its sweep needs no clamps at all: x*inv_c stays below hi + 1/2 (above lo - 1/2) for every
    // c >= c_base once |x| is below the bound of its sign; 1e-5 covers the rounding of inv_c and alpha_c.  A negative
    // value on a grid that starts at 0 is coded 0 by every scale: it is dropped whatever its size.
    const float a_first = __fmul_rn((float)(a.c_base + 1), g.step);
    const float pos_bound = (fhi + 0.5f) * a_first * 0.99999f, neg_bound = (0.5f - flo) * a_first * 0.99999f;
    const bool neg_free = flo == 0.f;
    int ncl_rest = (g.c_sat - a.c_base + 31) / 32;
    ncl_rest = max(0, min(CPT, ncl_rest));

    const long long n4_total = (a.n + 3) >> 2;
    const long long n4_full = a.n >> 2;
    const long long n_tiles = (n4_total + a.tile4 - 1) / a.tile4;
    const float4* x4 = reinterpret_cast<const float4*>(a.x);
    // |x| * thr_scale counts candidates; with a denormal step every value goes to all slots (Inf, or NaN for 0)
    const float thr_scale = g.tiny ? INFINITY : inv_thr;
    const bool flagging = a.flag_role == 1 && a.tile_flags != nullptr;
    const float flag_split = flagging ? a.flag_split : INFINITY;
    unsigned long long ev = 0ull;
    double sq_all = 0.0, sq1 = 0.0, sq2 = 0.0;       // squared sums: everything staged / first-slot-only / rest

    auto prefetch = [&](long long tl) {
        const long long base4 = tl * a.tile4;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int i = tid * 4 + j;
            if (base4 + i < n4_full) {
                const unsigned int dst = (unsigned int)__cvta_generic_to_shared(raw4 + i);
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(x4 + base4 + i) : "memory");
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    long long tl = blockIdx.x;
    if (tl < n_tiles) prefetch(tl);
    for (; tl < n_tiles; tl += gridDim.x) {
        const long long base4 = tl * a.tile4;
        asm volatile("cp.async.wait_all;" ::: "memory");
        float vals[16];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float4 v = make_float4(delta, delta, delta, delta);
            const int i = tid * 4 + j;
            if (base4 + i < n4_full) {
                v = raw4[i];
            } else {
                const long long e = (base4 + i) << 2;
                if (e < a.n) v.x = a.x[e];
                if (e + 1 < a.n) v.y = a.x[e + 1];
                if (e + 2 < a.n) v.z = a.x[e + 2];
            }
            vals[4 * j] = v.x - delta;
            vals[4 * j + 1] = v.y - delta;
            vals[4 * j + 2] = v.z - delta;
            vals[4 * j + 3] = v.w - delta;
        }
        if (tl + gridDim.x < n_tiles) prefetch(tl + gridDim.x);   // the slots are free again: next tile on its way
        // ---- three-way split: bit e of `first` / `rest` says where value e goes
        unsigned int first = 0u, rest = 0u;
        double tot = 0.0;                             // squared sum of everything this thread staged
        bool far = false;                             // a value that reaches the second sweep launch
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            const float x = vals[e];
            const float r = fabsf(x) * thr_scale - cbase_f;        // NaN for non-finite values: they go to the rest
            const bool needed = !(r <= 1.0f) && !(neg_free && x < 0.f);
            const bool may_sat = !(fabsf(x) < (x < 0.f ? neg_bound : pos_bound));
            const bool wide = needed && ((CPT > 1 && !(r <= 33.0f)) || may_sat);   // slot 1 needs x iff r > 32 + 1
            far |= !(r <= flag_split);
            first |= (needed && !wide ? 1u : 0u) << e;
            rest |= (wide ? 1u : 0u) << e;
            const double xd = (double)x;
            tot = fma(xd, xd, tot);
        }
        sq_all += tot;
        if (flagging && __any_sync(0xffffffffu, far) && lane == 0) {
            // a flag tile is a tile of the second launch: a multiple of 128 float4s, so a warp's 128 float4s lie in one
            const long long ft = (base4 + warp * 128) / a.flag_tile4;
            atomicOr(a.tile_flags + (ft >> 5), 1u << (ft & 31));
        }
        __syncwarp();                                 // the warp is done sweeping its previous share
        if (!__any_sync(0xffffffffu, (first | rest) != 0u)) continue;
        // ---- the two lists, thread-major (lane 0's values first): offsets from a warp scan of the counts
        const int packed = __popc(first) | (__popc(rest) << 16);
        int incl = packed;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int u = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += u;
        }
        const int totals = __shfl_sync(0xffffffffu, incl, 31);
        const int n1 = totals & 0xffff, n2 = totals >> 16;
        int o1 = (incl - packed) & 0xffff;                        // first list grows upwards from 0
        int o2 = region - 1 - ((incl - packed) >> 16);            // rest list grows downwards from the end
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            if ((first >> e) & 1u) reg[o1++] = vals[e];
        }
        if (n2 > 0) {
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                if ((rest >> e) & 1u) reg[o2--] = vals[e];
            }
        }
        // zero padding: the first list up to a multiple of 4, the rest list down to one
        const int n1p = (n1 + 3) & ~3, n2p = (n2 + 3) & ~3;
        if (lane < n1p - n1) reg[n1 + lane] = 0.f;
        if (lane < n2p - n2) reg[region - 1 - n2 - lane] = 0.f;
        __syncwarp();
        for (int i = lane; i < n1; i += 32) {
            const double xd = (double)reg[i];
            sq1 = fma(xd, xd, sq1);
        }
        for (int i = lane; i < n2; i += 32) {
            const double xd = (double)reg[region - 1 - i];
            sq2 = fma(xd, xd, sq2);
        }
        const float4* reg4 = reinterpret_cast<const float4*>(reg);
        if (n1 > 0) {
            sweep_range<CPT, 1, 0>(reg4, 0, n1p >> 2, inv2, na2, dacc, kMagic + flo, kMagic + fhi);
            ev += (unsigned long long)n1p;
        }
        if (n2 > 0) {
            sweep_ncl<CPT, CPT>(ncl_rest, reg4, (region - n2p) >> 2, region >> 2, inv2, na2, dacc, kMagic + flo, kMagic + fhi);
            ev += (unsigned long long)n2p * CPT;
        }
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    __syncthreads();
    if (warp > 0) {
#pragma unroll
        for (int sl = 0; sl < CPT; ++sl) xg[((warp - 1) * CPT + sl) * 32 + lane] = dacc[sl];
    }
    __syncthreads();
    if (warp == 0) {
        for (int w = 1; w < nwarp; ++w)
#pragma unroll
            for (int sl = 0; sl < CPT; ++sl) dacc[sl] += xg[((w - 1) * CPT + sl) * 32 + lane];
    }
    report_evaluations(a.evals, ev);
    long long zero = 0;
    block_sum2(sq_all, zero, dscratch);
    block_sum2(sq1, zero, dscratch);
    block_sum2(sq2, zero, dscratch);
    if (flagging && tid == 0) a.block_totals[blockIdx.x] = sq_all;
    const double sq0 = fmax(sq_all - sq1 - sq2, 0.0);   // what no slot evaluated
    if (warp == 0) {
#pragma unroll
        for (int sl = 0; sl < CPT; ++sl) {
            const int cl = sl * 32 + lane;
            if (cl < a.c_count)
                a.partials[(long long)blockIdx.x * a.n_cand + a.c_base + cl] = dacc[sl] + (sl == 0 ? sq0 : sq0 + sq1);
        }
    }
}

// Sums the per-block partial curves in block order.  Candidates below `split` were swept by a launch of n_blocks_lo
// blocks, the others by one of n_blocks_hi blocks.  A block of 256 threads handles 32 candidates: thread (j, c) adds
// the partials of blocks j, j+8, ... and the eight sums are combined in order.
__global__ void __launch_bounds__(256) tensor_curve_kernel(const TensorArgs a, int split, int n_blocks_lo, int n_blocks_hi) {
    __shared__ double part[8][33];
    const int cl = threadIdx.x & 31, j = threadIdx.x >> 5;
    const int c = blockIdx.x * 32 + cl;
    TensorState* st = a.st;
    const float mpos = __uint_as_float(st->mpos_bits), mneg = __uint_as_float(st->mneg_bits);
    const GridSetup g = grid_setup(mpos, mneg, a.hi_frac, a.n_cand, (float)a.lo, (float)a.hi);
    const float a_last = __fmul_rn((float)a.n_cand, g.step);
    const bool usable = (fmaxf(mpos, mneg) > 0.f) && (a_last >= FLT_MIN);
    double s = 0.0;
    if (usable && c < a.n_cand) {
        const int n_blocks = c < split ? n_blocks_lo : n_blocks_hi;
#pragma unroll 4
        for (int b = j; b < n_blocks; b += 8) s += __ldcg(&a.partials[(long long)b * a.n_cand + c]);
    }
    part[j][cl] = s;
    __syncthreads();
    if (j == 0 && c < a.n_cand) {
        double tot = INFINITY;
        if (usable) {
            tot = 0.0;
#pragma unroll
            for (int jj = 0; jj < 8; ++jj) tot += part[jj][cl];
            const float ac = __fmul_rn((float)(c + 1), g.step);
            if (!(ac >= FLT_MIN)) tot = INFINITY;
        }
        a.curve[c] = tot;
        if (a.curve_out) a.curve_out[c] = tot;
    }
}

// One block: argmin of the summed curve and the list of candidates inside the fp32 noise band of the minimum.
__global__ void __launch_bounds__(1024) tensor_finish_kernel(const TensorArgs a) {
    __shared__ double scratch[64];
    __shared__ int cnt;
    TensorState* st = a.st;
    const float mpos = __uint_as_float(st->mpos_bits), mneg = __uint_as_float(st->mneg_bits);
    const float m = fmaxf(mpos, mneg);
    const GridSetup g = grid_setup(mpos, mneg, a.hi_frac, a.n_cand, (float)a.lo, (float)a.hi);
    const float a_last = __fmul_rn((float)a.n_cand, g.step);
    const bool degenerate = !(m > 0.f) || !(a_last >= FLT_MIN);
    double bv = INFINITY;
    int bi = 0x7fffffff;
    if (!degenerate) {
        for (int c = threadIdx.x; c < a.n_cand; c += blockDim.x) {
            const double s = a.curve[c];
            if (s < bv) {
                bv = s;
                bi = c;
            }
        }
    }
    if (threadIdx.x == 0) cnt = 0;
    block_argmin(bv, bi, scratch);
    if (degenerate || bi == 0x7fffffff) {
        if (threadIdx.x == 0) {
            st->best_idx = -1;
            st->alpha = 0.f;
            st->n_list = 0;
            atomicOr(a.status, 2u);
        }
        return;
    }
    const double band = bv * (1.0 + kRescoreBand);
    for (int c = threadIdx.x; c < a.n_cand; c += blockDim.x) {
        if (a.curve[c] <= band) {
            a.list[atomicAdd(&cnt, 1)] = c;   // at most n_cand entries: the list holds them all
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        st->step = g.step;
        st->best_idx = bi;
        st->alpha = __fmul_rn((float)(bi + 1), g.step);
        st->n_list = cnt > 1 ? cnt : 0;   // a single candidate in the band needs no re-scoring
    }
}

// Grid-wide pass over the tensor; sums in fp64, codes equal to those of the IEEE division (see magic_code).
//   MODE 0 (rescore): squared error at each listed candidate; the last block picks the best.
//   MODE 1 (refine):  <x,q> and <q,q> at st->alpha; the last block sets alpha <- <x,q>/<q,q>.
//   MODE 2 (final):   squared error at st->alpha; the last block writes the outputs.
// Every block keeps its partial sums in its own slot of `partials`; blocks without a slot (a long list of
// candidates on a small scratch) leave at once and the others stride over the whole tensor.
template <int MODE>
__global__ void __launch_bounds__(256) tensor_pass_kernel(const TensorArgs a) {
    __shared__ double scratch[64];
    __shared__ bool is_last;
    TensorState* st = a.st;
    const float flo = (float)a.lo, fhi = (float)a.hi;
    const float clo = kMagic + flo, chi = kMagic + fhi;
    const float amb_thr = ambiguity_threshold(flo, fhi);
    const int n_list = MODE == 0 ? st->n_list : 1;
    if (MODE == 0 && n_list == 0) return;
    const float alpha_now = st->alpha;
    const float delta = st->delta;
    if (MODE == 1 && (!(alpha_now > 0.f) || st->polish_done)) return;
    const int slot = MODE == 0 ? ((n_list + 3) & ~3) : 1;                  // doubles per block
    const long long fit = a.partial_doubles / (slot + 1);
    const unsigned int nblk = (long long)gridDim.x < fit ? gridDim.x : (unsigned int)fit;
    if (blockIdx.x >= nblk) return;
    double* part_d = a.partials;                                           // [nblk][slot]
    long long* part_q = reinterpret_cast<long long*>(a.partials + (size_t)nblk * slot);   // [nblk]
    const long long stride = (long long)nblk * blockDim.x;
    const long long tid0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long n4 = a.n >> 2;
    const float4* x4 = reinterpret_cast<const float4*>(a.x);

    for (int l0 = 0; l0 < n_list; l0 += 4) {
        float al[4], inv[4];
        double ald[4];
        double acc[4] = {0.0, 0.0, 0.0, 0.0};
        long long sqq = 0;
        int sqq32 = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (MODE == 0) {
                const int c = (l0 + j < n_list) ? a.list[l0 + j] : a.list[l0];
                al[j] = __fmul_rn((float)(c + 1), st->step);
            } else {
                al[j] = alpha_now;
            }
            inv[j] = al[j] > 0.f ? __fdiv_rn(1.0f, al[j]) : 0.f;
            ald[j] = (double)al[j];
        }
        const int nj = MODE == 0 ? 4 : 1;
        auto element = [&](float x) {
            const double xd = (double)x;
#pragma unroll
            for (int j = 0; j < nj; ++j) {
                bool amb;
                float tc = magic_code(x, inv[j], clo, chi, amb_thr, amb);
                if (amb) tc = kMagic + (float)(al[j] > 0.f ? code_of(x, al[j], flo, fhi) : 0);   // rare: the division decides
                const int q = magic_int(tc);
                const double qd = int_double(q);
                if (MODE == 1) {
                    sqq32 += q * q;          // folded into the 64-bit sum after every float4 (q*q <= 2^14)
                    acc[j] = fma(xd, qd, acc[j]);
                } else {
                    const double d = fma(-ald[j], qd, xd);
                    acc[j] = fma(d, d, acc[j]);
                }
            }
        };
        auto four = [&](const float4& v) {
            element(v.x - delta);
            element(v.y - delta);
            element(v.z - delta);
            element(v.w - delta);
            sqq += sqq32;
            sqq32 = 0;
        };
        // four 128-bit loads in flight per thread before any of them is used
        long long i = tid0;
        for (; i + 3 * stride < n4; i += 4 * stride) {
            const float4 v0 = __ldg(x4 + i), v1 = __ldg(x4 + i + stride), v2 = __ldg(x4 + i + 2 * stride),
                         v3 = __ldg(x4 + i + 3 * stride);
            four(v0);
            four(v1);
            four(v2);
            four(v3);
        }
        for (; i < n4; i += stride) four(__ldg(x4 + i));
        for (long long e = (n4 << 2) + tid0; e < a.n; e += stride) element(a.x[e] - delta);
        sqq += sqq32;
        for (int j = 0; j < nj; ++j) {
            long long q = sqq;
            block_sum2(acc[j], q, scratch);
            if (threadIdx.x == 0) {
                part_d[(size_t)blockIdx.x * slot + l0 + j] = acc[j];
                if (MODE == 1) part_q[blockIdx.x] = q;
            }
        }
    }
    // ---- last block to arrive reduces the per-block partials (fixed order: thread t takes blocks t, t+256, ...,
    //      then the block-wide sum in lane and warp order)
    __threadfence();
    if (threadIdx.x == 0) {
        const unsigned int tk = atomicAdd(&st->ticket, 1u);
        is_last = (tk == nblk - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    double best_sse = INFINITY;     // MODE 0: this thread's best listed candidate
    int best = 0x7fffffff;
    double total = 0.0;             // MODE 1, 2
    long long total_q = 0;
    if (MODE == 0) {
        for (int l = threadIdx.x; l < n_list; l += blockDim.x) {
            double s = 0.0;
            for (unsigned int b = 0; b < nblk; ++b) s += __ldcg(&part_d[(size_t)b * slot + l]);
            const int c = a.list[l];
            if (s < best_sse || (s == best_sse && c < best)) {
                best_sse = s;
                best = c;
            }
        }
        block_argmin(best_sse, best, scratch);
    } else {
        for (unsigned int b = threadIdx.x; b < nblk; b += blockDim.x) {
            total += __ldcg(&part_d[b]);
            if (MODE == 1) total_q += __ldcg(&part_q[b]);
        }
        block_sum2(total, total_q, scratch);
    }
    if (threadIdx.x == 0) {
        st->ticket = 0u;
        if (MODE == 0) {
            st->best_idx = best;
            st->alpha = __fmul_rn((float)(best + 1), st->step);
        } else if (MODE == 1) {
            bool moved = false;
            if (total_q != 0) {
                const float a_new = (float)(total / (double)total_q);
                if (a_new >= FLT_MIN && a_new <= FLT_MAX && a_new != st->alpha) {
                    st->alpha = a_new;
                    moved = true;
                }
            }
            if (!moved) st->polish_done = 1;   // stopped or fixed point: the remaining polish launches have nothing to do
        } else {
            *a.alpha_out = st->alpha;
            if (a.delta_out) *a.delta_out = st->delta;
            *a.sse_out = (float)total;
            if (a.idx_out) *a.idx_out = st->best_idx;
        }
    }
}

// Key layers (Section 3.5): MSE of each layer = sum of its kernels' squared errors / elements, compared
// with the threshold tau.  One block per layer, fixed-order sum in fp64.
struct LayerError {
    const float* sse;        // [n_kernels] squared error per kernel, as the quantize calls output it
    long long n_kernels, kernel_len;
};

__global__ void __launch_bounds__(256) layer_mse_kernel(const LayerError* __restrict__ layers, float tau,
                                                         double* __restrict__ mse, int* __restrict__ is_key) {
    __shared__ double scratch[64];
    const LayerError L = layers[blockIdx.x];
    double s = 0.0;
    for (long long i = threadIdx.x; i < L.n_kernels; i += blockDim.x) s += (double)L.sse[i];
    long long zero = 0;
    block_sum2(s, zero, scratch);
    if (threadIdx.x == 0) {
        const double m = s / ((double)L.n_kernels * (double)L.kernel_len);
        mse[blockIdx.x] = m;
        if (is_key) is_key[blockIdx.x] = m > (double)tau ? 1 : 0;
    }
}

// Compression ratio of Section 3.5 for layers that hold one quantized tensor, or two where is_key is set:
// (codes at `bits` per element plus one binary32 scale per kernel, per quantized tensor) over the binary32 size.
__global__ void compression_ratio_kernel(const LayerError* __restrict__ layers, int n_layers, int bits,
                                         const int* __restrict__ is_key, double* __restrict__ cr) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    double q = 0.0, f = 0.0;
    for (int l = 0; l < n_layers; ++l) {
        const double n = (double)layers[l].n_kernels * (double)layers[l].kernel_len;
        q += (is_key[l] ? 2.0 : 1.0) * (n * (double)bits + 32.0 * (double)layers[l].n_kernels);
        f += 32.0 * n;
    }
    *cr = f > 0.0 ? q / f : 0.0;
}

// INT4 emission: byte e/2 holds element e (even) in bits 0-3 and element e+1 in bits 4-7.
__global__ void __launch_bounds__(256) pack_int4_kernel(const signed char* __restrict__ codes, long long n,
                                                         unsigned char* __restrict__ packed) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    const long long tid0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const bool aligned = ((reinterpret_cast<unsigned long long>(codes) & 15ull) == 0) &&
                         ((reinterpret_cast<unsigned long long>(packed) & 7ull) == 0);
    const long long n16 = aligned ? (n >> 4) : 0;
    for (long long i = tid0; i < n16; i += stride) {
        const int4 v = __ldg(reinterpret_cast<const int4*>(codes) + i);
        const unsigned int w[4] = {(unsigned)v.x, (unsigned)v.y, (unsigned)v.z, (unsigned)v.w};
        unsigned int out[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            unsigned int r = 0;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const unsigned int u = w[2 * h + j];   // four codes -> two bytes
                const unsigned int b0 = (u & 0xf) | ((u >> 4) & 0xf0);
                const unsigned int b1 = ((u >> 16) & 0xf) | ((u >> 20) & 0xf0);
                r |= (b0 | (b1 << 8)) << (16 * j);
            }
            out[h] = r;
        }
        reinterpret_cast<uint2*>(packed)[i] = make_uint2(out[0], out[1]);
    }
    const long long nb = (n + 1) >> 1;
    for (long long b = (n16 << 3) + tid0; b < nb; b += stride) {
        const unsigned int lo = (unsigned char)codes[2 * b] & 0xf;
        const unsigned int hi = (2 * b + 1 < n) ? ((unsigned char)codes[2 * b + 1] & 0xf) : 0u;
        packed[b] = (unsigned char)(lo | (hi << 4));
    }
}

}  // namespace omse
