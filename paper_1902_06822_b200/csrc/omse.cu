// Host side of the C interface declared in include/omse.h: argument checks, launch shapes, context.
// Every step of the method runs in the kernels of omse_rows.cuh / omse_tensor.cuh; there is no
// host arithmetic on tensor data and no CPU fallback.
#include "../../include/omse.h"

#include <algorithm>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#ifndef OMSE_ROWS_BIG_K
#define OMSE_ROWS_BIG_K 8192        /* rows at least this long use the larger block */
#endif
#ifndef OMSE_ROWS_THREADS_BIG
#define OMSE_ROWS_THREADS_BIG 512
#endif
#ifndef OMSE_ROWS_THREADS_MID
#define OMSE_ROWS_THREADS_MID 128
#endif

#ifndef OMSE_PRUNE
#define OMSE_PRUNE 1
#endif
#ifndef OMSE_SMALL_PRUNE_K
#define OMSE_SMALL_PRUNE_K 192      /* short rows at least this long are regrouped by magnitude class */
#endif
#ifndef OMSE_TINY_K
#define OMSE_TINY_K 32              /* rows up to this length, in large numbers, get one thread each */
#endif
#ifndef OMSE_SMALL_K
#define OMSE_SMALL_K 640            /* rows up to this length are batched per work unit */
#endif

#include "omse_rows.cuh"
#include "omse_tensor.cuh"
#include "omse_dual.cuh"

namespace {

constexpr size_t kPartialBytes = 16u << 20;   // per-block partial sums of the per-tensor search
constexpr int kMaxSmem = 231424;              // dynamic shared memory per block: the 227 KB opt-in limit of sm_100 less 1 KB for static use

struct Workspace {
    unsigned int status;
    unsigned int pad_[3];
    unsigned long long ticket[4];   // work-unit dispensers of the row kernels (self-resetting): a pair for launches on the
                                    // context's stream, a pair for the launch that runs beside them on the side stream
    unsigned long long evals;       // executed evaluations since the last omse_read_evaluations
    omse::TensorState tstate;
    double curve[OMSE_MAX_CANDIDATES];
    int list[OMSE_MAX_CANDIDATES];  // candidates of the per-tensor search that are re-scored in fp64
};

}  // namespace

struct LaunchShape { int cpt, threads; size_t smem; int occ; };

struct omse_ctx {
    int device;
    cudaStream_t stream;
    cudaStream_t side;                 // second launch of a batched call runs here, beside the first (fork and join by events)
    cudaEvent_t ev_fork, ev_join;
    int ticket_pair;                   // which dispenser pair the next row launch uses
    int n_sm;
    Workspace* ws;       // device
    double* partials;    // device, kPartialBytes
    omse::RowTensor* d_tensors;   // device, OMSE_MAX_BATCH descriptors of a batched launch
    // per-context launch bookkeeping (a context is used by one host thread at a time, so no lock)
    bool attr_rows[32], attr_tensor[4], attr_dual;   // opt-in shared-memory attribute set, per template instance
    LaunchShape seen[16];                           // blocks per SM of the row-kernel launch shapes met so far
    int n_seen, next_seen;
    int occ_sweep[2], occ_pass[3];                  // blocks per SM of the per-tensor kernels (0 = not yet asked)
    unsigned long long n_launches;                  // kernels launched since the last omse_read_launches
};

namespace {

// Makes the context's device current for the duration of a call and puts the caller's device back afterwards.
class DeviceScope {
public:
    explicit DeviceScope(int device) : prev_(-1), ok_(false) {
        if (cudaGetDevice(&prev_) != cudaSuccess) prev_ = -1;
        ok_ = (prev_ == device) || cudaSetDevice(device) == cudaSuccess;
        if (prev_ == device) prev_ = -1;   // nothing to restore
    }
    ~DeviceScope() {
        if (prev_ >= 0) cudaSetDevice(prev_);
    }
    bool ok() const { return ok_; }
private:
    int prev_;
    bool ok_;
};

int cpt_slot(int cpt) { return cpt == 1 ? 0 : cpt == 2 ? 1 : cpt == 4 ? 2 : 3; }

}  // namespace

namespace {

#ifndef OMSE_MAX_CPT
#define OMSE_MAX_CPT 8
#endif
int cpt_for(int n_cand) {
    const int c = n_cand <= 32 ? 1 : n_cand <= 64 ? 2 : n_cand <= 128 ? 4 : 8;
    return c > OMSE_MAX_CPT ? OMSE_MAX_CPT : c;
}

bool grid_ok(const omse_grid* g) {
    return g && g->n_cand >= 1 && g->n_cand <= OMSE_MAX_CANDIDATES && g->hi_frac > 0.f &&
           g->hi_frac <= 3.0e38f && g->refine_iters >= 0 && g->refine_iters <= 64;
}

void bounds(int bits, int is_signed, int* lo, int* hi) {
    if (is_signed) {
        *lo = -(1 << (bits - 1));
        *hi = (1 << (bits - 1)) - 1;
    } else {
        *lo = 0;
        *hi = (1 << bits) - 1;
    }
}

template <int CPT, bool EXT, int PATH>
int launch_rows_t(omse_ctx* ctx, omse::RowArgs& a, size_t smem) {
    const int slot = cpt_slot(CPT) + (EXT ? 4 : 0) + 8 * (PATH == 7 ? 0 : PATH == 1 ? 1 : PATH == 2 ? 2 : 3);
    if (!ctx->attr_rows[slot]) {
        if (cudaFuncSetAttribute(omse::rows_kernel<CPT, EXT, PATH>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem) != cudaSuccess)
            return OMSE_ECUDA;
        ctx->attr_rows[slot] = true;
    }
    const int threads = a.groups * a.tg;
    // blocks per SM for this launch shape (remembered: the query costs more than a small launch)
    int occ = 0;
    for (int i = 0; i < ctx->n_seen; ++i)
        if (ctx->seen[i].cpt == slot && ctx->seen[i].threads == threads && ctx->seen[i].smem == smem) occ = ctx->seen[i].occ;
    if (occ == 0) {
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, omse::rows_kernel<CPT, EXT, PATH>, threads, smem) != cudaSuccess || occ < 1)
            return OMSE_ECUDA;
        ctx->seen[ctx->next_seen] = LaunchShape{slot, threads, smem, occ};   // round robin once the table is full
        ctx->next_seen = (ctx->next_seen + 1) % 16;
        if (ctx->n_seen < 16) ++ctx->n_seen;
    }
    long long grid = (long long)ctx->n_sm * occ;
    if (grid > a.n_units) grid = a.n_units;
    omse::rows_kernel<CPT, EXT, PATH><<<(unsigned)grid, threads, smem, ctx->stream>>>(a);
    ++ctx->n_launches;
    return cudaGetLastError() == cudaSuccess ? OMSE_OK : OMSE_ECUDA;
}

// Launch shape for rows of at most max_k elements: threads per block, element groups, shared memory.
int launch_rows(omse_ctx* ctx, omse::RowArgs& a, long long max_k, size_t smem_small = 0, int path = 7) {
    const int cpt = cpt_for(a.n_cand);
    a.tg = (((a.n_cand + cpt - 1) / cpt) + 31) & ~31;
    const int k4 = (int)((max_k + 3) >> 2);
    a.max_k4 = k4;
    int target = max_k >= OMSE_ROWS_BIG_K ? OMSE_ROWS_THREADS_BIG : OMSE_ROWS_THREADS_MID;
    int groups = target / a.tg;
    if (groups > k4 / 8) groups = k4 / 8;
    if (groups < 1) groups = 1;
    a.groups = groups;
    // fixed part: reduction scratch, skipped sums, class table, misc
    const size_t fixed = (size_t)omse::kScratchDoubles * 8 + (size_t)cpt * 8 + 2 * (cpt + 1) * 4 + 8 * 4;
    auto smem_for = [&](int gr) {
        return (size_t)(a.keep_x0 ? 2 : 1) * k4 * 16 + (a.prune ? (size_t)k4 * 16 + (size_t)cpt * 16 : 0) +
               (size_t)(gr - 1) * cpt * a.tg * 8 + fixed;
    };
    // Regrouping by magnitude needs a second copy of the row on chip and 16-bit class counts; it is worth its
    // fixed cost only for long rows or for launches with several rows per SM.
    a.prune = (OMSE_PRUNE && max_k < 65536 && (max_k >= 1024 || a.n_units >= 4ll * ctx->n_sm)) ? 1 : 0;
    if (a.prune && smem_for(1) > (size_t)kMaxSmem) a.prune = 0;
    while (a.groups > 1 && smem_for(a.groups) > (size_t)kMaxSmem) a.groups >>= 1;
    size_t smem = smem_for(a.groups);
    if (smem > (size_t)kMaxSmem) return OMSE_EINVAL;
    if (smem_small > smem) smem = smem_small;
    a.ticket = ctx->ws->ticket + 2 * ctx->ticket_pair;
    a.status = &ctx->ws->status;
    a.evals = &ctx->ws->evals;
    // the extended kernel only where a launch needs what it adds
    bool ext = a.solver != 0 || a.n_delta > 0 || a.eps >= 0.f || a.sweeps_done != nullptr;
    if (a.tensors == nullptr) ext = ext || a.one.gate || a.one.prior_alpha;
    else ext = ext || a.ext_tensors;
    if (ext) {
        switch (cpt) {
            case 1: return launch_rows_t<1, true, 7>(ctx, a, smem);
            case 2: return launch_rows_t<2, true, 7>(ctx, a, smem);
            case 4: return launch_rows_t<4, true, 7>(ctx, a, smem);
            default: return launch_rows_t<8, true, 7>(ctx, a, smem);
        }
    }
    switch (cpt) {
        case 1: return launch_rows_t<1, false, 7>(ctx, a, smem);
        case 2: return launch_rows_t<2, false, 7>(ctx, a, smem);
        case 4: return launch_rows_t<4, false, 7>(ctx, a, smem);
        default:
            // single-path instantiations exist for the common case of eight candidates per thread
            if (path == 1) return launch_rows_t<8, false, 1>(ctx, a, smem);
            if (path == 2) return launch_rows_t<8, false, 2>(ctx, a, smem);
            if (path == 4) return launch_rows_t<8, false, 4>(ctx, a, smem);
            return launch_rows_t<8, false, 7>(ctx, a, smem);
    }
}

void fill_tensor(omse::RowTensor& t, const float* w, int64_t S, int64_t K, float* alpha, float* sse, int32_t* idx,
                 int8_t* codes, uint8_t* packed) {
    t.w = w;
    t.S = S;
    t.K = K;
    t.alpha = alpha;
    t.sse = sse;
    t.best_idx = idx;
    t.codes = reinterpret_cast<signed char*>(codes);
    t.packed = packed;
    t.delta = nullptr;
    t.prior_alpha = nullptr;
    t.gate = nullptr;
    t.unit_begin = 0;
    t.rows_per_unit = (packed && (K & 1)) ? 2 : 1;
    t.small = 0;
}

// Threads of one element group and whether a launch over rows of at most max_k elements runs a
// single group per block (the short-row path needs that).
int group_threads(int n_cand) {
    const int cpt = cpt_for(n_cand);
    return (((n_cand + cpt - 1) / cpt) + 31) & ~31;
}
bool single_group(int n_cand, long long max_k) {
    const int target = max_k >= OMSE_ROWS_BIG_K ? OMSE_ROWS_THREADS_BIG : OMSE_ROWS_THREADS_MID;
    return target / group_threads(n_cand) <= 1;
}

bool misaligned4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3) != 0; }

// ---- per-tensor search: the launches shared by omse_activation_scale* and the allocation-free entry point
struct TensorEnv {
    int n_sm;
    cudaStream_t stream;
    int* occ_sweep;      // [2] blocks per SM of the two sweep launch shapes (0 = not yet asked), cached by the caller
    int* occ_pass;       // [3] blocks per SM of the three pass kernels
    bool opt_in_smem;    // the sweep may ask for more than 48 KB of dynamic shared memory (context path only)
    bool* attr_tensor;   // [4] per CPT: opt-in attribute already set
    unsigned long long* launches;   // launch counter of the caller
};

template <int CPT, bool FINE>
int sweep_launch_t(const TensorEnv& env, omse::TensorArgs& a, size_t smem, int* n_blocks) {
    auto kernel = FINE ? omse::tensor_sweep_fine_kernel<CPT> : omse::tensor_sweep_kernel<CPT>;
    if (env.opt_in_smem && smem > 48 * 1024 && !env.attr_tensor[cpt_slot(CPT)]) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem) != cudaSuccess) return OMSE_ECUDA;
        env.attr_tensor[cpt_slot(CPT)] = true;
    }
    const int threads = a.groups * a.tg;
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, threads, smem) != cudaSuccess || occ < 1) return OMSE_ECUDA;
    const long long n4 = (a.n + 3) >> 2;
    const long long n_tiles = (n4 + a.tile4 - 1) / a.tile4;
    long long grid = (long long)env.n_sm * occ;
    const long long cap = a.partial_doubles / a.n_cand;
    if (grid > cap) grid = cap;
    if (grid > n_tiles) grid = n_tiles;
    if (grid < 1) grid = 1;
    *n_blocks = (int)grid;
    kernel<<<(unsigned)grid, threads, smem, env.stream>>>(a);
    ++*env.launches;
    return cudaGetLastError() == cudaSuccess ? OMSE_OK : OMSE_ECUDA;
}

// One sweep launch over the candidates [c_base, c_base + c_count) with `cpt` candidates per thread.
int sweep_launch(const TensorEnv& env, omse::TensorArgs a, int c_base, int c_count, int cpt, int* n_blocks) {
    a.c_base = c_base;
    a.c_count = c_count;
    a.tg = (((c_count + cpt - 1) / cpt) + 31) & ~31;
    a.groups = 256 / a.tg < 1 ? 1 : 256 / a.tg;
    a.tile4 = 4 * a.groups * a.tg;   // every thread stages exactly four float4s of a tile
    if (a.tg == 32) {
        // slots of 32 candidates: the warps of a block work on their own shares of a tile
        const size_t smem = (size_t)8 * (16 * 32 + 8) * 4 + (size_t)a.tile4 * 16;   // eight warp regions + landing zone
        switch (cpt) {
            case 1: return sweep_launch_t<1, true>(env, a, smem, n_blocks);
            case 2: return sweep_launch_t<2, true>(env, a, smem, n_blocks);
            case 4: return sweep_launch_t<4, true>(env, a, smem, n_blocks);
            default: return sweep_launch_t<8, true>(env, a, smem, n_blocks);
        }
    }
    // regrouped tile + landing zone of the asynchronous copies, which also holds the partial sums of the other groups
    // at the end
    const size_t regrouped = ((size_t)a.tile4 * 4 + 4 * cpt) * 4;
    const size_t landing = std::max((size_t)a.tile4 * 16, (size_t)(a.groups - 1) * cpt * a.tg * 8);
    const size_t smem = regrouped + landing;
    if (!env.opt_in_smem && smem + 1024 > 48 * 1024) return OMSE_ELIMIT;
    return sweep_launch_t<8, false>(env, a, smem, n_blocks);   // wide slots only occur with 8 candidates per thread
}

template <int MODE>
int pass_grid(const TensorEnv& env, long long n) {
    int& occ = env.occ_pass[MODE];
    if (occ == 0 && (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, omse::tensor_pass_kernel<MODE>, 256, 0) != cudaSuccess || occ < 1))
        occ = 4;
    long long grid = (n + 1023) / 1024;            // at least one float4 per thread
    if (grid > (long long)env.n_sm * occ) grid = (long long)env.n_sm * occ;   // one wave: every block is resident
    return grid < 1 ? 1 : (int)grid;
}

// Everything after the state has been cleared: maxima, sweep (one or two launches), curve, argmin, re-score, polish,
// final error.  `a` carries the buffers; grid fields are filled here.
int enqueue_tensor_search(const TensorEnv& env, omse::TensorArgs& a, int refine_iters) {
    cudaStream_t s = env.stream;
    const long long n = a.n;
    long long absmax_grid = (n + 1023) / 1024;
    if (absmax_grid > (long long)env.n_sm * 8) absmax_grid = (long long)env.n_sm * 8;
    if (absmax_grid < 1) absmax_grid = 1;
    const int kFine = 256;        // candidates of the first launch: 32 per slot
    int split = a.n_cand, nb_lo = 1, nb_hi = 1;
    if (n > 0) {
        // Two sweep launches share tile flags when they fit: a bit per tile of the SECOND launch in the (not yet
        // used) curve buffer, and the first launch's per-block squared sums in the (not yet used) candidate list.
        const bool two = a.n_cand > kFine;
        const int hi_tg = two ? ((((a.n_cand - kFine) + 7) / 8) + 31) & ~31 : 32;
        const long long flag_tile4 = 4ll * (256 / hi_tg < 1 ? 1 : 256 / hi_tg) * hi_tg;   // as sweep_launch sizes it
        const long long n_flag_tiles = (((n + 3) >> 2) + flag_tile4 - 1) / flag_tile4;
        // curve: n_cand doubles = 64*n_cand bits; list: n_cand/2 doubles, enough for three blocks per SM
        const bool flags = two && n_flag_tiles <= 64ll * a.n_cand && a.n_cand / 2 >= 3 * env.n_sm;
        const int flag_words = flags ? (int)((n_flag_tiles + 31) >> 5) : 0;
        omse::tensor_absmax_kernel<<<(unsigned)absmax_grid, 256, 0, s>>>(a.x, n, a.st, a.status,
                                                                      reinterpret_cast<unsigned int*>(a.curve), flag_words);
        ++*env.launches;
        if (a.delta_out) {
            omse::tensor_offset_kernel<<<1, 32, 0, s>>>(a.st);
            ++*env.launches;
        }
        int rc;
        if (!two) {
            rc = sweep_launch(env, a, 0, a.n_cand, cpt_for(a.n_cand), &nb_lo);
            nb_hi = nb_lo;
        } else {
            split = kFine;
            omse::TensorArgs lo = a;
            if (flags) {
                lo.tile_flags = reinterpret_cast<unsigned int*>(a.curve);
                lo.flag_words = flag_words;
                lo.flag_tile4 = (int)flag_tile4;
                lo.flag_role = 1;
                lo.flag_split = (float)(kFine + 1);
                lo.block_totals = reinterpret_cast<double*>(a.list);
                // the list holds n_cand ints = n_cand/2 doubles: one per block of the first launch
                const long long cap = (long long)(a.n_cand / 2) * a.n_cand;
                if (lo.partial_doubles > cap) lo.partial_doubles = cap;
            }
            rc = sweep_launch(env, lo, 0, kFine, 8, &nb_lo);
            omse::TensorArgs hi = a;
            if (flags) {
                hi.tile_flags = lo.tile_flags;
                hi.flag_words = flag_words;
                hi.flag_tile4 = lo.flag_tile4;
                hi.flag_role = 2;
                hi.block_totals = lo.block_totals;
                hi.n_totals = nb_lo;
            }
            if (rc == OMSE_OK) rc = sweep_launch(env, hi, kFine, a.n_cand - kFine, 8, &nb_hi);
        }
        if (rc != OMSE_OK) return rc;
    }
    omse::tensor_curve_kernel<<<(unsigned)((a.n_cand + 31) / 32), 256, 0, s>>>(a, split, nb_lo, nb_hi);
    omse::tensor_finish_kernel<<<1, 1024, 0, s>>>(a);
    omse::tensor_pass_kernel<0><<<(unsigned)pass_grid<0>(env, n), 256, 0, s>>>(a);
    const int g1 = pass_grid<1>(env, n);
    for (int it = 0; it < refine_iters; ++it) omse::tensor_pass_kernel<1><<<(unsigned)g1, 256, 0, s>>>(a);
    omse::tensor_pass_kernel<2><<<(unsigned)pass_grid<2>(env, n), 256, 0, s>>>(a);
    *env.launches += 4 + (unsigned long long)refine_iters;   // curve, finish, re-score, polish steps, final
    return cudaGetLastError() == cudaSuccess ? OMSE_OK : OMSE_ECUDA;
}

}  // namespace

namespace {

// How the scale of each row is found, for launches that do not use the default grid search with polish.
struct ListMode {
    int solver = 0, solver_iters = 0;   // comparison solvers of Section 3.4 (RowArgs::solver)
    int n_delta = 0;                    // offsets searched per row (0: none)
    float off_frac = 0.f;
};

// Launch for a list of weight tensors (bounds already set by the caller).
int quantize_list(omse_ctx* ctx, std::vector<omse::RowTensor>& list, long long max_k, int bits, int is_signed,
                  const omse_grid* grid, const ListMode& mode = ListMode()) {
    if (list.empty()) return OMSE_OK;
    DeviceScope dev(ctx->device);
    if (!dev.ok()) return OMSE_ECUDA;
    // Short rows are batched per work unit when the block is a single element group and the launch
    // still has a few work units per SM afterwards (otherwise one row per block fills the GPU better).
    size_t smem_small = 0;
    const bool plain = mode.solver == 0 && mode.n_delta == 0;   // the batched short-row paths implement the grid search only
    if (plain && single_group(grid->n_cand, max_k)) {
        const int cpt = cpt_for(grid->n_cand);
        const int ncs = cpt * group_threads(grid->n_cand);
        long long units_if_small = 0;
        // rows per work unit of the short-row path: eight rows of up to 128 elements amortise the unit's fixed costs,
        // but only a tensor with many rows has enough units left for an even finish; otherwise four
        auto small_batch = [&](const omse::RowTensor& t) { return (t.K <= 128 && t.S >= 16ll * ctx->n_sm) ? 8 : 4; };
        for (const auto& t : list) {
            const int b = t.K > OMSE_SMALL_K ? t.rows_per_unit : small_batch(t);
            units_if_small += (t.S + b - 1) / b;
        }
        // very short rows in large numbers: a thread per row, a block-sized batch of rows per unit
        const int threads = group_threads(grid->n_cand);
        for (auto& t : list) {
            if (t.K > OMSE_TINY_K || t.S < 64ll * ctx->n_sm || t.prior_alpha) continue;
            t.small = 4;
            t.rows_per_unit = threads;
            const size_t need = (size_t)((threads * t.K + 3) & ~3ll) * 4 + (size_t)((grid->n_cand + 3) & ~3) * 4 +
                                (size_t)threads * t.K + 16;
            if (need > smem_small) smem_small = need;
        }
        if (units_if_small >= 4ll * ctx->n_sm) {
            for (auto& t : list) {
                if (t.K > OMSE_SMALL_K || t.small) continue;
                const bool prune = OMSE_PRUNE && t.K >= OMSE_SMALL_PRUNE_K;
                t.small = prune ? 3 : 1;
                t.rows_per_unit = small_batch(t);
                const size_t kpad = (size_t)((t.K + 3) & ~3ll);
                // per row: the row, its error curve, its grid; when regrouping also skipped sums, class table, regrouped row
                const size_t need = (size_t)t.rows_per_unit *
                    (kpad * 4 + (size_t)ncs * 4 + 16 +
                     (prune ? (size_t)cpt * 8 + 2 * (cpt + 1) * 4 + (kpad + 4 * cpt) * 4 : 0));
                if (need > smem_small) smem_small = need;
            }
        }
    }
    // One launch per row path present in the list (block per row, batched short rows, thread per row): each launch
    // then runs the kernel instantiation that holds only its path.  Longest rows first inside a launch: the dispenser
    // hands out work in decreasing size and the tail is short.
    std::stable_sort(list.begin(), list.end(), [](const omse::RowTensor& x, const omse::RowTensor& y) { return x.K > y.K; });
    // With both long and short rows in the list, the launch of the short rows goes first, on the side stream (forked
    // from and joined to the context's stream by events, with its own work dispenser), and the long rows' launch runs
    // beside it: the blocks of the second fill the SMs as the blocks of the first run out of work, so only one tail
    // is left.  The two launches touch different tensors.
    int present = 0;
    for (const auto& t : list) present |= (t.small & 4) ? 4 : t.small ? 2 : 1;
    const bool beside = (present & 2) && (present & 5);
    bool forked = false;
    size_t desc_used = 0;
    const int path_order[3] = {2, 1, 4};
    int rc_all = OMSE_OK;
    for (int pi = 0; pi < 3 && rc_all == OMSE_OK; ++pi) {
        const int path = path_order[pi];
        std::vector<omse::RowTensor> sub;
        long long sub_max_k = 0;
        for (const auto& t : list) {
            const int p = (t.small & 4) ? 4 : t.small ? 2 : 1;
            if (p != path) continue;
            sub.push_back(t);
            if (t.K > sub_max_k) sub_max_k = t.K;
        }
        if (sub.empty()) continue;
        long long units = 0;
        for (auto& t : sub) {
            t.unit_begin = units;
            units += (t.S + t.rows_per_unit - 1) / t.rows_per_unit;
        }
        omse::RowArgs a;
        memset(&a, 0, sizeof(a));
        a.n_launch_tensors = (int)sub.size();
        a.n_units = units;
        for (const auto& t : sub) a.ext_tensors |= (t.gate || t.prior_alpha) ? 1 : 0;
        if (sub.size() == 1) {
            a.tensors = nullptr;
            a.one = sub[0];
        } else {
            omse::RowTensor* d_sub = ctx->d_tensors + desc_used;
            if (cudaMemcpyAsync(d_sub, sub.data(), sizeof(omse::RowTensor) * sub.size(), cudaMemcpyHostToDevice,
                                ctx->stream) != cudaSuccess) {
                rc_all = OMSE_ECUDA;
                break;
            }
            a.tensors = d_sub;
            desc_used += sub.size();
        }
        a.n_cand = grid->n_cand;
        a.hi_frac = grid->hi_frac;
        a.refine_iters = grid->refine_iters;
        a.n_tensors = 1;
        a.n_sweeps = 1;
        bounds(bits, is_signed, &a.lo[0], &a.hi[0]);
        a.solver = mode.solver;
        a.solver_iters = mode.solver_iters;
        a.n_delta = mode.n_delta;
        a.off_frac = mode.off_frac;
        a.eps = -1.f;
        a.keep_x0 = mode.n_delta > 0 ? 1 : 0;   // every offset is applied to the original row
        const bool on_side = beside && path == 2;
        cudaStream_t own = ctx->stream;
        if (on_side) {
            if (cudaEventRecord(ctx->ev_fork, own) != cudaSuccess || cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0) != cudaSuccess) {
                rc_all = OMSE_ECUDA;
                break;
            }
            forked = true;
            ctx->stream = ctx->side;
            ctx->ticket_pair = 1;
        }
        rc_all = launch_rows(ctx, a, sub_max_k, path == 1 ? 0 : smem_small, path);
        if (on_side) {
            ctx->stream = own;
            ctx->ticket_pair = 0;
        }
    }
    if (forked) {   // the side stream always rejoins, also after an error
        if (cudaEventRecord(ctx->ev_join, ctx->side) != cudaSuccess || cudaStreamWaitEvent(ctx->stream, ctx->ev_join, 0) != cudaSuccess)
            rc_all = rc_all == OMSE_OK ? OMSE_ECUDA : rc_all;
    }
    return rc_all;
}

}  // namespace

static int activation_impl(omse_ctx* ctx, const float* d_x, int64_t n, int bits, int is_signed, const omse_grid* grid,
                           float* d_alpha, float* d_delta, float* d_sse, int32_t* d_best_idx, double* d_sse_curve);

extern "C" {

const char* omse_status_string(int status) {
    switch (status) {
        case OMSE_OK: return "ok";
        case OMSE_EINVAL: return "invalid argument";
        case OMSE_ECUDA: return "CUDA runtime or launch failure";
        case OMSE_ENOMEM: return "out of device memory";
        case OMSE_ELIMIT: return "size beyond the fixed scratch of the allocation-free entry point";
        default: return "unknown status";
    }
}

int omse_create(omse_ctx** out, int device, void* cuda_stream) {
    if (!out) return OMSE_EINVAL;
    *out = nullptr;
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device < 0 || device >= n_dev) return OMSE_ECUDA;
    DeviceScope dev(device);
    if (!dev.ok()) return OMSE_ECUDA;
    omse_ctx* c = new (std::nothrow) omse_ctx;
    if (!c) return OMSE_ENOMEM;
    memset(c, 0, sizeof(*c));
    c->device = device;
    c->stream = static_cast<cudaStream_t>(cuda_stream);
    c->ws = nullptr;
    c->partials = nullptr;
    c->d_tensors = nullptr;
    if (cudaDeviceGetAttribute(&c->n_sm, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
        delete c;
        return OMSE_ECUDA;
    }
    if (cudaMalloc(&c->ws, sizeof(Workspace)) != cudaSuccess || cudaMalloc(&c->partials, kPartialBytes) != cudaSuccess ||
        cudaMalloc(&c->d_tensors, sizeof(omse::RowTensor) * OMSE_MAX_BATCH) != cudaSuccess) {
        cudaFree(c->ws);
        cudaFree(c->partials);
        delete c;
        cudaGetLastError();
        return OMSE_ENOMEM;
    }
    if (cudaMemsetAsync(c->ws, 0, sizeof(Workspace), c->stream) != cudaSuccess ||
        cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) != cudaSuccess) {
        if (c->ev_fork) cudaEventDestroy(c->ev_fork);
        if (c->side) cudaStreamDestroy(c->side);
        cudaFree(c->ws);
        cudaFree(c->partials);
        cudaFree(c->d_tensors);
        delete c;
        cudaGetLastError();
        return OMSE_ECUDA;
    }
    *out = c;
    return OMSE_OK;
}

int omse_destroy(omse_ctx* ctx) {
    if (!ctx) return OMSE_EINVAL;
    DeviceScope dev(ctx->device);
    cudaStreamSynchronize(ctx->stream);
    cudaStreamSynchronize(ctx->side);
    cudaEventDestroy(ctx->ev_fork);
    cudaEventDestroy(ctx->ev_join);
    cudaStreamDestroy(ctx->side);
    cudaFree(ctx->ws);
    cudaFree(ctx->partials);
    cudaFree(ctx->d_tensors);
    delete ctx;
    return OMSE_OK;
}

int omse_set_stream(omse_ctx* ctx, void* cuda_stream) {
    if (!ctx) return OMSE_EINVAL;
    ctx->stream = static_cast<cudaStream_t>(cuda_stream);
    return OMSE_OK;
}

size_t omse_workspace_bytes(int64_t n_kernels, int64_t kernel_len, int32_t n_cand, int32_t n_tensors) {
    // Rows are searched on chip, so the workspace does not grow with the problem: status and dispenser words, the
    // per-tensor search state and curve, per-block partial sums, descriptors of a batched launch.
    if (n_kernels < 0 || kernel_len < 1 || n_cand < 1 || n_cand > OMSE_MAX_CANDIDATES || n_tensors < 1 ||
        n_tensors > OMSE_MAX_TENSORS)
        return 0;
    return sizeof(Workspace) + kPartialBytes + sizeof(omse::RowTensor) * OMSE_MAX_BATCH;
}

int omse_last_device_status(omse_ctx* ctx, uint32_t* host_out) {
    if (!ctx || !host_out) return OMSE_EINVAL;
    DeviceScope dev(ctx->device);
    if (!dev.ok()) return OMSE_ECUDA;
    if (cudaMemcpyAsync(host_out, &ctx->ws->status, sizeof(uint32_t), cudaMemcpyDeviceToHost, ctx->stream) != cudaSuccess)
        return OMSE_ECUDA;
    if (cudaMemsetAsync(&ctx->ws->status, 0, sizeof(uint32_t), ctx->stream) != cudaSuccess) return OMSE_ECUDA;
    return cudaStreamSynchronize(ctx->stream) == cudaSuccess ? OMSE_OK : OMSE_ECUDA;
}

int omse_read_launches(omse_ctx* ctx, uint64_t* host_out) {
    if (!ctx || !host_out) return OMSE_EINVAL;
    *host_out = ctx->n_launches;
    ctx->n_launches = 0;
    return OMSE_OK;
}

int omse_read_evaluations(omse_ctx* ctx, uint64_t* host_out) {
    if (!ctx || !host_out) return OMSE_EINVAL;
    DeviceScope dev(ctx->device);
    if (!dev.ok()) return OMSE_ECUDA;
    unsigned long long v = 0;
    if (cudaMemcpyAsync(&v, &ctx->ws->evals, sizeof(v), cudaMemcpyDeviceToHost, ctx->stream) != cudaSuccess) return OMSE_ECUDA;
    if (cudaMemsetAsync(&ctx->ws->evals, 0, sizeof(v), ctx->stream) != cudaSuccess) return OMSE_ECUDA;
    if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return OMSE_ECUDA;
    *host_out = v;
    return OMSE_OK;
}

int omse_measure_fp32_peak(omse_ctx* ctx, int target_ms, double* host_out) {
    if (!ctx || !host_out || target_ms < 1 || target_ms > 5000) return OMSE_EINVAL;
    DeviceScope dev(ctx->device);
    if (!dev.ok()) return OMSE_ECUDA;
    const int blocks = ctx->n_sm * 4, threads = 256;
    float* out = reinterpret_cast<float*>(ctx->partials);        // blocks*threads floats, far below the 16 MB held
    // iterations for about target_ms at 128 lane operations per clock and SM at 2 GHz
    const double lane_ops_per_iter = (double)blocks * threads * omse::kPeakChains * 2.0;
    long long iters = (long long)((double)target_ms * 1e-3 * (double)ctx->n_sm * 128.0 * 2.0e9 / lane_ops_per_iter);
    if (iters < 1024) iters = 1024;
    if (iters > 0x7fffffff) iters = 0x7fffffff;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) {
        if (e0) cudaEventDestroy(e0);
        return OMSE_ECUDA;
    }
    omse::fma_peak_kernel<<<blocks, threads, 0, ctx->stream>>>(out, 4096, 1.0f);      // warm-up
    cudaEventRecord(e0, ctx->stream);
    omse::fma_peak_kernel<<<blocks, threads, 0, ctx->stream>>>(out, (int)iters, 1.0f);
    cudaEventRecord(e1, ctx->stream);
    float ms = 0.f;
    const bool ok = cudaEventSynchronize(e1) == cudaSuccess && cudaEventElapsedTime(&ms, e0, e1) == cudaSuccess &&
                    cudaGetLastError() == cudaSuccess && ms > 0.f;
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (!ok) return OMSE_ECUDA;
    *host_out = lane_ops_per_iter * (double)iters / ((double)ms * 1e-3);
    return OMSE_OK;
}

int omse_quantize_weights(omse_ctx* ctx, const float* d_w, int64_t n_kernels, int64_t kernel_len, int bits,
                          int is_signed, const omse_grid* grid, float* d_alpha, float* d_sse,
                          int32_t* d_best_idx, int8_t* d_codes, uint8_t* d_packed) {
    omse_weight_tensor t;
    t.d_w = d_w;
    t.n_kernels = n_kernels;
    t.kernel_len = kernel_len;
    t.d_alpha = d_alpha;
    t.d_sse = d_sse;
    t.d_best_idx = d_best_idx;
    t.d_codes = d_codes;
    t.d_packed = d_packed;
    return omse_quantize_weights_batched(ctx, &t, 1, bits, is_signed, grid);
}

int omse_quantize_weights_batched(omse_ctx* ctx, const omse_weight_tensor* tensors, int n_tensors, int bits,
                                  int is_signed, const omse_grid* grid) {
    if (!ctx || !grid_ok(grid) || bits < 2 || bits > 8 || n_tensors < 0 || n_tensors > OMSE_MAX_BATCH ||
        (n_tensors > 0 && !tensors))
        return OMSE_EINVAL;
    std::vector<omse::RowTensor> list;
    list.reserve((size_t)n_tensors);
    long long max_k = 0;
    for (int i = 0; i < n_tensors; ++i) {
        const omse_weight_tensor& u = tensors[i];
        if (u.n_kernels < 0 || u.kernel_len < 1 || u.kernel_len > OMSE_MAX_KERNEL_LEN || u.n_kernels > (int64_t)1 << 40)
            return OMSE_EINVAL;
        if (u.d_packed && bits > 4) return OMSE_EINVAL;
        if (u.n_kernels == 0) continue;
        if (!u.d_w || !u.d_alpha || !u.d_sse) return OMSE_EINVAL;
        if (misaligned4(u.d_w) || misaligned4(u.d_alpha) || misaligned4(u.d_sse) || misaligned4(u.d_best_idx))
            return OMSE_EINVAL;
        omse::RowTensor t;
        fill_tensor(t, u.d_w, u.n_kernels, u.kernel_len, u.d_alpha, u.d_sse, u.d_best_idx, u.d_codes, u.d_packed);
        list.push_back(t);
        if (u.kernel_len > max_k) max_k = u.kernel_len;
    }
    return quantize_list(ctx, list, max_k, bits, is_signed, grid);
}

int omse_quantize_weights_offset(omse_ctx* ctx, const float* d_w, int64_t n_kernels, int64_t kernel_len, int bits,
                                 const omse_grid* grid, float* d_alpha, float* d_delta, float* d_sse,
                                 int32_t* d_best_idx, int8_t* d_codes, uint8_t* d_packed) {
    if (!ctx || !grid_ok(grid) || bits < 2 || bits > 8 || n_kernels < 0 || kernel_len < 1 ||
        kernel_len > OMSE_MAX_KERNEL_LEN || n_kernels > (int64_t)1 << 40 || (d_packed && bits > 4))
        return OMSE_EINVAL;
    if (n_kernels == 0) return OMSE_OK;
    if (!d_w || !d_alpha || !d_sse || !d_delta) return OMSE_EINVAL;
    if (misaligned4(d_w) || misaligned4(d_alpha) || misaligned4(d_sse) || misaligned4(d_best_idx) || misaligned4(d_delta))
        return OMSE_EINVAL;
    std::vector<omse::RowTensor> list(1);
    fill_tensor(list[0], d_w, n_kernels, kernel_len, d_alpha, d_sse, d_best_idx, d_codes, d_packed);
    list[0].delta = d_delta;
    return quantize_list(ctx, list, kernel_len, bits, /*is_signed=*/0, grid);
}

int omse_residual_quantize(omse_ctx* ctx, const float* d_t, int64_t n_kernels, int64_t kernel_len, const int* bits,
                           int is_signed, const omse_grid* grid, int n_tensors, int n_sweeps, float* d_alpha,
                           float* d_sse, int8_t* d_codes, uint8_t* d_packed) {
    int flags[OMSE_MAX_TENSORS];
    for (int j = 0; j < OMSE_MAX_TENSORS; ++j) flags[j] = is_signed;
    return omse_alg1_quantize(ctx, d_t, n_kernels, kernel_len, bits, flags, grid, n_tensors, n_sweeps, d_alpha, d_sse,
                              nullptr, d_codes, d_packed);
}

static int alg1_impl(omse_ctx* ctx, const float* d_t, int64_t n_kernels, int64_t kernel_len, const int* bits,
                     const int* is_signed, const omse_grid* grid, int n_tensors, int n_sweeps, float eps, float* d_alpha,
                     float* d_sse, float* d_sse_history, int32_t* d_sweeps_done, int8_t* d_codes, uint8_t* d_packed) {
    if (!ctx || !grid_ok(grid) || !bits || !is_signed || n_tensors < 1 || n_tensors > OMSE_MAX_TENSORS || n_sweeps < 1 ||
        n_sweeps > 64 || n_kernels < 0 || kernel_len < 1 || kernel_len > OMSE_MAX_KERNEL_LEN ||
        n_kernels > (int64_t)1 << 40)
        return OMSE_EINVAL;
    for (int j = 0; j < n_tensors; ++j) {
        if (bits[j] < 2 || bits[j] > 8) return OMSE_EINVAL;
        if (d_packed && bits[j] > 4) return OMSE_EINVAL;
    }
    if (n_sweeps > 1 && (!d_codes || kernel_len > OMSE_MAX_KERNEL_LEN_MULTISWEEP)) return OMSE_EINVAL;
    if (n_kernels == 0) return OMSE_OK;
    if (!d_t || !d_alpha || !d_sse) return OMSE_EINVAL;
    if (misaligned4(d_t) || misaligned4(d_alpha) || misaligned4(d_sse) || misaligned4(d_sse_history) ||
        misaligned4(d_sweeps_done))
        return OMSE_EINVAL;
    DeviceScope dev(ctx->device);
    if (!dev.ok()) return OMSE_ECUDA;
    omse::RowArgs a;
    memset(&a, 0, sizeof(a));
    fill_tensor(a.one, d_t, n_kernels, kernel_len, d_alpha, d_sse, nullptr, d_codes, d_packed);
    a.tensors = nullptr;
    a.n_launch_tensors = 1;
    a.n_units = (n_kernels + a.one.rows_per_unit - 1) / a.one.rows_per_unit;
    a.n_cand = grid->n_cand;
    a.hi_frac = grid->hi_frac;
    a.refine_iters = grid->refine_iters;
    a.n_tensors = n_tensors;
    a.n_sweeps = n_sweeps;
    for (int j = 0; j < n_tensors; ++j) bounds(bits[j], is_signed[j], &a.lo[j], &a.hi[j]);
    a.keep_x0 = n_sweeps > 1 ? 1 : 0;
    a.sse_history = d_sse_history;
    a.eps = eps;
    a.sweeps_done = d_sweeps_done;
    return launch_rows(ctx, a, kernel_len, 0, /*path=*/1);   // Algorithm 1 always takes the block-per-row path
}

int omse_alg1_quantize(omse_ctx* ctx, const float* d_t, int64_t n_kernels, int64_t kernel_len, const int* bits,
                       const int* is_signed, const omse_grid* grid, int n_tensors, int n_sweeps, float* d_alpha,
                       float* d_sse, float* d_sse_history, int8_t* d_codes, uint8_t* d_packed) {
    return alg1_impl(ctx, d_t, n_kernels, kernel_len, bits, is_signed, grid, n_tensors, n_sweeps, -1.f, d_alpha, d_sse,
                     d_sse_history, nullptr, d_codes, d_packed);
}

int omse_alg1_quantize_converge(omse_ctx* ctx, const float* d_t, int64_t n_kernels, int64_t kernel_len, const int* bits,
                                const int* is_signed, const omse_grid* grid, int n_tensors, int max_sweeps, float eps,
                                float* d_alpha, float* d_sse, float* d_sse_history, int32_t* d_sweeps_done,
                                int8_t* d_codes, uint8_t* d_packed) {
    if (!(eps >= 0.f)) return OMSE_EINVAL;
    return alg1_impl(ctx, d_t, n_kernels, kernel_len, bits, is_signed, grid, n_tensors, max_sweeps, eps, d_alpha, d_sse,
                     d_sse_history, d_sweeps_done, d_codes, d_packed);
}

int omse_quantize_weights_solver(omse_ctx* ctx, const float* d_w, int64_t n_kernels, int64_t kernel_len, int bits,
                                 int is_signed, int solver, int n_iter, const omse_grid* grid, float* d_alpha,
                                 float* d_sse, int32_t* d_best_idx, int8_t* d_codes, uint8_t* d_packed) {
    if (solver == OMSE_SOLVER_GRID)
        return omse_quantize_weights(ctx, d_w, n_kernels, kernel_len, bits, is_signed, grid, d_alpha, d_sse, d_best_idx,
                                     d_codes, d_packed);
    if (!ctx || !grid_ok(grid) || bits < 2 || bits > 8 || n_kernels < 0 || kernel_len < 1 ||
        kernel_len > OMSE_MAX_KERNEL_LEN || n_kernels > (int64_t)1 << 40 || (d_packed && bits > 4) ||
        solver < OMSE_SOLVER_UNIFORM || solver > OMSE_SOLVER_GOLDEN || n_iter < 0 || n_iter > 1024)
        return OMSE_EINVAL;
    if (n_kernels == 0) return OMSE_OK;
    if (!d_w || !d_alpha || !d_sse) return OMSE_EINVAL;
    if (misaligned4(d_w) || misaligned4(d_alpha) || misaligned4(d_sse) || misaligned4(d_best_idx)) return OMSE_EINVAL;
    std::vector<omse::RowTensor> list(1);
    fill_tensor(list[0], d_w, n_kernels, kernel_len, d_alpha, d_sse, d_best_idx, d_codes, d_packed);
    ListMode mode;
    mode.solver = solver;
    mode.solver_iters = n_iter;
    return quantize_list(ctx, list, kernel_len, bits, is_signed, grid, mode);
}

int omse_quantize_weights_affine(omse_ctx* ctx, const float* d_w, int64_t n_kernels, int64_t kernel_len, int bits,
                                 const omse_grid* grid, const omse_offset_grid* offsets, float* d_alpha, float* d_delta,
                                 float* d_sse, int32_t* d_best_idx, int8_t* d_codes, uint8_t* d_packed) {
    if (!ctx || !grid_ok(grid) || !offsets || offsets->n_delta < 1 || offsets->n_delta > OMSE_MAX_OFFSETS ||
        !(offsets->off_frac >= 0.f) || !(offsets->off_frac <= 1.f) || bits < 2 || bits > 8 || n_kernels < 0 ||
        kernel_len < 1 || kernel_len > OMSE_MAX_KERNEL_LEN_MULTISWEEP || n_kernels > (int64_t)1 << 40 ||
        (d_packed && bits > 4) || (int64_t)offsets->n_delta * grid->n_cand > 0x7fffffff)
        return OMSE_EINVAL;
    if (n_kernels == 0) return OMSE_OK;
    if (!d_w || !d_alpha || !d_sse || !d_delta) return OMSE_EINVAL;
    if (misaligned4(d_w) || misaligned4(d_alpha) || misaligned4(d_sse) || misaligned4(d_best_idx) || misaligned4(d_delta))
        return OMSE_EINVAL;
    std::vector<omse::RowTensor> list(1);
    fill_tensor(list[0], d_w, n_kernels, kernel_len, d_alpha, d_sse, d_best_idx, d_codes, d_packed);
    list[0].delta = d_delta;
    ListMode mode;
    mode.n_delta = offsets->n_delta;
    mode.off_frac = offsets->off_frac;
    return quantize_list(ctx, list, kernel_len, bits, /*is_signed=*/0, grid, mode);
}

int omse_quantize_key_layers(omse_ctx* ctx, const omse_key_layer* layers, int n_layers, int bits, int is_signed,
                             const omse_grid* grid, float tau, double* d_mse, int32_t* d_is_key, double* d_cr) {
    if (!ctx || !grid_ok(grid) || bits < 2 || bits > 8 || n_layers < 0 || n_layers > OMSE_MAX_BATCH ||
        (n_layers > 0 && (!layers || !d_mse || !d_is_key)) || !(tau >= 0.f))
        return OMSE_EINVAL;
    if ((reinterpret_cast<uintptr_t>(d_mse) & 7) || (reinterpret_cast<uintptr_t>(d_cr) & 7) || misaligned4(d_is_key))
        return OMSE_EINVAL;
    std::vector<omse_weight_tensor> first((size_t)n_layers);
    std::vector<omse_layer_error> errs((size_t)n_layers);
    for (int l = 0; l < n_layers; ++l) {
        const omse_key_layer& L = layers[l];
        if (L.first.n_kernels < 1 || L.first.kernel_len < 1 || L.first.kernel_len > OMSE_MAX_KERNEL_LEN ||
            !L.d_alpha2 || !L.d_sse2 || misaligned4(L.d_alpha2) || misaligned4(L.d_sse2) || (L.d_packed2 && bits > 4))
            return OMSE_EINVAL;
        first[l] = L.first;
        errs[l].d_sse = L.first.d_sse;
        errs[l].n_kernels = L.first.n_kernels;
        errs[l].kernel_len = L.first.kernel_len;
    }
    if (n_layers == 0) return OMSE_OK;
    // 1. every layer with one quantized tensor; 2. MSE per layer against tau
    int rc = omse_quantize_weights_batched(ctx, first.data(), n_layers, bits, is_signed, grid);
    if (rc != OMSE_OK) return rc;
    rc = omse_select_key_layers(ctx, errs.data(), n_layers, tau, d_mse, d_is_key);
    if (rc != OMSE_OK) return rc;
    // 3. one launch over all layers for the second tensor: blocks skip the layers whose flag is 0, so the host
    //    never reads the flags; each row's residual is rebuilt on chip from the first scale
    std::vector<omse::RowTensor> list((size_t)n_layers);
    long long max_k = 0;
    for (int l = 0; l < n_layers; ++l) {
        const omse_key_layer& L = layers[l];
        fill_tensor(list[l], L.first.d_w, L.first.n_kernels, L.first.kernel_len, L.d_alpha2, L.d_sse2, nullptr,
                    L.d_codes2, L.d_packed2);
        list[l].prior_alpha = L.first.d_alpha;
        list[l].gate = d_is_key + l;
        if (L.first.kernel_len > max_k) max_k = L.first.kernel_len;
    }
    rc = quantize_list(ctx, list, max_k, bits, is_signed, grid);
    if (rc != OMSE_OK) return rc;
    // 4. compression ratio of the result (one or two quantized tensors per layer)
    if (d_cr) {
        DeviceScope dev(ctx->device);
        if (!dev.ok()) return OMSE_ECUDA;
        std::vector<omse::LayerError> shape((size_t)n_layers);
        for (int l = 0; l < n_layers; ++l) {
            shape[l].sse = nullptr;
            shape[l].n_kernels = layers[l].first.n_kernels;
            shape[l].kernel_len = layers[l].first.kernel_len;
        }
        omse::LayerError* d_layers = reinterpret_cast<omse::LayerError*>(ctx->d_tensors);
        if (cudaMemcpyAsync(d_layers, shape.data(), sizeof(omse::LayerError) * shape.size(), cudaMemcpyHostToDevice,
                            ctx->stream) != cudaSuccess)
            return OMSE_ECUDA;
        omse::compression_ratio_kernel<<<1, 32, 0, ctx->stream>>>(d_layers, n_layers, bits, d_is_key, d_cr);
        ++ctx->n_launches;
        if (cudaGetLastError() != cudaSuccess) return OMSE_ECUDA;
    }
    return OMSE_OK;
}

int omse_dual_quantize(omse_ctx* ctx, const float* d_t, int64_t n_kernels, int64_t kernel_len, int bits1, int bits2,
                       int is_signed, const omse_dual_grid* grid, float* d_alpha, float* d_sse, int32_t* d_best_idx,
                       int8_t* d_codes, uint8_t* d_packed) {
    if (!ctx || !grid || grid->n_cand1 < 1 || grid->n_cand2 < 1 || grid->n_cand1 > OMSE_DUAL_MAX_CANDIDATES ||
        grid->n_cand2 > OMSE_DUAL_MAX_CANDIDATES || !(grid->hi_frac1 > 0.f) || !(grid->hi_frac2 > 0.f) ||
        !(grid->hi_frac1 <= 3.0e38f) || !(grid->hi_frac2 <= 3.0e38f) || bits1 < 2 || bits1 > 8 || bits2 < 2 ||
        bits2 > 8 || n_kernels < 0 || kernel_len < 1 || kernel_len > OMSE_MAX_KERNEL_LEN || n_kernels > (int64_t)1 << 40)
        return OMSE_EINVAL;
    if (d_packed && (bits1 > 4 || bits2 > 4)) return OMSE_EINVAL;
    if (n_kernels == 0) return OMSE_OK;
    if (!d_t || !d_alpha || !d_sse) return OMSE_EINVAL;
    if (misaligned4(d_t) || misaligned4(d_alpha) || misaligned4(d_sse) || misaligned4(d_best_idx)) return OMSE_EINVAL;
    DeviceScope dev(ctx->device);
    if (!dev.ok()) return OMSE_ECUDA;
    omse::DualArgs a;
    memset(&a, 0, sizeof(a));
    a.t = d_t;
    a.S = n_kernels;
    a.K = kernel_len;
    a.n_cand1 = grid->n_cand1;
    a.n_cand2 = grid->n_cand2;
    a.hi_frac1 = grid->hi_frac1;
    a.hi_frac2 = grid->hi_frac2;
    bounds(bits1, is_signed, &a.lo1, &a.hi1);
    bounds(bits2, is_signed, &a.lo2, &a.hi2);
    a.alpha = d_alpha;
    a.sse = d_sse;
    a.best_idx = d_best_idx;
    a.codes = reinterpret_cast<signed char*>(d_codes);
    a.packed = d_packed;
    a.status = &ctx->ws->status;
    a.rows_per_unit = (d_packed && (kernel_len & 1)) ? 2 : 1;
    const size_t smem = (size_t)((kernel_len + 3) & ~3ll) * 4 + 64 * 8 + omse::kDualListCap * 4 + 4 * 4;
    if (!ctx->attr_dual) {
        if (cudaFuncSetAttribute(omse::dual_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem) != cudaSuccess)
            return OMSE_ECUDA;
        ctx->attr_dual = true;
    }
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, omse::dual_kernel, omse::kDualThreads, smem) != cudaSuccess || occ < 1)
        return OMSE_ECUDA;
    const long long n_units = (n_kernels + a.rows_per_unit - 1) / a.rows_per_unit;
    long long blocks = (long long)ctx->n_sm * occ;
    if (blocks > n_units) blocks = n_units;
    // every block keeps the fp32 grid of its current row in the context workspace
    const long long cap = (long long)(kPartialBytes / ((size_t)grid->n_cand1 * grid->n_cand2 * 4));
    if (blocks > cap) blocks = cap;
    if (blocks < 1) return OMSE_EINVAL;
    a.curve = reinterpret_cast<float*>(ctx->partials);
    a.evals = &ctx->ws->evals;
    omse::dual_kernel<<<(unsigned)blocks, omse::kDualThreads, smem, ctx->stream>>>(a);
    ++ctx->n_launches;
    return cudaGetLastError() == cudaSuccess ? OMSE_OK : OMSE_ECUDA;
}

int omse_select_key_layers(omse_ctx* ctx, const omse_layer_error* layers, int n_layers, float tau, double* d_mse,
                           int32_t* d_is_key) {
    if (!ctx || n_layers < 0 || n_layers > OMSE_MAX_BATCH || (n_layers > 0 && (!layers || !d_mse)) || !(tau >= 0.f))
        return OMSE_EINVAL;
    if ((reinterpret_cast<uintptr_t>(d_mse) & 7) || misaligned4(d_is_key)) return OMSE_EINVAL;
    static_assert(sizeof(omse::LayerError) <= sizeof(omse::RowTensor), "descriptor buffer too small");
    std::vector<omse::LayerError> list((size_t)n_layers);
    for (int i = 0; i < n_layers; ++i) {
        if (!layers[i].d_sse || layers[i].n_kernels < 1 || layers[i].kernel_len < 1 || misaligned4(layers[i].d_sse))
            return OMSE_EINVAL;
        list[i].sse = layers[i].d_sse;
        list[i].n_kernels = layers[i].n_kernels;
        list[i].kernel_len = layers[i].kernel_len;
    }
    if (n_layers == 0) return OMSE_OK;
    DeviceScope dev(ctx->device);
    if (!dev.ok()) return OMSE_ECUDA;
    omse::LayerError* d_layers = reinterpret_cast<omse::LayerError*>(ctx->d_tensors);
    if (cudaMemcpyAsync(d_layers, list.data(), sizeof(omse::LayerError) * list.size(), cudaMemcpyHostToDevice,
                        ctx->stream) != cudaSuccess)
        return OMSE_ECUDA;
    omse::layer_mse_kernel<<<(unsigned)n_layers, 256, 0, ctx->stream>>>(d_layers, tau, d_mse, d_is_key);
    ++ctx->n_launches;
    return cudaGetLastError() == cudaSuccess ? OMSE_OK : OMSE_ECUDA;
}

double omse_compression_ratio(const int64_t* n_kernels, const int64_t* kernel_len, const int* bits, const int* n_tensors,
                              int n_layers) {
    if (!n_kernels || !kernel_len || !bits || !n_tensors || n_layers < 1) return -1.0;
    double q = 0.0, f = 0.0;
    for (int l = 0; l < n_layers; ++l) {
        if (n_kernels[l] < 0 || kernel_len[l] < 1 || bits[l] < 1 || n_tensors[l] < 1) return -1.0;
        const double n = (double)n_kernels[l] * (double)kernel_len[l];
        q += (double)n_tensors[l] * (n * (double)bits[l] + 32.0 * (double)n_kernels[l]);
        f += 32.0 * n;
    }
    return f > 0.0 ? q / f : -1.0;
}

int omse_activation_scale(omse_ctx* ctx, const float* d_x, int64_t n, int bits, int is_signed, const omse_grid* grid,
                          float* d_alpha, float* d_sse, int32_t* d_best_idx, double* d_sse_curve) {
    return activation_impl(ctx, d_x, n, bits, is_signed, grid, d_alpha, nullptr, d_sse, d_best_idx, d_sse_curve);
}

int omse_activation_scale_offset(omse_ctx* ctx, const float* d_x, int64_t n, int bits, const omse_grid* grid,
                                 float* d_alpha, float* d_delta, float* d_sse, int32_t* d_best_idx,
                                 double* d_sse_curve) {
    if (!d_delta || misaligned4(d_delta)) return OMSE_EINVAL;
    return activation_impl(ctx, d_x, n, bits, /*is_signed=*/0, grid, d_alpha, d_delta, d_sse, d_best_idx, d_sse_curve);
}

}  // extern "C"

static int activation_impl(omse_ctx* ctx, const float* d_x, int64_t n, int bits, int is_signed, const omse_grid* grid,
                           float* d_alpha, float* d_delta, float* d_sse, int32_t* d_best_idx, double* d_sse_curve) {
    if (!ctx || !grid_ok(grid) || bits < 2 || bits > 8 || n < 0 || !d_alpha || !d_sse) return OMSE_EINVAL;
    if (n > 0 && !d_x) return OMSE_EINVAL;
    if ((reinterpret_cast<uintptr_t>(d_x) & 15) || (reinterpret_cast<uintptr_t>(d_alpha) & 3) ||
        (reinterpret_cast<uintptr_t>(d_sse) & 3) || (reinterpret_cast<uintptr_t>(d_best_idx) & 3) ||
        (reinterpret_cast<uintptr_t>(d_sse_curve) & 7))
        return OMSE_EINVAL;
    DeviceScope dev(ctx->device);
    if (!dev.ok()) return OMSE_ECUDA;
    omse::TensorArgs a;
    memset(&a, 0, sizeof(a));
    a.x = d_x;
    a.n = n;
    a.n_cand = grid->n_cand;
    a.hi_frac = grid->hi_frac;
    bounds(bits, is_signed, &a.lo, &a.hi);
    a.st = &ctx->ws->tstate;
    a.partials = ctx->partials;
    a.partial_doubles = (long long)(kPartialBytes / 8);
    a.list = ctx->ws->list;
    a.curve = ctx->ws->curve;
    a.curve_out = d_sse_curve;
    a.alpha_out = d_alpha;
    a.sse_out = d_sse;
    a.idx_out = d_best_idx;
    a.delta_out = d_delta;
    a.evals = &ctx->ws->evals;
    a.status = &ctx->ws->status;
    omse::tensor_init_kernel<<<1, 32, 0, ctx->stream>>>(a.st);
    ++ctx->n_launches;
    const TensorEnv env = {ctx->n_sm, ctx->stream, ctx->occ_sweep, ctx->occ_pass, true, ctx->attr_tensor, &ctx->n_launches};
    return enqueue_tensor_search(env, a, grid->refine_iters);
}

extern "C" {

int omse_pack_int4(omse_ctx* ctx, const int8_t* d_codes, int64_t n, int is_signed, uint8_t* d_packed) {
    (void)is_signed;
    if (!ctx || n < 0) return OMSE_EINVAL;
    if (n == 0) return OMSE_OK;
    if (!d_codes || !d_packed) return OMSE_EINVAL;
    DeviceScope dev(ctx->device);
    if (!dev.ok()) return OMSE_ECUDA;
    long long grid = (n / 16 + 255) / 256;
    if (grid > (long long)ctx->n_sm * 16) grid = (long long)ctx->n_sm * 16;
    if (grid < 1) grid = 1;
    omse::pack_int4_kernel<<<(unsigned)grid, 256, 0, ctx->stream>>>(reinterpret_cast<const signed char*>(d_codes), n, d_packed);
    ++ctx->n_launches;
    return cudaGetLastError() == cudaSuccess ? OMSE_OK : OMSE_ECUDA;
}

}  // extern "C"

// -------------------------------------------------------------------------------------------------
// Allocation-free per-tensor search (omse_activation_scale_static).  The scratch that
// omse_activation_scale takes from the context workspace lives here in a fixed device array; every
// GPU that loads the library holds OMSE_STATIC_SCRATCH_BYTES of it until the process exits.
// -------------------------------------------------------------------------------------------------
namespace {

constexpr size_t kStaticPartialDoubles = 1u << 19;   // 4 MiB of per-block partial sums

struct StaticScratch {
    unsigned int status;
    unsigned int pad_[3];
    omse::TensorState tstate;
    double curve[OMSE_STATIC_MAX_CANDIDATES];
    int list[OMSE_STATIC_MAX_CANDIDATES];
    double partials[kStaticPartialDoubles];
};
static_assert(sizeof(StaticScratch) <= OMSE_STATIC_SCRATCH_BYTES, "static scratch larger than documented");

// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[OMSE_STATIC_SCRATCH_BYTES];

struct StaticDevice {
    StaticScratch* ptr;   // device address of g_static_scratch on this device
    int n_sm;
    bool ready;
    int occ_sweep[2], occ_pass[3];
    bool attr_unused[4];
};
StaticDevice g_static_dev[64];
std::mutex g_static_mutex;

// Everything that must start from zero: the array keeps the previous call's contents.
__global__ void static_begin_kernel(StaticScratch* s) {
    if (threadIdx.x == 0) {
        s->status = 0u;
        s->tstate.mpos_bits = 0u;
        s->tstate.mneg_bits = 0u;
        s->tstate.ticket = 0u;
        s->tstate.best_idx = -1;
        s->tstate.alpha = 0.f;
        s->tstate.step = 0.f;
        s->tstate.n_list = 0;
        s->tstate.list_overflow = 0;
        s->tstate.polish_done = 0;
        s->tstate.key_min = 0x7fffffff;
        s->tstate.key_max = (int)0x80000000;
        s->tstate.delta = 0.f;
    }
}

__global__ void static_end_kernel(const StaticScratch* s, unsigned int* d_status) {
    if (threadIdx.x == 0 && d_status) *d_status = s->status;
}

}  // namespace

extern "C" int omse_activation_scale_static(int device, void* cuda_stream, const float* d_x, int64_t n, int bits,
                                            int is_signed, const omse_grid* grid, float* d_alpha, float* d_sse,
                                            int32_t* d_best_idx, double* d_sse_curve, uint32_t* d_status) {
    if (!grid_ok(grid) || bits < 2 || bits > 8 || n < 0 || !d_alpha || !d_sse || device < 0 || device >= 64)
        return OMSE_EINVAL;
    if (grid->n_cand > OMSE_STATIC_MAX_CANDIDATES) return OMSE_ELIMIT;
    if (n > 0 && !d_x) return OMSE_EINVAL;
    if ((reinterpret_cast<uintptr_t>(d_x) & 15) || (reinterpret_cast<uintptr_t>(d_alpha) & 3) ||
        (reinterpret_cast<uintptr_t>(d_sse) & 3) || (reinterpret_cast<uintptr_t>(d_best_idx) & 3) ||
        (reinterpret_cast<uintptr_t>(d_sse_curve) & 7) || (reinterpret_cast<uintptr_t>(d_status) & 3))
        return OMSE_EINVAL;
    DeviceScope dev(device);
    if (!dev.ok()) return OMSE_ECUDA;
    StaticDevice& sd = g_static_dev[device];
    {
        // once per device, with that device current: the device address of the array
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!sd.ready) {
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return OMSE_ECUDA;
            if (cudaDeviceGetAttribute(&sd.n_sm, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) return OMSE_ECUDA;
            sd.ptr = static_cast<StaticScratch*>(p);
            sd.ready = true;
        }
    }
    StaticScratch* sc = sd.ptr;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    omse::TensorArgs a;
    memset(&a, 0, sizeof(a));
    a.x = d_x;
    a.n = n;
    a.n_cand = grid->n_cand;
    a.hi_frac = grid->hi_frac;
    bounds(bits, is_signed, &a.lo, &a.hi);
    a.st = &sc->tstate;
    a.partials = sc->partials;
    a.partial_doubles = (long long)kStaticPartialDoubles;
    a.list = sc->list;
    a.curve = sc->curve;
    a.curve_out = d_sse_curve;
    a.alpha_out = d_alpha;
    a.sse_out = d_sse;
    a.idx_out = d_best_idx;
    a.status = &sc->status;

    static_begin_kernel<<<1, 32, 0, s>>>(sc);
    // the sweep stays below 48 KB of dynamic shared memory, so no attribute call is needed here
    unsigned long long not_counted = 0;
    const TensorEnv env = {sd.n_sm, s, sd.occ_sweep, sd.occ_pass, false, sd.attr_unused, &not_counted};
    const int rc = enqueue_tensor_search(env, a, grid->refine_iters);
    if (rc != OMSE_OK) return rc;
    static_end_kernel<<<1, 32, 0, s>>>(sc, d_status);
    return cudaGetLastError() == cudaSuccess ? OMSE_OK : OMSE_ECUDA;
}

