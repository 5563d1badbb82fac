/*
 * omse.h - C interface of the B200 (sm_100a) constrained-MMSE quantization library.
 *
 * The library computes the data-parallel part of "Low-bit Quantization of Neural Networks
 * for Efficient Inference" (Choukroun et al., arXiv:1902.06822): for a tensor T and a
 * b-bit integer range Z_p it finds the scale alpha minimising ||T - alpha*[T/alpha]_Zp||_F^2
 * (Section 3.4) by evaluating a grid of candidate scales and polishing the best one with
 * the closed-form least-squares update; kernel-wise for weights (Section 3.3), per tensor
 * for activations (Section 3.7); optionally as a sum of several low-precision tensors
 * (Section 3.5, Algorithm 1; Section 3.7 residual form); and it emits INT4 codes.
 *
 * Conventions that hold for every entry point
 *   - Every pointer named d_* is DEVICE memory owned by the caller.  It must stay valid until
 *     the work queued by the call has finished on the context's stream.  The library keeps
 *     no pointer after the work completes.  float/int32 buffers must be 4-byte aligned,
 *     double buffers 8-byte aligned; only omse_activation_scale* asks for more (16 bytes for
 *     d_x).  Rows of odd length and views at odd offsets are therefore accepted as they are.
 *   - Pointers without the d_ prefix are HOST memory, read before the call returns.
 *   - Calls only enqueue work on the context's CUDA stream and return; nothing synchronises
 *     except omse_last_device_status(), omse_read_evaluations() and omse_destroy().  A call
 *     whose list holds both long and short kernels runs one of its two launches on a second
 *     stream that the context owns, forked from the context's stream and joined back to it by
 *     events inside the call: for the caller everything stays ordered on the context's stream.
 *   - All work queued through one context shares that context's device workspace (work-unit
 *     dispenser, search state, partial sums).  It must therefore be stream-ordered: after
 *     omse_set_stream() the caller makes the new stream wait for the work already queued on the
 *     old one (an event), otherwise two calls of one context may overlap on the GPU and corrupt
 *     each other.  Use one context per stream for concurrent work.
 *   - Every call makes the context's device current while it runs and restores the caller's
 *     current device before it returns.
 *   - The return value is OMSE_OK or a negative omse_status.  Invalid arguments are
 *     rejected before anything is enqueued.  Data-dependent conditions (NaN/Inf in the
 *     input, an all-zero segment) never fail a call: they set bits in the device status
 *     word (omse_last_device_status) and produce the outputs documented below.
 *   - There is no CPU fallback: without a CUDA device omse_create() fails.
 *
 * Quantization range (Section 3.1): signed Z_p = {-2^(p-1) .. 2^(p-1)-1}, unsigned
 * Z_p = {0 .. 2^p-1}.  [.]_Zp is IEEE binary32 division by alpha, round to nearest with
 * ties to even, then saturation to the range.
 */
#ifndef OMSE_H
#define OMSE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    OMSE_OK = 0,
    OMSE_EINVAL = -1, /* NULL pointer, size or parameter out of range                 */
    OMSE_ECUDA = -2,  /* a CUDA runtime call or a kernel launch failed                */
    OMSE_ENOMEM = -3, /* the context workspace could not be allocated                 */
    OMSE_ELIMIT = -4  /* a size exceeds the fixed scratch of omse_activation_scale_static */
} omse_status;

/* bits of the device status word */
#define OMSE_DEV_NONFINITE 1u  /* a NaN or Inf was read from an input tensor                          */
#define OMSE_DEV_DEGENERATE 2u /* a segment had max|x| = 0 (or below FLT_MIN*C): alpha=0, codes 0 */

/* Largest supported sizes. */
#define OMSE_MAX_CANDIDATES 4096   /* n_cand                                                        */
#define OMSE_MAX_KERNEL_LEN 28672  /* kernel_len of the kernel-wise entry points (one row on chip) */
#define OMSE_MAX_KERNEL_LEN_MULTISWEEP 25600 /* with n_sweeps > 1 (row and residual both on chip)       */
#define OMSE_MAX_TENSORS 4         /* n_tensors of omse_residual_quantize                           */
#define OMSE_MAX_BATCH 1024        /* weight tensors per omse_quantize_weights_batched call         */

/* The grid of the line search of Section 3.4 (the paper fixes neither its range nor its spacing):
 * n_cand scales spaced linearly in (0, hi_frac*max|x|], candidate c (0-based) being
 * fl(fl(c+1) * fl(fl(hi_frac*max|x|)/fl(n_cand))) in binary32.  refine_iters is the number of
 * closed-form polish steps (alpha <- <x,q>/<q,q> with q = [x/alpha]_Zp) applied to the best
 * candidate; a step that reproduces the scale bit for bit ends the polish early (later steps would
 * repeat it), as does <q,q> = 0 or a scale that is not a normal positive number. */
typedef struct {
    int32_t n_cand;       /* 1 .. OMSE_MAX_CANDIDATES                    */
    float hi_frac;        /* > 0; 1.0 puts the last candidate at max|x| */
    int32_t refine_iters; /* 0 .. 64                                     */
} omse_grid;

typedef struct omse_ctx omse_ctx;

/* Creates a context bound to CUDA device `device` and to `cuda_stream` (a cudaStream_t, borrowed,
 * NULL = the legacy default stream).  Allocates the device workspace (omse_workspace_bytes).  One
 * context must not be used from two host threads at once; different contexts are independent.
 * Returns OMSE_ECUDA if the device is absent. */
int omse_create(omse_ctx** out, int device, void* cuda_stream);

/* Waits for the stream, frees the workspace and the context. */
int omse_destroy(omse_ctx* ctx);

/* Replaces the stream later calls enqueue on (borrowed).  See the stream-ordering rule above. */
int omse_set_stream(omse_ctx* ctx, void* cuda_stream);

/* Bytes of device workspace a context allocates for calls of the given size (n_kernels rows of
 * kernel_len elements, n_cand candidates, n_tensors quantized tensors per row).  Rows are searched
 * on chip, so the answer is the same for every valid size (about 16.5 MB); 0 for invalid arguments. */
size_t omse_workspace_bytes(int64_t n_kernels, int64_t kernel_len, int32_t n_cand, int32_t n_tensors);

/*
 * Kernel-wise MMSE quantization of a weight tensor (Sections 3.3 and 3.4).
 * d_w is row-major [n_kernels][kernel_len] binary32: row k is kernel W_lk flattened
 * (kernel_len = c*w*h).  Each row gets its own scale.  bits in 2..8.
 * Outputs (each nullable except d_alpha and d_sse):
 *   d_alpha   [n_kernels] float  final scale (0 for a degenerate row)
 *   d_sse     [n_kernels] float  ||W_lk - alpha*q||^2 at the final scale (accumulated in binary64)
 *   d_best_idx[n_kernels] int32  winning grid index, lowest index among equal errors (-1 degenerate)
 *   d_codes   [n_kernels*kernel_len] int8   the codes q
 *   d_packed  [ceil(n_kernels*kernel_len/2)] uint8  the same codes as nibbles (layout: omse_pack_int4);
 *             only for bits <= 4.
 * Limits: 1 <= kernel_len <= OMSE_MAX_KERNEL_LEN, n_kernels >= 0 (0 enqueues nothing).
 */
int omse_quantize_weights(omse_ctx* ctx, const float* d_w, int64_t n_kernels, int64_t kernel_len,
                          int bits, int is_signed, const omse_grid* grid, float* d_alpha,
                          float* d_sse, int32_t* d_best_idx, int8_t* d_codes, uint8_t* d_packed);

/*
 * The same operation on a set of weight tensors (the layers W_1..W_L of a network, Section 3.1) in
 * ONE launch: kernels of all tensors are handed out to the thread blocks longest first, so the GPU
 * stays full across layer boundaries.  `tensors` is a HOST array of n_tensors descriptors (read
 * before the call returns); each descriptor's fields have the meaning and nullability of the
 * arguments of omse_quantize_weights.  bits / is_signed / grid apply to every tensor.
 * 0 <= n_tensors <= OMSE_MAX_BATCH; tensors with n_kernels == 0 are skipped.
 */
typedef struct {
    const float* d_w;
    int64_t n_kernels, kernel_len;
    float* d_alpha;
    float* d_sse;
    int32_t* d_best_idx;
    int8_t* d_codes;
    uint8_t* d_packed;
} omse_weight_tensor;

int omse_quantize_weights_batched(omse_ctx* ctx, const omse_weight_tensor* tensors, int n_tensors,
                                  int bits, int is_signed, const omse_grid* grid);

/*
 * Per-tensor MMSE scale for an activation tensor (Section 3.7, first equation): one scale for
 * all n elements of d_x.  Outputs: d_alpha[1], d_sse[1] (float), d_best_idx[1] (nullable),
 * d_sse_curve[n_cand] (nullable, double): the squared error at every candidate, i.e. the curve of
 * Figure 1, accumulated in binary32 blocks of 128 elements folded into binary64.
 * n >= 0 (0 is treated as a degenerate tensor).  d_x must be 16-byte aligned (128-bit loads).
 */
int omse_activation_scale(omse_ctx* ctx, const float* d_x, int64_t n, int bits, int is_signed,
                          const omse_grid* grid, float* d_alpha, float* d_sse,
                          int32_t* d_best_idx, double* d_sse_curve);

/*
 * Multiple-tensor quantization T ~ sum_j alpha_j q^j (Section 3.5, Algorithm 1), kernel-wise.
 * All alpha_j and q^j start at zero; each of the n_sweeps sweeps visits j = 1..n_tensors and
 * replaces (alpha_j, q^j) by the MMSE quantization (as in omse_quantize_weights, bits[j]) of the
 * residual T - sum_{i != j} alpha_i q^i, formed in binary32 by fused multiply-adds in increasing i.
 * n_sweeps = 1 is the residual scheme of Section 3.7 (second equation).
 * bits: HOST array [n_tensors].  Outputs are for the last sweep, tensor-major:
 *   d_alpha [n_tensors][n_kernels], d_sse [n_tensors][n_kernels] (error after tensors 1..j updated),
 *   d_codes [n_tensors][n_kernels*kernel_len] int8 (nullable when n_sweeps == 1),
 *   d_packed[n_tensors][ceil(n_kernels*kernel_len/2)] (nullable; needs every bits[j] <= 4).
 * Limits: 1 <= n_tensors <= OMSE_MAX_TENSORS; 1 <= n_sweeps <= 64; n_sweeps > 1 needs d_codes
 * (the codes of the other tensors are read back from it) and
 * kernel_len <= OMSE_MAX_KERNEL_LEN_MULTISWEEP.
 */
int omse_residual_quantize(omse_ctx* ctx, const float* d_t, int64_t n_kernels, int64_t kernel_len,
                           const int* bits, int is_signed, const omse_grid* grid, int n_tensors,
                           int n_sweeps, float* d_alpha, float* d_sse, int8_t* d_codes,
                           uint8_t* d_packed);

/*
 * Quantization with offset (Section 3.1, first displayed scheme: T^ = alpha*[(T - delta)/alpha]_Zp + delta,
 * delta = min_i T_i, unsigned range Z_p = {0..2^p-1}) with the scale found by the MMSE search of
 * Section 3.4 instead of the (max - delta)/(2^p - 1) rule.  Each kernel (omse_quantize_weights_offset) or
 * the whole tensor (omse_activation_scale_offset) is shifted by its minimum in binary32, fl(T_i - delta),
 * and searched on the unsigned grid; d_delta receives the offsets ([n_kernels] or [1]).  The reported
 * error is that of the shifted values.  Codes are unsigned: for bits = 8 the int8 buffer holds the byte.
 * Everything else as in omse_quantize_weights / omse_activation_scale.
 */
int omse_quantize_weights_offset(omse_ctx* ctx, const float* d_w, int64_t n_kernels, int64_t kernel_len,
                                 int bits, const omse_grid* grid, float* d_alpha, float* d_delta,
                                 float* d_sse, int32_t* d_best_idx, int8_t* d_codes, uint8_t* d_packed);
int omse_activation_scale_offset(omse_ctx* ctx, const float* d_x, int64_t n, int bits,
                                 const omse_grid* grid, float* d_alpha, float* d_delta, float* d_sse,
                                 int32_t* d_best_idx, double* d_sse_curve);

/*
 * omse_residual_quantize with one signedness flag per quantized tensor and the convergence history of
 * Algorithm 1 (Section 3.5).  is_signed: HOST array [n_tensors] (a non-negative
 * tensor may take an unsigned first tensor and a signed tensor for its residual, whose rounding errors
 * have both signs).  d_sse_history (nullable): [n_sweeps][n_tensors][n_kernels] float, the squared
 * error after every update, in the order the updates are made; its last [n_tensors][n_kernels] block
 * equals d_sse.  Everything else as in omse_residual_quantize.
 */
int omse_alg1_quantize(omse_ctx* ctx, const float* d_t, int64_t n_kernels, int64_t kernel_len,
                       const int* bits, const int* is_signed, const omse_grid* grid, int n_tensors,
                       int n_sweeps, float* d_alpha, float* d_sse, float* d_sse_history,
                       int8_t* d_codes, uint8_t* d_packed);

/*
 * Algorithm 1 with its loop condition (Section 3.5, Algorithm 1: the sweeps go on until the error stops
 * improving by more than a threshold).  The paper does not define the rate; here it is the relative decrease of a kernel's
 * squared error over one sweep, (E_prev - E_cur)/E_prev, E being the error after the last tensor's update and
 * E_0 = ||T_k||^2.  Each kernel stops on its own after the first sweep whose rate is not above eps, or after
 * max_sweeps sweeps.  d_sweeps_done (nullable) [n_kernels] int32: sweeps that ran; history entries of sweeps
 * that did not run repeat the last error.  eps >= 0; everything else as in omse_alg1_quantize with
 * n_sweeps = max_sweeps.
 */
int omse_alg1_quantize_converge(omse_ctx* ctx, const float* d_t, int64_t n_kernels, int64_t kernel_len,
                                const int* bits, const int* is_signed, const omse_grid* grid, int n_tensors,
                                int max_sweeps, float eps, float* d_alpha, float* d_sse, float* d_sse_history,
                                int32_t* d_sweeps_done, int8_t* d_codes, uint8_t* d_packed);

/*
 * The other ways of choosing the scale that Section 3.4 compares the grid search with (the columns of its table
 * of quantization methods), on the same objective and with the same outputs as omse_quantize_weights:
 *   OMSE_SOLVER_GRID         the line search itself (identical to omse_quantize_weights; n_iter unused);
 *   OMSE_SOLVER_UNIFORM      the no-offset uniform quantizer of Section 3.1, alpha = max|W_k| / L with L the
 *                            largest code of the range (2^(bits-1)-1 signed, 2^bits-1 unsigned);
 *   OMSE_SOLVER_ALTERNATING  alternating optimisation from that scale: n_iter least-squares steps
 *                            alpha <- <x,q>/<q,q>, q = [x/alpha]_Zp;
 *   OMSE_SOLVER_GOLDEN       golden-section search on the bracket [0, grid->hi_frac*max|W_k|] with n_iter
 *                            shrink steps.  The paper gives neither bracket nor stopping rule; this library's:
 *                            scales in binary32, rho = 0.618034f, interior points x1 = b - rho*(b-a) and
 *                            x2 = a + rho*(b-a) (every operation rounded), the bracket becomes [a, x2] when
 *                            f(x1) <= f(x2) and [x1, b] otherwise, the result is the interior point with the
 *                            smaller error (x1 on equal errors), errors accumulated in binary64.
 * grid->refine_iters further least-squares steps follow every solver (0 for the plain methods); grid->n_cand is
 * used by the grid solver only.  d_best_idx receives 0 (-1 for a degenerate kernel) for the other solvers.
 * 0 <= n_iter <= 1024.
 */
typedef enum {
    OMSE_SOLVER_GRID = 0,
    OMSE_SOLVER_UNIFORM = 1,
    OMSE_SOLVER_ALTERNATING = 2,
    OMSE_SOLVER_GOLDEN = 3
} omse_solver;

int omse_quantize_weights_solver(omse_ctx* ctx, const float* d_w, int64_t n_kernels, int64_t kernel_len, int bits,
                                 int is_signed, int solver, int n_iter, const omse_grid* grid, float* d_alpha,
                                 float* d_sse, int32_t* d_best_idx, int8_t* d_codes, uint8_t* d_packed);

/*
 * Quantization with offset (Section 3.1, first displayed scheme) with the offset searched as well as the scale.
 * The paper fixes delta = min_i T_i; for a kernel with long tails on both sides the smallest error needs the low
 * end clipped too.  With lo = min W_k, R = fl(max W_k - lo) the offsets are
 *     delta_d = fl(lo + fl(fl(d) * fl(fl(off_frac*R)/fl(n_delta)))),   d = 0 .. n_delta-1
 * (d = 0 is the paper's choice); for each, the shifted kernel fl(W_k - delta_d) goes through the line search of
 * Section 3.4 on the unsigned range.  The (offset, scale) pair with the smallest error wins, lowest
 * d*n_cand + c on equal errors; grid->refine_iters polish steps of the scale follow, the offset staying fixed.
 * Outputs as omse_quantize_weights_offset; d_best_idx receives d*n_cand + c.  The kernel stays on chip while all
 * offsets are tried, so the cost is n_delta line searches from one read of the tensor.
 * Limits: 1 <= n_delta <= OMSE_MAX_OFFSETS, 0 <= off_frac <= 1, kernel_len <= OMSE_MAX_KERNEL_LEN_MULTISWEEP.
 */
#define OMSE_MAX_OFFSETS 64
typedef struct {
    int32_t n_delta; /* offsets on the grid                                  */
    float off_frac;  /* they span [min, min + off_frac*(max-min))            */
} omse_offset_grid;

int omse_quantize_weights_affine(omse_ctx* ctx, const float* d_w, int64_t n_kernels, int64_t kernel_len, int bits,
                                 const omse_grid* grid, const omse_offset_grid* offsets, float* d_alpha,
                                 float* d_delta, float* d_sse, int32_t* d_best_idx, int8_t* d_codes,
                                 uint8_t* d_packed);

/*
 * Dual line search for two quantized tensors (Section 3.5, the special case n = 2, third displayed
 * equation of the section): T ~ alpha1*Q1 + alpha2*Q2, kernel-wise.  The pair of scales is searched on
 * a two-dimensional grid; for every pair each element picks its first code by enumerating all of
 * Z_bits1, the second code being the rounding of the rest,
 *     min over t in Z_bits1 of ( T_j - alpha1*t - alpha2*[ (T_j - alpha1*t)/alpha2 ]_Z_bits2 )^2,
 * decided in binary32 (fused multiply-adds, IEEE division, lowest t on equal errors).  The paper gives
 * no grid; this library's is alpha1_c = (c+1)/n_cand1 * hi_frac1 * max|T_k| and, for each alpha1,
 * alpha2_d = (d+1)/n_cand2 * hi_frac2 * alpha1_c, in the binary32 form of omse_grid.  The pair with
 * the smallest error wins, lowest c*n_cand2+d among equal errors; there is no polish step.
 * The cost is n_cand1*n_cand2*2^bits1 evaluations per element: meant for small tensors (Section 3.5).
 * Outputs: d_alpha [2][n_kernels], d_sse [n_kernels] (binary64 accumulation of the objective),
 * d_best_idx [n_kernels] (nullable; -1 for a degenerate kernel), d_codes [2][n_kernels*kernel_len]
 * (nullable), d_packed [2][ceil(n_kernels*kernel_len/2)] (nullable; needs bits1, bits2 <= 4).
 * Limits: 1 <= n_cand1, n_cand2 <= OMSE_DUAL_MAX_CANDIDATES; bits1, bits2 in 2..8;
 * 1 <= kernel_len <= OMSE_MAX_KERNEL_LEN.
 */
#define OMSE_DUAL_MAX_CANDIDATES 1024
typedef struct {
    int32_t n_cand1, n_cand2;
    float hi_frac1; /* alpha1 grid reaches hi_frac1 * max|T_k|  */
    float hi_frac2; /* alpha2 grid reaches hi_frac2 * alpha1     */
} omse_dual_grid;

int omse_dual_quantize(omse_ctx* ctx, const float* d_t, int64_t n_kernels, int64_t kernel_len,
                       int bits1, int bits2, int is_signed, const omse_dual_grid* grid,
                       float* d_alpha, float* d_sse, int32_t* d_best_idx, int8_t* d_codes,
                       uint8_t* d_packed);

/*
 * Key-layer rule of Section 3.5: a layer whose MSE exceeds a threshold tau gets a second quantized tensor.
 * For each layer l this call sums the per-kernel squared errors that
 * omse_quantize_weights wrote (d_sse, [n_kernels] float) in binary64 in a fixed order, divides by the
 * layer's element count and compares with tau: d_mse[l] = sum / (n_kernels*kernel_len),
 * d_is_key[l] = (d_mse[l] > tau).  `layers` is a HOST array read before the call returns; d_mse
 * [n_layers] double and d_is_key [n_layers] int32 (nullable) are device buffers.
 * 0 <= n_layers <= OMSE_MAX_BATCH, tau >= 0.
 */
typedef struct {
    const float* d_sse;
    int64_t n_kernels, kernel_len;
} omse_layer_error;

int omse_select_key_layers(omse_ctx* ctx, const omse_layer_error* layers, int n_layers, float tau,
                           double* d_mse, int32_t* d_is_key);

/*
 * The key-layer procedure of Section 3.5 in one call, with no host read in between:
 *   1. every layer is quantized kernel-wise with one tensor (as omse_quantize_weights_batched on layers[l].first);
 *   2. d_mse[l] and d_is_key[l] = (d_mse[l] > tau) as in omse_select_key_layers;
 *   3. one more launch over all layers gives the layers with d_is_key[l] = 1 their second tensor: each kernel's
 *      residual fl(W_k - alpha1*q1) is rebuilt on chip from the first scale and quantized the same way
 *      (Algorithm 1, one sweep); blocks skip the other layers, whose second outputs stay untouched;
 *      d_alpha2 / d_sse2 [n_kernels] (error after both tensors), d_codes2 / d_packed2 (nullable) are the second
 *      tensor's outputs;
 *   4. d_cr[0] (nullable, double) = compression ratio of the result, one or two tensors per layer.
 * d_mse [n_layers] double and d_is_key [n_layers] int32 are required.  0 <= n_layers <= OMSE_MAX_BATCH.
 */
typedef struct {
    omse_weight_tensor first;
    float* d_alpha2;
    float* d_sse2;
    int8_t* d_codes2;
    uint8_t* d_packed2;
} omse_key_layer;

int omse_quantize_key_layers(omse_ctx* ctx, const omse_key_layer* layers, int n_layers, int bits, int is_signed,
                             const omse_grid* grid, float tau, double* d_mse, int32_t* d_is_key, double* d_cr);

/*
 * Compression ratio (Section 3.5): size of the quantized model - bits[l] per code and one binary32
 * scale per kernel, times n_tensors[l] quantized tensors - over the size of the binary32 model.
 * Host arithmetic on HOST arrays of n_layers entries; returns -1 on invalid arguments.
 */
double omse_compression_ratio(const int64_t* n_kernels, const int64_t* kernel_len, const int* bits,
                              const int* n_tensors, int n_layers);

/*
 * INT4 code emission.  The paper deploys INT4 tensors but fixes no byte layout; this library's is:
 * element e (flat index) goes to byte e/2, even e in bits 0-3 and odd e in bits 4-7, the nibble
 * being the low four bits of the two's-complement code; if n is odd, bits 4-7 of the last byte are 0.
 * d_codes [n] int8 -> d_packed [ceil(n/2)] uint8.  is_signed is accepted for symmetry with the
 * other calls and does not change the bytes.
 */
int omse_pack_int4(omse_ctx* ctx, const int8_t* d_codes, int64_t n, int is_signed,
                   uint8_t* d_packed);

/*
 * omse_activation_scale without any allocation.  (The paper has no counterpart: this is a property
 * of the library, not of the method.)
 *
 * Who needs it: code that may not call cudaMalloc when it wants a scale - a plugin running inside a
 * host application whose memory pool already owns all device memory, a real-time or safety-certified
 * loop that forbids allocation after start-up, a caller holding a lock under which the allocator
 * could deadlock.  Such code cannot even create an omse_ctx, because omse_create allocates the
 * workspace.  This entry point takes no context: the scratch of the search (search state, summed
 * error curve, per-block partial sums) is a fixed array inside the library, OMSE_STATIC_SCRATCH_BYTES
 * per GPU, present on every GPU that loads the library until the process exits.  The call itself
 * performs no cudaMalloc / cudaFree and calls no allocating routine; inputs and outputs are still
 * the caller's device buffers.
 *
 * Arguments are those of omse_activation_scale, with `device` / `cuda_stream` instead of the context
 * and d_status (device, nullable): receives the OMSE_DEV_* bits of THIS call when its work completes.
 * Limits: grid->n_cand <= OMSE_STATIC_MAX_CANDIDATES, otherwise OMSE_ELIMIT is returned and nothing
 * is enqueued; device < 64.
 * First call on a device: looks up the array's device address (cudaGetSymbolAddress) and the SM
 * count and caches them; make that first call outside any stream capture.
 * Sharing: all calls on a device use the same array.  Each call re-initialises what must start
 * at zero, so calls that follow one another on one stream are independent; calls that can overlap
 * on the GPU (different streams, different threads) race on the array and give wrong results.
 * Results equal omse_activation_scale's up to the grouping of partial sums (same tolerances).
 */
#define OMSE_STATIC_MAX_CANDIDATES 2048
#define OMSE_STATIC_SCRATCH_BYTES (4u * 1024u * 1024u + 32u * 1024u)
int omse_activation_scale_static(int device, void* cuda_stream, const float* d_x, int64_t n, int bits,
                                 int is_signed, const omse_grid* grid, float* d_alpha, float* d_sse,
                                 int32_t* d_best_idx, double* d_sse_curve, uint32_t* d_status);

/* Synchronises the stream, copies the device status word (OMSE_DEV_* bits OR-ed over all calls
 * since the last read) to *host_out and clears it. */
int omse_last_device_status(omse_ctx* ctx, uint32_t* host_out);

/* Instrumentation (no counterpart in the paper): synchronises the stream and returns in *host_out how many
 * (element, candidate) evaluations the search kernels of this context actually executed since the last read,
 * then clears the counter.  The algorithmic count of a call is n_cand * elements (* quantized tensors); the
 * kernels execute fewer because a candidate skips, exactly, the elements it is known to code as zero.  For
 * omse_dual_quantize the unit is (element, pair, first code).  omse_activation_scale_static does not count. */
int omse_read_evaluations(omse_ctx* ctx, uint64_t* host_out);

/* Instrumentation (no counterpart in the paper): the number of kernels the calls on this context have launched since
 * the last read (host-side count, no synchronisation), then cleared.  A batched weight call launches one kernel per
 * row path present (rows longer than 640 elements, shorter rows, very short rows), the per-tensor search ten or so. */
int omse_read_launches(omse_ctx* ctx, uint64_t* host_out);

/* Instrumentation (no counterpart in the paper): runs a register-only loop of independent fma.rn.f32x2 on every SM
 * for about target_ms milliseconds (1..5000) on the context's stream, synchronises, and returns in *host_out the
 * measured FP32 lane operations per second of the FMA pipe (a packed instruction counts as two).  This is the
 * arithmetic roof the candidate sweep is compared with: an evaluation the sweep executes costs 4 such operations. */
int omse_measure_fp32_peak(omse_ctx* ctx, int target_ms, double* host_out);

/* Static description of a return value. */
const char* omse_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* OMSE_H */
