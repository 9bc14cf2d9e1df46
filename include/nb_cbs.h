/*
 * nb_cbs.h -- C ABI of the B200 (sm_100a) Conv2d -> BatchNorm(training-mode batch statistics) -> SiLU
 * block: forward, data gradient, weight gradient, and the stand-alone batch statistics.
 *
 * Conventions follow the paper's description of its C ABI (Sec. 4): nb_* names, opaque caller-owned
 * handles with explicit destructors, runtime dtype tags, status codes plus a thread-local error
 * string, additive versioning (struct_size field).  The operators are the ones the paper's case
 * study uses (Sec. 6: convolutions with SiLU activations; Sec. 3.2 and Table 2 row 2: batch
 * normalisation kept in F32 while convolutions run in 16-bit).  The paper prints no formula for
 * them; the definitions below are those of the works it cites for BN and SiLU.
 *
 * Shapes and layouts (all tensors dense, innermost dimension contiguous):
 *   x      [N][H][W][Cin]        input activation, NHWC
 *   w      [Cout][k][k][Cin]     filter, k in {1,3}, cross-correlation (no flip), zero pad P = k/2
 *   y,a,g,dy [N][Ho][Wo][Cout]   Ho = (H + 2P - k)/stride + 1, likewise Wo;  M = N*Ho*Wo rows
 *   dx     like x, dw like w (always fp32)
 *   gamma, beta, mean, invstd, running_*, dgamma, dbeta: fp32 [Cout]
 *
 * Element types by mode:
 *   NB_MODE_BF16_TC : x, w, a, g, dy, dx are bf16; the saved convolution output y is IEEE fp16
 *                     (an internal tensor: same bytes as bf16, 8x finer, saturated at +-65504);
 *                     accumulation and all BN/SiLU arithmetic in fp32; dw, dgamma, dbeta fp32.
 *   NB_MODE_F32_REF : every tensor fp32, plain FMA arithmetic (no tensor cores, no TF32).
 *   NB_MODE_F16_TC  : as NB_MODE_BF16_TC with IEEE fp16 in place of bf16 for x, w, a, g, dy, dx (the paper's own
 *                     mixed-precision policy, Sec. 3.2: F16 convolutions, F32 BN, dynamic loss scaling -- the scaler
 *                     is nb_sgd_clip_nesterov_step_scaled).  Same tensor-core kernels with fp16 operand formats;
 *                     16-bit stores saturate at +-65504 and the tensor-core epilogues count saturations in the
 *                     status block.
 *
 * Every pointer is a DEVICE pointer on the plan's device unless its name starts with `host_`; the
 * caller owns all memory, including the workspace.  Tensor pointers must be 16-byte aligned.
 * Compute calls enqueue work on `stream` (a cudaStream_t passed as void*; NULL = default stream)
 * and return without synchronising; they make the plan's device current while they run and restore the
 * caller's current device before returning (`stream` must belong to the plan's device).  Outputs are
 * overwritten, never accumulated into.  Calls on one plan must not run concurrently, neither on the host
 * (they share the plan's cached tensor maps) nor on the device (its status block, the accumulators in which a
 * default plan sums the BatchNorm statistics, and the workspace).  Two exceptions on the device:
 * nb_conv_bn_silu_bwd_weight uses of the plan only the atomic error words of the status block, so on a stream of
 * its own, with a workspace of its own and ordered after the call that produced dy, it may overlap any other
 * call of this or another plan; and a plan created with NB_CBS_FLAG_SEPARATE_FINALIZE keeps all scratch of a
 * call in the workspace that call was given, so its calls may overlap on different streams when their
 * workspaces differ.  Calls of DIFFERENT plans may always overlap: no kernel waits for another block or kernel.
 * On invalid arguments nothing is launched and a non-zero status is returned; nb_last_error()
 * then describes the problem.
 */
#ifndef NB_CBS_H
#define NB_CBS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define NB_CBS_ABI_VERSION 3u /* 2: adds the evaluation-mode / plain calls (additive); 3: flag 2 is NB_CBS_FLAG_SEPARATE_FINALIZE,
                                  the grid-barrier test hook is gone with the barriers, nb_cbs_plan_set_bwd_residual is new */

typedef int32_t nb_status;
enum {
    NB_OK = 0,
    NB_ERR_INVALID_ARG = 1, /* NULL pointer, non-positive extent, bad enum, struct_size mismatch */
    NB_ERR_UNSUPPORTED = 2, /* shape outside what the mode supports (see nb_cbs_plan_create) */
    NB_ERR_WORKSPACE = 3,   /* workspace NULL or smaller than nb_cbs_workspace_bytes reports */
    NB_ERR_ALIGNMENT = 4,   /* a tensor pointer is not 16-byte aligned */
    NB_ERR_CUDA = 5,        /* a CUDA runtime/driver call failed (no device, launch error, ...) */
    NB_ERR_ARCH = 6,        /* the device is not compute capability 10.x */
    NB_ERR_TIMEOUT = 7,     /* a kernel gave up a bounded wait (reported by nb_cbs_poll_status) */
    NB_ERR_INTERNAL = 8
};

typedef enum { NB_DTYPE_F32 = 0, NB_DTYPE_BF16 = 1, NB_DTYPE_F16 = 2 } nb_dtype;
typedef enum { NB_MODE_BF16_TC = 0, NB_MODE_F32_REF = 1, NB_MODE_F16_TC = 2 } nb_mode;

/* nb_cbs_desc.flags */
#define NB_CBS_FLAG_FORCE_SIMT 1u /* BF16 mode: run the three convolutions on the CUDA-core kernels
                                     (same arithmetic contract; for testing and as a cross-check) */
#define NB_CBS_FLAG_SEPARATE_FINALIZE 2u /* the BatchNorm statistics are finished by separate small kernels that add
                                     per-block partial sums in a fixed order, so that they come out bit-identical from
                                     run to run (a few microseconds more per call).  By default the kernels that sum
                                     (the tensor-core forward convolution, the backward reduce pass) add their block
                                     sums to fp64 accumulators with atomics and the pass that follows derives its
                                     coefficients from the totals: the same values, except that a total may differ
                                     in its last fp64 bit with the order of the additions (seen in an fp32 result
                                     only if the total sits within 2^-50 of a rounding boundary).  No kernel of either
                                     kind waits for another block or kernel, so calls of different plans may share
                                     the GPU (other streams, other processes) with or without this flag. */

typedef struct nb_cbs_desc {
    uint32_t struct_size; /* = sizeof(nb_cbs_desc) */
    int32_t n, h, w, c_in, c_out;
    int32_t ksize;  /* 1 or 3; pad = ksize/2 */
    int32_t stride; /* 1 or 2 */
    float eps;      /* added to the biased batch variance; 1e-3 in every benchmark configuration */
    float momentum; /* running-statistics momentum; read only when running_* pointers are given */
    int32_t mode;   /* nb_mode */
    uint32_t flags;
} nb_cbs_desc;

typedef struct nb_cbs_plan_s* nb_cbs_plan;

/* ABI revision of the loaded library (NB_CBS_ABI_VERSION at build time). */
uint32_t nb_abi_version(void);

/* Description of the last failure on the calling thread ("" if none); valid until the next nb_* call
 * on this thread. */
const char* nb_last_error(void);

/* Create a plan for one block shape on CUDA device `device`.  Allocates a small (<= 4 KB) device
 * status block; all other memory is the caller's.  Requirements: all extents > 0; ksize in {1,3};
 * stride in {1,2}; BF16 mode: c_out % 8 == 0; F32 mode: c_out % 4 == 0; N*Ho*Wo >= 2.
 * Errors: NB_ERR_INVALID_ARG, NB_ERR_UNSUPPORTED, NB_ERR_CUDA (no usable device), NB_ERR_ARCH. */
nb_status nb_cbs_plan_create(const nb_cbs_desc* desc, int device, nb_cbs_plan* out_plan);

/* Free the plan and its status block.  NULL is accepted. */
nb_status nb_cbs_plan_destroy(nb_cbs_plan plan);

/* Output extents Ho, Wo of the plan's shape. */
nb_status nb_cbs_out_shape(nb_cbs_plan plan, int32_t* ho, int32_t* wo);

/* Minimum workspace sizes in bytes for the forward call (also enough for nb_bn_stats) and for the two
 * backward calls.  The workspace needs no initialisation and may be shared between plans whose calls
 * do not overlap on the device; it must be 256-byte aligned. */
nb_status nb_cbs_workspace_bytes(nb_cbs_plan plan, size_t* fwd_bytes, size_t* bwd_bytes);

/* Channel-slice operands for chained blocks (split / concat without copies): declare that, in the three TRAINING calls
 * of this plan, the input x, the output a_out and the upstream gradient g are channel slices of wider NHWC tensors:
 * the pointer passed to the call addresses the slice's first channel and consecutive pixels are ld_* elements apart
 * (0 = dense; otherwise at least the channel count and a multiple of 8 elements -- 4 in F32 mode -- so that slices stay
 * 16-byte aligned).  x is read with this pitch by the forward and the weight-gradient call, a_out is written with ld_a,
 * g is read with ld_g by the data-gradient call; every other tensor (y, dy, dx, dw, ...) stays dense.
 * NB_ERR_UNSUPPORTED if ld_x is given and the plan's forward or weight gradient does not run on the tensor-core kernels
 * (their TMA descriptors carry the pitch).  The evaluation-mode, plain and host-buffer calls refuse a pitched plan. */
nb_status nb_cbs_plan_set_pitches(nb_cbs_plan plan, int64_t ld_x, int64_t ld_a, int64_t ld_g);

/* Residual connection performed by the block that feeds it (the bottlenecks of the detector's C2f units, Sec. 6): with
 * res != NULL, nb_conv_bn_silu_fwd of this plan writes a_out = SiLU(z) + res, where res is a tensor of a_out's shape and
 * type, dense or a channel slice with pixels ld_res elements apart (0 = dense); the sum is formed in fp32 and rounded
 * once.  Everything the backward calls need (y_saved, mean, invstd) is unchanged: the gradient of the sum is the
 * gradient of both summands.  res must stay valid while calls of the plan may run; NULL restores the plain block.
 * The evaluation-mode, plain and host-buffer calls refuse such a plan. */
nb_status nb_cbs_plan_set_fwd_residual(nb_cbs_plan plan, const void* res, int64_t ld_res);

/* Backward counterpart of nb_cbs_plan_set_fwd_residual: the gradient that reaches the sum a_out = SiLU(z) + res is the
 * gradient of both summands, so with gres != NULL nb_conv_bn_silu_bwd_data of this plan also hands its incoming
 * gradient g to the shortcut: gres (a tensor of g's shape and type, dense or a channel slice with pixels ld_gres
 * elements apart; 0 = dense) receives gres + g when accumulate = 1 (fp32 sum rounded once to the 16-bit type, exactly
 * as a separate accumulation pass would) or a copy of g when accumulate = 0.  The dy pass, which reads g anyway, does
 * it.  gres must not overlap g, dy or dx, and must stay valid while calls of the plan may run; NULL switches it off.
 * NB_ERR_UNSUPPORTED in fp32 mode and for NB_CBS_FLAG_SEPARATE_FINALIZE plans.  The host-buffer call refuses such a plan. */
nb_status nb_cbs_plan_set_bwd_residual(nb_cbs_plan plan, void* gres, int64_t ld_gres, int32_t accumulate);

/* Gradient accumulation at fan-out without a separate pass: declare that, in nb_conv_bn_silu_bwd_data of this plan, dx is
 * a channel slice of a wider NHWC tensor (pointer = the slice's first channel, pixels ld_dx elements apart; 0 = dense) and,
 * with accumulate = 1, that the data gradient is ADDED to what dx holds instead of overwriting it (a tensor with several
 * consumers receives the sum of their gradients, Sec. 6 dataflow; each addition rounds once to the 16-bit type, exactly as
 * a separate accumulation pass would).  The epilogue then issues TMA reductions instead of TMA stores.
 * NB_ERR_UNSUPPORTED unless the plan's data gradient runs on the tensor-core kernel of a stride-1 layer; ld_dx at least
 * c_in and a multiple of 8 elements.  (0, 0) restores the default.  The plain and host-buffer calls refuse such a plan. */
nb_status nb_cbs_plan_set_dx_target(nb_cbs_plan plan, int64_t ld_dx, int32_t accumulate);

/* Which implementation each convolution of this plan runs on: writes three ints (fprop, dgrad, wgrad),
 * 1 = tcgen05 tensor-core kernel, 0 = CUDA-core kernel. */
nb_status nb_cbs_plan_paths(nb_cbs_plan plan, int32_t* paths3);

/* Synchronise `stream`, then report whether any kernel launched through this plan gave up a bounded
 * wait (NB_ERR_TIMEOUT) or saturated an fp16 store (still NB_OK; see nb_last_error()).  Clears the
 * status block. */
nb_status nb_cbs_poll_status(nb_cbs_plan plan, void* stream);

/* Diagnostics (the paper has no counterpart; they exist for the benchmark's per-kernel roofline figures).
 * nb_cbs_launch_count: number of CUDA kernels this library has launched in this process so far.
 * nb_cbs_profile_enable(plan, 1): from now on every kernel site of calls on this plan is bracketed by CUDA
 *   events and the call WAITS for the kernel, accumulating its device time; enable = 0 turns it off again;
 *   either call clears the accumulators.  Not for use inside stream capture.
 * nb_cbs_profile_site_name(i): name of kernel site i, NULL once i is past the last site.
 * nb_cbs_profile_read: accumulated milliseconds and launch count of one site since the last enable call. */
unsigned long long nb_cbs_launch_count(void);
nb_status nb_cbs_profile_enable(nb_cbs_plan plan, int32_t enable);
const char* nb_cbs_profile_site_name(int32_t site);
nb_status nb_cbs_profile_read(nb_cbs_plan plan, int32_t site, double* total_ms, int64_t* launches);

/* Forward (Sec. 6 operators; BN in fp32 per Sec. 3.2 / Table 2 row 2):
 *   y[n,p,q,c'] = sum_{r,t,c} x[n, p*s-P+r, q*s-P+t, c] * w[c',r,t,c]        (zero outside the image)
 *   mean_c = (1/M) sum y ; var_c = (1/M) sum (y-mean_c)^2 (biased) ; invstd_c = (var_c + eps)^-1/2
 *   a = z * sigmoid(z),  z = gamma_c * (y - mean_c) * invstd_c + beta_c
 *   optional: running_mean <- (1-m) running_mean + m mean ; running_var <- (1-m) running_var + m var*M/(M-1)
 * x, w, gamma, beta: inputs.  running_mean/running_var: both NULL or both given (in/out).
 * y_saved, save_mean, save_invstd: outputs that the backward calls need.  a_out: the block's output. */
nb_status nb_conv_bn_silu_fwd(nb_cbs_plan plan, const void* x, const void* w, const float* gamma, const float* beta,
                              float* running_mean, float* running_var, void* y_saved, float* save_mean,
                              float* save_invstd, void* a_out, void* workspace, size_t workspace_bytes, void* stream);

/* Stand-alone training-mode batch statistics of a [M][Cout] tensor (M = N*Ho*Wo of the plan):
 * mean and invstd as in the forward call; optionally also the raw per-channel sum and sum of squares.
 * y_dtype: NB_DTYPE_F16 in BF16 mode (the saved y), NB_DTYPE_F32 in F32 mode; anything else is
 * NB_ERR_UNSUPPORTED.  sum / sumsq may be NULL. */
nb_status nb_bn_stats(nb_cbs_plan plan, const void* y, int32_t y_dtype, float* mean, float* invstd, float* sum,
                      float* sumsq, void* workspace, size_t workspace_bytes, void* stream);

/* Backward with respect to the block's input, gamma and beta, given g = dL/da:
 *   s = sigmoid(z) ; dz = g * s * (1 + z*(1-s))                               (z recomputed from y_saved)
 *   dbeta_c = sum dz ; dgamma_c = sum dz*xhat,  xhat = (y-mean_c)*invstd_c
 *   dy = gamma_c*invstd_c * (dz - dbeta_c/M - xhat*dgamma_c/M)                 -> dy_out (kept for bwd_weight)
 *   dx[n,h,w,c] = sum over (p,q,r,t,c') with p*s-P+r = h, q*s-P+t = w of dy[n,p,q,c'] * w[c',r,t,c]
 * dx may be NULL (first layer of a network): then only dy_out, dgamma and dbeta are produced. */
nb_status nb_conv_bn_silu_bwd_data(nb_cbs_plan plan, const void* g, const void* y_saved, const float* save_mean,
                                   const float* save_invstd, const float* gamma, const float* beta, const void* w,
                                   void* dx, float* dgamma, float* dbeta, void* dy_out, void* workspace,
                                   size_t workspace_bytes, void* stream);

/* Backward with respect to the filter:
 *   dw[c',r,t,c] = sum_{n,p,q} dy[n,p,q,c'] * x[n, p*s-P+r, q*s-P+t, c]        (fp32 output)
 * dy is the tensor nb_conv_bn_silu_bwd_data wrote to dy_out (ordering on the stream is the caller's). */
nb_status nb_conv_bn_silu_bwd_weight(nb_cbs_plan plan, const void* x, const void* dy, float* dw, void* workspace,
                                     size_t workspace_bytes, void* stream);

/* ---- Evaluation-mode and plain variants of the block (inference; nothing is saved, nothing is updated) ----
 * The paper's reproduction protocol found that validation must normalise with the RUNNING statistics (Table 2 row 9),
 * and its detector's head ends in convolutions that carry a bias and no normalisation (Table 2 row 3).
 *
 * Workspace size of the three calls below and whether they run as ONE kernel: `*fused` (may be NULL) is 1 when the
 * convolution runs on the tensor-core kernel with the per-channel scale/shift and the activation applied to the fp32
 * accumulators in its epilogue (BF16 mode, c_in % 16 == 0, c_out % 16 == 0; also the 3 -> 48 channel 3x3 stride-2
 * first layer, whose own kernel has the same epilogue); 0 when the plan falls back to
 * convolution -> coefficient kernel -> elementwise pass, whose workspace also holds the convolution output. */
nb_status nb_cbs_infer_workspace_bytes(nb_cbs_plan plan, size_t* bytes, int32_t* fused);

/* Evaluation-mode forward:
 *   y = conv(x, w) as in nb_conv_bn_silu_fwd
 *   z = gamma_c * (y - running_mean_c) / sqrt(running_var_c + eps) + beta_c ;  a = z * sigmoid(z)  -> a_out
 * The per-channel scale gamma/sqrt(var+eps) and shift beta - mean*scale are formed in fp64 and applied in fp32.
 * Layouts and dtypes as in the training forward (a_out bf16 in BF16 mode, fp32 in F32 mode). */
nb_status nb_conv_bn_silu_infer(nb_cbs_plan plan, const void* x, const void* w, const float* gamma, const float* beta,
                                const float* running_mean, const float* running_var, void* a_out, void* workspace,
                                size_t workspace_bytes, void* stream);

/* Convolution with a per-channel bias and no normalisation:
 *   z = conv(x, w) + bias_c (bias may be NULL: zero) ;  out = act ? z * sigmoid(z) : z     (act: 0 = none, 1 = SiLU)
 * With the outputs of nb_bn_fold as (w, bias) and act = 1 this is the evaluation-mode block with BN folded away. */
nb_status nb_conv_bias_act(nb_cbs_plan plan, const void* x, const void* w, const float* bias, int32_t act, void* out,
                           void* workspace, size_t workspace_bytes, void* stream);

/* Backward of the plain convolution with bias (act = 0), given dout = dL/d out:
 *   dx = conv^T(dout, w) (may be NULL), dw[c',r,t,c] = sum_{n,p,q} dout[n,p,q,c'] * x[...] (fp32), dbias_c' = sum dout (may be NULL).
 * The same data-gradient and weight-gradient kernels as the block's backward calls; workspace of the backward size. */
nb_status nb_conv_bias_bwd(nb_cbs_plan plan, const void* x, const void* w, const void* dout, void* dx, float* dw,
                           float* dbias, void* workspace, size_t workspace_bytes, void* stream);

/* Fold evaluation-mode BN into the filter that feeds it: with s_c' = gamma_c' / sqrt(running_var_c' + eps),
 *   w_folded[c',r,t,c] = s_c' * w[c',r,t,c]   (the plan's activation dtype, rounded once)
 *   bias_folded[c']    = beta_c' - running_mean_c' * s_c'                                   (fp32)
 * No workspace.  w_folded may not alias w. */
nb_status nb_bn_fold(nb_cbs_plan plan, const void* w, const float* gamma, const float* beta, const float* running_mean,
                     const float* running_var, void* w_folded, float* bias_folded, void* stream);

/* Batch statistics for callers that cannot allocate device memory.  (The paper has no counterpart of this entry
 * point.)  Some hosts of this library must not call cudaMalloc -- code running under a framework's caching allocator
 * that forbids raw allocations, real-time or plug-in code with a fixed memory budget, or code that would have to size
 * a workspace before it knows the tensor -- and nb_bn_stats needs both a plan (whose creation allocates a status
 * block) and a caller-provided workspace.  This variant computes the same mean / invstd / sum / sumsq of a dense
 * [m][c] tensor, with no plan and no workspace: its partial sums live in an array built into the library
 * (2 MiB, file-scope device memory, held by every GPU that loads the library until the process exits).
 *   Limits: c <= 1024 channels, c % 8 == 0 for NB_DTYPE_F16, c % 4 == 0 for NB_DTYPE_F32, m >= 2; anything beyond
 *   returns NB_ERR_UNSUPPORTED (or NB_ERR_INVALID_ARG) with a message and launches nothing.
 *   It runs on the CURRENT device.  The first call on each device looks up the array's device address (one
 *   cudaGetSymbolAddress); make that first call before any stream capture begins.  The address is cached per
 *   device for the life of the process: after a cudaDeviceReset of that device it is stale, and this entry point
 *   must not be used again in that process.
 *   It calls no cudaMalloc / cudaFree and no allocating library routine.
 *   Every call on a device shares the one array, which keeps the previous call's contents; each call overwrites
 *   every entry it later reads, so nothing needs clearing -- but two calls whose kernels overlap on the GPU
 *   (different streams, no ordering between them) race on it and give wrong results.  Serialise such calls.
 * y, mean, invstd (and sum, sumsq when not NULL) are device pointers, 16-byte aligned; results are written
 * asynchronously on `stream`. */
nb_status nb_bn_stats_static(const void* y, int32_t y_dtype, int64_t m, int32_t c, float eps, float* mean, float* invstd,
                             float* sum, float* sumsq, void* stream);

/* One whole training step of the block from HOST buffers (the end-to-end path of a caller whose data
 * lives in host memory): copies host_x, host_w, host_gamma, host_beta, host_g to the device, runs the
 * forward call and the two backward calls above, and copies a, dx (unless host_dx is NULL), dw, dgamma,
 * dbeta back, all on `stream`; returns after enqueueing (host buffers should be pinned for the copies to
 * be asynchronous, and must stay valid until the stream is synchronised).  device_scratch is a device
 * buffer of at least nb_cbs_step_host_scratch_bytes() bytes, 256-byte aligned, owned by the caller; it
 * holds the device copies, the saved tensors and the workspace.  The paper has no counterpart of this
 * entry point; it exists so that the host-to-host cost of the path can be measured. */
nb_status nb_cbs_step_host_scratch_bytes(nb_cbs_plan plan, size_t* bytes);
nb_status nb_conv_bn_silu_step_host(nb_cbs_plan plan, const void* host_x, const void* host_w, const float* host_gamma,
                                    const float* host_beta, const void* host_g, void* host_a, void* host_dx,
                                    float* host_dw, float* host_dgamma, float* host_dbeta, void* device_scratch,
                                    size_t scratch_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* NB_CBS_H */
