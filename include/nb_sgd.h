/*
 * nb_sgd.h -- C ABI of the fused optimiser step that consumes the gradients of the Conv-BN-SiLU calls
 * (include/nb_cbs.h): global-norm gradient clipping over ALL gradient tensors followed by SGD with Nesterov
 * momentum, per-group learning rate and weight decay, in two kernel launches for any number of tensors.
 *
 * The paper (Sec. 3.2 "Optimization", Table 1 "Optimization", Table 2 rows 6-7) describes the step: SGD with Nesterov
 * momentum 0.937, three parameter groups (decayed weights, undecayed normalisation gains, undecayed biases),
 * fused multi-tensor update paths, and global-norm clipping at 10.0 every step done as one squared-norm accumulation
 * across all 243 gradient tensors instead of 243 per-tensor synchronisations.  It prints no formula; the
 * semantics are the dominant framework's defaults, which the paper says it keeps:
 *
 *   total = sqrt(sum over every tensor and element of g^2);  c = min(max_norm / (total + 1e-6), 1)
 *   d   = c*g + weight_decay[group] * p
 *   buf = d                       when first_step != 0 (the buffer's previous contents are ignored)
 *   buf = momentum * buf + d      otherwise
 *   p   = p - lr[group] * (d + momentum * buf)
 *   param_bf16 = round-to-nearest-even bf16 of the new p     (when the tensor has a working copy)
 *
 * Here the norm never leaves the device: the update kernel reads the per-block partial sums of the norm kernel
 * itself (no device-to-host readback at all, where the paper needs one).  Sums are taken in a fixed order, so
 * results are bitwise reproducible for a given tensor list and device.
 *
 * All tensor pointers are DEVICE pointers on the current device, 16-byte aligned, fp32 unless stated; the caller
 * owns everything including the workspace.  Calls enqueue on `stream` and return without synchronising.  Status
 * codes and nb_last_error() are those of nb_cbs.h.
 */
#ifndef NB_SGD_H
#define NB_SGD_H

#include "nb_cbs.h"

#ifdef __cplusplus
extern "C" {
#endif

#define NB_SGD_GROUPS 3 /* 0: weights (decayed), 1: normalisation gains, 2: biases -- only lr/weight_decay differ */

typedef struct nb_sgd_tensor {
    const float* grad; /* [numel] gradient (dw, dgamma, dbeta of the block calls); read only */
    float* param;      /* [numel] fp32 master parameter, updated in place */
    float* momentum;   /* [numel] momentum buffer, updated in place */
    void* param_bf16;  /* NULL, or [numel] 16-bit working copy (what the convolution calls read), rewritten */
    int64_t numel;     /* > 0 */
    int32_t group;     /* 0 .. NB_SGD_GROUPS-1 */
    int32_t copy_dtype; /* type of the working copy: 0 or NB_DTYPE_BF16 = bf16, NB_DTYPE_F16 = IEEE fp16 (saturating) */
} nb_sgd_tensor;

typedef struct nb_sgd_hyper {
    uint32_t struct_size; /* = sizeof(nb_sgd_hyper) */
    float momentum;       /* 0.937 in the paper's recipe (0.8 -> 0.937 during warm-up) */
    float max_norm;       /* 10.0 in the paper's recipe; <= 0 or +inf disables clipping */
    float lr[NB_SGD_GROUPS];
    float weight_decay[NB_SGD_GROUPS];
    int32_t first_step;   /* non-zero: the momentum buffers hold nothing yet */
} nb_sgd_hyper;

/* Dynamic loss scaling (Sec. 3.2 "Mixed precision"; Table 1: initial scale 2^16; Table 2 row 4: a FLOOR keeps repeated
 * overflows from driving the scale towards zero).  The state lives in DEVICE memory and never visits the host:
 * the gradients handed to the step are the gradients of (scale * loss). */
typedef struct nb_loss_scaler {
    float scale;            /* current loss scale; initialise (e.g. 65536) before the first step */
    int32_t growth_tracker; /* consecutive good steps since the last change; initialise to 0 */
    int32_t skipped;        /* written by every step: 1 if it was skipped because a gradient was inf or NaN */
    int32_t reserved;
} nb_loss_scaler;

typedef struct nb_scaler_hyper {
    uint32_t struct_size;  /* = sizeof(nb_scaler_hyper) */
    float growth_factor;   /* 2.0 */
    float backoff_factor;  /* 0.5 */
    float floor_scale;     /* the scale never drops below this (0 = no floor) */
    int32_t growth_interval; /* good steps before the scale grows (2000) */
} nb_scaler_hyper;

typedef struct nb_sgd_plan_s* nb_sgd_plan; /* opaque, caller-owned, host memory only */

/* Validate a tensor list (a HOST array of `count` entries holding DEVICE pointers on device `device`) and build
 * the chunk table that spreads the elements of all tensors over the blocks.  Allocates host memory only.
 * Errors: NB_ERR_INVALID_ARG (NULL, count <= 0, numel <= 0, bad group, NULL grad/param/momentum),
 * NB_ERR_ALIGNMENT (a tensor pointer is not 16-byte aligned), NB_ERR_CUDA (device query failed). */
nb_status nb_sgd_plan_create(const nb_sgd_tensor* host_tensors, int32_t count, int device, nb_sgd_plan* out_plan);

/* Free the plan.  NULL is accepted.  Not before the copy of nb_sgd_upload has completed. */
nb_status nb_sgd_plan_destroy(nb_sgd_plan plan);

/* Bytes of device workspace (256-byte aligned, caller-owned): a device copy of the list and of the chunk
 * table, and the norm's per-block partial sums. */
nb_status nb_sgd_workspace_bytes(nb_sgd_plan plan, size_t* bytes);

/* Copy the list and the chunk table into the workspace (one asynchronous copy on `stream` from memory the plan
 * owns).  Once per workspace; the optimiser state itself lives in the caller's param / momentum tensors.
 * Errors: NB_ERR_INVALID_ARG, NB_ERR_WORKSPACE, NB_ERR_CUDA. */
nb_status nb_sgd_upload(nb_sgd_plan plan, void* workspace, size_t workspace_bytes, void* stream);

/* One optimiser step over the plan's tensors: two launches (squared-norm partials; clip + update), ordered on
 * `stream` after the upload.  total_norm (device pointer, may be NULL) receives the gradient norm before
 * clipping.  Safe to capture into a CUDA graph.
 * Errors: NB_ERR_INVALID_ARG (NULL, struct_size mismatch), NB_ERR_WORKSPACE, NB_ERR_ALIGNMENT, NB_ERR_CUDA. */
nb_status nb_sgd_clip_nesterov_step(nb_sgd_plan plan, void* workspace, size_t workspace_bytes, const nb_sgd_hyper* hyper,
                                    float* total_norm, void* stream);

/* The same step for gradients that arrive multiplied by state->scale: they are unscaled (g / scale) on the fly, the
 * clip threshold applies to the unscaled norm (which total_norm receives), and if any gradient element is inf or NaN
 * the step is SKIPPED: parameters, momentum and working copies stay untouched.  Then the state is advanced:
 *   skipped:  scale = max(scale * backoff_factor, floor_scale), growth_tracker = 0, skipped = 1
 *   otherwise growth_tracker += 1; when it reaches growth_interval: scale *= growth_factor, growth_tracker = 0; skipped = 0
 * Three launches (norm partials; clip + update; scaler state), no host readback; `state` is a device pointer, 16-byte
 * aligned.  Errors as nb_sgd_clip_nesterov_step, plus NB_ERR_INVALID_ARG for a NULL state or scaler. */
nb_status nb_sgd_clip_nesterov_step_scaled(nb_sgd_plan plan, void* workspace, size_t workspace_bytes, const nb_sgd_hyper* hyper,
                                           const nb_scaler_hyper* scaler, nb_loss_scaler* state, float* total_norm, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* NB_SGD_H */
