/*
 * nb_glue.h -- the elementwise glue that chaining Conv-BN-SiLU blocks into the detector's C2f / PAN structure needs
 * (Sec. 6: the case-study detector is built from such blocks joined by channel splits, concatenations and residual
 * additions; in the backward pass a tensor with several consumers receives the SUM of their gradients).
 * One call covers all of them because every operand is a channel slice of an NHWC tensor:
 *
 *   out[r][c] = (accumulate ? out[r][c] : 0) + a[r][c] + (b ? b[r][c] : 0),   0 <= r < rows, 0 <= c < channels
 *
 * with out, a, b pointing at the FIRST channel of their slice and ld_* the row pitch of the tensor they live in
 * (elements; ld >= channels).  Uses: copy a slice (split / concat), residual add (b given), gradient accumulation
 * (accumulate = 1).  The sum is formed in fp32 and rounded once to the element type.
 *
 * Device pointers on the current device; 16-byte vector accesses are used when pointers and pitches allow, scalar
 * accesses otherwise (any element-aligned slice works).  out may alias a or b only element for element (same
 * pointer and pitch).  Enqueues on `stream`; status codes and nb_last_error() as in nb_cbs.h.
 * Errors: NB_ERR_INVALID_ARG (NULL out/a, non-positive sizes, pitch < channels, unknown dtype), NB_ERR_ALIGNMENT,
 * NB_ERR_CUDA.
 */
#ifndef NB_GLUE_H
#define NB_GLUE_H

#include "nb_cbs.h"

#ifdef __cplusplus
extern "C" {
#endif

nb_status nb_slice_add(int32_t dtype /* nb_dtype */, int64_t rows, int32_t channels, void* out, int64_t ld_out,
                       const void* a, int64_t ld_a, const void* b /* nullable */, int64_t ld_b, int32_t accumulate,
                       void* stream);

#ifdef __cplusplus
}
#endif
#endif /* NB_GLUE_H */
