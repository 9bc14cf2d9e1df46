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

/* 5x5 max-pool, stride 1, padding 2 over x [n][h][w][c] (the detector's SPPF unit chains three of them); padding never
 * wins.  idx (may be NULL; one byte per element, same shape) receives r*5 + t of the FIRST maximum of each window in
 * row-major order (r, t = 0..4 from the window's corner at (p-2, q-2)): the record the backward call needs.
 * ld_x / ld_y: elements between consecutive pixels of x / y (0 = dense, else >= c): either may be a channel slice of a
 * wider tensor (the SPPF concatenation buffer holds the pools side by side); idx is always dense.
 * 16-byte accesses for 16-bit types when c and the pitches are multiples of 8 and x, y are 16-byte aligned. */
nb_status nb_maxpool5_fwd(int32_t dtype, int32_t n, int32_t h, int32_t w, int32_t c, const void* x, void* y, uint8_t* idx,
                          int64_t ld_x, int64_t ld_y, void* stream);

/* Gradient of nb_maxpool5_fwd: dx[n][i][j][c] = [dx +] sum of g over the windows whose recorded maximum is (i, j)
 * (fp32 sum in a fixed order, one rounding; accumulate != 0 adds to dx for tensors with several consumers).
 * ld_g / ld_dx: pixel pitches of g and dx as above. */
nb_status nb_maxpool5_bwd(int32_t dtype, int32_t n, int32_t h, int32_t w, int32_t c, const void* g, const uint8_t* idx,
                          void* dx, int32_t accumulate, int64_t ld_g, int64_t ld_dx, void* stream);

/* Nearest-neighbour 2x upsampling of [n][h][w][c] (the extents of the SMALL tensor):
 *   backward == 0: dst[n][2i+a][2j+b][c] = src[n][i][j][c]                       (src small, dst large)
 *   backward != 0: dst[n][i][j][c] = [dst +] sum_{a,b} src[n][2i+a][2j+b][c]      (src large, dst small)
 * ld_small / ld_large: elements between consecutive pixels of the small / the large tensor (0 = dense, else >= c): either
 * may be a channel slice of a wider tensor, e.g. the large one a part of the concatenation buffer it feeds. */
nb_status nb_upsample2(int32_t dtype, int32_t n, int32_t h, int32_t w, int32_t c, const void* src, void* dst,
                       int32_t backward, int32_t accumulate, int64_t ld_small, int64_t ld_large, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* NB_GLUE_H */
