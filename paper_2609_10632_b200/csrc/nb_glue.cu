// C ABI of the glue between chained blocks (see include/nb_glue.h): channel-slice add / copy / accumulate, 5x5 max-pool,
// 2x nearest upsampling.  Everything runs on the current device; no memory is allocated.
#include <algorithm>
#include <cstring>
#include <new>
#include <vector>

#include "api_common.cuh"
#include "common.cuh"
#include "glue.cuh"

using namespace nbcbs;
using namespace nbapi;

// ---------------------------------------------------------------- glue between chained blocks (include/nb_glue.h)
namespace {
template <typename T>
nb_status run_slice_add(void* out, long long ld_out, const void* a, long long ld_a, const void* b, long long ld_b, long long rows, int channels,
                        int accumulate, cudaStream_t st) {
    constexpr int V = 16 / (int)sizeof(T);
    const bool vec = channels % V == 0 && ld_out % V == 0 && ld_a % V == 0 && (!b || ld_b % V == 0) &&
                     !((reinterpret_cast<uintptr_t>(out) | reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(b)) & 15u);
    const long long total = rows * (vec ? channels / V : channels);
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const unsigned blocks = (unsigned)std::max<long long>(1, std::min<long long>((total + 255) / 256, (long long)sms * 16));
    const bool small = total + 256LL * blocks < (1LL << 32);  // indices (one grid stride past the end included) fit 32 bits
#define NB_SLICE_LAUNCH(VECF, IDX)                                                                                                         \
    launch_k(slice_add_kernel<T, VECF, IDX>, dim3(blocks), dim3(256), 0, st, 1, static_cast<T*>(out), ld_out, static_cast<const T*>(a), ld_a, \
             static_cast<const T*>(b), ld_b, rows, channels, accumulate)
    if (vec && small) NB_SLICE_LAUNCH(true, unsigned);
    else if (vec) NB_SLICE_LAUNCH(true, long long);
    else if (small) NB_SLICE_LAUNCH(false, unsigned);
    else NB_SLICE_LAUNCH(false, long long);
#undef NB_SLICE_LAUNCH
    return launch_ok("slice_add");
}
}  // namespace

extern "C" nb_status nb_slice_add(int32_t dtype, int64_t rows, int32_t channels, void* out, int64_t ld_out, const void* a, int64_t ld_a,
                                  const void* b, int64_t ld_b, int32_t accumulate, void* stream) {
    g_err.clear();
    if (!out || !a) return fail(NB_ERR_INVALID_ARG, "out and a must not be NULL");
    if (rows <= 0 || channels <= 0) return fail(NB_ERR_INVALID_ARG, "rows and channels must be positive");
    if (ld_out < channels || ld_a < channels || (b && ld_b < channels)) return fail(NB_ERR_INVALID_ARG, "a row pitch is smaller than the channel count");
    const size_t es = dtype == NB_DTYPE_F32 ? 4 : 2;
    if ((reinterpret_cast<uintptr_t>(out) | reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(b)) & (es - 1))
        return fail(NB_ERR_ALIGNMENT, "a pointer is not aligned to its element size");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    switch (dtype) {
        case NB_DTYPE_F32: return run_slice_add<float>(out, ld_out, a, ld_a, b, ld_b, rows, channels, accumulate != 0, st);
        case NB_DTYPE_BF16: return run_slice_add<__nv_bfloat16>(out, ld_out, a, ld_a, b, ld_b, rows, channels, accumulate != 0, st);
        case NB_DTYPE_F16: return run_slice_add<__half>(out, ld_out, a, ld_a, b, ld_b, rows, channels, accumulate != 0, st);
        default: return fail(NB_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    }
}

namespace {
unsigned glue_blocks(long long total) {
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    return (unsigned)std::max<long long>(1, std::min<long long>((total + 255) / 256, (long long)sms * 8));
}
nb_status check_nhwc(int32_t n, int32_t h, int32_t w, int32_t c) {
    if (n <= 0 || h <= 0 || w <= 0 || c <= 0) return fail(NB_ERR_INVALID_ARG, "extents must be positive");
    return NB_OK;
}
template <typename T>
nb_status run_maxpool_fwd(const void* x, void* y, uint8_t* idx, int n, int h, int w, int c, long long ld_x, long long ld_y, cudaStream_t st) {
    const bool vec = sizeof(T) == 2 && c % 8 == 0 && ld_x % 8 == 0 && ld_y % 8 == 0 && !((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(y)) & 15u);
    if (vec) {
        const long long total = (long long)n * h * w * (c / 8);
        launch_k(maxpool5_fwd_kernel<T, 8>, dim3(glue_blocks(total)), dim3(256), 0, st, 1, static_cast<const T*>(x), static_cast<T*>(y), idx, n, h, w, c, ld_x, ld_y);
    } else {
        const long long total = (long long)n * h * w * c;
        launch_k(maxpool5_fwd_kernel<T, 1>, dim3(glue_blocks(total)), dim3(256), 0, st, 1, static_cast<const T*>(x), static_cast<T*>(y), idx, n, h, w, c, ld_x, ld_y);
    }
    return launch_ok("maxpool5_fwd");
}
}  // namespace

extern "C" {

nb_status nb_maxpool5_fwd(int32_t dtype, int32_t n, int32_t h, int32_t w, int32_t c, const void* x, void* y, uint8_t* idx, int64_t ld_x, int64_t ld_y,
                          void* stream) {
    g_err.clear();
    if (!x || !y) return fail(NB_ERR_INVALID_ARG, "x and y must not be NULL");
    NB_TRY(check_nhwc(n, h, w, c));
    if (ld_x == 0) ld_x = c;
    if (ld_y == 0) ld_y = c;
    if (ld_x < c || ld_y < c) return fail(NB_ERR_INVALID_ARG, "a pixel pitch must be 0 (dense) or at least c");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    switch (dtype) {
        case NB_DTYPE_F32: return run_maxpool_fwd<float>(x, y, idx, n, h, w, c, (long long)ld_x, (long long)ld_y, st);
        case NB_DTYPE_BF16: return run_maxpool_fwd<__nv_bfloat16>(x, y, idx, n, h, w, c, (long long)ld_x, (long long)ld_y, st);
        case NB_DTYPE_F16: return run_maxpool_fwd<__half>(x, y, idx, n, h, w, c, (long long)ld_x, (long long)ld_y, st);
        default: return fail(NB_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    }
}

nb_status nb_maxpool5_bwd(int32_t dtype, int32_t n, int32_t h, int32_t w, int32_t c, const void* g, const uint8_t* idx, void* dx, int32_t accumulate,
                          int64_t ld_g, int64_t ld_dx, void* stream) {
    g_err.clear();
    if (!g || !idx || !dx) return fail(NB_ERR_INVALID_ARG, "g, idx and dx must not be NULL");
    NB_TRY(check_nhwc(n, h, w, c));
    if (ld_g == 0) ld_g = c;
    if (ld_dx == 0) ld_dx = c;
    if (ld_g < c || ld_dx < c) return fail(NB_ERR_INVALID_ARG, "a pixel pitch must be 0 (dense) or at least c");
    if ((long long)n * h * w >= (1LL << 32)) return fail(NB_ERR_UNSUPPORTED, "more than 2^32 pixels");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool vec = dtype != NB_DTYPE_F32 && c % 8 == 0 && ld_g % 8 == 0 && ld_dx % 8 == 0 &&
                     !((reinterpret_cast<uintptr_t>(g) | reinterpret_cast<uintptr_t>(dx)) & 15u) && !(reinterpret_cast<uintptr_t>(idx) & 7u);
    const unsigned blocks = glue_blocks((long long)n * h * w * (vec ? c / 8 : c));
#define NB_POOLB(T)                                                                                                                               \
    do {                                                                                                                                          \
        if (vec) launch_k(maxpool5_bwd_kernel<T, 8>, dim3(blocks), dim3(256), 0, st, 1, static_cast<const T*>(g), idx, static_cast<T*>(dx), n, h, w, c, accumulate != 0, (long long)ld_g, (long long)ld_dx); \
        else launch_k(maxpool5_bwd_kernel<T, 1>, dim3(blocks), dim3(256), 0, st, 1, static_cast<const T*>(g), idx, static_cast<T*>(dx), n, h, w, c, accumulate != 0, (long long)ld_g, (long long)ld_dx);     \
    } while (0)
    switch (dtype) {
        case NB_DTYPE_F32: NB_POOLB(float); break;
        case NB_DTYPE_BF16: NB_POOLB(__nv_bfloat16); break;
        case NB_DTYPE_F16: NB_POOLB(__half); break;
        default: return fail(NB_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    }
#undef NB_POOLB
    return launch_ok("maxpool5_bwd");
}

nb_status nb_upsample2(int32_t dtype, int32_t n, int32_t h, int32_t w, int32_t c, const void* src, void* dst, int32_t backward, int32_t accumulate,
                       int64_t ld_small, int64_t ld_large, void* stream) {
    g_err.clear();
    if (!src || !dst) return fail(NB_ERR_INVALID_ARG, "src and dst must not be NULL");
    NB_TRY(check_nhwc(n, h, w, c));
    if (ld_small == 0) ld_small = c;
    if (ld_large == 0) ld_large = c;
    if (ld_small < c || ld_large < c) return fail(NB_ERR_INVALID_ARG, "a pixel pitch must be 0 (dense) or at least c");
    if ((long long)n * h * w >= (1LL << 32)) return fail(NB_ERR_UNSUPPORTED, "more than 2^32 pixels");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool vec = dtype != NB_DTYPE_F32 && c % 8 == 0 && ld_small % 8 == 0 && ld_large % 8 == 0 && !((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15u);
    const unsigned blocks = glue_blocks((long long)n * h * w * (vec ? c / 8 : c));
#define NB_UPS1(T, BW, VV) launch_k(upsample2_kernel<T, BW, VV>, dim3(blocks), dim3(256), 0, st, 1, static_cast<const T*>(src), static_cast<T*>(dst), n, h, w, c, accumulate != 0, (long long)ld_small, (long long)ld_large)
#define NB_UPS(T)                                   \
    do {                                            \
        if (backward && vec) NB_UPS1(T, true, 8);   \
        else if (backward) NB_UPS1(T, true, 1);     \
        else if (vec) NB_UPS1(T, false, 8);         \
        else NB_UPS1(T, false, 1);                  \
    } while (0)
    switch (dtype) {
        case NB_DTYPE_F32: NB_UPS(float); break;
        case NB_DTYPE_BF16: NB_UPS(__nv_bfloat16); break;
        case NB_DTYPE_F16: NB_UPS(__half); break;
        default: return fail(NB_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    }
#undef NB_UPS
#undef NB_UPS1
    return launch_ok("upsample2");
}

}  // extern "C"
