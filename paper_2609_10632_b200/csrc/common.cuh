// Shared device/host helpers of the nb_cbs library: shape record, status block, small conversions.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

namespace nbcbs {

// Geometry of one Conv(k, stride, pad k/2) block; plain ints so it can be passed by value to kernels.
struct Geom {
    int n, h, w, c_in, c_out, k, stride, pad, ho, wo;
    long long m;  // n*ho*wo
    int kdim;     // k*k*c_in
};

// Device status block owned by a plan (ints): [0] error code, [1] where, [2] detail, [3] fp16 saturation count.
enum { ST_ERR = 0, ST_WHERE = 1, ST_DETAIL = 2, ST_SAT = 3, ST_WORDS = 16 };

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <> __device__ __forceinline__ float to_f32<__half>(__half v) { return __half2float(v); }

template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }
// fp16 stores saturate instead of producing inf (the saved conv output must stay finite for BN).
template <> __device__ __forceinline__ __half from_f32<__half>(float v) {
    return __float2half_rn(fminf(fmaxf(v, -65504.f), 65504.f));
}

// 16-byte vector of VT elements (8 x 16-bit or 4 x fp32).
template <typename T> struct Vec16 {
    static constexpr int N = 16 / sizeof(T);
    T v[N];
};
template <typename T> __device__ __forceinline__ Vec16<T> ld16(const T* p) {
    Vec16<T> r;
    *reinterpret_cast<uint4*>(&r) = *reinterpret_cast<const uint4*>(p);
    return r;
}
template <typename T> __device__ __forceinline__ void st16(T* p, const Vec16<T>& r) {
    *reinterpret_cast<uint4*>(p) = *reinterpret_cast<const uint4*>(&r);
}
// Streaming variants: data touched once should not displace reusable lines in L1.
template <typename T> __device__ __forceinline__ Vec16<T> ld16_stream(const T* p) {
    Vec16<T> r;
    *reinterpret_cast<uint4*>(&r) = __ldcs(reinterpret_cast<const uint4*>(p));
    return r;
}
template <typename T> __device__ __forceinline__ void st16_stream(T* p, const Vec16<T>& r) {
    __stcs(reinterpret_cast<uint4*>(p), *reinterpret_cast<const uint4*>(&r));
}

// Programmatic dependent launch.  Every kernel of the library starts with pdl_launch_dependents() and executes pdl_wait()
// before its first access to global memory: the next kernel in the stream may then become resident and run its prologue
// (barrier set-up, TMEM allocation, descriptor prefetch) while this one drains, and still sees all of its results.
// Because every kernel waits before it finishes, completion of the previous kernel implies completion of all earlier ones.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

inline bool pdl_enabled() {
    static const bool on = !(getenv("NB_PDL") && atoi(getenv("NB_PDL")) == 0);
    return on;
}

// Launches `kernel` on `st` with the programmatic-serialization attribute (and a cluster of `cluster_x` CTAs when > 1).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, int cluster_x, Args&&... args) {
    cudaLaunchConfig_t lc;
    memset(&lc, 0, sizeof lc);
    lc.gridDim = grid;
    lc.blockDim = block;
    lc.dynamicSmemBytes = smem;
    lc.stream = st;
    cudaLaunchAttribute at[2];
    unsigned n = 0;
    if (pdl_enabled()) {
        at[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    if (cluster_x > 1) {
        at[n].id = cudaLaunchAttributeClusterDimension;
        at[n].val.clusterDim.x = (unsigned)cluster_x;
        at[n].val.clusterDim.y = 1;
        at[n].val.clusterDim.z = 1;
        ++n;
    }
    lc.attrs = at;
    lc.numAttrs = n;
    return cudaLaunchKernelEx(&lc, kernel, static_cast<KArgs>(args)...);
}

// Rearranged filter for dgrad: for parity class `cls` (a list of taps), wt[c][ti][c'] = w[c'][r_ti][t_ti][c].
struct WtClass {
    int ntaps;
    int r[9], t[9];
    size_t offset;  // element offset of this class's matrix in the output buffer
};
struct WtParams {
    int c_in, c_out, k, nclasses;
    WtClass cls[4];
};
// One thread per output element, output-contiguous (c' fastest); `block` of `nblocks` blocks of blockDim.x threads.
__device__ __forceinline__ void wt_transform_blocks(const __nv_bfloat16* __restrict__ w, __nv_bfloat16* __restrict__ wt, const WtParams& P, int block,
                                                    int nblocks) {
    const size_t total = (size_t)P.c_in * P.k * P.k * P.c_out;
    for (size_t e = (size_t)block * blockDim.x + threadIdx.x; e < total; e += (size_t)nblocks * blockDim.x) {
        int cls = 0;
        while (cls + 1 < P.nclasses && e >= P.cls[cls + 1].offset) ++cls;
        const WtClass& C = P.cls[cls];
        size_t le = e - C.offset;
        const int co = (int)(le % P.c_out);
        le /= P.c_out;
        const int ti = (int)(le % C.ntaps);
        const int c = (int)(le / C.ntaps);
        wt[e] = w[(((size_t)co * P.k + C.r[ti]) * P.k + C.t[ti]) * P.c_in + c];
    }
}
__global__ void dgrad_weight_transform_kernel(const __nv_bfloat16* __restrict__ w, __nv_bfloat16* __restrict__ wt, WtParams P) {
    pdl_launch_dependents();
    pdl_wait();
    wt_transform_blocks(w, wt, P, (int)blockIdx.x, (int)gridDim.x);
}

}  // namespace nbcbs
