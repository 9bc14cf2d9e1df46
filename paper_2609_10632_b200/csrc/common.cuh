// Shared device/host helpers of the nb_cbs library: shape record, status block, small conversions.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include "../../include/nb_cbs.h"

namespace nbcbs {

// Geometry of one Conv(k, stride, pad k/2) block; plain ints so it can be passed by value to kernels.
struct Geom {
    int n, h, w, c_in, c_out, k, stride, pad, ho, wo;
    long long m;  // n*ho*wo
    int kdim;     // k*k*c_in
};

// Device status block owned by a plan (ints): [0] error code, [1] where, [2] detail, [3] fp16 saturation count.
// Words 8 and 10 count the blocks of the normalise + SiLU pass / the dy pass that have read the fp64 channel
// accumulators (see ChanAcc); each is zero whenever no kernel of the plan is running.
enum { ST_ERR = 0, ST_WHERE = 1, ST_DETAIL = 2, ST_SAT = 3, ST_READERS_FWD = 8, ST_READERS_BWD = 10, ST_WORDS = 16 };
// Sites that a give-up is reported from (ST_WHERE): 1-5 the roles of the implicit-GEMM kernel (A producer, accumulator
// free, operands ready, accumulator ready, B producer), 11-15 the same roles of the weight-gradient kernel.

// Every wait in the library (all of them waits of a CTA on its own mbarriers: no kernel waits for another CTA's or
// another kernel's flag) is bounded: about two seconds.
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

// Records a give-up in a plan's status block (first one wins): error code, site, detail.
__device__ __forceinline__ void report_timeout(int* status, int site, int detail) {
    if (atomicCAS(status + ST_ERR, 0, (int)NB_ERR_TIMEOUT) == 0) {
        status[ST_WHERE] = site;
        status[ST_DETAIL] = detail;
    }
}

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

// Two fp32 values per instruction (fma / mul / add .f32x2 of sm_100): each half is the IEEE round-to-nearest result of the
// scalar operation, so a loop written with these gives the same bits as its scalar form with half the arithmetic issue slots.
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) {
    float2 d;
    asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmov.b64 rc, {%6, %7};\n\t"
        "fma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d.x), "=f"(d.y)
        : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y), "f"(c.x), "f"(c.y));
    return d;
}
__device__ __forceinline__ float2 mul2(float2 a, float2 b) {
    float2 d;
    asm("{\n\t.reg .b64 ra, rb, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmul.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d.x), "=f"(d.y)
        : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return d;
}
__device__ __forceinline__ float2 add2(float2 a, float2 b) {
    float2 d;
    asm("{\n\t.reg .b64 ra, rb, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tadd.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d.x), "=f"(d.y)
        : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return d;
}
__device__ __forceinline__ float2 splat2(float v) { return make_float2(v, v); }

// Elements 2j and 2j+1 of a vector as fp32, and back (round to nearest; fp16 saturates like from_f32<__half>).
template <typename T> __device__ __forceinline__ float2 pair_to_f32(const T* v);
template <> __device__ __forceinline__ float2 pair_to_f32<float>(const float* v) { return make_float2(v[0], v[1]); }
template <> __device__ __forceinline__ float2 pair_to_f32<__nv_bfloat16>(const __nv_bfloat16* v) {
    return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(v));
}
template <> __device__ __forceinline__ float2 pair_to_f32<__half>(const __half* v) { return __half22float2(*reinterpret_cast<const __half2*>(v)); }
template <typename T> __device__ __forceinline__ void pair_from_f32(T* v, float2 f);
template <> __device__ __forceinline__ void pair_from_f32<float>(float* v, float2 f) {
    v[0] = f.x;
    v[1] = f.y;
}
template <> __device__ __forceinline__ void pair_from_f32<__nv_bfloat16>(__nv_bfloat16* v, float2 f) {
    *reinterpret_cast<__nv_bfloat162*>(v) = __float22bfloat162_rn(f);
}
template <> __device__ __forceinline__ void pair_from_f32<__half>(__half* v, float2 f) {
    f.x = fminf(fmaxf(f.x, -65504.f), 65504.f);
    f.y = fminf(fmaxf(f.y, -65504.f), 65504.f);
    *reinterpret_cast<__half2*>(v) = __float22half2_rn(f);
}

// 16-byte vector of VT elements (8 x 16-bit or 4 x fp32).
template <typename T> struct __align__(16) Vec16 {
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

// Programmatic dependent launch.  Every kernel starts with pdl_launch_dependents() and executes pdl_wait() before its
// first access to global memory: the next kernel in the stream may then become resident and run its prologue (barrier
// set-up, TMEM allocation, descriptor prefetch) while this one drains, and still sees all of its results.  Because every
// kernel waits before it finishes, completion of the previous kernel implies completion of all earlier ones.  This is
// safe because no block of any kernel waits for another block: a resident block of the next kernel can delay blocks of
// this one, never stop them.
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
// Tiled transpose through shared memory: per (class, tap) the [c_out][c_in] slice of the filter (c_in contiguous) becomes
// [c_in][c_out] (c_out contiguous).  A tile is 32 c_out rows x 64 c_in columns; it is fetched with 16-byte cp.async copies
// (no registers held, so a kernel can start the fetch, do its own work and finish the tile later) and written back as
// 16-byte vectors of eight c_out values.  Channel counts are multiples of 8 on this path.
constexpr int WT_PITCH = 72;  // elements per shared-memory row of a tile (64 + padding, rows stay 16-byte aligned)
typedef __nv_bfloat16 WtTileBuf[32][WT_PITCH];
struct WtTile {
    int cls, tap, r0, c0;
};
__device__ __forceinline__ int wt_num_tiles(const WtParams& P) {
    int taps = 0;
    for (int cls = 0; cls < P.nclasses; ++cls) taps += P.cls[cls].ntaps;
    return taps * ((P.c_out + 31) / 32) * ((P.c_in + 63) / 64);
}
__device__ __forceinline__ WtTile wt_tile_decode(const WtParams& P, int t) {
    const int tc = (P.c_in + 63) / 64, per_tap = ((P.c_out + 31) / 32) * tc;
    WtTile T;
    T.tap = t / per_tap;
    const int rem = t - T.tap * per_tap;
    T.r0 = (rem / tc) * 32;
    T.c0 = (rem - (rem / tc) * tc) * 64;
    T.cls = 0;
    while (T.tap >= P.cls[T.cls].ntaps) T.tap -= P.cls[T.cls++].ntaps;
    return T;
}
// Starts the copies of one tile (all threads of the block take part); complete them with wt_async_wait() + __syncthreads().
__device__ __forceinline__ void wt_tile_load_async(const __nv_bfloat16* __restrict__ w, const WtParams& P, const WtTile& T, WtTileBuf& tile) {
    const WtClass& C = P.cls[T.cls];
    const int src_tap = C.r[T.tap] * P.k + C.t[T.tap], kk = P.k * P.k;
    for (int e = threadIdx.x; e < 256; e += blockDim.x) {
        const int i = e >> 3, v = e & 7;  // row (c_out) and 16-byte vector (eight c_in) within the tile
        const bool ok = T.r0 + i < P.c_out && T.c0 + v * 8 < P.c_in;
        const __nv_bfloat16* src = ok ? w + ((size_t)(T.r0 + i) * kk + src_tap) * P.c_in + T.c0 + v * 8 : w;
        const unsigned dst = (unsigned)__cvta_generic_to_shared(&tile[i][v * 8]);
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(ok ? 16 : 0) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
}
__device__ __forceinline__ void wt_async_wait() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
// Writes one fetched tile transposed (call after the copies have landed and the block has synchronised).
__device__ __forceinline__ void wt_tile_store(__nv_bfloat16* __restrict__ wt, const WtParams& P, const WtTile& T, const WtTileBuf& tile) {
    const WtClass& C = P.cls[T.cls];
    for (int e = threadIdx.x; e < 256; e += blockDim.x) {
        const int j = e >> 2, v = e & 3;  // column (c_in) within the tile and vector of eight c_out rows
        if (T.c0 + j < P.c_in && T.r0 + v * 8 < P.c_out) {
            Vec16<__nv_bfloat16> o;
#pragma unroll
            for (int i = 0; i < 8; ++i) o.v[i] = tile[v * 8 + i][j];
            st16(wt + C.offset + ((size_t)(T.c0 + j) * C.ntaps + T.tap) * P.c_out + T.r0 + v * 8, o);
        }
    }
}
// The whole rearrangement by `nblocks` blocks, tiles dealt round-robin (all threads of a block take part).
__device__ __forceinline__ void wt_transform_blocks(const __nv_bfloat16* __restrict__ w, __nv_bfloat16* __restrict__ wt, const WtParams& P, int block,
                                                    int nblocks, int first_round = 0) {
    __shared__ __align__(16) WtTileBuf tile;
    const int ntiles = wt_num_tiles(P);
    for (int t = block + first_round * nblocks; t < ntiles; t += nblocks) {
        const WtTile T = wt_tile_decode(P, t);
        wt_tile_load_async(w, P, T, tile);
        wt_async_wait();
        __syncthreads();
        wt_tile_store(wt, P, T, tile);
        __syncthreads();
    }
}
static __global__ void dgrad_weight_transform_kernel(const __nv_bfloat16* __restrict__ w, __nv_bfloat16* __restrict__ wt, WtParams P) {
    pdl_launch_dependents();
    pdl_wait();
    wt_transform_blocks(w, wt, P, (int)blockIdx.x, (int)gridDim.x);
}

}  // namespace nbcbs
