// CUDA-core implicit GEMMs for the three convolutions (fprop, dgrad, wgrad): any shape, fp32 or bf16 inputs,
// fp32 accumulation flushed into fp64 every 1024 terms.  They carry the fp32 reference mode and every shape
// the tensor-core kernels do not take; they are not tuned.
#pragma once
#include "common.cuh"

namespace nbcbs {

// out[i][j] = sum_kk A(i,kk) * B(kk,j).  A policy supplies the extents and element loaders.
template <typename TX, typename TW> struct FpropProblem {
    const TX* x;
    const TW* w;
    Geom g;
    static constexpr bool A_KCONTIG = true, B_KCONTIG = true;
    __device__ long long I() const { return g.m; }
    __device__ int J() const { return g.c_out; }
    __device__ long long KK() const { return g.kdim; }
    __device__ float loadA(long long i, long long kk) const {
        const int q = (int)(i % g.wo);
        const long long t1 = i / g.wo;
        const int p = (int)(t1 % g.ho), n = (int)(t1 / g.ho);
        const int c = (int)(kk % g.c_in);
        const int t2 = (int)(kk / g.c_in);
        const int t = t2 % g.k, r = t2 / g.k;
        const int h = p * g.stride - g.pad + r, ww = q * g.stride - g.pad + t;
        if (h < 0 || h >= g.h || ww < 0 || ww >= g.w) return 0.f;
        return to_f32(x[(((size_t)n * g.h + h) * g.w + ww) * g.c_in + c]);
    }
    __device__ float loadB(long long kk, int j) const { return to_f32(w[(size_t)j * g.kdim + kk]); }
};

template <typename TD, typename TW> struct DgradProblem {
    const TD* dy;
    const TW* w;
    Geom g;
    static constexpr bool A_KCONTIG = true, B_KCONTIG = false;
    __device__ long long I() const { return (long long)g.n * g.h * g.w; }
    __device__ int J() const { return g.c_in; }
    __device__ long long KK() const { return (long long)g.k * g.k * g.c_out; }
    __device__ float loadA(long long i, long long kk) const {
        const int ww = (int)(i % g.w);
        const long long t1 = i / g.w;
        const int h = (int)(t1 % g.h), n = (int)(t1 / g.h);
        const int co = (int)(kk % g.c_out);
        const int t2 = (int)(kk / g.c_out);
        const int t = t2 % g.k, r = t2 / g.k;
        const int hp = h + g.pad - r, wq = ww + g.pad - t;
        if (hp < 0 || wq < 0 || (hp % g.stride) != 0 || (wq % g.stride) != 0) return 0.f;
        const int p = hp / g.stride, q = wq / g.stride;
        if (p >= g.ho || q >= g.wo) return 0.f;
        return to_f32(dy[(((size_t)n * g.ho + p) * g.wo + q) * g.c_out + co]);
    }
    __device__ float loadB(long long kk, int j) const {
        const int co = (int)(kk % g.c_out);
        const int rt = (int)(kk / g.c_out);
        return to_f32(w[((size_t)co * g.k * g.k + rt) * g.c_in + j]);
    }
};

template <typename TD, typename TX> struct WgradProblem {
    const TD* dy;
    const TX* x;
    Geom g;
    static constexpr bool A_KCONTIG = false, B_KCONTIG = false;
    __device__ long long I() const { return g.c_out; }
    __device__ int J() const { return g.kdim; }
    __device__ long long KK() const { return g.m; }
    __device__ float loadA(long long i, long long kk) const { return to_f32(dy[(size_t)kk * g.c_out + i]); }
    __device__ float loadB(long long kk, int j) const {
        const int q = (int)(kk % g.wo);
        const long long t1 = kk / g.wo;
        const int p = (int)(t1 % g.ho), n = (int)(t1 / g.ho);
        const int c = j % g.c_in;
        const int t2 = j / g.c_in;
        const int t = t2 % g.k, r = t2 / g.k;
        const int h = p * g.stride - g.pad + r, ww = q * g.stride - g.pad + t;
        if (h < 0 || h >= g.h || ww < 0 || ww >= g.w) return 0.f;
        return to_f32(x[(((size_t)n * g.h + h) * g.w + ww) * g.c_in + c]);
    }
};

constexpr int SIMT_BM = 64, SIMT_BN = 64, SIMT_BK = 16, SIMT_FLUSH = 64;

// grid (ceil(I/64), ceil(J/64), splits); block 256.  With splits > 1, `out` is a float partial buffer
// [splits][I][J] and slice z covers kk in [z*kchunk, (z+1)*kchunk).
template <class P, typename TO>
__global__ void __launch_bounds__(256) simt_gemm_kernel(P prob, TO* __restrict__ out, long long kchunk) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ float As[SIMT_BK][SIMT_BM + 4];
    __shared__ float Bs[SIMT_BK][SIMT_BN + 4];
    const long long I = prob.I();
    const int J = prob.J();
    const long long KK = prob.KK();
    const long long i0 = (long long)blockIdx.x * SIMT_BM;
    const int j0 = blockIdx.y * SIMT_BN;
    const long long kbeg = (long long)blockIdx.z * kchunk;
    const long long kend = (kbeg + kchunk < KK) ? kbeg + kchunk : KK;
    const int tid = threadIdx.x, ty = tid / 16, tx = tid % 16;
    float acc[4][4];
    double dacc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            acc[a][b] = 0.f;
            dacc[a][b] = 0.0;
        }
    int since = 0;
    for (long long k0 = kbeg; k0 < kend; k0 += SIMT_BK) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int idx = tid + e * 256;
            int il, kl;
            if (P::A_KCONTIG) { kl = idx % SIMT_BK; il = idx / SIMT_BK; } else { il = idx % SIMT_BM; kl = idx / SIMT_BM; }
            As[kl][il] = (i0 + il < I && k0 + kl < kend) ? prob.loadA(i0 + il, k0 + kl) : 0.f;
            int jl, kb;
            if (P::B_KCONTIG) { kb = idx % SIMT_BK; jl = idx / SIMT_BK; } else { jl = idx % SIMT_BN; kb = idx / SIMT_BN; }
            Bs[kb][jl] = (j0 + jl < J && k0 + kb < kend) ? prob.loadB(k0 + kb, j0 + jl) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < SIMT_BK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                a[u] = As[kk][ty * 4 + u];
                b[u] = Bs[kk][tx * 4 + u];
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int v = 0; v < 4; ++v) acc[u][v] = fmaf(a[u], b[v], acc[u][v]);
        }
        __syncthreads();
        if (++since == SIMT_FLUSH) {
            since = 0;
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    dacc[u][v] += (double)acc[u][v];
                    acc[u][v] = 0.f;
                }
        }
    }
    TO* o = out + (size_t)blockIdx.z * (size_t)I * (size_t)J;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const long long i = i0 + ty * 4 + u;
        if (i >= I) continue;
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            const int j = j0 + tx * 4 + v;
            if (j < J) o[(size_t)i * J + j] = from_f32<TO>((float)(dacc[u][v] + (double)acc[u][v]));
        }
    }
}

// out[e] = sum_z partial[z][e], summed in fp64 in slice order (four elements per thread when the count allows).
// Eight slices are loaded before any is added so that a thread keeps eight independent 16-byte loads in flight:
// the kernel is tiny and otherwise bound by one memory latency per slice.
__global__ void __launch_bounds__(256) splitk_reduce_kernel(const float* __restrict__ partial, int splits, size_t elems, float* __restrict__ out) {
    pdl_launch_dependents();
    pdl_wait();
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    if ((elems & 3) == 0) {
        const size_t nv = elems >> 2;
        const float4* p4 = reinterpret_cast<const float4*>(partial);
        for (size_t v = (size_t)blockIdx.x * blockDim.x + threadIdx.x; v < nv; v += stride) {
            double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
            for (int z0 = 0; z0 < splits; z0 += 8) {
                float4 a[8];
#pragma unroll
                for (int u = 0; u < 8; ++u)
                    if (z0 + u < splits) a[u] = p4[(size_t)(z0 + u) * nv + v];
#pragma unroll
                for (int u = 0; u < 8; ++u)
                    if (z0 + u < splits) {
                        s0 += (double)a[u].x;
                        s1 += (double)a[u].y;
                        s2 += (double)a[u].z;
                        s3 += (double)a[u].w;
                    }
            }
            reinterpret_cast<float4*>(out)[v] = make_float4((float)s0, (float)s1, (float)s2, (float)s3);
        }
    } else {
        for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < elems; e += stride) {
            double s = 0.0;
            for (int z = 0; z < splits; ++z) s += (double)partial[(size_t)z * elems + e];
            out[e] = (float)s;
        }
    }
}

// The same sum for many slices of few elements (the first layer's weight gradient: ~1200 slices of 1296 values): a block of
// 32 x 32 threads takes 32 consecutive elements; thread (e, zg) adds slices zg, zg + 32, ... in that order in fp64 (coalesced
// 128-byte rows, eight loads in flight), and the 32 partial sums of an element are combined in the order of zg.
__global__ void __launch_bounds__(1024) splitk_reduce_tall_kernel(const float* __restrict__ partial, int splits, size_t elems, float* __restrict__ out) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ double red[32][33];
    const int ex = threadIdx.x & 31, zg = threadIdx.x >> 5;
    const size_t e = (size_t)blockIdx.x * 32 + ex;
    double acc = 0.0;
    if (e < elems) {
        for (int z0 = zg; z0 < splits; z0 += 256) {
            float a[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) a[u] = z0 + 32 * u < splits ? partial[(size_t)(z0 + 32 * u) * elems + e] : 0.f;
#pragma unroll
            for (int u = 0; u < 8; ++u) acc += (double)a[u];
        }
    }
    red[zg][ex] = acc;
    __syncthreads();
    if (zg == 0 && e < elems) {
        double s = 0.0;
#pragma unroll 8
        for (int k = 0; k < 32; ++k) s += red[k][ex];
        out[e] = (float)s;
    }
}

}  // namespace nbcbs
