// Direct CUDA-core kernels for the network's first layer: 3 input channels, 3x3, stride 2, pad 1.
// A 3-channel bf16 pixel is 6 bytes, which no TMA descriptor can address (strides must be multiples of 16 bytes),
// and with K = 27 the layer is bound by HBM traffic, not by arithmetic: these kernels keep the filter in shared
// memory as fp32, one thread per output pixel (fprop), per pair of input pixels (dgrad), or per 4x3 patch of the
// filter gradient (wgrad).  COUT is a template parameter (48 for the detector's stem).
#pragma once
#include "common.cuh"

namespace nbcbs {

constexpr int STEM_CIN = 3, STEM_K = 3, STEM_TAPS = 9, STEM_KDIM = 27;

// y[n,p,q,:] = sum_{r,t,c} x[n,2p-1+r,2q-1+t,c] * w[:,r,t,c]   (fp16 output, fp32 accumulate)
template <int COUT>
__global__ void __launch_bounds__(128) stem_fprop_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ w,
                                                         __half* __restrict__ y, Geom g) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ __align__(16) float ws[STEM_KDIM][COUT];  // ws[k][c'] = w[c'][k]
    for (int e = threadIdx.x; e < STEM_KDIM * COUT; e += blockDim.x) {
        const int co = e / STEM_KDIM, k = e % STEM_KDIM;
        ws[k][co] = __bfloat162float(w[e]);
    }
    __syncthreads();
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long m = (long long)blockIdx.x * blockDim.x + threadIdx.x; m < g.m; m += stride) {
        const int q = (int)(m % g.wo);
        const long long t1 = m / g.wo;
        const int p = (int)(t1 % g.ho), n = (int)(t1 / g.ho);
        float xin[STEM_KDIM];
#pragma unroll
        for (int r = 0; r < 3; ++r) {
            const int h = 2 * p - 1 + r;
#pragma unroll
            for (int t = 0; t < 3; ++t) {
                const int ww = 2 * q - 1 + t;
                const bool ok = h >= 0 && h < g.h && ww >= 0 && ww < g.w;
                const __nv_bfloat16* px = x + (((size_t)n * g.h + (ok ? h : 0)) * g.w + (ok ? ww : 0)) * 3;
#pragma unroll
                for (int c = 0; c < 3; ++c) xin[(r * 3 + t) * 3 + c] = ok ? __bfloat162float(px[c]) : 0.f;
            }
        }
        float acc[COUT];
#pragma unroll
        for (int c = 0; c < COUT; ++c) acc[c] = 0.f;
#pragma unroll
        for (int k = 0; k < STEM_KDIM; ++k) {
            const float xv = xin[k];
#pragma unroll
            for (int c = 0; c < COUT; c += 4) {
                const float4 wv = *reinterpret_cast<const float4*>(&ws[k][c]);
                acc[c] = fmaf(xv, wv.x, acc[c]);
                acc[c + 1] = fmaf(xv, wv.y, acc[c + 1]);
                acc[c + 2] = fmaf(xv, wv.z, acc[c + 2]);
                acc[c + 3] = fmaf(xv, wv.w, acc[c + 3]);
            }
        }
        __half* yo = y + (size_t)m * COUT;
#pragma unroll
        for (int c = 0; c < COUT; c += 8) {
            Vec16<__half> v;
#pragma unroll
            for (int i = 0; i < 8; ++i) v.v[i] = from_f32<__half>(acc[c + i]);
            st16(yo + c, v);
        }
    }
}

// dx for two horizontally adjacent input pixels (w = 2*w2, 2*w2+1) per thread; H and W even.
// Input column 2*w2 sees filter column t=1 at output column w2; column 2*w2+1 sees t=0 at w2+1 and t=2 at w2.
// Input row h even sees filter row r=1 at output row h/2; h odd sees r=0 at (h+1)/2 and r=2 at (h-1)/2.
template <int COUT>
__global__ void __launch_bounds__(128) stem_dgrad_kernel(const __nv_bfloat16* __restrict__ dy, const __nv_bfloat16* __restrict__ w,
                                                         __nv_bfloat16* __restrict__ dx, Geom g) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ __align__(16) float ws[STEM_TAPS][COUT][4];  // ws[tap][c'][c], c padded to 4
    for (int e = threadIdx.x; e < STEM_TAPS * COUT; e += blockDim.x) {
        const int tap = e / COUT, co = e % COUT;
#pragma unroll
        for (int c = 0; c < 3; ++c) ws[tap][co][c] = __bfloat162float(w[((size_t)co * STEM_TAPS + tap) * 3 + c]);
        ws[tap][co][3] = 0.f;
    }
    __syncthreads();
    const int w2n = g.w / 2;
    const long long total = (long long)g.n * g.h * w2n;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += stride) {
        const int w2 = (int)(idx % w2n);
        const long long t1 = idx / w2n;
        const int h = (int)(t1 % g.h), n = (int)(t1 / g.h);
        float e0 = 0.f, e1 = 0.f, e2 = 0.f;  // pixel (h, 2*w2)
        float o0 = 0.f, o1 = 0.f, o2 = 0.f;  // pixel (h, 2*w2+1)
        const int nrows = (h & 1) ? 2 : 1;
        for (int ri = 0; ri < nrows; ++ri) {
            int r, p;
            if (h & 1) {
                r = ri == 0 ? 0 : 2;
                p = ri == 0 ? (h + 1) / 2 : (h - 1) / 2;
            } else {
                r = 1;
                p = h / 2;
            }
            if (p >= g.ho) continue;
            const __nv_bfloat16* row = dy + (((size_t)n * g.ho + p) * g.wo) * COUT;
            const __nv_bfloat16* dA = row + (size_t)w2 * COUT;  // output column w2
            const bool hasB = w2 + 1 < g.wo;
            const __nv_bfloat16* dB = row + (size_t)(hasB ? w2 + 1 : w2) * COUT;  // output column w2+1
#pragma unroll
            for (int c0 = 0; c0 < COUT; c0 += 8) {
                const Vec16<__nv_bfloat16> va = ld16(dA + c0);
                const Vec16<__nv_bfloat16> vb = ld16(dB + c0);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float a = __bfloat162float(va.v[i]);
                    const float b = hasB ? __bfloat162float(vb.v[i]) : 0.f;
                    const float4 w1 = *reinterpret_cast<const float4*>(ws[r * 3 + 1][c0 + i]);  // t = 1
                    const float4 w0 = *reinterpret_cast<const float4*>(ws[r * 3 + 0][c0 + i]);  // t = 0
                    const float4 w2v = *reinterpret_cast<const float4*>(ws[r * 3 + 2][c0 + i]); // t = 2
                    e0 = fmaf(a, w1.x, e0); e1 = fmaf(a, w1.y, e1); e2 = fmaf(a, w1.z, e2);
                    o0 = fmaf(b, w0.x, o0); o1 = fmaf(b, w0.y, o1); o2 = fmaf(b, w0.z, o2);
                    o0 = fmaf(a, w2v.x, o0); o1 = fmaf(a, w2v.y, o1); o2 = fmaf(a, w2v.z, o2);
                }
            }
        }
        // six consecutive bf16 values (12 bytes) at a 4-byte aligned address
        __nv_bfloat16* o = dx + (((size_t)n * g.h + h) * g.w + 2 * (size_t)w2) * 3;
        __nv_bfloat162* o2p = reinterpret_cast<__nv_bfloat162*>(o);
        o2p[0] = __floats2bfloat162_rn(e0, e1);
        o2p[1] = __floats2bfloat162_rn(e2, o0);
        o2p[2] = __floats2bfloat162_rn(o1, o2);
    }
}

// dw partials: block b accumulates dw over its pixel range; thread (cg, tap) owns dw[4*cg .. 4*cg+3][tap][0..2].
// partial layout [gridDim.x][COUT][27].
template <int COUT>
__global__ void __launch_bounds__(128) stem_wgrad_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ dy,
                                                         float* __restrict__ partial, Geom g, long long pix_per_block) {
    pdl_launch_dependents();
    pdl_wait();
    constexpr int P = 32;  // pixels per staged chunk
    constexpr int NCG = COUT / 4;
    __shared__ __align__(16) float dys[P][COUT];
    __shared__ float xs[P][STEM_KDIM + 1];
    const int tid = threadIdx.x;
    const int cg = tid / STEM_TAPS, tap = tid % STEM_TAPS;
    const bool compute = tid < NCG * STEM_TAPS;
    float acc[4][3];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int c = 0; c < 3; ++c) acc[a][c] = 0.f;
    const long long m_begin = (long long)blockIdx.x * pix_per_block;
    const long long m_end = (m_begin + pix_per_block < g.m) ? m_begin + pix_per_block : g.m;
    for (long long m0 = m_begin; m0 < m_end; m0 += P) {
        const int np = (int)((m_end - m0 < P) ? (m_end - m0) : P);
        // stage dy (COUT/8 vectors per pixel) and the 27 input values of every pixel
        for (int e = tid; e < P * (COUT / 8); e += blockDim.x) {
            const int pi = e / (COUT / 8), v = e % (COUT / 8);
            if (pi < np) {
                const Vec16<__nv_bfloat16> q = ld16(dy + (size_t)(m0 + pi) * COUT + v * 8);
#pragma unroll
                for (int i = 0; i < 8; ++i) dys[pi][v * 8 + i] = __bfloat162float(q.v[i]);
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) dys[pi][v * 8 + i] = 0.f;
            }
        }
        for (int e = tid; e < P * STEM_TAPS; e += blockDim.x) {
            const int pi = e / STEM_TAPS, tp = e % STEM_TAPS;
            float v0 = 0.f, v1 = 0.f, v2 = 0.f;
            if (pi < np) {
                const long long m = m0 + pi;
                const int q = (int)(m % g.wo);
                const long long t1 = m / g.wo;
                const int p = (int)(t1 % g.ho), n = (int)(t1 / g.ho);
                const int h = 2 * p - 1 + tp / 3, ww = 2 * q - 1 + tp % 3;
                if (h >= 0 && h < g.h && ww >= 0 && ww < g.w) {
                    const __nv_bfloat16* px = x + (((size_t)n * g.h + h) * g.w + ww) * 3;
                    v0 = __bfloat162float(px[0]);
                    v1 = __bfloat162float(px[1]);
                    v2 = __bfloat162float(px[2]);
                }
            }
            xs[pi][tp * 3] = v0;
            xs[pi][tp * 3 + 1] = v1;
            xs[pi][tp * 3 + 2] = v2;
        }
        __syncthreads();
        if (compute) {
#pragma unroll 8
            for (int pi = 0; pi < P; ++pi) {
                const float4 d = *reinterpret_cast<const float4*>(&dys[pi][cg * 4]);
                const float x0 = xs[pi][tap * 3], x1 = xs[pi][tap * 3 + 1], x2 = xs[pi][tap * 3 + 2];
                acc[0][0] = fmaf(d.x, x0, acc[0][0]); acc[0][1] = fmaf(d.x, x1, acc[0][1]); acc[0][2] = fmaf(d.x, x2, acc[0][2]);
                acc[1][0] = fmaf(d.y, x0, acc[1][0]); acc[1][1] = fmaf(d.y, x1, acc[1][1]); acc[1][2] = fmaf(d.y, x2, acc[1][2]);
                acc[2][0] = fmaf(d.z, x0, acc[2][0]); acc[2][1] = fmaf(d.z, x1, acc[2][1]); acc[2][2] = fmaf(d.z, x2, acc[2][2]);
                acc[3][0] = fmaf(d.w, x0, acc[3][0]); acc[3][1] = fmaf(d.w, x1, acc[3][1]); acc[3][2] = fmaf(d.w, x2, acc[3][2]);
            }
        }
        __syncthreads();
    }
    if (compute) {
        float* o = partial + (size_t)blockIdx.x * COUT * STEM_KDIM;
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int c = 0; c < 3; ++c) o[(size_t)(cg * 4 + a) * STEM_KDIM + tap * 3 + c] = acc[a][c];
    }
}

}  // namespace nbcbs
