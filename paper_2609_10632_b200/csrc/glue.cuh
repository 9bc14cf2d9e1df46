// Glue between chained blocks: out[r][c] = (accumulate ? out[r][c] : 0) + a[r][c] (+ b[r][c]) over `rows` pixels and
// `channels` channels, where every operand is a CHANNEL SLICE of an NHWC tensor (its own row pitch in elements, its
// pointer already advanced to the slice's first channel).  One kernel covers what a chained C2f / PAN block needs:
// channel split and concat (copy into / out of a slice), the residual add, and the accumulation of gradients that fan
// out to several consumers.  Sums are formed in fp32 and rounded once.
#pragma once
#include "common.cuh"

namespace nbcbs {

// IdxT = unsigned when the vector count fits 32 bits (cheap divisions), long long otherwise.  (A variant with four
// iterations in flight per thread and a quarter of the blocks was measured slower inside the chained detector: these
// tensors mostly sit in L2, where more resident blocks beat deeper per-thread pipelines.)
template <typename T, bool VEC, typename IdxT>
__global__ void __launch_bounds__(256) slice_add_kernel(T* __restrict__ out, long long ld_out, const T* __restrict__ a, long long ld_a,
                                                        const T* __restrict__ b, long long ld_b, long long rows, int channels, int accumulate) {
    pdl_launch_dependents();
    pdl_wait();
    constexpr int V = VEC ? Vec16<T>::N : 1;
    const IdxT cv = (IdxT)(channels / V);  // vectors per row
    const IdxT total = (IdxT)rows * cv, stride = (IdxT)gridDim.x * (IdxT)blockDim.x;
    for (IdxT i = (IdxT)blockIdx.x * (IdxT)blockDim.x + (IdxT)threadIdx.x; i < total; i += stride) {
        const long long r = (long long)(i / cv);
        const int c = (int)(i - (IdxT)r * cv) * V;
        if (VEC) {
            const Vec16<T> va = ld16(a + r * ld_a + c);
            Vec16<T> vb, vo, res;
            if (b) vb = ld16(b + r * ld_b + c);
            if (accumulate) vo = ld16(out + r * ld_out + c);
#pragma unroll
            for (int k = 0; k < V; ++k) {
                float s = to_f32(va.v[k]);
                if (b) s += to_f32(vb.v[k]);
                if (accumulate) s += to_f32(vo.v[k]);
                res.v[k] = from_f32<T>(s);
            }
            st16(out + r * ld_out + c, res);
        } else {
            float s = to_f32(a[r * ld_a + c]);
            if (b) s += to_f32(b[r * ld_b + c]);
            if (accumulate) s += to_f32(out[r * ld_out + c]);
            out[r * ld_out + c] = from_f32<T>(s);
        }
    }
}


}  // namespace nbcbs

namespace nbcbs {

// 5x5 max-pool, stride 1, padding 2 over NHWC (the SPPF unit chains three of them).  One thread per 8-channel (16-byte)
// vector of an output pixel, or per element when C % 8 != 0.  idx (optional, one byte per element) = r*5 + t of the FIRST
// maximum of the window in row-major order: comparisons are strict, elements outside the image never win.
template <typename T, int V>
__global__ void __launch_bounds__(256) maxpool5_fwd_kernel(const T* __restrict__ x, T* __restrict__ y, uint8_t* __restrict__ idx, int N, int H, int W, int C,
                                                           long long ld_x, long long ld_y /* pixel pitches of x and y; idx is dense */) {
    pdl_launch_dependents();
    pdl_wait();
    const int cv = C / V;
    const long long total = (long long)N * H * W * cv;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(i % cv) * V;
        long long t1 = i / cv;
        const int q = (int)(t1 % W);
        t1 /= W;
        const int p = (int)(t1 % H);
        const long long n = t1 / H;
        float best[V];
        int bi[V];
#pragma unroll
        for (int k = 0; k < V; ++k) {
            best[k] = -__int_as_float(0x7f800000);
            bi[k] = 0;
        }
        for (int r = 0; r < 5; ++r) {
            const int h = p - 2 + r;
            if (h < 0 || h >= H) continue;
            for (int t = 0; t < 5; ++t) {
                const int w = q - 2 + t;
                if (w < 0 || w >= W) continue;
                const T* src = x + (((n * H + h) * W + w) * ld_x + c);
                T v[V];
                if (V == 8) *reinterpret_cast<uint4*>(v) = *reinterpret_cast<const uint4*>(src); else v[0] = src[0];
#pragma unroll
                for (int k = 0; k < V; ++k) {
                    const float f = to_f32(v[k]);
                    if (f > best[k]) {
                        best[k] = f;
                        bi[k] = r * 5 + t;
                    }
                }
            }
        }
        const long long pixo = (n * H + p) * W + q;
        const long long o = pixo * (long long)C + c, oy = pixo * ld_y + c;
#pragma unroll
        for (int k = 0; k < V; ++k) {
            y[oy + k] = from_f32<T>(best[k]);  // the maximum of stored values is itself a stored value: exact
            if (idx) idx[o + k] = (uint8_t)bi[k];
        }
    }
}

// dx[n][h][w][c] = sum of g over the (at most 25) windows whose recorded maximum is this element; fp32 sum in fixed
// (row-major window) order, one rounding.  accumulate != 0 adds the result to dx instead of overwriting it.  One thread per
// V channels of an input pixel (V = 8 with 16-byte loads of g and 8-byte loads of the recorded positions, or 1).
template <typename T, int V>
__global__ void __launch_bounds__(256) maxpool5_bwd_kernel(const T* __restrict__ g, const uint8_t* __restrict__ idx, T* __restrict__ dx, int N, int H, int W,
                                                           int C, int accumulate, long long ld_g, long long ld_dx /* pixel pitches of g and dx; idx is dense */) {
    pdl_launch_dependents();
    pdl_wait();
    const unsigned cv = (unsigned)(C / V);
    const long long total = (long long)N * H * W * cv;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const unsigned pix = (unsigned)(i / cv);  // fewer than 2^32 pixels (checked by the caller)
        const int c = (int)((unsigned)(i - (long long)pix * cv)) * V;
        const unsigned t1 = pix / (unsigned)W;
        const int w = (int)(pix - t1 * (unsigned)W);
        const unsigned n = t1 / (unsigned)H;
        const int h = (int)(t1 - n * (unsigned)H);
        float s[V];
#pragma unroll
        for (int k = 0; k < V; ++k) s[k] = 0.f;
        for (int r = 4; r >= 0; --r) {  // the window at output row p = h + 2 - r sees this element at offset r
            const int p = h + 2 - r;
            if (p < 0 || p >= H) continue;
            for (int t = 4; t >= 0; --t) {
                const int q = w + 2 - t;
                if (q < 0 || q >= W) continue;
                const long long pixo = ((long long)n * H + p) * W + q;
                const long long o = pixo * (long long)C + c, og = pixo * ld_g + c;
                const int code = r * 5 + t;
                if (V == 8) {
                    const uint2 ib = *reinterpret_cast<const uint2*>(idx + o);
                    const uint32_t pat = (uint32_t)code * 0x01010101u;
                    if (((ib.x ^ pat) & 0xffu) && ((ib.x ^ pat) & 0xff00u) && ((ib.x ^ pat) & 0xff0000u) && ((ib.x ^ pat) & 0xff000000u) &&
                        ((ib.y ^ pat) & 0xffu) && ((ib.y ^ pat) & 0xff00u) && ((ib.y ^ pat) & 0xff0000u) && ((ib.y ^ pat) & 0xff000000u))
                        continue;  // none of the eight channels of this window points here
                    const Vec16<T> gv = ld16(g + og);
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const uint32_t byte = ((k < 4 ? ib.x : ib.y) >> (8 * (k & 3))) & 0xffu;
                        if (byte == (uint32_t)code) s[k] += to_f32(gv.v[k]);
                    }
                } else if (idx[o] == code) {
                    s[0] += to_f32(g[og]);
                }
            }
        }
        const long long oi = (long long)pix * ld_dx + c;
        if (V == 8) {
            Vec16<T> res;
            if (accumulate) {
                const Vec16<T> old = ld16(dx + oi);
#pragma unroll
                for (int k = 0; k < 8; ++k) s[k] += to_f32(old.v[k]);
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) res.v[k] = from_f32<T>(s[k]);
            st16(dx + oi, res);
        } else {
            if (accumulate) s[0] += to_f32(dx[oi]);
            dx[oi] = from_f32<T>(s[0]);
        }
    }
}

// Nearest-neighbour 2x upsampling y[n][2h+a][2w+b][c] = x[n][h][w][c] (BWD = false), and its adjoint
// dx[n][h][w][c] = sum of the four g (BWD = true; fp32 sum, one rounding; accumulate adds to dx).  x / dx is [N][H][W][C];
// one thread per V channels of a small-tensor pixel (V = 8: 16-byte accesses, or 1).
template <typename T, bool BWD, int V>
__global__ void __launch_bounds__(256) upsample2_kernel(const T* __restrict__ src, T* __restrict__ dst, int N, int H, int W, int C, int accumulate,
                                                        long long ld_s /* pixel pitch of the small tensor */, long long ld_l /* of the large one */) {
    pdl_launch_dependents();
    pdl_wait();
    const unsigned cv = (unsigned)(C / V);
    const long long total = (long long)N * H * W * cv;
    const long long row2 = 2LL * W * ld_l, nx = ld_l;  // one row down / one pixel to the right in the large tensor
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const unsigned pix = (unsigned)(i / cv);
        const int c = (int)((unsigned)(i - (long long)pix * cv)) * V;
        const unsigned t1 = pix / (unsigned)W;
        const int w = (int)(pix - t1 * (unsigned)W);
        const unsigned n = t1 / (unsigned)H;
        const int h = (int)(t1 - n * (unsigned)H);
        const long long os = (long long)pix * ld_s + c;                                   // in the small tensor
        const long long o = (((long long)n * 2 * H + 2 * h) * 2 * W + 2 * w) * ld_l + c;  // (2h, 2w) in the large tensor
        if (V == 8) {
            if (BWD) {
                const Vec16<T> a0 = ld16(src + o), a1 = ld16(src + o + nx), a2 = ld16(src + o + row2), a3 = ld16(src + o + row2 + nx);
                Vec16<T> old, res;
                if (accumulate) old = ld16(dst + os);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    float sum = (to_f32(a0.v[k]) + to_f32(a1.v[k])) + (to_f32(a2.v[k]) + to_f32(a3.v[k]));
                    if (accumulate) sum += to_f32(old.v[k]);
                    res.v[k] = from_f32<T>(sum);
                }
                st16(dst + os, res);
            } else {
                const Vec16<T> v = ld16(src + os);
                st16(dst + o, v);
                st16(dst + o + nx, v);
                st16(dst + o + row2, v);
                st16(dst + o + row2 + nx, v);
            }
        } else if (BWD) {
            float sum = (to_f32(src[o]) + to_f32(src[o + nx])) + (to_f32(src[o + row2]) + to_f32(src[o + row2 + nx]));
            if (accumulate) sum += to_f32(dst[os]);
            dst[os] = from_f32<T>(sum);
        } else {
            const T v = src[os];
            dst[o] = v;
            dst[o + nx] = v;
            dst[o + row2] = v;
            dst[o + row2 + nx] = v;
        }
    }
}

}  // namespace nbcbs
