// Glue between chained blocks: out[r][c] = (accumulate ? out[r][c] : 0) + a[r][c] (+ b[r][c]) over `rows` pixels and
// `channels` channels, where every operand is a CHANNEL SLICE of an NHWC tensor (its own row pitch in elements, its
// pointer already advanced to the slice's first channel).  One kernel covers what a chained C2f / PAN block needs:
// channel split and concat (copy into / out of a slice), the residual add, and the accumulation of gradients that fan
// out to several consumers.  Sums are formed in fp32 and rounded once.
#pragma once
#include "common.cuh"

namespace nbcbs {

template <typename T, bool VEC>
__global__ void __launch_bounds__(256) slice_add_kernel(T* __restrict__ out, long long ld_out, const T* __restrict__ a, long long ld_a,
                                                        const T* __restrict__ b, long long ld_b, long long rows, int channels, int accumulate) {
    pdl_launch_dependents();
    pdl_wait();
    constexpr int V = VEC ? Vec16<T>::N : 1;
    const int cv = channels / V;  // vectors per row
    const long long total = rows * cv;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const long long r = i / cv;
        const int c = (int)(i - r * cv) * V;
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
