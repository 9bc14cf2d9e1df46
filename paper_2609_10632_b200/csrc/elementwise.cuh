// HBM-bound passes over [M][C] NHWC tensors: batch statistics, normalise+affine+SiLU, and their backward.
// All of them walk the tensor as a flat array of 16-byte vectors with a stride that is a multiple of the
// number of vectors per row, so a thread always sees the same channel group: per-channel parameters and
// accumulators live in registers, loads are fully coalesced, and reductions have a fixed order
// (bitwise reproducible run to run: no floating-point atomics anywhere).
#pragma once
#include "common.cuh"

namespace nbcbs {

// sigmoid(z).  The fast form is 0.5*tanh(z/2) + 0.5 with the hardware tanh approximation (one special-function
// instruction instead of an exponential and a reciprocal; absolute error about 2.5e-4, far below the bf16 rounding of
// the results it feeds); these passes issue enough instructions per byte that the special-function unit matters.
template <bool FAST> __device__ __forceinline__ float sigmoid_f(float z) {
    if (FAST) {
        float t;
        asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(0.5f * z));
        return fmaf(0.5f, t, 0.5f);
    } else {
        return 1.f / (1.f + expf(-z));
    }
}

// The same for two values at once, and dz = g * s * (1 + z*(1 - s)) with s = sigmoid(z) (the derivative of SiLU times g);
// the operations and their order are those of the scalar expressions the passes used to spell out, so the bits agree.
template <bool FAST> __device__ __forceinline__ float2 sigmoid2(float2 z) {
    if (FAST) {
        const float2 hz = mul2(splat2(0.5f), z);
        float2 t;
        asm("tanh.approx.f32 %0, %1;" : "=f"(t.x) : "f"(hz.x));
        asm("tanh.approx.f32 %0, %1;" : "=f"(t.y) : "f"(hz.y));
        return fma2(splat2(0.5f), t, splat2(0.5f));
    } else {
        return make_float2(sigmoid_f<false>(z.x), sigmoid_f<false>(z.y));
    }
}
template <bool FAST> __device__ __forceinline__ float2 silu_bwd_dz2(float2 z, float2 g) {
    const float2 s = sigmoid2<FAST>(z);
    const float2 oms = fma2(s, splat2(-1.f), splat2(1.f));  // 1 - s, exactly
    return mul2(mul2(g, s), fma2(z, oms, splat2(1.f)));
}

// ------------------------------------------------------------------ per-channel sum and sum of squares
// partials layout: [gridDim.x][2][C]; blockDim.x = (C/V) * R.
template <typename YT>
__global__ void __launch_bounds__(288, 3) bn_stats_partial_kernel(const YT* __restrict__ y, long long total_vecs, int C,
                                                                float* __restrict__ partials) {
    pdl_launch_dependents();
    pdl_wait();
    constexpr int V = Vec16<YT>::N;
    extern __shared__ float red[];  // [blockDim.x][V]
    const int tid = threadIdx.x;
    const int cgs = C / V;
    float s[V], ss[V];
#pragma unroll
    for (int i = 0; i < V; ++i) s[i] = ss[i] = 0.f;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long v = (long long)blockIdx.x * blockDim.x + tid; v < total_vecs; v += stride) {
        const Vec16<YT> q = ld16(y + v * V);
#pragma unroll
        for (int i = 0; i < V; ++i) {
            const float f = to_f32(q.v[i]);
            s[i] += f;
            ss[i] = fmaf(f, f, ss[i]);
        }
    }
    const int R = blockDim.x / cgs;
    for (int pass = 0; pass < 2; ++pass) {
#pragma unroll
        for (int i = 0; i < V; ++i) red[tid * V + i] = pass ? ss[i] : s[i];
        __syncthreads();
        for (int c = tid; c < C; c += blockDim.x) {
            const int g = c / V, e = c % V;
            float acc = 0.f;
            for (int r = 0; r < R; ++r) acc += red[(r * cgs + g) * V + e];
            partials[((size_t)blockIdx.x * 2 + pass) * C + c] = acc;
        }
        __syncthreads();
    }
}

// Both sums of channel c at once: s0 = sum over b of partials[b][0][c], s1 = the same for [b][1][c].  Lane l takes
// b = l, l+32, ... (all loads of a step are issued before any is used), then a butterfly over the 32 lanes, in fp64.
// The order is fixed, so the result is bitwise reproducible.
// L2 = read around L1 (the partials were written by other CTAs of the same launch).
// Sixteen loads (eight slices x two quantities) are issued before the first is used, so up to 256 slices cost one
// memory round trip; the fused finalize steps at the tail of other kernels sit on the critical path.
template <bool L2 = false>
__device__ __forceinline__ void warp_sum_partials2(const float* __restrict__ partials, int nparts, int C, int c, int lane, double& s0, double& s1) {
    double a0 = 0.0, a1 = 0.0, b0 = 0.0, b1 = 0.0;
    const float* base = partials + c;
    const size_t step = (size_t)2 * C;
    for (int b = lane; b < nparts; b += 256) {
        float u[8], v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int bk = b + 32 * k;
            const float* q = base + (size_t)bk * step;
            u[k] = bk < nparts ? (L2 ? __ldcg(q) : *q) : 0.f;
            v[k] = bk < nparts ? (L2 ? __ldcg(q + C) : q[C]) : 0.f;
        }
#pragma unroll
        for (int k = 0; k < 8; k += 2) {
            a0 += (double)u[k];
            b0 += (double)v[k];
            a1 += (double)u[k + 1];
            b1 += (double)v[k + 1];
        }
    }
    double s = a0 + a1, q = b0 + b1;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        s += __shfl_xor_sync(0xffffffffu, s, o);
        q += __shfl_xor_sync(0xffffffffu, q, o);
    }
    s0 = s;
    s1 = q;
}

// The finalize of one channel by one warp (also called from the tail of the tensor-core forward kernel).
template <bool L2>
__device__ __forceinline__ void bn_finalize_channel(const float* __restrict__ partials, int nparts, int C, int c, int lane, double M, float eps,
                                                    float momentum, const float* __restrict__ gamma, const float* __restrict__ beta, float* mean,
                                                    float* invstd, float* scale, float* shift, float* rmean, float* rvar, float* sum_out,
                                                    float* sumsq_out) {
    // the per-channel inputs of the last step are requested first so that they arrive while the partials are summed
    const float ga = scale ? gamma[c] : 0.f, be = scale ? beta[c] : 0.f;
    const float rm = rmean ? rmean[c] : 0.f, rv = rmean ? rvar[c] : 0.f;
    double s, q;
    warp_sum_partials2<L2>(partials, nparts, C, c, lane, s, q);
    if (lane == 0) {
        // (this chain sits on the critical path of the forward kernel's tail: one reciprocal serves all divisions by M,
        // and the inverse square root is the library's, accurate to within two units in the last place of fp64)
        const double inv_m = 1.0 / M;
        const double mu = s * inv_m;
        double var = q * inv_m - mu * mu;
        if (var < 0.0) var = 0.0;
        const double is = rsqrt(var + (double)eps);
        if (mean) mean[c] = (float)mu;
        if (invstd) invstd[c] = (float)is;
        if (scale) {
            const double sc = (double)ga * is;
            scale[c] = (float)sc;
            shift[c] = (float)((double)be - mu * sc);
        }
        if (sum_out) sum_out[c] = (float)s;
        if (sumsq_out) sumsq_out[c] = (float)q;
        if (rmean) {
            rmean[c] = (float)((1.0 - (double)momentum) * (double)rm + (double)momentum * mu);
            rvar[c] = (float)((1.0 - (double)momentum) * (double)rv + (double)momentum * var * M / (M - 1.0));
        }
    }
}

// Combine partials [nparts][2][C] and derive the per-channel quantities.  One warp per channel, 8 channels per block.
// Outputs (any may be NULL): mean, invstd, scale = gamma*invstd, shift = beta - mean*scale, raw sums,
// running statistics (in place; unbiased variance, momentum).
__global__ void __launch_bounds__(256) bn_finalize_kernel(const float* __restrict__ partials, int nparts, int C, double M, float eps,
                                                          float momentum, const float* __restrict__ gamma, const float* __restrict__ beta,
                                                          float* mean, float* invstd, float* scale, float* shift, float* rmean, float* rvar,
                                                          float* sum_out, float* sumsq_out) {
    pdl_launch_dependents();
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const int c = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (c >= C) return;
    bn_finalize_channel<false>(partials, nparts, C, c, lane, M, eps, momentum, gamma, beta, mean, invstd, scale, shift, rmean, rvar, sum_out, sumsq_out);
}

// V consecutive per-channel floats (V = 4 or 8) with 16-byte loads.
template <int V> __device__ __forceinline__ void load_params(const float* __restrict__ p, int cg, float (&out)[V]) {
    const float4* q = reinterpret_cast<const float4*>(p + (size_t)cg * V);
#pragma unroll
    for (int i = 0; i < V / 4; ++i) {
        const float4 t = q[i];
        out[4 * i] = t.x;
        out[4 * i + 1] = t.y;
        out[4 * i + 2] = t.z;
        out[4 * i + 3] = t.w;
    }
}

template <int V> __device__ __forceinline__ void load_params(const float* __restrict__ p, int cg, float2 (&out)[V / 2]) {  // as pairs
    const float4* q = reinterpret_cast<const float4*>(p + (size_t)cg * V);
#pragma unroll
    for (int i = 0; i < V / 4; ++i) {
        const float4 t = q[i];
        out[2 * i] = make_float2(t.x, t.y);
        out[2 * i + 1] = make_float2(t.z, t.w);
    }
}

// ------------------------------------------------------------------ per-channel sums kept in fp64 accumulators
// The kernel that produces per-channel sums (the convolution's epilogue, the backward reduce pass) adds every block's
// fp32 partial sums to `acc` with fp64 atomics, and every block of the kernel that consumes them (the normalise + SiLU
// pass, the dy pass) reads the totals and derives its coefficients itself.  No block waits for another one: the
// producer needs neither a grid-wide barrier nor a resident grid, and the only ordering is the kernel boundary.
// acc holds `copies` sets of [2][C] doubles (block b adds to set b mod copies, so the cache lines of one set are not
// the target of every block at once).  The sets are zero when the producer starts: the last block of the consumer to
// have read them (counted in *readers) zeroes them again.  Adding a few hundred fp32 values in fp64 is exact unless
// their magnitudes differ by more than 2^29, so the totals do not depend on the order in which the atomics land.
struct ChanAcc {
    double* acc;   // NULL: the consumer reads coefficients that a finalize kernel has written
    int* readers;
    int copies;
};
__device__ __forceinline__ void chan_acc_add(const ChanAcc& ca, int C, int which, int c, float v) {
    atomicAdd(ca.acc + ((size_t)((int)blockIdx.x % ca.copies) * 2 + which) * C + c, (double)v);
}
// totals of channels c and c + 1 (c even) of both sums; read from L2, where the atomics were performed, with the loads
// of four sets in flight at a time (the consuming pass starts with this latency)
__device__ __forceinline__ void chan_acc_total2(const ChanAcc& ca, int C, int c, double2& t0, double2& t1) {
    t0 = t1 = make_double2(0.0, 0.0);
    const size_t set = (size_t)2 * C;
    const double* base = ca.acc + c;
    int k = 0;
    for (; k + 4 <= ca.copies; k += 4) {
        double2 a[4], b[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            a[i] = __ldcg(reinterpret_cast<const double2*>(base + (k + i) * set));
            b[i] = __ldcg(reinterpret_cast<const double2*>(base + (k + i) * set + C));
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            t0.x += a[i].x; t0.y += a[i].y;
            t1.x += b[i].x; t1.y += b[i].y;
        }
    }
    for (; k < ca.copies; ++k) {
        const double2 a = __ldcg(reinterpret_cast<const double2*>(base + k * set)), b = __ldcg(reinterpret_cast<const double2*>(base + k * set + C));
        t0.x += a.x; t0.y += a.y;
        t1.x += b.x; t1.y += b.y;
    }
}
// One thread per block, after the block's reads of acc (and a block-level barrier): returns the number of blocks that
// had read before this one.  The value is needed only at the end of the kernel.  No fence: the block's reads have
// delivered their values (they were used before the barrier), and the zeroes are written only by the block that sees
// every other block's increment.
__device__ __forceinline__ int chan_acc_reader_arrive(const ChanAcc& ca) { return atomicAdd(ca.readers, 1); }
// All threads of the block, `last` block-uniform: the last reader leaves the sets and the counter zeroed.
__device__ __forceinline__ void chan_acc_reset_if(const ChanAcc& ca, int C, bool last) {
    if (!last) return;
    const int n = ca.copies * 2 * C;
    for (int i = threadIdx.x; i < n; i += blockDim.x) ca.acc[i] = 0.0;
    if (threadIdx.x == 0) *ca.readers = 0;
}

// 1/sqrt(v) for v well inside the fp32 range: the fp32 approximation refined by one Newton step in fp64 (relative error
// below 2^-44, i.e. exact once rounded to fp32 but for values within 2^-20 units in the last place of a rounding
// boundary).  The library's fp64 rsqrt is a chain three times as long, and every block of the consuming pass waits for it.
__device__ __forceinline__ double rsqrt_refined(double v) {
    const float vf = (float)v;
    if (!(vf > 1e-30f && vf < 1e30f)) return rsqrt(v);
    const double r = (double)rsqrtf(vf);
    const double e = fma(-(v * r), r, 1.0);
    return fma(0.5 * r, e, r);
}

// What a block of the normalise + SiLU pass needs to turn the totals (sum y, sum y^2) into scale and shift; block 0
// also writes the batch statistics and updates the running ones (the same fp64 chain as bn_finalize_channel).
struct FwdFin {
    double inv_m, unbias;  // 1/M and M/(M-1)
    float eps, momentum;
    const float *gamma, *beta;
    float *mean, *invstd, *rmean, *rvar;
};
__device__ __forceinline__ void fwd_coef_from_acc(const ChanAcc& ca, const FwdFin& f, int C, float* s_coef /*[2][C] shared*/) {
    const bool writer = blockIdx.x == 0;
    // two channels per thread and round (kept rolled: the fp64 chains must not crowd the registers of the streaming loop)
#pragma unroll 1
    for (int c = 2 * (int)threadIdx.x; c < C; c += 2 * (int)blockDim.x) {
        const float2 ga = *reinterpret_cast<const float2*>(f.gamma + c), be = *reinterpret_cast<const float2*>(f.beta + c);
        double2 s, q;
        chan_acc_total2(ca, C, c, s, q);
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const double mu = (j ? s.y : s.x) * f.inv_m;
            double var = (j ? q.y : q.x) * f.inv_m - mu * mu;
            if (var < 0.0) var = 0.0;
            const double is = rsqrt_refined(var + (double)f.eps);
            const double sc = (double)(j ? ga.y : ga.x) * is;
            s_coef[c + j] = (float)sc;
            s_coef[C + c + j] = (float)((double)(j ? be.y : be.x) - mu * sc);
            if (writer) {
                f.mean[c + j] = (float)mu;
                f.invstd[c + j] = (float)is;
                if (f.rmean) {
                    f.rmean[c + j] = (float)((1.0 - (double)f.momentum) * (double)f.rmean[c + j] + (double)f.momentum * mu);
                    f.rvar[c + j] = (float)((1.0 - (double)f.momentum) * (double)f.rvar[c + j] + (double)f.momentum * var * f.unbias);
                }
            }
        }
    }
}
template <int V> __device__ __forceinline__ void load_params_shared(const float* s, int cg, float2 (&out)[V / 2]) {
    const float4* q = reinterpret_cast<const float4*>(s + (size_t)cg * V);
#pragma unroll
    for (int i = 0; i < V / 4; ++i) {
        const float4 t = q[i];
        out[2 * i] = make_float2(t.x, t.y);
        out[2 * i + 1] = make_float2(t.z, t.w);
    }
}

// ------------------------------------------------------------------ a = SiLU(y*scale + shift)  (ACT = false: no SiLU)
// RES: a = SiLU(...) + res with res a (possibly pitched) tensor of the output's type -- the residual connection of a
// bottleneck performed by the block that feeds it; the sum is formed in fp32 and rounded once.
// FIN: scale and shift are derived here from the totals in `ca` (dynamic shared memory: 2*C floats); else they are read.
template <typename YT, typename AT, bool FAST, bool ACT = true, bool PITCHED = false, bool RES = false, bool FIN = false>
__global__ void __launch_bounds__(288, 3) bn_silu_apply_kernel(const YT* __restrict__ y, AT* __restrict__ a,
                                                             long long total_vecs, int C, const float* __restrict__ scale,
                                                             const float* __restrict__ shift, long long ld_a, const AT* __restrict__ res, long long ld_r,
                                                             ChanAcc ca, FwdFin fin) {
    pdl_launch_dependents();
    pdl_wait();
    constexpr int V = Vec16<YT>::N;
    static_assert(V == Vec16<AT>::N, "y and a must have the same element size");
    const int cg = threadIdx.x % (C / V);
    float2 sc[V / 2], sh[V / 2];
    extern __shared__ __align__(16) float s_coef[];
    __shared__ int s_last;
    int readers_before = 0;
    if (FIN) {
        fwd_coef_from_acc(ca, fin, C, s_coef);
        __syncthreads();
        if (threadIdx.x == 0) readers_before = chan_acc_reader_arrive(ca);
        load_params_shared<V>(s_coef, cg, sc);
        load_params_shared<V>(s_coef + C, cg, sh);
    } else {
        load_params<V>(scale, cg, sc);
        load_params<V>(shift, cg, sh);
    }
    const long long stride = (long long)gridDim.x * blockDim.x;
    // a may be a channel slice of a wider tensor: row pitch ld_a elements (the stride is a whole number of rows, so the
    // output offset advances by a constant)
    const int cgs = C / V;
    const long long v0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    long long oa = PITCHED ? (v0 / cgs) * ld_a + (long long)cg * V : v0 * V;  // (dense: the flat offset, no division)
    const long long oa_step = PITCHED ? (stride / cgs) * ld_a : stride * V;
    long long orr = RES ? (v0 / cgs) * ld_r + (long long)cg * V : 0;
    const long long or_step = RES ? (stride / cgs) * ld_r : 0;
    for (long long v = v0; v < total_vecs; v += stride, oa += oa_step, orr += or_step) {
        if (v + 2 * stride < total_vecs) asm volatile("prefetch.global.L2 [%0];" ::"l"(y + (v + 2 * stride) * V));  // see the reduce kernel
        const Vec16<YT> q = ld16(y + v * V);
        Vec16<AT> o, r;
        if (RES) r = ld16(res + orr);
#pragma unroll
        for (int j = 0; j < V / 2; ++j) {
            const float2 z = fma2(pair_to_f32(q.v + 2 * j), sc[j], sh[j]);
            float2 out = ACT ? mul2(z, sigmoid2<FAST>(z)) : z;
            if (RES) out = add2(out, pair_to_f32(r.v + 2 * j));
            pair_from_f32(o.v + 2 * j, out);
        }
        st16(a + oa, o);
    }
    if (FIN) {
        if (threadIdx.x == 0) s_last = readers_before == (int)gridDim.x - 1;
        __syncthreads();
        chan_acc_reset_if(ca, C, s_last != 0);
    }
}

// ------------------------------------------------------------------ evaluation-mode coefficients and BN folding
// scale_c = gamma_c / sqrt(rvar_c + eps), shift_c = beta_c - rmean_c*scale_c (fp64 arithmetic, like the training-mode
// finalize).  gamma NULL: scale 1; rmean NULL: no normalisation (shift = beta, or 0 when beta is NULL too).
__device__ __forceinline__ void bn_eval_coef(const float* gamma, const float* beta, const float* rmean, const float* rvar, float eps, int c, double& sc,
                                             double& sh) {
    sc = gamma ? (double)gamma[c] : 1.0;
    sh = beta ? (double)beta[c] : 0.0;
    if (rmean) {
        sc /= sqrt((double)rvar[c] + (double)eps);
        sh -= (double)rmean[c] * sc;
    }
}
__global__ void __launch_bounds__(256) bn_eval_coef_kernel(const float* __restrict__ gamma, const float* __restrict__ beta, const float* __restrict__ rmean,
                                                           const float* __restrict__ rvar, float eps, int C, float* __restrict__ scale,
                                                           float* __restrict__ shift) {
    pdl_launch_dependents();
    pdl_wait();
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= C) return;
    double sc, sh;
    bn_eval_coef(gamma, beta, rmean, rvar, eps, c, sc, sh);
    scale[c] = (float)sc;
    shift[c] = (float)sh;
}
// Folded filter w'[co][t] = scale_co * w[co][t] (rounded to WT once) and bias'[co] = shift_co; K = taps per output channel.
template <typename WT>
__global__ void __launch_bounds__(256) bn_fold_kernel(const WT* __restrict__ w, long long K, int C, const float* __restrict__ gamma,
                                                      const float* __restrict__ beta, const float* __restrict__ rmean, const float* __restrict__ rvar,
                                                      float eps, WT* __restrict__ w_folded, float* __restrict__ bias_folded) {
    pdl_launch_dependents();
    pdl_wait();
    const long long total = (long long)C * K;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const int co = (int)(i / K);
        double sc, sh;
        bn_eval_coef(gamma, beta, rmean, rvar, eps, co, sc, sh);
        w_folded[i] = from_f32<WT>((float)((double)to_f32(w[i]) * sc));
        if (i - (long long)co * K == 0) bias_folded[co] = (float)sh;
    }
}

// partials [nparts][2][C] (sum dz, sum dz*y) -> dbeta, dgamma (fp32) and four per-channel coefficients for the dy pass:
//   coef[0] = a = gamma*invstd, coef[1] = b = beta - mean*a                      (z = y*a + b)
//   coef[2] = p1 = a*invstd*dgamma/M, coef[3] = p0 = p1*mean - a*dbeta/M        (dy = a*dz - p1*y + p0)
// which is dy = a*(dz - dbeta/M - xhat*dgamma/M) with xhat = (y - mean)*invstd written out in terms of y.
template <bool L2>
__device__ __forceinline__ void bn_bwd_finalize_channel(const float* __restrict__ partials, int nparts, int C, int c, int lane, double M,
                                                        const float* __restrict__ mean, const float* __restrict__ invstd,
                                                        const float* __restrict__ gamma, const float* __restrict__ beta, float* dgamma, float* dbeta,
                                                        float* coef /*[4][C]*/) {
    const float mu_f = mean[c], is_f = invstd[c], ga = gamma[c], be = beta[c];  // requested before the partials are summed
    double s0, s1;
    warp_sum_partials2<L2>(partials, nparts, C, c, lane, s0, s1);
    if (lane == 0) {
        const double mu = (double)mu_f, is = (double)is_f;
        const double inv_m = 1.0 / M;
        const double dg = is * (s1 - mu * s0);
        const double a = (double)ga * is;
        const double p1 = a * is * dg * inv_m;
        dbeta[c] = (float)s0;
        dgamma[c] = (float)dg;
        coef[c] = (float)a;
        coef[C + c] = (float)((double)be - mu * a);
        coef[2 * C + c] = (float)p1;
        coef[3 * C + c] = (float)(p1 * mu - a * s0 * inv_m);
    }
}

// ------------------------------------------------------------------ backward reductions: sum dz, sum dz*y
// z = y*a + b with a = gamma*invstd, b = beta - mean*a (recomputed here from the saved statistics).  The second
// sum is taken against y itself; sum dz*xhat = invstd*(sum dz*y - mean*sum dz) is formed in fp64 by the finalize
// kernel, so this pass needs only two per-channel values per element.
// Extras of the reduce kernel: with acc.acc != NULL the block sums go to the fp64 accumulators (and `partials` is not
// written); w / wt: filter and its rearranged copy for the data-gradient GEMM (wt = NULL: nothing to rearrange), work
// that the blocks of this kernel carry along because the memory latency of a few filter tiles costs them nothing.
struct BwdFused {
    ChanAcc acc;
    const __nv_bfloat16* w;
    __nv_bfloat16* wt;
};
template <typename YT, typename AT, bool FAST, bool PITCHED = false>
__global__ void __launch_bounds__(288, 3) bn_silu_bwd_reduce_kernel(const AT* __restrict__ g, const YT* __restrict__ y,
                                                                  long long total_vecs, int C, const float* __restrict__ mean,
                                                                  const float* __restrict__ invstd, const float* __restrict__ gamma,
                                                                  const float* __restrict__ beta, float* __restrict__ partials, BwdFused fb,
                                                                  WtParams wtp, long long ld_g) {
    pdl_launch_dependents();
    pdl_wait();
    constexpr int V = Vec16<YT>::N;
    static_assert(V == Vec16<AT>::N, "g and y must have the same element size");
    extern __shared__ float red[];
    const int tid = threadIdx.x;
    const int cgs = C / V;
    const int cg = tid % cgs;
    // The first two filter tiles of this block (for the data-gradient GEMM's rearranged filter) are requested now with
    // cp.async and written back after the streaming loop, so their memory latency costs nothing.
    __shared__ __align__(16) WtTileBuf wtile[2];
    const int wt_tiles = fb.wt ? wt_num_tiles(wtp) : 0;
    if (wt_tiles > 0) {
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const int t = (int)blockIdx.x + k * (int)gridDim.x;
            if (t < wt_tiles) wt_tile_load_async(fb.w, wtp, wt_tile_decode(wtp, t), wtile[k]);
        }
    }
    float2 a[V / 2], b[V / 2], sb[V / 2], sy[V / 2];
    {
        float mu[V], is[V], ga[V], be[V];
        load_params<V>(mean, cg, mu);
        load_params<V>(invstd, cg, is);
        load_params<V>(gamma, cg, ga);
        load_params<V>(beta, cg, be);
#pragma unroll
        for (int j = 0; j < V / 2; ++j) {
            a[j] = make_float2(ga[2 * j] * is[2 * j], ga[2 * j + 1] * is[2 * j + 1]);
            b[j] = make_float2(fmaf(-mu[2 * j], a[j].x, be[2 * j]), fmaf(-mu[2 * j + 1], a[j].y, be[2 * j + 1]));
            sb[j] = sy[j] = splat2(0.f);
        }
    }
    const long long stride = (long long)gridDim.x * blockDim.x;
    // g may be a channel slice of a wider tensor (row pitch ld_g elements); the stride is a whole number of rows
    const long long v0 = (long long)blockIdx.x * blockDim.x + tid;
    long long og = PITCHED ? (v0 / cgs) * ld_g + (long long)cg * V : v0 * V;  // (dense: the flat offset)
    const long long og_step = PITCHED ? (stride / cgs) * ld_g : stride * V;
    for (long long v = v0; v < total_vecs; v += stride, og += og_step) {
        // ask L2 for the lines this thread reads two iterations from now: more DRAM requests in flight without holding
        // registers (measured on 157 MB tensors: 93 -> 79 us; no effect on tensors that already sit in L2)
        if (v + 2 * stride < total_vecs) {
            asm volatile("prefetch.global.L2 [%0];" ::"l"(y + (v + 2 * stride) * V));
            asm volatile("prefetch.global.L2 [%0];" ::"l"(g + og + 2 * og_step));
        }
        const Vec16<YT> qy = ld16(y + v * V);
        const Vec16<AT> qg = ld16(g + og);
#pragma unroll
        for (int j = 0; j < V / 2; ++j) {
            const float2 yv = pair_to_f32(qy.v + 2 * j);
            const float2 dz = silu_bwd_dz2<FAST>(fma2(yv, a[j], b[j]), pair_to_f32(qg.v + 2 * j));
            sb[j] = add2(sb[j], dz);
            sy[j] = fma2(dz, yv, sy[j]);
        }
    }
    const int R = blockDim.x / cgs;
    for (int pass = 0; pass < 2; ++pass) {
#pragma unroll
        for (int j = 0; j < V / 2; ++j) *reinterpret_cast<float2*>(&red[tid * V + 2 * j]) = pass ? sy[j] : sb[j];
        __syncthreads();
        for (int c = tid; c < C; c += blockDim.x) {
            const int gq = c / V, e = c % V;
            float acc = 0.f;
            for (int r = 0; r < R; ++r) acc += red[(r * cgs + gq) * V + e];
            // pass 0: sum dz, pass 1: sum dz*y
            if (fb.acc.acc) chan_acc_add(fb.acc, C, pass, c, acc);
            else partials[((size_t)blockIdx.x * 2 + pass) * C + c] = acc;
        }
        __syncthreads();
    }
    if (wt_tiles > 0) {
        wt_async_wait();
        __syncthreads();
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const int t = (int)blockIdx.x + k * (int)gridDim.x;
            if (t < wt_tiles) wt_tile_store(fb.wt, wtp, wt_tile_decode(wtp, t), wtile[k]);
        }
        if (wt_tiles > 2 * (int)gridDim.x) wt_transform_blocks(fb.w, fb.wt, wtp, (int)blockIdx.x, (int)gridDim.x, 2);  // rare: very large filters
    }
}

__global__ void __launch_bounds__(256) bn_bwd_finalize_kernel(const float* __restrict__ partials, int nparts, int C, double M,
                                                              const float* __restrict__ mean, const float* __restrict__ invstd,
                                                              const float* __restrict__ gamma, const float* __restrict__ beta,
                                                              float* dgamma, float* dbeta, float* coef /*[4][C]*/, int fin_blocks,
                                                              const __nv_bfloat16* __restrict__ w, __nv_bfloat16* __restrict__ wt, WtParams wtp) {
    pdl_launch_dependents();
    pdl_wait();
    // Blocks past the first `fin_blocks` rearrange the filter for the data-gradient GEMM that follows this call's dy pass
    // (independent work that fills the otherwise idle GPU while the short finalize chain runs).
    if ((int)blockIdx.x >= fin_blocks) {
        wt_transform_blocks(w, wt, wtp, (int)blockIdx.x - fin_blocks, (int)gridDim.x - fin_blocks);
        return;
    }
    const int lane = threadIdx.x & 31;
    const int c = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (c >= C) return;
    bn_bwd_finalize_channel<false>(partials, nparts, C, c, lane, M, mean, invstd, gamma, beta, dgamma, dbeta, coef);
}

// ------------------------------------------------------------------ dy = a*dz - p1*y + p0
// What a block of the dy pass needs to turn the totals (sum dz, sum dz*y) into its four coefficients; block 0 also
// writes dgamma and dbeta (the same fp64 chain as bn_bwd_finalize_channel).
struct BwdFin {
    double inv_m;
    const float *mean, *invstd, *gamma, *beta;
    float *dgamma, *dbeta;
};
__device__ __forceinline__ void bwd_coef_from_acc(const ChanAcc& ca, const BwdFin& f, int C, float* s_coef /*[4][C] shared*/) {
    const bool writer = blockIdx.x == 0;
#pragma unroll 1
    for (int c = 2 * (int)threadIdx.x; c < C; c += 2 * (int)blockDim.x) {  // two channels per thread and round, see fwd_coef_from_acc
        const float2 mu_f = *reinterpret_cast<const float2*>(f.mean + c), is_f = *reinterpret_cast<const float2*>(f.invstd + c);
        const float2 ga = *reinterpret_cast<const float2*>(f.gamma + c), be = *reinterpret_cast<const float2*>(f.beta + c);
        double2 t0, t1;
        chan_acc_total2(ca, C, c, t0, t1);
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const double mu = (double)(j ? mu_f.y : mu_f.x), is = (double)(j ? is_f.y : is_f.x);
            const double s0 = j ? t0.y : t0.x, s1 = j ? t1.y : t1.x;
            const double dg = is * (s1 - mu * s0);
            const double a = (double)(j ? ga.y : ga.x) * is;
            const double p1 = a * is * dg * f.inv_m;
            s_coef[c + j] = (float)a;
            s_coef[C + c + j] = (float)((double)(j ? be.y : be.x) - mu * a);
            s_coef[2 * C + c + j] = (float)p1;
            s_coef[3 * C + c + j] = (float)(p1 * mu - a * s0 * f.inv_m);
            if (writer) {
                f.dbeta[c + j] = (float)s0;
                f.dgamma[c + j] = (float)dg;
            }
        }
    }
}
// FIN: the coefficients are derived here from the totals in `ca` (dynamic shared memory: 4*C floats); else read from coef.
// GRES: the incoming gradient g is also the gradient of a residual connection's shortcut: the pass adds it to (or, with
// gres_add = 0, copies it into) `gres`, a tensor of g's shape with pixels ld_gres elements apart -- the backward
// counterpart of the RES form of the normalise + SiLU pass (fp32 sum, rounded once, like a separate accumulation pass).
template <typename YT, typename AT, bool FAST, bool PITCHED = false, bool FIN = false, bool GRES = false>
__global__ void __launch_bounds__(288, 3) bn_silu_bwd_dy_kernel(const AT* __restrict__ g, const YT* __restrict__ y,
                                                              AT* __restrict__ dy, long long total_vecs, int C,
                                                              const float* __restrict__ coef, long long ld_g, ChanAcc ca, BwdFin fin,
                                                              AT* __restrict__ gres, long long ld_gres, int gres_add) {
    pdl_launch_dependents();
    pdl_wait();
    constexpr int V = Vec16<YT>::N;
    const int cg = threadIdx.x % (C / V);
    float2 a[V / 2], b[V / 2], np1[V / 2], p0[V / 2];
    extern __shared__ __align__(16) float s_coef[];
    __shared__ int s_last;
    int readers_before = 0;
    if (FIN) {
        bwd_coef_from_acc(ca, fin, C, s_coef);
        __syncthreads();
        if (threadIdx.x == 0) readers_before = chan_acc_reader_arrive(ca);
        load_params_shared<V>(s_coef, cg, a);
        load_params_shared<V>(s_coef + C, cg, b);
        load_params_shared<V>(s_coef + 2 * C, cg, np1);
        load_params_shared<V>(s_coef + 3 * C, cg, p0);
    } else {
        load_params<V>(coef, cg, a);
        load_params<V>(coef + C, cg, b);
        load_params<V>(coef + 2 * C, cg, np1);
        load_params<V>(coef + 3 * C, cg, p0);
    }
#pragma unroll
    for (int j = 0; j < V / 2; ++j) np1[j] = make_float2(-np1[j].x, -np1[j].y);
    const long long stride = (long long)gridDim.x * blockDim.x;
    const int cgs = C / V;
    const long long v0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    long long og = PITCHED ? (v0 / cgs) * ld_g + (long long)cg * V : v0 * V;  // g may be a channel slice (row pitch ld_g), see the reduce kernel
    const long long og_step = PITCHED ? (stride / cgs) * ld_g : stride * V;
    long long ogr = GRES ? (v0 / cgs) * ld_gres + (long long)cg * V : 0;
    const long long ogr_step = GRES ? (stride / cgs) * ld_gres : 0;
    for (long long v = v0; v < total_vecs; v += stride, og += og_step, ogr += ogr_step) {
        if (v + 2 * stride < total_vecs) {  // L2 prefetch two iterations ahead (see the reduce kernel)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(y + (v + 2 * stride) * V));
            asm volatile("prefetch.global.L2 [%0];" ::"l"(g + og + 2 * og_step));
        }
        const Vec16<YT> qy = ld16(y + v * V);
        const Vec16<AT> qg = ld16(g + og);
        if (GRES) {
            Vec16<AT> r = qg;
            if (gres_add) {
                const Vec16<AT> old = ld16(gres + ogr);
#pragma unroll
                for (int j = 0; j < V / 2; ++j) pair_from_f32(r.v + 2 * j, add2(pair_to_f32(old.v + 2 * j), pair_to_f32(qg.v + 2 * j)));
            }
            st16(gres + ogr, r);
        }
        Vec16<AT> o;
#pragma unroll
        for (int j = 0; j < V / 2; ++j) {
            const float2 yv = pair_to_f32(qy.v + 2 * j);
            const float2 dz = silu_bwd_dz2<FAST>(fma2(yv, a[j], b[j]), pair_to_f32(qg.v + 2 * j));
            pair_from_f32(o.v + 2 * j, fma2(a[j], dz, fma2(np1[j], yv, p0[j])));
        }
        st16(dy + v * V, o);
    }
    if (FIN) {
        if (threadIdx.x == 0) s_last = readers_before == (int)gridDim.x - 1;
        __syncthreads();
        chan_acc_reset_if(ca, C, s_last != 0);
    }
}

}  // namespace nbcbs
