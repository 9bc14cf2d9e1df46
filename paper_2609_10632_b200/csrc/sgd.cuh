// Fused optimiser step: global-norm clipping over a list of gradient tensors, then SGD with Nesterov momentum
// (see include/nb_sgd.h for the arithmetic).  Two kernels for any number of tensors: the elements of all tensors are
// cut into chunks of SGD_CHUNK elements, chunk i belongs to block i % gridDim.x, and both kernels walk the same table.
#pragma once
#include "../../include/nb_sgd.h"
#include "common.cuh"

namespace nbcbs {

constexpr int SGD_CHUNK = 4096;    // elements per chunk (a multiple of 4: chunks start 16-byte aligned)
constexpr int SGD_THREADS = 256;
constexpr int SGD_VPT = SGD_CHUNK / 4 / SGD_THREADS;  // 16-byte vectors per thread and chunk
constexpr int SGD_MAX_BLOCKS = 2048;
constexpr uint32_t SGD_MAGIC = 0x6e627367u;

struct SgdChunk {
    int32_t tensor;
    int32_t len;     // elements of this chunk (<= SGD_CHUNK)
    int64_t start;   // first element inside the tensor
};
struct SgdHeader {  // first 256 bytes of the workspace
    uint32_t magic;
    int32_t count, nchunks, grid;
    uint64_t off_tensors, off_chunks, off_partials, total_bytes;
};

__device__ __forceinline__ double block_sum_fixed_order(double v, double* red /*[SGD_THREADS/32]*/) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) red[warp] = v;
    __syncthreads();
    double t = 0.0;
    if (threadIdx.x == 0)
        for (int w = 0; w < SGD_THREADS / 32; ++w) t += red[w];
    return t;  // valid in thread 0
}

// partials[b] = sum of g^2 over the chunks of block b (fp32 per thread over at most a few hundred elements, fp64 above).
__global__ void __launch_bounds__(SGD_THREADS) sgd_sqnorm_kernel(const uint8_t* __restrict__ ws) {
    pdl_launch_dependents();
    pdl_wait();
    const SgdHeader& H = *reinterpret_cast<const SgdHeader*>(ws);
    const nb_sgd_tensor* T = reinterpret_cast<const nb_sgd_tensor*>(ws + H.off_tensors);
    const SgdChunk* C = reinterpret_cast<const SgdChunk*>(ws + H.off_chunks);
    double* partials = reinterpret_cast<double*>(const_cast<uint8_t*>(ws) + H.off_partials);
    __shared__ double red[SGD_THREADS / 32];
    double acc = 0.0;
    for (int c = blockIdx.x; c < H.nchunks; c += gridDim.x) {
        const SgdChunk ch = C[c];
        const float* g = T[ch.tensor].grad + ch.start;
        const int n4 = ch.len >> 2;
        float s = 0.f;
        // a chunk is at most SGD_VPT vectors per thread: all of them are requested before the first is used
        float4 v[SGD_VPT];
#pragma unroll
        for (int k = 0; k < SGD_VPT; ++k) {
            const int i = threadIdx.x + k * SGD_THREADS;
            v[k] = i < n4 ? reinterpret_cast<const float4*>(g)[i] : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int k = 0; k < SGD_VPT; ++k) {
            s = fmaf(v[k].x, v[k].x, s); s = fmaf(v[k].y, v[k].y, s); s = fmaf(v[k].z, v[k].z, s); s = fmaf(v[k].w, v[k].w, s);
        }
        for (int i = (n4 << 2) + threadIdx.x; i < ch.len; i += SGD_THREADS) s = fmaf(g[i], g[i], s);
        acc += (double)s;
    }
    const double t = block_sum_fixed_order(acc, red);
    if (threadIdx.x == 0) partials[blockIdx.x] = t;
}

struct SgdScalars {
    float momentum, max_norm;
    float lr[NB_SGD_GROUPS], wd[NB_SGD_GROUPS];
    int first_step;
    // dynamic loss scaling (scaler == NULL: gradients are unscaled): the gradients arrive multiplied by scaler->scale
    const nb_loss_scaler* scaler;
};

__device__ __forceinline__ void sgd_one(float g, float& p, float& b, float coef, float lr, float wd, float mom, bool first) {
    const float d = fmaf(wd, p, g * coef);
    b = first ? d : fmaf(mom, b, d);
    p = fmaf(-lr, fmaf(mom, b, d), p);
}

__global__ void __launch_bounds__(SGD_THREADS) sgd_update_kernel(const uint8_t* __restrict__ ws, SgdScalars hs, float* __restrict__ total_norm_out) {
    pdl_launch_dependents();
    pdl_wait();
    const SgdHeader& H = *reinterpret_cast<const SgdHeader*>(ws);
    const nb_sgd_tensor* T = reinterpret_cast<const nb_sgd_tensor*>(ws + H.off_tensors);
    const SgdChunk* C = reinterpret_cast<const SgdChunk*>(ws + H.off_chunks);
    const double* partials = reinterpret_cast<const double*>(ws + H.off_partials);
    // every block forms the clip coefficient itself from the norm kernel's partial sums, in one fixed order
    __shared__ double red[SGD_THREADS / 32];
    __shared__ float s_coef;
    double acc = 0.0;
    for (int i = threadIdx.x; i < H.grid; i += SGD_THREADS) acc += partials[i];
    const double t = block_sum_fixed_order(acc, red);
    __shared__ int s_skip;
    if (threadIdx.x == 0) {
        // the state is read here and rewritten only by the scaler kernel that runs after this one
        const double inv = hs.scaler ? 1.0 / (double)hs.scaler->scale : 1.0;
        const double total = sqrt(t) * inv;  // norm of the unscaled gradients; inf or NaN if any gradient element is
        double c = 1.0;
        if (hs.max_norm > 0.f && hs.max_norm < __int_as_float(0x7f800000)) c = fmin((double)hs.max_norm / (total + 1e-6), 1.0);
        s_coef = (float)(c * inv);
        s_skip = (hs.scaler && !isfinite(t)) ? 1 : 0;
        if (blockIdx.x == 0 && total_norm_out) *total_norm_out = (float)total;
    }
    __syncthreads();
    if (s_skip) return;  // overflow under loss scaling: parameters and momentum stay as they are
    const float coef = s_coef, mom = hs.momentum;
    const bool first = hs.first_step != 0;
    for (int c = blockIdx.x; c < H.nchunks; c += gridDim.x) {
        const SgdChunk ch = C[c];
        const nb_sgd_tensor t_ = T[ch.tensor];
        const int grp = t_.group;  // selects, not indexing: the scalars stay in the parameter bank
        const float lr = grp == 0 ? hs.lr[0] : grp == 1 ? hs.lr[1] : hs.lr[2];
        const float wd = grp == 0 ? hs.wd[0] : grp == 1 ? hs.wd[1] : hs.wd[2];
        const float* g = t_.grad + ch.start;
        float* p = t_.param + ch.start;
        float* b = t_.momentum + ch.start;
        __nv_bfloat16* lp = t_.param_bf16 ? static_cast<__nv_bfloat16*>(t_.param_bf16) + ch.start : nullptr;  // (or __half: same size)
        const bool lp_f16 = t_.copy_dtype == NB_DTYPE_F16;
        const int n4 = ch.len >> 2;
        // all loads of the chunk first (up to 3 x SGD_VPT vectors in flight per thread), then the arithmetic and the stores
        float4 gv[SGD_VPT], pv[SGD_VPT], bv[SGD_VPT];
        const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int k = 0; k < SGD_VPT; ++k) {
            const int i = threadIdx.x + k * SGD_THREADS;
            const bool in = i < n4;
            gv[k] = in ? reinterpret_cast<const float4*>(g)[i] : zero4;
            pv[k] = in ? reinterpret_cast<const float4*>(p)[i] : zero4;
            bv[k] = (in && !first) ? reinterpret_cast<const float4*>(b)[i] : zero4;
        }
#pragma unroll
        for (int k = 0; k < SGD_VPT; ++k) {
            const int i = threadIdx.x + k * SGD_THREADS;
            if (i >= n4) break;
            sgd_one(gv[k].x, pv[k].x, bv[k].x, coef, lr, wd, mom, first);
            sgd_one(gv[k].y, pv[k].y, bv[k].y, coef, lr, wd, mom, first);
            sgd_one(gv[k].z, pv[k].z, bv[k].z, coef, lr, wd, mom, first);
            sgd_one(gv[k].w, pv[k].w, bv[k].w, coef, lr, wd, mom, first);
            reinterpret_cast<float4*>(p)[i] = pv[k];
            reinterpret_cast<float4*>(b)[i] = bv[k];
            if (lp) {
                uint2 o;
                if (lp_f16) {
                    const __half a0 = from_f32<__half>(pv[k].x), a1 = from_f32<__half>(pv[k].y), a2 = from_f32<__half>(pv[k].z), a3 = from_f32<__half>(pv[k].w);
                    o.x = (uint32_t)__half_as_ushort(a0) | ((uint32_t)__half_as_ushort(a1) << 16);
                    o.y = (uint32_t)__half_as_ushort(a2) | ((uint32_t)__half_as_ushort(a3) << 16);
                } else {
                    const __nv_bfloat162 lo = __floats2bfloat162_rn(pv[k].x, pv[k].y), hi = __floats2bfloat162_rn(pv[k].z, pv[k].w);
                    o.x = *reinterpret_cast<const uint32_t*>(&lo);
                    o.y = *reinterpret_cast<const uint32_t*>(&hi);
                }
                reinterpret_cast<uint2*>(lp)[i] = o;
            }
        }
        for (int i = (n4 << 2) + threadIdx.x; i < ch.len; i += SGD_THREADS) {
            float pv = p[i], bv = first ? 0.f : b[i];
            sgd_one(g[i], pv, bv, coef, lr, wd, mom, first);
            p[i] = pv;
            b[i] = bv;
            if (lp) {
                if (lp_f16) reinterpret_cast<__half*>(lp)[i] = from_f32<__half>(pv);
                else lp[i] = __float2bfloat16_rn(pv);
            }
        }
    }
}

// After the update kernel: the scaler's state for the next step (one thread).  found_inf is recomputed from the same
// partial sums in the same order.
__global__ void sgd_scaler_kernel(const uint8_t* __restrict__ ws, nb_loss_scaler* state, float growth_factor, float backoff_factor, float floor_scale,
                                  int growth_interval) {
    pdl_launch_dependents();
    pdl_wait();
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    const SgdHeader& H = *reinterpret_cast<const SgdHeader*>(ws);
    const double* partials = reinterpret_cast<const double*>(ws + H.off_partials);
    double t = 0.0;
    for (int i = 0; i < H.grid; ++i) t += partials[i];
    if (!isfinite(t)) {
        state->scale = fmaxf(state->scale * backoff_factor, floor_scale);
        state->growth_tracker = 0;
        state->skipped = 1;
    } else {
        state->skipped = 0;
        if (++state->growth_tracker >= growth_interval) {
            state->scale *= growth_factor;
            state->growth_tracker = 0;
        }
    }
}

}  // namespace nbcbs
