// Kernels for the network's first layer: 3 input channels, 3x3, stride 2, pad 1.
// A 3-channel bf16 pixel is 6 bytes, which no TMA descriptor can address (strides must be multiples of 16 bytes), and
// K = 27 is far too short for the tcgen05 pipeline: the forward and the weight gradient run on warp-level mma.sync tiles of
// 16 pixels, the data gradient (3 output channels) on register-tiled CUDA-core FMAs.  COUT is a template parameter
// (48 for the detector's stem).
#pragma once
#include "common.cuh"

namespace nbcbs {

constexpr int STEM_CIN = 3, STEM_K = 3, STEM_TAPS = 9, STEM_KDIM = 27;

// ---- tensor-core forward for the stem.  K = 27 is far too short for the tcgen05 pipeline (and a 6-byte pixel cannot be
// fetched by TMA), so this kernel uses warp-level mma.sync (m16n8k16, bf16 -> fp32): a warp computes 16 consecutive output
// pixels x COUT channels with K padded to 32.  The filter fragments stay in registers for the whole kernel; a thread
// gathers the 2 x 8 input values of its fragment rows with 2-byte loads (the 3 x 3 x 3 patch of a pixel is three runs of 9
// contiguous values, L1-resident across neighbouring pixels) and writes its accumulator pairs as fp16.
template <typename T> __device__ __forceinline__ void mma_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1);
template <> __device__ __forceinline__ void mma_16816<__nv_bfloat16>(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
template <> __device__ __forceinline__ void mma_16816<__half>(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// Per-channel epilogue of the evaluation-mode / plain forward: out = act(acc*scale_c + shift_c), coefficients as bn_eval_coef.
struct StemEpi {
    const float *gamma, *beta, *rmean, *rvar;
    float eps;
    int act;
};
// EPI = false: y = the convolution output in fp16 (training forward).  EPI = true: OutT = bf16 activations, see StemEpi.
// InT = the 16-bit type of x and w (bf16, or IEEE fp16).
template <int COUT, typename OutT = __half, bool EPI = false, typename InT = __nv_bfloat16>
__global__ void __launch_bounds__(128) stem_fprop_mma_kernel(const InT* __restrict__ x, const InT* __restrict__ w,
                                                             OutT* __restrict__ y, Geom g, StemEpi ep) {
    pdl_launch_dependents();
    pdl_wait();
    static_assert(COUT % 8 == 0, "whole n-blocks");
    constexpr int NB = COUT / 8;
    const int lane = threadIdx.x & 31, gq = lane >> 2, tq = lane & 3;
    const unsigned short* xs = reinterpret_cast<const unsigned short*>(x);
    const unsigned short* wsrc = reinterpret_cast<const unsigned short*>(w);
    // the eight K indices of this lane's A / B fragment elements: k-step s, register half j, element e
    int koff[8];   // element offset of K index k inside the input relative to the patch origin, or -1 for the padding (k >= 27)
    int kr[8], kt[8];  // filter row and column of k (bounds checks)
    uint32_t bfrag[2][NB][2];
#pragma unroll
    for (int s2 = 0; s2 < 2; ++s2)
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int k = s2 * 16 + j * 8 + tq * 2 + e, i = s2 * 4 + j * 2 + e;
                const int r = k / 9, kp = k - r * 9;
                kr[i] = r;
                kt[i] = kp / 3;
                koff[i] = k < STEM_KDIM ? r * g.w * 3 + kp : -1;
            }
#pragma unroll
    for (int s2 = 0; s2 < 2; ++s2)
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int k = s2 * 16 + j * 8 + tq * 2, n = nb * 8 + gq;
                const uint32_t lo = k < STEM_KDIM ? wsrc[n * STEM_KDIM + k] : 0u, hi = k + 1 < STEM_KDIM ? wsrc[n * STEM_KDIM + k + 1] : 0u;
                bfrag[s2][nb][j] = lo | (hi << 16);
            }
    // this lane's accumulator columns are nb*8 + 2*tq and the next one: their (scale, shift) pairs stay in registers
    float esc[EPI ? NB : 1][2], esh[EPI ? NB : 1][2];
    if (EPI) {
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                double sc, sh;
                bn_eval_coef(ep.gamma, ep.beta, ep.rmean, ep.rvar, ep.eps, nb * 8 + tq * 2 + e, sc, sh);
                esc[nb][e] = (float)sc;
                esh[nb][e] = (float)sh;
            }
    }
    __shared__ __align__(16) OutT stage[4][16 * COUT];
    const long long ntiles = (g.m + 15) / 16;
    const long long wstride = (long long)gridDim.x * (blockDim.x >> 5);
    for (long long tile = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); tile < ntiles; tile += wstride) {
        const long long m0 = tile * 16;
        uint32_t a[2][4];
#pragma unroll
        for (int half = 0; half < 2; ++half) {  // fragment rows gq and gq + 8
            const long long m = m0 + gq + half * 8;
            const bool row_ok = m < g.m;
            const unsigned mm = row_ok ? (unsigned)m : 0u;  // the stem has fewer than 2^31 output pixels: 32-bit divisions
            const unsigned t1 = mm / (unsigned)g.wo;
            const int q = (int)(mm - t1 * (unsigned)g.wo);
            const int n = (int)(t1 / (unsigned)g.ho), p = (int)(t1 - (unsigned)n * (unsigned)g.ho);
            const int h0 = 2 * p - 1, w0 = 2 * q - 1;
            const long long origin = (((long long)n * g.h + h0) * g.w + w0) * 3;  // may point before the image; only used when in bounds
            unsigned short v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int h = h0 + kr[i], ww = w0 + kt[i];
                const bool ok = row_ok && koff[i] >= 0 && h >= 0 && h < g.h && ww >= 0 && ww < g.w;
                v[i] = ok ? xs[origin + koff[i]] : (unsigned short)0;
            }
            // registers of m16n8k16 A: a0 = (row g, k 2t..2t+1), a1 = (row g+8, same k), a2 = (row g, k 2t+8..), a3 = (row g+8, k 2t+8..)
            a[0][half] = (uint32_t)v[0] | ((uint32_t)v[1] << 16);
            a[0][2 + half] = (uint32_t)v[2] | ((uint32_t)v[3] << 16);
            a[1][half] = (uint32_t)v[4] | ((uint32_t)v[5] << 16);
            a[1][2 + half] = (uint32_t)v[6] | ((uint32_t)v[7] << 16);
        }
        float acc[NB][4];
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
            acc[nb][0] = acc[nb][1] = acc[nb][2] = acc[nb][3] = 0.f;
            mma_16816<InT>(acc[nb], a[0], bfrag[0][nb][0], bfrag[0][nb][1]);
            mma_16816<InT>(acc[nb], a[1], bfrag[1][nb][0], bfrag[1][nb][1]);
        }
        // accumulator registers: c0, c1 = (row g, columns 2t, 2t+1), c2, c3 = (row g+8, same columns).  The 16 x COUT tile is one
        // contiguous run of the output, so it is staged in shared memory and written with coalesced 16-byte stores.
        OutT* st = stage[threadIdx.x >> 5];
#pragma unroll
        for (int half = 0; half < 2; ++half)
#pragma unroll
            for (int nb = 0; nb < NB; ++nb) {
                float v0 = acc[nb][2 * half], v1 = acc[nb][2 * half + 1];
                if (EPI) {
                    v0 = fmaf(v0, esc[nb][0], esh[nb][0]);
                    v1 = fmaf(v1, esc[nb][1], esh[nb][1]);
                    if (ep.act) {
                        v0 *= sigmoid_f<true>(v0);
                        v1 *= sigmoid_f<true>(v1);
                    }
                }
                OutT* dst = st + (gq + half * 8) * COUT + nb * 8 + tq * 2;
                dst[0] = from_f32<OutT>(v0);
                dst[1] = from_f32<OutT>(v1);
            }
        __syncwarp();
        const long long rows_left = g.m - m0;
        const int nvec = (int)(rows_left >= 16 ? 16 : rows_left) * COUT / 8;  // 16-byte pieces of the tile that exist
        for (int v = lane; v < nvec; v += 32) st16(y + (size_t)m0 * COUT + v * 8, ld16(st + v * 8));
        __syncwarp();
    }
}

// Data gradient, register-tiled: a thread produces the 2 x 4 input pixels (rows 2i, 2i+1, columns 4jp .. 4jp+3) that the
// six dy pixels (rows i, i+1, columns 2jp .. 2jp+2) feed, so one broadcast read of a channel's 27 filter values serves
// 54 FMAs (a one-pair-per-thread version read three float4 per nine FMAs and was bound by shared-memory reads: 246 us
// against 175 us on the 16 x 640 x 640 stem).
// With pixel (2i+a, 2j+b): (0,0) <- dy[i][j] w11;  (0,1) <- dy[i][j+1] w10 + dy[i][j] w12;  (1,0) <- dy[i+1][j] w01 + dy[i][j] w21;
// (1,1) <- dy[i+1][j+1] w00 + dy[i+1][j] w02 + dy[i][j+1] w20 + dy[i][j] w22   (w_rt = filter tap (r,t); H and W even).
template <typename T> __device__ __forceinline__ uint32_t stem_pack2(float a, float b) {
    const T lo = from_f32<T>(a), hi = from_f32<T>(b);
    return (uint32_t)(*reinterpret_cast<const unsigned short*>(&lo)) | ((uint32_t)(*reinterpret_cast<const unsigned short*>(&hi)) << 16);
}
template <int COUT, typename T = __nv_bfloat16>
__global__ void __launch_bounds__(128) stem_dgrad_tiled_kernel(const T* __restrict__ dy, const T* __restrict__ w, T* __restrict__ dx, Geom g) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ __align__(16) float ws[COUT][28];  // ws[c'][tap*3 + c]
    for (int e = threadIdx.x; e < COUT * STEM_KDIM; e += blockDim.x) ws[e / STEM_KDIM][e % STEM_KDIM] = to_f32(w[e]);
    __syncthreads();
    const int npair = (g.wo + 1) / 2;
    const long long total = (long long)g.n * g.ho * npair;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += stride) {
        const int jp = (int)(idx % npair);
        const long long t1 = idx / npair;
        const int i = (int)(t1 % g.ho), n = (int)(t1 / g.ho);
        const int j = 2 * jp;
        const bool row1 = i + 1 < g.ho, col1 = j + 1 < g.wo, col2 = j + 2 < g.wo;
        const T* r0 = dy + (((size_t)n * g.ho + i) * g.wo + j) * COUT;
        const T* r1 = r0 + (size_t)g.wo * COUT;
        float acc[2][4][3];  // [row a][column 0..3 of the 4 produced][channel]
#pragma unroll
        for (int a = 0; a < 2; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) acc[a][b][0] = acc[a][b][1] = acc[a][b][2] = 0.f;
        Vec16<T> zero;
#pragma unroll
        for (int e = 0; e < 8; ++e) zero.v[e] = from_f32<T>(0.f);
#pragma unroll 1
        for (int c0 = 0; c0 < COUT; c0 += 8) {
            const Vec16<T> v00 = ld16(r0 + c0);
            const Vec16<T> v01 = col1 ? ld16(r0 + COUT + c0) : zero;
            const Vec16<T> v02 = col2 ? ld16(r0 + 2 * COUT + c0) : zero;
            const Vec16<T> v10 = row1 ? ld16(r1 + c0) : zero;
            const Vec16<T> v11 = (row1 && col1) ? ld16(r1 + COUT + c0) : zero;
            const Vec16<T> v12 = (row1 && col2) ? ld16(r1 + 2 * COUT + c0) : zero;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float d00 = to_f32(v00.v[e]), d01 = to_f32(v01.v[e]), d02 = to_f32(v02.v[e]);
                const float d10 = to_f32(v10.v[e]), d11 = to_f32(v11.v[e]), d12 = to_f32(v12.v[e]);
                float wv[28];
#pragma unroll
                for (int q = 0; q < 7; ++q) *reinterpret_cast<float4*>(wv + 4 * q) = *reinterpret_cast<const float4*>(&ws[c0 + e][4 * q]);
#pragma unroll
                for (int c = 0; c < 3; ++c) {
                    const float w00 = wv[0 + c], w01 = wv[3 + c], w02 = wv[6 + c], w10 = wv[9 + c], w11 = wv[12 + c], w12 = wv[15 + c];
                    const float w20 = wv[18 + c], w21 = wv[21 + c], w22 = wv[24 + c];
                    // first 2 x 2 group (dy column j), second (dy column j+1)
                    acc[0][0][c] = fmaf(d00, w11, acc[0][0][c]);
                    acc[0][1][c] = fmaf(d01, w10, fmaf(d00, w12, acc[0][1][c]));
                    acc[1][0][c] = fmaf(d10, w01, fmaf(d00, w21, acc[1][0][c]));
                    acc[1][1][c] = fmaf(d11, w00, fmaf(d10, w02, fmaf(d01, w20, fmaf(d00, w22, acc[1][1][c]))));
                    acc[0][2][c] = fmaf(d01, w11, acc[0][2][c]);
                    acc[0][3][c] = fmaf(d02, w10, fmaf(d01, w12, acc[0][3][c]));
                    acc[1][2][c] = fmaf(d11, w01, fmaf(d01, w21, acc[1][2][c]));
                    acc[1][3][c] = fmaf(d12, w00, fmaf(d11, w02, fmaf(d02, w20, fmaf(d01, w22, acc[1][3][c]))));
                }
            }
        }
        // rows 2i and 2i+1, columns 4jp .. 4jp+3 (the last two only when dy column j+1 exists): 12 bf16 = 24 bytes per row, 8-byte aligned
#pragma unroll
        for (int a = 0; a < 2; ++a) {
            T* o = dx + (((size_t)n * g.h + 2 * i + a) * g.w + 4 * (size_t)jp) * 3;
            uint32_t* o2 = reinterpret_cast<uint32_t*>(o);
            o2[0] = stem_pack2<T>(acc[a][0][0], acc[a][0][1]);
            o2[1] = stem_pack2<T>(acc[a][0][2], acc[a][1][0]);
            o2[2] = stem_pack2<T>(acc[a][1][1], acc[a][1][2]);
            if (col1) {
                o2[3] = stem_pack2<T>(acc[a][2][0], acc[a][2][1]);
                o2[4] = stem_pack2<T>(acc[a][2][2], acc[a][3][0]);
                o2[5] = stem_pack2<T>(acc[a][3][1], acc[a][3][2]);
            }
        }
    }
}

// ---- tensor-core weight gradient for the stem: dw[c'][k] = sum over pixels of dy[pixel][c'] * patch[pixel][k] as
// mma.sync tiles of 16 pixels (the reduction index): A = dy^T (the 16 x COUT piece of dy is one contiguous run: staged in
// shared memory with 16-byte loads and read back transposed with ldmatrix), B = the pixels' patch values (gathered like
// in the forward kernel).  A block sums its pixel range; its four warps are combined in a fixed order into the block's
// slice of `partial` [gridDim.x][COUT][27].
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* smem_row) {
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(smem_row);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
template <int COUT, typename T = __nv_bfloat16>
__global__ void __launch_bounds__(128) stem_wgrad_mma_kernel(const T* __restrict__ x, const T* __restrict__ dy,
                                                             float* __restrict__ partial, Geom g, long long pix_per_block) {
    pdl_launch_dependents();
    pdl_wait();
    static_assert(COUT % 16 == 0, "whole m-blocks");
    constexpr int MB = COUT / 16, NBK = 4;  // accumulator blocks: MB x 16 channels by NBK x 8 filter positions (27 padded to 32)
    __shared__ __align__(16) T dys[4][16 * COUT];
    __shared__ float red[4][COUT][33];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gq = lane >> 2, tq = lane & 3;
    const unsigned short* xs = reinterpret_cast<const unsigned short*>(x);
    // B fragment element (k = pixel 2t.., n = 8*nb + g): filter position n of the pixel's patch
    int koff[NBK], kr[NBK], kt[NBK];
#pragma unroll
    for (int nb = 0; nb < NBK; ++nb) {
        const int k = nb * 8 + gq, r = k / 9, kp = k - r * 9;
        kr[nb] = r;
        kt[nb] = kp / 3;
        koff[nb] = k < STEM_KDIM ? r * g.w * 3 + kp : -1;
    }
    float acc[MB][NBK][4];
#pragma unroll
    for (int a = 0; a < MB; ++a)
#pragma unroll
        for (int b = 0; b < NBK; ++b) acc[a][b][0] = acc[a][b][1] = acc[a][b][2] = acc[a][b][3] = 0.f;
    const long long m_begin = (long long)blockIdx.x * pix_per_block;
    const long long m_end = (m_begin + pix_per_block < g.m) ? m_begin + pix_per_block : g.m;
    T* st = dys[warp];
    for (long long m0 = m_begin + warp * 16; m0 < m_end; m0 += 64) {
        const int np = (int)((m_end - m0 < 16) ? (m_end - m0) : 16);  // pixels of this tile inside the block's range
        // stage dy[m0 .. m0+15][:] (zeros past the range)
        for (int v = lane; v < 16 * COUT / 8; v += 32) {
            Vec16<T> q;
            if (v * 8 < np * COUT) {
                q = ld16(dy + (size_t)m0 * COUT + v * 8);
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) q.v[i] = from_f32<T>(0.f);
            }
            st16(st + v * 8, q);
        }
        // B fragments: four pixels of the tile (2t, 2t+1, 2t+8, 2t+9) x NBK filter positions
        uint32_t bfr[NBK][2];
        unsigned short v4[4][NBK];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int pl = tq * 2 + (j & 1) + (j >> 1) * 8;
            const bool row_ok = pl < np;
            const unsigned mm = row_ok ? (unsigned)(m0 + pl) : 0u;
            const unsigned t1 = mm / (unsigned)g.wo;
            const int q = (int)(mm - t1 * (unsigned)g.wo);
            const int n = (int)(t1 / (unsigned)g.ho), p = (int)(t1 - (unsigned)n * (unsigned)g.ho);
            const int h0 = 2 * p - 1, w0 = 2 * q - 1;
            const long long origin = (((long long)n * g.h + h0) * g.w + w0) * 3;
#pragma unroll
            for (int nb = 0; nb < NBK; ++nb) {
                const int h = h0 + kr[nb], ww = w0 + kt[nb];
                const bool ok = row_ok && koff[nb] >= 0 && h >= 0 && h < g.h && ww >= 0 && ww < g.w;
                v4[j][nb] = ok ? xs[origin + koff[nb]] : (unsigned short)0;
            }
        }
#pragma unroll
        for (int nb = 0; nb < NBK; ++nb) {
            bfr[nb][0] = (uint32_t)v4[0][nb] | ((uint32_t)v4[1][nb] << 16);
            bfr[nb][1] = (uint32_t)v4[2][nb] | ((uint32_t)v4[3][nb] << 16);
        }
        __syncwarp();  // the staged dy rows are complete
#pragma unroll
        for (int mb = 0; mb < MB; ++mb) {
            // A = dy^T: matrix i of the x4 load is [8 pixels][8 channels] of the staged tile, read transposed:
            // i = 0: pixels 0-7, channels 16mb+0..7 (a0), 1: pixels 0-7, channels +8 (a1), 2: pixels 8-15, channels +0 (a2), 3: pixels 8-15, +8 (a3)
            uint32_t afr[4];
            const int mi = lane >> 3, mr = lane & 7;
            ldmatrix_x4_trans(afr, st + (mr + (mi >> 1) * 8) * COUT + mb * 16 + (mi & 1) * 8);
#pragma unroll
            for (int nb = 0; nb < NBK; ++nb) mma_16816<T>(acc[mb][nb], afr, bfr[nb][0], bfr[nb][1]);
        }
        __syncwarp();  // before the next tile overwrites the staged rows
    }
    // accumulator registers: c0, c1 = (channel 16mb+g, positions 8nb+2t, +1), c2, c3 = (channel 16mb+g+8, same positions)
#pragma unroll
    for (int mb = 0; mb < MB; ++mb)
#pragma unroll
        for (int nb = 0; nb < NBK; ++nb) {
            red[warp][mb * 16 + gq][nb * 8 + tq * 2] = acc[mb][nb][0];
            red[warp][mb * 16 + gq][nb * 8 + tq * 2 + 1] = acc[mb][nb][1];
            red[warp][mb * 16 + gq + 8][nb * 8 + tq * 2] = acc[mb][nb][2];
            red[warp][mb * 16 + gq + 8][nb * 8 + tq * 2 + 1] = acc[mb][nb][3];
        }
    __syncthreads();
    float* o = partial + (size_t)blockIdx.x * COUT * STEM_KDIM;
    for (int e = threadIdx.x; e < COUT * STEM_KDIM; e += blockDim.x) {
        const int c = e / STEM_KDIM, k = e - c * STEM_KDIM;
        o[e] = ((red[0][c][k] + red[1][c][k]) + red[2][c][k]) + red[3][c][k];
    }
}

}  // namespace nbcbs
