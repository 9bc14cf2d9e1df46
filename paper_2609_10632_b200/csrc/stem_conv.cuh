// Kernels for the network's first layer: 3 input channels, 3x3, stride 2, pad 1, even H and W.
// A 3-channel 16-bit pixel is 6 bytes, which no TMA descriptor can address (strides must be multiples of 16 bytes), and
// K = 27 is far too short for the tcgen05 pipeline, so all three convolutions run on warp-level mma.sync tiles
// (m16n8k16, fp32 accumulation).  All three are HBM-bound by design (157 MB of y / dy against 39 MB of x / dx at batch
// 16, 640 x 640): every global access is a coalesced 16-byte (or 4-byte) vector; the 3 x 3 x 3 patches are never gathered
// from global memory but cut out of input rows staged in shared memory.
// Work unit of every kernel: a STRIP of up to 64 consecutive output pixels of one output row (16 per warp); the forward
// kernel takes strips of up to 320 pixels on wide images (five tiles per warp).
// COUT is a template parameter (48 for the detector's stem).
#pragma once
#include "common.cuh"

namespace nbcbs {

constexpr int STEM_CIN = 3, STEM_K = 3, STEM_TAPS = 9, STEM_KDIM = 27;
constexpr int STEM_TQ = 64;        // output pixels per strip (data and weight gradient; forward of narrow images)
constexpr int STEM_TQ_WIDE = 320;  // the forward kernel's strip on wide images: per-strip work is shared by 20 tiles instead of 4
__host__ __device__ constexpr int stem_xchunks(int tq) {  // 16-byte chunks per staged input row: columns 2*q0-1 .. 2*q0+2*tq-1, plus the alignment shift (<= 7)
    return ((2 * tq + 1) * STEM_CIN + 7 + 7) / 8;
}
constexpr int STEM_XCHUNKS = stem_xchunks(STEM_TQ);
constexpr int STEM_XPITCH = STEM_XCHUNKS * 8;

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
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* smem_row) {
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(smem_row);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* smem_row) {
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(smem_row);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}

// Strip number -> image n, output row p, first output column q0.  `sh` is filled by the kernels that stage input rows:
// the alignment shifts of the strip's three staged rows, 3 bits each (see stem_stage_rows_async).
struct StemStrip {
    int n, p, q0, sh;
};
template <int TQ = STEM_TQ> __device__ __forceinline__ StemStrip stem_strip(long long t, const Geom& g, int strips_per_row) {
    // (32-bit divisions: the plan admits fewer than 2^31 output pixels; 64-bit ones cost about a hundred instructions each,
    // and these kernels are bound by instruction issue)
    StemStrip s;
    const unsigned tt = (unsigned)t, t1 = tt / (unsigned)strips_per_row;
    s.q0 = (int)(tt - t1 * (unsigned)strips_per_row) * TQ;
    s.n = (int)(t1 / (unsigned)g.ho);
    s.p = (int)(t1 - (unsigned)s.n * (unsigned)g.ho);
    s.sh = 0;
    return s;
}
// A block visits strips blockIdx.x, + gridDim.x, + 2 gridDim.x, ...: the stride is decomposed once (two divisions), and
// every further strip follows from the one before it by additions and two carries.
struct StemWalk {
    int dq0, dp, dn, row_len, ho;  // stride in first-column units / rows / images; strips_per_row * strip width; output rows
};
template <int TQ = STEM_TQ> __device__ __forceinline__ StemWalk stem_walk(const Geom& g, int strips_per_row) {
    StemWalk k;
    const unsigned d = gridDim.x, d1 = d / (unsigned)strips_per_row;
    k.dq0 = (int)(d - d1 * (unsigned)strips_per_row) * TQ;
    k.dn = (int)(d1 / (unsigned)g.ho);
    k.dp = (int)(d1 - (unsigned)k.dn * (unsigned)g.ho);
    k.row_len = strips_per_row * TQ;
    k.ho = g.ho;
    return k;
}
__device__ __forceinline__ StemStrip stem_advance(StemStrip s, const StemWalk& k) {
    s.q0 += k.dq0;
    if (s.q0 >= k.row_len) {
        s.q0 -= k.row_len;
        ++s.p;
    }
    s.p += k.dp;  // (p < ho, dp < ho and one carry: a single subtraction brings it back into range)
    if (s.p >= k.ho) {
        s.p -= k.ho;
        ++s.n;
    }
    s.n += k.dn;
    return s;
}
__host__ __device__ inline long long stem_num_strips(const Geom& g, int tq = STEM_TQ) { return (long long)g.n * g.ho * ((g.wo + tq - 1) / tq); }

// 16-byte asynchronous copy global -> shared; bytes past `src_bytes` (0..16) are written as zeros.
__device__ __forceinline__ void cp_async16_zfill(void* smem_dst, const void* gsrc, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait_pending() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }  // at most N groups still in flight

// The three input rows 2p-1, 2p, 2p+1 of a strip, columns 2*q0-1 .. 2*q0+2*TQ-1, are staged in shared memory as aligned
// 16-byte chunks of the flat tensor: element k of staged row r -- input column 2*q0-1 + k/3, channel k%3 -- is
// xrow[r][shift[r] + k].  Row -1 (p = 0) is written as zeros; column -1 (q0 = 0) holds whatever precedes the row in memory
// and is masked when the fragments of the strip's first pixel are built; values past the image's last column belong to output pixels that do not
// exist and are never used.  The copies are asynchronous (cp.async) and run several strips ahead of the arithmetic (a ring
// of NS buffers, NS - 1 strips in flight per block): with one strip in flight the kernels were bound by memory latency
// (bytes in flight per SM x 148 / latency was far below the HBM rate), not by bandwidth.  `total` = number of elements of x.
__device__ __forceinline__ int stem_row_start(const Geom& g, const StemStrip& s, int r, int& shift) {
    // (int arithmetic: the plan admits fewer than 2^31 input elements; e0 is negative only inside the padding, and in two's
    // complement the masks below round towards minus infinity there too)
    const int e0 = ((s.n * g.h + (2 * s.p - 1 + r)) * g.w + (2 * s.q0 - 1)) * 3;
    shift = e0 & 7;
    return e0 & ~7;
}
// WHOLE = false stages only what the strip's own pixels read (a wide strip of a narrower row); what lies behind in the buffer
// is then stale, which only a kernel whose tiles' rows are independent of one another may ignore.
template <int TQ = STEM_TQ, bool WHOLE = true>
__device__ __forceinline__ int stem_stage_rows_async(const unsigned short* __restrict__ x, const Geom& g, int total, const StemStrip& s,
                                                     unsigned short (*xrow)[stem_xchunks(TQ) * 8]) {
    int shifts = 0;  // returned: the three rows' shifts, 3 bits each
    const int width = g.wo - s.q0 < TQ ? g.wo - s.q0 : TQ;  // output pixels the strip really has
#pragma unroll
    for (int r = 0; r < 3; ++r) {
        int sh;
        const int a0 = stem_row_start(g, s, r, sh);
        shifts |= sh << (3 * r);
        const bool row_ok = 2 * s.p - 1 + r >= 0;
        const int nchunks = WHOLE ? stem_xchunks(TQ) : ((2 * width + 1) * STEM_CIN + sh + 7) >> 3;
        for (int ci = threadIdx.x; ci < nchunks; ci += blockDim.x) {
            const int start = a0 + 8 * ci;
            int bytes = 0;  // a chunk before the tensor's start (a0 < 0: only padding lies there), in row -1 or past the end: zeros
            if (row_ok && start >= 0 && start < total) bytes = total - start >= 8 ? 16 : (total - start) * 2;
            cp_async16_zfill(&xrow[r][8 * ci], bytes ? x + start : x, bytes);
        }
    }
    return shifts;
}

// Two fp32 values rounded to a pair of 16-bit values (fp16 saturates at the largest finite value), and back.
template <typename T> __device__ __forceinline__ uint32_t stem_pack2(float2 v);
template <> __device__ __forceinline__ uint32_t stem_pack2<__half>(float2 v) {
    uint32_t r;
    asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(v.y), "f"(v.x));
    return r;
}
template <> __device__ __forceinline__ uint32_t stem_pack2<__nv_bfloat16>(float2 v) {
    const __nv_bfloat162 b = __float22bfloat162_rn(v);
    return *reinterpret_cast<const uint32_t*>(&b);
}
template <typename T> __device__ __forceinline__ float2 stem_unpack2(uint32_t v);
template <> __device__ __forceinline__ float2 stem_unpack2<__half>(uint32_t v) { return __half22float2(*reinterpret_cast<const __half2*>(&v)); }
template <> __device__ __forceinline__ float2 stem_unpack2<__nv_bfloat16>(uint32_t v) { return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v)); }

// Per-channel epilogue of the evaluation-mode / plain forward: out = act(acc*scale_c + shift_c), coefficients as bn_eval_coef.
struct StemEpi {
    const float *gamma, *beta, *rmean, *rvar;
    float eps;
    int act;
};
// Forward.  A warp computes 16 output pixels x COUT channels with K padded to 32 (two k-steps); the filter fragments stay
// in registers for the whole kernel; the A fragments are read from the staged rows (2-byte shared-memory loads: the nine
// values of one filter row of a pixel are contiguous there).  The 16 x COUT output tile is one contiguous run: staged and
// written with 16-byte stores.
// EPI = false: y = the convolution output in fp16 (training forward), and with `partials` != NULL the block also writes the
// per-channel sum and sum of squares of the ROUNDED values it stored to partials[blockIdx.x][2][COUT], or with `acc` != NULL
// adds them to accumulator set blockIdx.x mod acc_copies of [acc_copies][2][COUT] doubles (batch statistics
// without a second pass over y; fixed order, bitwise reproducible).  EPI = true: OutT = activations, see StemEpi.
// InT = the 16-bit type of x and w (bf16, or IEEE fp16).
template <int COUT, typename OutT = __half, bool EPI = false, typename InT = __nv_bfloat16, int TQ = STEM_TQ>
__global__ void __launch_bounds__(128, 4) stem_fprop_mma_kernel(const InT* __restrict__ x, const InT* __restrict__ w, OutT* __restrict__ y, Geom g,
                                                                StemEpi ep, float* __restrict__ partials, double* __restrict__ acc, int acc_copies) {
    pdl_launch_dependents();
    pdl_wait();
    static_assert(COUT % 8 == 0, "whole n-blocks");
    static_assert(TQ % 64 == 0, "whole 16-pixel tiles for each of the four warps");
    constexpr int NB = COUT / 8, XPITCH = stem_xchunks(TQ) * 8;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gq = lane >> 2, tq = lane & 3;
    const unsigned short* xs = reinterpret_cast<const unsigned short*>(x);
    const unsigned short* wsrc = reinterpret_cast<const unsigned short*>(w);
    // the eight K indices of this lane's A fragment elements: k-step s2, register half j, element e -> filter row and offset
    // inside the nine contiguous values of that row (-1: the padding k >= 27)
    // (a padding index k >= 27 meets a zero filter value: it reads the patch's centre, a value the pixel depends on anyway)
    int krow[8], koff[8];    // filter row of k, and its offset in the staged rows relative to the pixel's first element
    unsigned left_mask = 0;  // bit i: element i lies in the patch's left column (zero padding for the image's first column)
    uint32_t bfrag[2][NB][2];
#pragma unroll
    for (int s2 = 0; s2 < 2; ++s2)
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int k = s2 * 16 + j * 8 + tq * 2 + e, i = s2 * 4 + j * 2 + e;
                krow[i] = k < STEM_KDIM ? k / 9 : 1;
                koff[i] = krow[i] * XPITCH + (k < STEM_KDIM ? k % 9 : 3);
                if (k < STEM_KDIM && k % 9 < 3) left_mask |= 1u << i;
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
    float2 ssum[EPI ? 1 : NB], ssq[EPI ? 1 : NB];  // running channel sums of this lane's two columns per n-block over its rows
    if (!EPI) {
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) ssum[nb] = ssq[nb] = make_float2(0.f, 0.f);
    }
    constexpr int NS = TQ == STEM_TQ ? 4 : 3;  // ring of staged strips
    __shared__ __align__(16) unsigned short xrow[NS][3][XPITCH];
    __shared__ __align__(16) OutT stage[4][16 * COUT];
    const int total = g.n * g.h * g.w * 3;
    const int strips_per_row = (g.wo + TQ - 1) / TQ;
    const long long nstrips = stem_num_strips(g, TQ);
    const StemWalk walk = stem_walk<TQ>(g, strips_per_row);
    StemStrip ahead[NS - 1];  // the strips whose rows are in flight, decoded once
#pragma unroll
    for (int k = 0; k < NS - 1; ++k) {  // (one group per strip, empty when the block has no such strip)
        const long long tk = blockIdx.x + (long long)k * gridDim.x;
        ahead[k] = k == 0 ? stem_strip<TQ>(tk < nstrips ? tk : 0, g, strips_per_row) : stem_advance(ahead[k > 0 ? k - 1 : 0], walk);
        if (tk < nstrips) ahead[k].sh = stem_stage_rows_async<TQ, TQ == STEM_TQ>(xs, g, total, ahead[k], xrow[k]);
        cp_async_commit();
    }
    int buf = 0;
    for (long long t = blockIdx.x; t < nstrips; t += gridDim.x, buf = (buf + 1) % NS) {
        const StemStrip s = ahead[0];
#pragma unroll
        for (int k = 0; k + 1 < NS - 1; ++k) ahead[k] = ahead[k + 1];
        cp_async_wait_pending<NS - 2>();
        __syncthreads();  // this strip's rows have landed; the buffer refilled below (the previous strip's) has been consumed
        const long long tn = t + (long long)(NS - 1) * gridDim.x;
        if (tn < nstrips) {  // (then strip tn - gridDim.x, which ahead[NS - 2] still holds, was decoded too)
            ahead[NS - 2] = stem_advance(ahead[NS - 2], walk);
            ahead[NS - 2].sh = stem_stage_rows_async<TQ, TQ == STEM_TQ>(xs, g, total, ahead[NS - 2], xrow[(buf + NS - 1) % NS]);
        }
        cp_async_commit();
        // per strip: where this lane's eight fragment elements sit in the staged rows, relative to a pixel's first element
        int addr[8];
        {
            int sh[3];
#pragma unroll
            for (int r = 0; r < 3; ++r) sh[r] = (s.sh >> (3 * r)) & 7;
#pragma unroll
            for (int i = 0; i < 8; ++i) addr[i] = koff[i] + (krow[i] == 0 ? sh[0] : krow[i] == 1 ? sh[1] : sh[2]);
        }
        const long long mrow = ((long long)s.n * g.ho + s.p) * g.wo;  // first output pixel of the strip's row
#pragma unroll 1
        for (int tile = warp; tile < TQ / 16; tile += 4) {  // (one tile per warp with 64-pixel strips)
            const int qw = s.q0 + tile * 16;  // first output column of this tile's 16 pixels
            if (qw >= g.wo) break;
            const unsigned short* xr = &xrow[buf][0][0] + 6 * (tile * 16 + gq);
            uint32_t a[2][4];
            bool row_ok[2];
#pragma unroll
            for (int half = 0; half < 2; ++half) {  // fragment rows gq and gq + 8
                row_ok[half] = qw + gq + half * 8 < g.wo;  // (pixels past the row's end compute on whatever the buffer holds there and are dropped below)
                unsigned short v[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) v[i] = xr[addr[i] + 48 * half];
                if (half == 0 && qw + gq == 0) {  // the image's first column: its left neighbours are zero padding
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        if ((left_mask >> i) & 1u) v[i] = 0;
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
            // accumulator registers: c0, c1 = (row g, columns 2t, 2t+1), c2, c3 = (row g+8, same columns)
            OutT* st = stage[warp];
#pragma unroll
            for (int half = 0; half < 2; ++half)
#pragma unroll
                for (int nb = 0; nb < NB; ++nb) {
                    float2 v = make_float2(acc[nb][2 * half], acc[nb][2 * half + 1]);
                    if (EPI) {
                        v.x = fmaf(v.x, esc[nb][0], esh[nb][0]);
                        v.y = fmaf(v.y, esc[nb][1], esh[nb][1]);
                        if (ep.act) v = mul2(v, sigmoid2<true>(v));
                    }
                    const uint32_t pk = stem_pack2<OutT>(v);  // the two rounded values: one 4-byte store
                    *reinterpret_cast<uint32_t*>(st + (gq + half * 8) * COUT + nb * 8 + tq * 2) = pk;
                    if (!EPI && row_ok[half]) {
                        const float2 r = stem_unpack2<OutT>(pk);
                        ssum[nb] = add2(ssum[nb], r);
                        ssq[nb] = fma2(r, r, ssq[nb]);
                    }
                }
            __syncwarp();
            const int rows = g.wo - qw < 16 ? g.wo - qw : 16;
            const int nvec = rows * COUT / 8;  // 16-byte pieces of the tile that exist
            OutT* yt = y + (size_t)(mrow + qw) * COUT;
            for (int v = lane; v < nvec; v += 32) st16(yt + v * 8, ld16(st + v * 8));
            __syncwarp();
        }
    }
    if (!EPI && (partials || acc)) {
        // lanes with the same tq hold the same columns for different rows: add over gq (fixed butterfly), then over the warps
        __shared__ float wsum[4][2][COUT];
        __syncthreads();
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                float sv = e ? ssum[nb].y : ssum[nb].x, qv = e ? ssq[nb].y : ssq[nb].x;
#pragma unroll
                for (int o = 4; o < 32; o <<= 1) {
                    sv += __shfl_xor_sync(0xffffffffu, sv, o);
                    qv += __shfl_xor_sync(0xffffffffu, qv, o);
                }
                if (gq == 0) {
                    wsum[warp][0][nb * 8 + tq * 2 + e] = sv;
                    wsum[warp][1][nb * 8 + tq * 2 + e] = qv;
                }
            }
        __syncthreads();
        for (int e = threadIdx.x; e < 2 * COUT; e += blockDim.x) {
            const int which = e / COUT, c = e - which * COUT;
            const float v = ((wsum[0][which][c] + wsum[1][which][c]) + wsum[2][which][c]) + wsum[3][which][c];
            if (acc) atomicAdd(acc + ((size_t)((int)blockIdx.x % acc_copies) * 2 + which) * COUT + c, (double)v);  // the plan's fp64 accumulators (see ChanAcc)
            else partials[(size_t)blockIdx.x * 2 * COUT + e] = v;
        }
    }
}

// Data gradient as mma.sync tiles.  For dy position (i, j) the four input pixels (2i+a, 2j+b) receive
//   (0,0) <- dy[i][j] w11;  (0,1) <- dy[i][j+1] w10 + dy[i][j] w12;  (1,0) <- dy[i+1][j] w01 + dy[i][j] w21;
//   (1,1) <- dy[i+1][j+1] w00 + dy[i+1][j] w02 + dy[i][j+1] w20 + dy[i][j] w22        (w_rt = filter tap (r,t)),
// i.e. per parity class a GEMM [16 positions x COUT] x [COUT x 3] per tap with the dy tile shifted by (0|1, 0|1).  An MMA
// has eight output columns and a tap fills three, so two taps that read the same shifted tile share an MMA: columns 0-2
// belong to a class of output row parity 0, columns 3-5 to the class of parity 1 with the same column parity.  Two
// accumulators (column parity 0 and 1) and six MMAs per 16 channels of dy instead of four accumulators and nine:
//   parity b = 0:  dy[i][j] x [w11 | w21],  dy[i+1][j] x [0 | w01]
//   parity b = 1:  dy[i][j] x [w12 | w22],  dy[i][j+1] x [w10 | w20],  dy[i+1][j] x [0 | w02],  dy[i+1][j+1] x [0 | w00].
// A block stages rows i and i+1 of a 64-position strip (plus one column) in shared memory with 16-byte loads (pixel
// pitch 112 bytes: conflict-free ldmatrix), the 18 filter fragments stay in registers, and the 2 x 32 output pixels of a
// warp are staged and written as 4-byte words (coalesced).  Five blocks are resident per SM (96 registers, a ring of four
// staged rows of 7.3 KB per block).  Grid: stem_dgrad_grid().
constexpr int STEM_DYPITCH = 56;  // elements per staged dy pixel (48 channels + padding)
// Blocks and rows per block of the data-gradient kernel: the bands (image x 64-column strip) are cut into as many row
// segments as keep the grid within one wave of `slots` resident blocks; more bands than slots: whole bands, several waves.
inline int stem_dgrad_grid(const Geom& g, int slots, int* seg_rows) {
    const long long bands = (long long)g.n * ((g.wo + STEM_TQ - 1) / STEM_TQ);
    const long long segs_wanted = bands < slots ? slots / bands : 1;
    *seg_rows = (int)((g.ho + segs_wanted - 1) / segs_wanted);
    const long long segs = (g.ho + *seg_rows - 1) / *seg_rows;
    return (int)(bands * segs);
}
template <int COUT, typename T = __nv_bfloat16>
__global__ void __launch_bounds__(128, 5) stem_dgrad_mma_kernel(const T* __restrict__ dy, const T* __restrict__ w, T* __restrict__ dx, Geom g, int seg_rows) {
    pdl_launch_dependents();
    pdl_wait();
    static_assert(COUT % 16 == 0 && COUT + 8 <= STEM_DYPITCH, "whole k-steps; pitch holds a pixel");
    constexpr int KS = COUT / 16;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gq = lane >> 2, tq = lane & 3;
    const unsigned short* wsrc = reinterpret_cast<const unsigned short*>(w);
    // B fragments of the six MMAs: element (k = channel c' of dy, n = output column gq): columns 0-2 take filter tap
    // pair[m][0], columns 3-5 tap pair[m][1] (tap = r*3 + t; -1: zeros), input channel gq % 3; columns 6, 7 are padding
    constexpr int kPair[6][2] = {{4, 7}, {-1, 1}, {5, 8}, {3, 6}, {-1, 2}, {-1, 0}};
    uint32_t bfrag[6][KS][2];
    {
        const int slot = gq >= 3 ? 1 : 0, ch = gq - 3 * slot;
#pragma unroll
        for (int m = 0; m < 6; ++m) {
            const int tap = gq < 6 ? (slot ? kPair[m][1] : kPair[m][0]) : -1;
#pragma unroll
            for (int ks = 0; ks < KS; ++ks)
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const int c0 = ks * 16 + j * 8 + tq * 2;
                    const uint32_t lo = tap >= 0 ? wsrc[c0 * STEM_KDIM + tap * 3 + ch] : 0u, hi = tap >= 0 ? wsrc[(c0 + 1) * STEM_KDIM + tap * 3 + ch] : 0u;
                    bfrag[m][ks][j] = lo | (hi << 16);
                }
        }
    }
    // Work unit of a block: output row pairs [p_lo, p_hi) of one 64-column band of one image.  Consecutive strips of a band
    // share a dy row, so the block keeps a ring of single rows and every dy row travels to the SM once per band instead of
    // twice; the strip arithmetic is one addition.
    constexpr int NR = 4;  // ring of staged dy rows: two in use, two on their way
    __shared__ __align__(16) T dyrow[NR][(STEM_TQ + 1) * STEM_DYPITCH];  // [buffer][pixel][channel]
    __shared__ __align__(16) T outs[4][2][32 * 3];
    const int strips_per_row = (g.wo + STEM_TQ - 1) / STEM_TQ;
    const int bands = g.n * strips_per_row;
    const int seg = (int)blockIdx.x / bands, band = (int)blockIdx.x - seg * bands;  // (neighbouring blocks: neighbouring bands of the same rows)
    StemStrip s;
    s.n = band / strips_per_row;
    s.q0 = (band - s.n * strips_per_row) * STEM_TQ;
    s.sh = 0;
    const int p_lo = seg * seg_rows, p_hi = p_lo + seg_rows < g.ho ? p_lo + seg_rows : g.ho;
    constexpr int VPP = COUT / 8;  // 16-byte vectors per pixel
    // asynchronous staging of dy[row][q0 .. q0+64][:] (zeros past the last row / column).  A row's 65 pixels are one
    // contiguous run of 65 * VPP vectors in global memory; in shared memory pixels are STEM_DYPITCH apart.  A thread copies
    // vector `vec` of pixels px0, px0 + PXSTEP, ...: both addresses advance by constants (no division per copy).
    constexpr int PXSTEP = 128 / VPP, PXITER = (STEM_TQ + 1 + PXSTEP - 1) / PXSTEP;
    const int px0 = threadIdx.x / VPP, vec = threadIdx.x - px0 * VPP;
    const bool stager = px0 < PXSTEP;  // (128 threads = PXSTEP whole pixels and a remainder that stays idle)
    const int npx = g.wo - s.q0;       // pixels of a row from q0 on
    const T* const col0 = dy + ((size_t)s.n * g.ho * g.wo + s.q0 + px0) * COUT + vec * 8;
    auto stage_row_async = [&](int row) {  // rows beyond p_hi are not needed by this block: an empty group
        if (stager && row <= p_hi) {
            const bool row_ok = row < g.ho;
            const T* src = col0 + (size_t)row * g.wo * COUT;
            T* d = &dyrow[row & (NR - 1)][px0 * STEM_DYPITCH + vec * 8];
#pragma unroll
            for (int it = 0; it < PXITER; ++it) {
                const int px = px0 + it * PXSTEP;
                if (px <= STEM_TQ) {
                    const bool ok = row_ok && px < npx;
                    cp_async16_zfill(d + it * PXSTEP * STEM_DYPITCH, ok ? src + it * PXSTEP * COUT : dy, ok ? 16 : 0);
                }
            }
        }
        cp_async_commit();
    };
    stage_row_async(p_lo);
    stage_row_async(p_lo + 1);
    stage_row_async(p_lo + 2);
    for (s.p = p_lo; s.p < p_hi; ++s.p) {
        cp_async_wait_pending<1>();  // all groups but the newest: rows p and p + 1 have landed
        __syncthreads();             // ... for every thread, and the buffer refilled below (row p - 1's) has been consumed
        stage_row_async(s.p + 3);
        const int buf = s.p & (NR - 1), buf1 = (s.p + 1) & (NR - 1);
        const int jw = s.q0 + warp * 16;  // first dy column of this warp's 16 positions
        if (jw < g.wo) {
            float acc[2][4];  // column parity b: columns 0-2 = row parity 0, columns 3-5 = row parity 1
#pragma unroll
            for (int c = 0; c < 2; ++c) acc[c][0] = acc[c][1] = acc[c][2] = acc[c][3] = 0.f;
            const int mi = lane >> 3, mr = lane & 7;  // ldmatrix: matrix and row this lane addresses
            const T* d0 = dyrow[buf];
            const T* d1 = dyrow[buf1];
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                uint32_t a00[4], a01[4], a10[4], a11[4];  // dy tile shifted by (di, dj)
                const int px = warp * 16 + mr + (mi & 1) * 8, ko = ks * 16 + (mi >> 1) * 8;
                ldmatrix_x4(a00, &d0[px * STEM_DYPITCH + ko]);
                ldmatrix_x4(a01, &d0[(px + 1) * STEM_DYPITCH + ko]);
                ldmatrix_x4(a10, &d1[px * STEM_DYPITCH + ko]);
                ldmatrix_x4(a11, &d1[(px + 1) * STEM_DYPITCH + ko]);
                mma_16816<T>(acc[0], a00, bfrag[0][ks][0], bfrag[0][ks][1]);  // b = 0: dy[i][j]     x [w11 | w21]
                mma_16816<T>(acc[1], a00, bfrag[2][ks][0], bfrag[2][ks][1]);  // b = 1: dy[i][j]     x [w12 | w22]
                mma_16816<T>(acc[0], a10, bfrag[1][ks][0], bfrag[1][ks][1]);  // b = 0: dy[i+1][j]   x [ 0  | w01]
                mma_16816<T>(acc[1], a01, bfrag[3][ks][0], bfrag[3][ks][1]);  // b = 1: dy[i][j+1]   x [w10 | w20]
                mma_16816<T>(acc[1], a10, bfrag[4][ks][0], bfrag[4][ks][1]);  //        dy[i+1][j]   x [ 0  | w02]
                mma_16816<T>(acc[1], a11, bfrag[5][ks][0], bfrag[5][ks][1]);  //        dy[i+1][j+1] x [ 0  | w00]
            }
            // accumulator registers: c0, c1 = (position gq, columns 2tq, 2tq+1), c2, c3 = (position gq+8, same columns);
            // column c < 6 = row parity c / 3, input channel c % 3
            T(*o)[32 * 3] = outs[warp];
            if (tq < 3) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int col = 2 * tq + e, a = col >= 3 ? 1 : 0, ch = col - 3 * a;
#pragma unroll
                    for (int b = 0; b < 2; ++b)
#pragma unroll
                        for (int half = 0; half < 2; ++half) o[a][(2 * (gq + half * 8) + b) * 3 + ch] = from_f32<T>(acc[b][2 * half + e]);
                }
            }
            __syncwarp();
            const int npos = g.wo - jw < 16 ? g.wo - jw : 16;
            const int nwords = npos * 3;  // 4-byte words per output row segment (2*npos pixels x 3 channels x 2 bytes)
#pragma unroll
            for (int a = 0; a < 2; ++a) {
                uint32_t* dst = reinterpret_cast<uint32_t*>(dx + (((size_t)s.n * g.h + 2 * s.p + a) * g.w + 2 * (size_t)jw) * 3);
                const uint32_t* src = reinterpret_cast<const uint32_t*>(o[a]);
                for (int v = lane; v < nwords; v += 32) dst[v] = src[v];
            }
            __syncwarp();
        }
    }
}

// Weight gradient: dw[c'][k] = sum over pixels of dy[pixel][c'] * patch[pixel][k] as mma.sync tiles of 16 pixels (the
// reduction index): A = dy^T (the 16 x COUT piece of dy is one contiguous run: staged in shared memory with 16-byte loads
// and read back transposed with ldmatrix), B = the pixels' patch values cut out of the staged input rows.  A block sums
// the strips it is dealt; its four warps are combined in a fixed order into the block's slice of `partial`
// [gridDim.x][COUT][27].
// TQ = strip width: STEM_TQ, or STEM_TQ_WGRAD on wide images (two tiles per warp and strip: the per-strip work -- staging
// loops, strip arithmetic, one block-wide barrier -- is shared by twice as many tiles).  Dynamic shared memory:
// stem_wgrad_smem_bytes<COUT, T, TQ>().
constexpr int STEM_TQ_WGRAD = 128;
template <int COUT, typename T, int TQ> struct StemWgradRing {
    static constexpr int NS = TQ == STEM_TQ ? 4 : 3;  // ring of staged strips
    unsigned short xrow[NS][3][stem_xchunks(TQ) * 8];
    T dys[NS][TQ * COUT];  // the strip's TQ x COUT piece of dy (one contiguous run), per buffer
};
template <int COUT, typename T, int TQ> constexpr size_t stem_wgrad_smem_bytes() {
    return sizeof(StemWgradRing<COUT, T, TQ>) > 4 * sizeof(float[COUT][33]) ? sizeof(StemWgradRing<COUT, T, TQ>) : 4 * sizeof(float[COUT][33]);
}
template <int COUT, typename T = __nv_bfloat16, int TQ = STEM_TQ>
__global__ void __launch_bounds__(128, 4) stem_wgrad_mma_kernel(const T* __restrict__ x, const T* __restrict__ dy, float* __restrict__ partial, Geom g) {
    pdl_launch_dependents();
    pdl_wait();
    static_assert(COUT % 16 == 0, "whole m-blocks");
    static_assert(TQ % 64 == 0, "whole 16-pixel tiles for each of the four warps");
    constexpr int MB = COUT / 16, NBK = 4;  // accumulator blocks: MB x 16 channels by NBK x 8 filter positions (27 padded to 32)
    typedef StemWgradRing<COUT, T, TQ> Ring;
    constexpr int NS = Ring::NS, XPITCH = stem_xchunks(TQ) * 8;
    typedef float Red[COUT][33];
    extern __shared__ __align__(16) unsigned char raw[];  // the ring while strips are processed, then the four warps' sums
    Ring& ring = *reinterpret_cast<Ring*>(raw);
    Red* red = reinterpret_cast<Red*>(raw);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gq = lane >> 2, tq = lane & 3;
    const unsigned short* xs = reinterpret_cast<const unsigned short*>(x);
    // B fragment element (k = pixel 2t.., n = 8*nb + g): filter position n of the pixel's patch -> filter row, offset in the row
    // (positions n >= 27 are accumulator columns that are never stored: they read the patch's centre)
    int krow[NBK], koff[NBK];
    unsigned left_mask = 0;  // bit nb: the position lies in the patch's left column (zero padding for the image's first column)
#pragma unroll
    for (int nb = 0; nb < NBK; ++nb) {
        const int k = nb * 8 + gq;
        krow[nb] = k < STEM_KDIM ? k / 9 : 1;
        koff[nb] = krow[nb] * XPITCH + (k < STEM_KDIM ? k % 9 : 3);
        if (k < STEM_KDIM && k % 9 < 3) left_mask |= 1u << nb;
    }
    float acc[MB][NBK][4];
#pragma unroll
    for (int a = 0; a < MB; ++a)
#pragma unroll
        for (int b = 0; b < NBK; ++b) acc[a][b][0] = acc[a][b][1] = acc[a][b][2] = acc[a][b][3] = 0.f;
    const int total = g.n * g.h * g.w * 3;
    const int strips_per_row = (g.wo + TQ - 1) / TQ;
    const long long nstrips = stem_num_strips(g, TQ);
    // asynchronous staging of a strip: the three input rows and dy[strip][:] (zeros past the row's end: those pixels then
    // contribute nothing)
    auto stage_async = [&](const StemStrip& s, int b) -> int {
        const int shifts = stem_stage_rows_async<TQ, true>(xs, g, total, s, ring.xrow[b]);  // (whole: pixels past the row's end must read defined values)
        const T* src = dy + (((size_t)s.n * g.ho + s.p) * g.wo + s.q0) * COUT;
        const int nv = (g.wo - s.q0 < TQ ? g.wo - s.q0 : TQ) * (COUT / 8);  // 16-byte vectors of dy that exist
#pragma unroll
        for (int it = 0; it < TQ * COUT / 8 / 128; ++it) {
            const int v = threadIdx.x + it * 128;
            const bool ok = v < nv;
            cp_async16_zfill(&ring.dys[b][v * 8], ok ? src + v * 8 : dy, ok ? 16 : 0);
        }
        return shifts;
    };
    const StemWalk walk = stem_walk<TQ>(g, strips_per_row);
    StemStrip ahead[NS - 1];  // the strips whose data are in flight, decoded once
#pragma unroll
    for (int k = 0; k < NS - 1; ++k) {
        const long long tk = blockIdx.x + (long long)k * gridDim.x;
        ahead[k] = k == 0 ? stem_strip<TQ>(tk < nstrips ? tk : 0, g, strips_per_row) : stem_advance(ahead[k > 0 ? k - 1 : 0], walk);
        if (tk < nstrips) ahead[k].sh = stage_async(ahead[k], k);
        cp_async_commit();
    }
    int buf = 0;
    for (long long t = blockIdx.x; t < nstrips; t += gridDim.x, buf = (buf + 1) % NS) {
        const StemStrip s = ahead[0];
#pragma unroll
        for (int k = 0; k + 1 < NS - 1; ++k) ahead[k] = ahead[k + 1];
        cp_async_wait_pending<NS - 2>();
        __syncthreads();
        const long long tn = t + (long long)(NS - 1) * gridDim.x;
        if (tn < nstrips) {  // (then strip tn - gridDim.x, which ahead[NS - 2] still holds, was decoded too)
            ahead[NS - 2] = stem_advance(ahead[NS - 2], walk);
            ahead[NS - 2].sh = stage_async(ahead[NS - 2], (buf + NS - 1) % NS);
        }
        cp_async_commit();
        int addr[NBK];  // per strip: where this lane's filter positions sit in the staged rows, relative to a pixel's first element
        {
            int sh[3];
#pragma unroll
            for (int r = 0; r < 3; ++r) sh[r] = (s.sh >> (3 * r)) & 7;
#pragma unroll
            for (int nb = 0; nb < NBK; ++nb) addr[nb] = koff[nb] + (krow[nb] == 0 ? sh[0] : krow[nb] == 1 ? sh[1] : sh[2]);
        }
#pragma unroll 1
        for (int tile = warp; tile < TQ / 16; tile += 4) {  // (one tile per warp with 64-pixel strips)
            const int qw = s.q0 + tile * 16;
            if (qw >= g.wo) break;
            const unsigned short* xr = &ring.xrow[buf][0][0] + 6 * (tile * 16 + tq * 2);
            const T* st = &ring.dys[buf][tile * 16 * COUT];
            // B fragments: four pixels of the tile (2t, 2t+1, 2t+8, 2t+9) x NBK filter positions.  (Pixels past the row's
            // end meet zero dy rows, so whatever defined values they read contribute nothing.)
            uint32_t bfr[NBK][2];
            unsigned short v4[4][NBK];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
#pragma unroll
                for (int nb = 0; nb < NBK; ++nb) v4[j][nb] = xr[addr[nb] + 6 * ((j & 1) + (j >> 1) * 8)];
            }
            if (qw + tq == 0) {  // the image's first column (pixel j = 0 of this lane): its left neighbours are zero padding
#pragma unroll
                for (int nb = 0; nb < NBK; ++nb)
                    if ((left_mask >> nb) & 1u) v4[0][nb] = 0;
            }
#pragma unroll
            for (int nb = 0; nb < NBK; ++nb) {
                bfr[nb][0] = (uint32_t)v4[0][nb] | ((uint32_t)v4[1][nb] << 16);
                bfr[nb][1] = (uint32_t)v4[2][nb] | ((uint32_t)v4[3][nb] << 16);
            }
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
        }
    }
    // accumulator registers: c0, c1 = (channel 16mb+g, positions 8nb+2t, +1), c2, c3 = (channel 16mb+g+8, same positions)
    cp_async_wait_pending<0>();
    __syncthreads();  // every warp is done with the ring: its space now holds the warps' sums
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
