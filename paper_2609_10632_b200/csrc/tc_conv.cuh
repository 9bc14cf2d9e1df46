// Tensor-core convolution kernels for sm_100a: an implicit GEMM whose A operand (activation pixels x channels of
// one filter tap) is fetched by TMA in im2col mode, whose B operand (filter rows) is fetched by tiled TMA, whose
// products are issued as tcgen05.mma by one thread with fp32 accumulators in TMEM, and whose epilogue (eight warps)
// reads the accumulators back with tcgen05.ld, converts, stages the tile in shared memory, takes per-channel sums
// for the batch statistics and hands the rows to TMA stores.  The same kernel computes fprop (A = x, B = w) and dgrad
// (A = dy, B = the filter rearranged per output-parity class).  No multicast anywhere; every wait is bounded.
#pragma once
#include <atomic>
#include <cuda.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <string>

#include "../../include/nb_cbs.h"
#include "common.cuh"
#include "ptx_sm100.cuh"
#include "simt_conv.cuh"

namespace nbcbs {

// ------------------------------------------------------------------------------------------ kernel parameters
struct IgemmParams {
    CUtensorMap tmA;     // im2col map over the activation [N][Hs][Ws][Ca]
    CUtensorMap tmB[4];  // per class: tiled map over the filter matrix [rowsB][ntaps*Ca], K contiguous
    // Ca mod 64 in (0, 32]: the last k-block of every tap is 32 channels wide, fetched through these maps (same tensors,
    // boxes of 32 channels in the 64-byte swizzle) and multiplied by two MMAs instead of four.
    int tail32;
    CUtensorMap tmA_t;
    CUtensorMap tmB_t[4];
    long long M;      // rows of the GEMM: n * Hq * Wq
    int Hq, Wq;       // traversal grid per image
    int ts;           // traversal stride (input pixels per grid step)
    int lo_w, lo_h;   // input coordinate of grid position 0 for tap offset 0
    // A launch covers up to four "classes" that share A, the tiling and the output tensor but have their own filter
    // matrix, tap list and output offset (the four output-parity classes of a stride-2 data gradient); for the order of
    // the tiles see igemm_tile_class.
    int nclasses, tiles_per_class;
    int cls_interleave;          // four classes: the classes of one [m][n] tile are neighbours in the tile order
    int cls_ntaps[4], cls_oa[4], cls_ob[4];
    int Ca, KC, kc_per_tap;
    int kpb;                     // k-blocks (of KC channels) per pipeline stage
    uint32_t a_sub_bytes, b_sub_bytes;  // bytes of one k-block of A / B inside a stage
    int BN, n_tiles, m_tiles;
    int mh;                      // 128-row sub-tiles per tile (1 or 2): the tile is [128*mh x BN]
    int acc_bufs;                // accumulator sets in TMEM (2 when 2*mh*acc_stride <= 512)
    int ncol_a;                  // columns of a tile that epilogue team 0 handles (team 1: the other BN - ncol_a)
    int stage_cw;                // columns per staging pass of a team (<= 64)
    // When GEMM row == output row (everything but a stride-2 dgrad) a warp hands each staged [32 x width] piece
    // to TMA: tmOut[i] is a tiled map over the output [M][ldo] with box {out_w[i], 32}; clipping at M is the map's.
    int tma_store;
    int out_accumulate;  // the TMA stores are reductions: the tile is added to what the output tensor holds (data gradient into a shared gradient buffer)
    int out_w[3];
    CUtensorMap tmOut[3];
    // Statistics variant: with acc.acc != NULL every CTA adds its channel sums to the plan's fp64 accumulators (the
    // normalise + SiLU pass derives mean, invstd, scale and shift from them, see ChanAcc); else it writes them to
    // `partials` for a separate finalize kernel.
    ChanAcc acc;
    float fin_eps;
    const float *fin_gamma, *fin_beta, *fin_rmean, *fin_rvar;
    // Fused per-channel epilogue (EPI variant: evaluation-mode BN or a bias, then optionally SiLU, applied to the fp32
    // accumulators before they are rounded): out = act(acc*scale_c + shift_c).  The CTA derives the coefficients itself
    // from fin_gamma / fin_beta / fin_rmean / fin_rvar / fin_eps (gamma NULL: scale 1; rmean NULL: shift = beta or 0).
    int epi_act;
    int stages, acc_stride, tmem_cols;
    uint32_t umma_swizzle, sbo, a_stage_bytes, b_stage_bytes, idesc;
    int a_tiled;                 // 1: A is a plain [M][Ca] matrix fetched with a tiled 2-D map (1x1 stride-1 convolutions)
    int ldo;                     // channels per output pixel
    int Hout, Wout, os;          // GEMM row (n,i,j) -> output pixel (n, i*os+oa, j*os+ob) of an Hout x Wout image
    void* out;
    float* partials;  // [gridDim.x][2][ldo] per-CTA channel sums and sums of squares (statistics variant only)
    int* status;
    uint16_t off_w[4][9], off_h[4][9];
};

// Tile number -> (class, tile within the class).  Default order: class by class, classes with more taps first.  With
// cls_interleave (set for the four parity classes of a stride-2 data gradient) the four classes of one [m][n] tile are
// neighbours in the order, so the dy rows they share are fetched from DRAM once and found in L2 three times instead of being
// streamed once per class; the class of position r is rotated by the round of the persistent loop so that a worker
// (whose tile numbers are nworkers apart) still cycles through heavy and light classes.
// CLS4 = the launch has the four classes (a template parameter: every other launch has one class and pays nothing for
// the decoding, which sits in the producer, MMA and epilogue loops).
template <bool CLS4> __device__ __forceinline__ void igemm_tile_class(const IgemmParams& p, int tile, int nworkers, int& cls, int& lt) {
    if (!CLS4) {
        cls = 0;
        lt = tile;
    } else if (p.cls_interleave) {
        const int r = tile & 3;
        const int round = (tile - r) / nworkers;
        cls = (r + ((nworkers & 1) ? 0 : round)) & 3;
        lt = tile >> 2;
    } else {
        cls = tile / p.tiles_per_class;
        lt = tile - cls * p.tiles_per_class;
    }
}

constexpr int TC_BM = 128;
constexpr int IG_THREADS = 352;  // implicit-GEMM kernel: the roles below plus a second epilogue team in warps 7-10
constexpr int TC_THREADS = 224;  // warp 0: TMA producer for A, warp 1: MMA issuer + TMEM owner, warps 2-5: epilogue, warp 6: TMA producer for B

__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// Bounded mbarrier wait: gives up after `limit_ns` (or as soon as another role has given up), records the site.
__device__ __noinline__ bool wait_bar(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status, int site, uint64_t limit_ns = kWaitLimitNs) {
    uint64_t t0 = 0;
    for (uint32_t i = 0;; ++i) {
        if (ptx::mbar_try_wait_parked(bar, parity, 4000u)) return true;
        if ((i & 127u) == 127u) {
            if (*abort_flag) return false;
            const uint64_t now = global_timer_ns();
            if (t0 == 0) {
                t0 = now;
            } else if (now - t0 > limit_ns) {
                *abort_flag = 1;
                report_timeout(status, site, (int)blockIdx.x);
                return false;
            }
        }
    }
}

// Fast path inline (the barrier is usually complete already), slow bounded path out of line.
// Called by all 32 lanes of a producer or MMA warp; the lanes leave together with the same answer.
__device__ __forceinline__ bool wait_bar_fast(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status, int site) {
    bool ok = ptx::mbar_try_wait(bar, parity);
    if (!ok) ok = wait_bar(bar, parity, abort_flag, status, site);
    return __all_sync(0xffffffffu, ok) != 0;
}

__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
// The same over the 256 threads of the implicit-GEMM kernel's two epilogue teams.
__device__ __forceinline__ void epi2_bar_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
__device__ __forceinline__ bool epi2_bar_and(bool ok) {
    uint32_t r;
    asm volatile(
        "{\n\t"
        ".reg .pred p, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "bar.red.and.pred q, 1, 256, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t"
        "}\n"
        : "=r"(r)
        : "r"((uint32_t)ok)
        : "memory");
    return r != 0;
}
// Barrier over the 128 epilogue threads that also ANDs a predicate, so that all of them take the same decision.
__device__ __forceinline__ bool epi_bar_and(bool ok) {
    uint32_t r;
    asm volatile(
        "{\n\t"
        ".reg .pred p, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "bar.red.and.pred q, 1, 128, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t"
        "}\n"
        : "=r"(r)
        : "r"((uint32_t)ok)
        : "memory");
    return r != 0;
}

template <typename OutT> __device__ __forceinline__ uint32_t pack2(float a, float b, int* sat);
template <> __device__ __forceinline__ uint32_t pack2<__nv_bfloat16>(float a, float b, int*) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&v);
}
// fp16 stores saturate to the largest finite value; `sat` collects, per 16-bit half, a flag bit (bit 15 / 31) that is set
// when a stored magnitude is 65504 (0x7bff) or an exceptional pattern above it.
template <> __device__ __forceinline__ uint32_t pack2<__half>(float a, float b, int* sat) {
    uint32_t v;
    asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(v) : "f"(b), "f"(a));
    if (sat) *sat |= (int)((v & 0x7fff7fffu) + 0x04010401u);  // (sat is a compile-time NULL where the caller tracks saturation otherwise)
    return v;
}

// One epilogue pass of NP columns (16, 32, 48 or 64) by one warp when the output goes through TMA: this thread's
// accumulator row segment travels TMEM -> registers -> dense staging rows (row pitch NP*2 bytes; 128-byte rows in the
// 128-byte swizzle), `release` is called as soon as the registers hold the data (the accumulator may be reused), lane 0
// hands the 32 x NP piece to TMA, and with STATS the warp adds the piece's per-channel sums of the rounded values to its
// running sums (a lane owns two adjacent channels).  Everything is unrolled on NP: constant offsets, no predicates.
// With EPI the accumulators first become act(acc*scale + shift) with the pass's per-channel (scale, shift) pairs read
// from shared memory (`coef`, the same address in every lane: a broadcast; per channel pair scale, scale, shift, shift).
template <typename OutT, bool STATS, int NP, int EPI, class Release>
__device__ __forceinline__ void epi_pass_tma(uint32_t taddr, uint8_t* wrows, int lane, bool& store_pending, int& sat, const CUtensorMap* tm, int col,
                                             int grow, float* stat_s, float* stat_q, const float2* coef, int act, bool accumulate, Release release) {
    constexpr bool SWZ = NP == 64;
    constexpr int PITCH = NP * 2;
    uint32_t r[NP];
#pragma unroll
    for (int hh = 0; hh < NP / 16; ++hh) ptx::tmem_ld_32x32b_x16(taddr + (uint32_t)(16 * hh), r + 16 * hh);
    ptx::tmem_ld_wait();
    release();
    if (EPI) {
        if (act) {
#pragma unroll
            for (int j = 0; j < NP; j += 2) {
                const float4 cf = *reinterpret_cast<const float4*>(coef + j);
                const float2 z = fma2(make_float2(__uint_as_float(r[j]), __uint_as_float(r[j + 1])), make_float2(cf.x, cf.y), make_float2(cf.z, cf.w));
                const float2 o = mul2(z, sigmoid2<true>(z));
                r[j] = __float_as_uint(o.x);
                r[j + 1] = __float_as_uint(o.y);
            }
        } else {
#pragma unroll
            for (int j = 0; j < NP; j += 2) {
                const float4 cf = *reinterpret_cast<const float4*>(coef + j);
                const float2 z = fma2(make_float2(__uint_as_float(r[j]), __uint_as_float(r[j + 1])), make_float2(cf.x, cf.y), make_float2(cf.z, cf.w));
                r[j] = __float_as_uint(z.x);
                r[j + 1] = __float_as_uint(z.y);
            }
        }
    }
    if (store_pending) {  // the previous TMA store must have read the staging rows before they are overwritten
        if (lane == 0) ptx::tma_store_wait_read<0>();
        __syncwarp();
    }
    uint8_t* const my_row = wrows + lane * PITCH;
    int sat_bits = 0;
    // (With STATS a saturated value is recognised below from the sums of squares, which costs nothing per element.)
    int* const sat_track = STATS ? nullptr : &sat_bits;
#pragma unroll
    for (int j = 0; j < NP / 8; ++j) {
        uint4 v;
        v.x = pack2<OutT>(__uint_as_float(r[8 * j + 0]), __uint_as_float(r[8 * j + 1]), sat_track);
        v.y = pack2<OutT>(__uint_as_float(r[8 * j + 2]), __uint_as_float(r[8 * j + 3]), sat_track);
        v.z = pack2<OutT>(__uint_as_float(r[8 * j + 4]), __uint_as_float(r[8 * j + 5]), sat_track);
        v.w = pack2<OutT>(__uint_as_float(r[8 * j + 6]), __uint_as_float(r[8 * j + 7]), sat_track);
        *reinterpret_cast<uint4*>(my_row + (SWZ ? (j ^ (lane & 7)) : j) * 16) = v;
    }
    if (sat_bits & (int)0x80008000u) ++sat;  // this thread's row segment of the pass held a saturated value
    ptx::fence_async_smem();  // writes visible to the async proxy before the store is issued
    __syncwarp();
    if (lane == 0) {
        if (accumulate) ptx::tma_reduce_add_2d(tm, wrows, col, grow); else ptx::tma_store_2d(tm, wrows, col, grow);
        ptx::tma_store_commit();
    }
    store_pending = true;
    if (STATS) {
        if (lane < NP / 2) {
            float2 sa = make_float2(0.f, 0.f), sb = sa, qa = sa, qb = sa;
            const int cj = lane >> 2;
            const uint8_t* base = wrows + (lane & 3) * 4;
#pragma unroll
            for (int rr = 0; rr < 32; rr += 2) {
                const float2 f0 = __half22float2(*reinterpret_cast<const __half2*>(base + rr * PITCH + (SWZ ? (cj ^ (rr & 7)) : cj) * 16));
                const float2 f1 = __half22float2(*reinterpret_cast<const __half2*>(base + (rr + 1) * PITCH + (SWZ ? (cj ^ ((rr + 1) & 7)) : cj) * 16));
                sa = add2(sa, f0);  // packed fp32 pairs: the same sums in half the issue slots
                sb = add2(sb, f1);
                qa = fma2(f0, f0, qa);
                qb = fma2(f1, f1, qb);
            }
            // a stored +-65504 puts at least 65504^2 into its channel's sum of squares over these 32 rows; nothing else
            // does unless the 32 values average above 11585, i.e. sit within a factor of six of the fp16 range
            const float qx = qa.x + qb.x, qy = qa.y + qb.y;
            if (fmaxf(qx, qy) >= 4290774016.f) ++sat;
            float2* ps = reinterpret_cast<float2*>(stat_s + 2 * lane);
            float2* pq = reinterpret_cast<float2*>(stat_q + 2 * lane);
            float2 a2 = *ps, b2 = *pq;
            a2.x += sa.x + sb.x; a2.y += sa.y + sb.y;
            b2.x += qa.x + qb.x; b2.y += qa.y + qb.y;
            *ps = a2;
            *pq = b2;
        }
        __syncwarp();  // staged rows read before the next pass overwrites them
    }
}

// CG2 = the CTAs run as pairs (clusters of two): rank 0 issues tcgen05.mma.cta_group::2 with M = 256; each CTA owns 128
// of the rows (its own A tile, accumulator and epilogue) and fetches half of the B tile, which halves the filter
// bytes written to and read from each SM's shared memory.
// EPI = 1: the epilogue applies a per-channel scale and shift (evaluation-mode BN or a bias) and optionally SiLU to the
// accumulators, so the kernel writes the block's final activations (no statistics, no second pass); TMA stores only.
// STATS (forward of a training block): TMA stores only; the epilogue also sums every channel's values and squares.
template <typename OutT, bool STATS, bool CG2, int EPI = 0, bool CLS4 = false>
__global__ void __launch_bounds__(IG_THREADS, 1) tc_igemm_kernel(const __grid_constant__ IgemmParams p) {
    static_assert(!CLS4 || (!STATS && !EPI), "four classes: the stride-2 data gradient only");
    static_assert(!EPI || !STATS, "the fused per-channel epilogue is a forward-only variant without statistics");
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* sA = smem;
    uint8_t* sB = sA + (size_t)p.stages * p.a_stage_bytes;
    uint8_t* stg = sB + (size_t)p.stages * p.b_stage_bytes;  // staging: per epilogue team [128 rows][ncol_a columns] of OutT, row pitch ncol_a*2+16 bytes
    const int cw = p.stage_cw;  // columns per staging pass (<= 64)
    const int pitch = cw * 2 + 16;
    float* wstat = reinterpret_cast<float*>(stg + (size_t)2 * TC_BM * pitch);  // per team [4 warps][2][its columns of every n-tile]: warp-private channel sums
    uint64_t* bars = reinterpret_cast<uint64_t*>(wstat + ((STATS || EPI) ? 8 * p.ldo : 0));  // EPI: wstat holds [ldo] (scale, shift) pairs
    uint64_t* full = bars;                // [stages]
    uint64_t* empty = bars + p.stages;    // [stages]
    uint64_t* tfull = empty + p.stages;   // [2]
    uint64_t* tempty = tfull + 2;         // [2]
    uint64_t* drain = tempty + 2;         // [1]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    // the next kernel of the stream may become resident and run its prologue right away
    pdl_launch_dependents();
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;  // warp index in a form the compiler knows to be uniform
    const int total_tiles = p.nclasses * p.tiles_per_class;
    const int mh = p.mh;          // 128-row sub-tiles per tile (1 or 2); both share every B stage
    const int nbuf = p.acc_bufs;  // accumulator sets in TMEM (2 = the epilogue of a tile overlaps the next tile's MMAs)
    const uint32_t rank = CG2 ? (blockIdx.x & 1u) : 0u;                       // position in the CTA pair (clusters are (2,1,1))
    const int worker = CG2 ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;        // tile-loop start
    const int nworkers = CG2 ? (int)(gridDim.x >> 1) : (int)gridDim.x;        // tile-loop stride

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            ptx::mbar_init(full + s, 2);  // the A and the B producer arrive once each with their byte counts (pairs: rank 0's
                                          // producers announce the bytes of both CTAs, the peer only issues its loads)
            ptx::mbar_init(empty + s, 1);
        }
        ptx::mbar_init(tfull, 1);
        ptx::mbar_init(tfull + 1, 1);
        ptx::mbar_init(tempty, CG2 ? 16 : 256);  // pairs: one arrival per epilogue warp of both CTAs
        ptx::mbar_init(tempty + 1, CG2 ? 16 : 256);
        ptx::mbar_init(drain, 1);
        *abort_flag = 0;
        ptx::fence_mbar_init();
    }
    // the tensor maps live in the kernel's parameters: their fetch can run while this kernel still waits for its predecessor
    if (lane == 0) {
        if (warp == 0) ptx::prefetch_tmap(&p.tmA);
        if (warp == 6)
            for (int c = 0; c < p.nclasses; ++c) ptx::prefetch_tmap(&p.tmB[c]);
        if (warp == 2 && p.tma_store)
            for (int i = 0; i < 3; ++i)
                if (p.out_w[i]) ptx::prefetch_tmap(&p.tmOut[i]);
    }
    if (STATS) {
        for (int c = threadIdx.x; c < 8 * p.ldo; c += IG_THREADS) wstat[c] = 0.f;
    }
    if (warp == 1) {
        if (CG2) {
            ptx::tmem_alloc_cg2(tmem_slot, (uint32_t)p.tmem_cols);
            ptx::tmem_relinquish_cg2();
        } else {
            ptx::tmem_alloc(tmem_slot, (uint32_t)p.tmem_cols);
            ptx::tmem_relinquish();
        }
    }
    ptx::tc_fence_before();
    if (CG2) ptx::cluster_sync_all(); else __syncthreads();  // barriers of both CTAs are initialised before any remote arrive
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // Everything above touched only shared memory, TMEM and kernel parameters.  Each role waits for the previous kernel
    // (griddepcontrol.wait) itself, as late as it can: the producers after they have read their parameters, right before
    // the first load; the epilogue warps before their first access to global memory; the MMA issuer touches none.
    if (EPI) {
        pdl_wait();
        // per-channel coefficients of the fused epilogue, in fp64 like the training-mode finalize
        // (stored per channel pair as scale, scale, shift, shift: the operands of the packed fp32 multiply-add)
        for (int c = threadIdx.x; c < p.ldo; c += IG_THREADS) {
            double sc, sh;
            bn_eval_coef(p.fin_gamma, p.fin_beta, p.fin_rmean, p.fin_rvar, p.fin_eps, c, sc, sh);
            wstat[4 * (c >> 1) + (c & 1)] = (float)sc;
            wstat[4 * (c >> 1) + 2 + (c & 1)] = (float)sh;
        }
        __syncthreads();
    }

    if (warp == 0 || warp == 6) {
        // ------------------------------------------------------------------ TMA producers: warp 0 feeds A, warp 6 feeds B
        // Both producer warps run their loops converged; `leader` predicates the instructions that must be issued once.
        const uint32_t leader = ptx::elect_one() ? 1u : 0u;
        const bool isA = warp == 0;
        int s = 0;
        uint32_t ph = 0;
        long long issued = 0;
        bool ok = true;
        const int bn_own = CG2 ? p.BN / 2 : p.BN;  // rows of the B tile this CTA fetches
        const uint32_t kb_bytes = isA ? (uint32_t)(TC_BM * mh * p.KC * 2) : (uint32_t)(bn_own * p.KC * 2);
        const int kc_tail = p.tail32 ? p.kc_per_tap - 1 : -1;  // index of the 32-channel k-block inside a tap (-1: none)
        // loop-invariant values in registers: this thread's instruction stream is on the critical path
        const int kpb = p.kpb, stages = p.stages, KC = p.KC, kc_per_tap = p.kc_per_tap, Ca = p.Ca, BN = p.BN, n_tiles = p.n_tiles;
        const int Wq = p.Wq, Hq = p.Hq, ts = p.ts, a_tiled = p.a_tiled;
        const uint32_t stage_bytes = isA ? p.a_stage_bytes : p.b_stage_bytes, sub_bytes = isA ? p.a_sub_bytes : p.b_sub_bytes;
        // pairs: loads of both CTAs are counted on the rank-0 CTA's full barriers (the MMA issuer waits there)
        const uint32_t base_u32 = ptx::smem_u32(isA ? sA : sB);
        const uint32_t full_u32 = CG2 ? ptx::mapa_u32(ptx::smem_u32(full), 0u) : ptx::smem_u32(full);
        pdl_wait();
        for (int tile = worker; ok && tile < total_tiles; tile += nworkers) {
            int cls, lt;
            igemm_tile_class<CLS4>(p, tile, nworkers, cls, lt);
            const CUtensorMap* tm_full = isA ? &p.tmA : &p.tmB[cls];
            const CUtensorMap* tm_tail = isA ? &p.tmA_t : &p.tmB_t[cls];
            const int kblocks = p.cls_ntaps[cls] * kc_per_tap;
            const int m_tile = lt / n_tiles, n_tile = lt - m_tile * n_tiles;
            const int m0 = (CG2 ? m_tile * 2 + (int)rank : m_tile) * TC_BM * mh;
            int cw0 = 0, ch0 = 0, n0 = 0;
            if (isA && !a_tiled) {
                const int j0 = m0 % Wq, t1 = m0 / Wq;
                const int i0 = t1 % Hq;
                n0 = t1 / Hq;
                cw0 = p.lo_w + j0 * ts;
                ch0 = p.lo_h + i0 * ts;
            }
            const int brow = n_tile * BN + (CG2 ? (int)rank * bn_own : 0);
            // each CTA starts its K loop at a different k-block so that the CTAs do not all ask L2 for the same
            // filter lines at the same moment
            const int ntaps_c = p.cls_ntaps[cls];
            const int rot = (int)(((unsigned)worker * 7u) % (unsigned)kblocks);
            int tap = rot / kc_per_tap, kc = rot - tap * kc_per_tap;
            for (int kb0 = 0; kb0 < kblocks; kb0 += kpb) {
                const int nkb = (kblocks - kb0 < kpb) ? kblocks - kb0 : kpb;
                if (!wait_bar_fast(empty + s, ph ^ 1u, abort_flag, p.status, isA ? 1 : 5)) {
                    ok = false;
                    break;
                }
                const uint32_t bar = full_u32 + 8u * (uint32_t)s;
                uint32_t tx_bytes = kb_bytes * (uint32_t)nkb;
                if (kc_tail >= 0) {  // a 32-channel k-block brings half the bytes
                    int kq = kc;
                    for (int j = 0; j < nkb; ++j) {
                        if (kq == kc_tail) tx_bytes -= kb_bytes >> 1;
                        if (++kq == kc_per_tap) kq = 0;
                    }
                }
                if (!CG2) ptx::mbar_expect_tx_u32_if(leader, bar, tx_bytes);
                else if (rank == 0) ptx::mbar_expect_tx_u32_if(leader, ptx::smem_u32(full) + 8u * (uint32_t)s, 2u * tx_bytes);
                uint32_t dst = base_u32 + (uint32_t)s * stage_bytes;
                for (int j = 0; j < nkb; ++j) {
                    const CUtensorMap* tm = kc == kc_tail ? tm_tail : tm_full;
                    if (isA) {
                        if (a_tiled) {
                            if (CG2) ptx::tma_load_2d_cg2_if(leader, dst, tm, bar, kc * KC, m0); else ptx::tma_load_2d_u32_if(leader, dst, tm, bar, kc * KC, m0);
                        } else {
                            if (CG2)
                                ptx::tma_load_im2col_4d_cg2_if(leader, dst, tm, bar, kc * KC, cw0, ch0, n0, p.off_w[cls][tap], p.off_h[cls][tap]);
                            else
                                ptx::tma_load_im2col_4d_u32_if(leader, dst, tm, bar, kc * KC, cw0, ch0, n0, p.off_w[cls][tap], p.off_h[cls][tap]);
                        }
                    } else {
                        if (CG2) ptx::tma_load_2d_cg2_if(leader, dst, tm, bar, tap * Ca + kc * KC, brow); else ptx::tma_load_2d_u32_if(leader, dst, tm, bar, tap * Ca + kc * KC, brow);
                    }
                    dst += sub_bytes;
                    if (++kc == kc_per_tap) {
                        kc = 0;
                        if (++tap == ntaps_c) tap = 0;
                    }
                }
                ++issued;
                if (++s == stages) {
                    s = 0;
                    ph ^= 1u;
                }
            }
        }
        if (!ok) {
            // Gave up: wait (bounded) for the loads still in flight so that nothing lands after the CTA has exited.
            const int back = issued < (long long)p.stages ? (int)issued : p.stages;
            for (int b = 0; b < back; ++b) {
                s = (s == 0) ? p.stages - 1 : s - 1;
                if (s == p.stages - 1) ph ^= 1u;
                for (int i = 0; i < 100000 && !ptx::mbar_try_wait(full + s, ph); ++i) {
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (one thread; in a pair only rank 0)
        const uint32_t leader = ptx::elect_one() ? 1u : 0u;  // the whole warp runs the loop, this lane issues
        if (rank == 0) {
            int s = 0, acc = 0;
            uint32_t ph = 0, acc_ph = 0;
            bool ok = true;
            const int ksteps = p.KC / 16, kpb = p.kpb, stages = p.stages;
            const uint32_t idesc = p.idesc, acc_stride = (uint32_t)p.acc_stride;
            const uint64_t a_sub16 = (uint64_t)(p.a_sub_bytes >> 4), b_sub16 = (uint64_t)(p.b_sub_bytes >> 4);
            const uint64_t a_stage16 = (uint64_t)(p.a_stage_bytes >> 4), b_stage16 = (uint64_t)(p.b_stage_bytes >> 4);
            const uint64_t a_half16 = (uint64_t)((TC_BM * p.KC * 2) >> 4);  // second 128-row sub-tile inside a k-block of A
            // 32-channel k-block: rows of 64 bytes in the 64-byte swizzle; same start address, other stride and swizzle fields
            const uint64_t tail_flip = ptx::make_smem_desc(0u, 16, p.sbo, p.umma_swizzle) ^ ptx::make_smem_desc(0u, 16, p.sbo >> 1, (uint32_t)ptx::kSwizzle64);
            const int kc_tail = p.tail32 ? p.kc_per_tap - 1 : -1;
            const uint64_t da0 = ptx::make_smem_desc(ptx::smem_u32(sA), 16, p.sbo, p.umma_swizzle);
            const uint64_t db0 = ptx::make_smem_desc(ptx::smem_u32(sB), 16, p.sbo, p.umma_swizzle);
            const uint32_t empty_u32 = ptx::smem_u32(empty);
            uint64_t da_s = da0, db_s = db0;  // descriptors of the current stage
            const int kc_per_tap = p.kc_per_tap;
            const uint32_t tfull_u32 = ptx::smem_u32(tfull);
            for (int tile = worker; ok && tile < total_tiles; tile += nworkers) {
                int cls_mma, lt_mma;
                igemm_tile_class<CLS4>(p, tile, nworkers, cls_mma, lt_mma);
                const int kblocks = p.cls_ntaps[cls_mma] * kc_per_tap;
                if (!wait_bar_fast(tempty + acc, acc_ph ^ 1u, abort_flag, p.status, 2)) break;
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * mh) * acc_stride;
                uint32_t accumulate = 0;
                int kc = (int)(((unsigned)worker * 7u) % (unsigned)kblocks) % kc_per_tap;  // the producers' starting k-block
                for (int kb0 = 0; kb0 < kblocks; kb0 += kpb) {
                    const int nkb = (kblocks - kb0 < kpb) ? kblocks - kb0 : kpb;
                    if (!wait_bar_fast(full + s, ph, abort_flag, p.status, 3)) {
                        ok = false;
                        break;
                    }
                    ptx::tc_fence_after();
                    uint64_t da = da_s, db = db_s;
                    for (int j = 0; j < nkb; ++j) {
                        const bool tail = kc == kc_tail;
                        if (++kc == kc_per_tap) kc = 0;
                        for (int h = 0; h < mh; ++h) {
                            const uint64_t dah = da + (uint64_t)h * a_half16;
                            const uint32_t dt = d_tmem + (uint32_t)h * acc_stride;
                            if (tail) {
                                const uint64_t dat = (da + (uint64_t)h * (a_half16 >> 1)) ^ tail_flip, dbt = db ^ tail_flip;
                                if (CG2) {
                                    ptx::umma_f16_cg2_if(leader, dt, dat, dbt, idesc, accumulate);
                                    ptx::umma_f16_cg2_if(leader, dt, dat + 2, dbt + 2, idesc, 1u);
                                } else {
                                    ptx::umma_f16_if(leader, dt, dat, dbt, idesc, accumulate);
                                    ptx::umma_f16_if(leader, dt, dat + 2, dbt + 2, idesc, 1u);
                                }
                            } else if (CG2) {
                                ptx::umma_f16_cg2_if(leader, dt, dah, db, idesc, accumulate);
                                ptx::umma_f16_cg2_if(leader, dt, dah + 2, db + 2, idesc, 1u);
                                ptx::umma_f16_cg2_if(leader, dt, dah + 4, db + 4, idesc, 1u);
                                ptx::umma_f16_cg2_if(leader, dt, dah + 6, db + 6, idesc, 1u);
                            } else if (ksteps == 4) {
                                ptx::umma_f16_if(leader, dt, dah, db, idesc, accumulate);
                                ptx::umma_f16_if(leader, dt, dah + 2, db + 2, idesc, 1u);
                                ptx::umma_f16_if(leader, dt, dah + 4, db + 4, idesc, 1u);
                                ptx::umma_f16_if(leader, dt, dah + 6, db + 6, idesc, 1u);
                            } else {
                                for (int k = 0; k < ksteps; ++k)
                                    ptx::umma_f16_if(leader, dt, dah + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, (k | (int)accumulate) ? 1u : 0u);
                            }
                        }
                        accumulate = 1u;
                        da += a_sub16;
                        db += b_sub16;
                    }
                    if (CG2) ptx::umma_commit_cg2_mc_if(leader, empty_u32 + 8u * (uint32_t)s, 3); else ptx::umma_commit_u32_if(leader, empty_u32 + 8u * (uint32_t)s);
                    da_s += a_stage16;
                    db_s += b_stage16;
                    if (++s == stages) {
                        s = 0;
                        ph ^= 1u;
                        da_s = da0;
                        db_s = db0;
                    }
                }
                if (!ok) break;
                if (CG2) ptx::umma_commit_cg2_mc_if(leader, tfull_u32 + 8u * (uint32_t)acc, 3); else ptx::umma_commit_u32_if(leader, tfull_u32 + 8u * (uint32_t)acc);
                if (++acc == nbuf) {
                    acc = 0;
                    acc_ph ^= 1u;
                }
            }
            // Make sure every MMA issued by this thread has retired before TMEM is released.
            if (CG2) ptx::umma_commit_cg2_if(leader, ptx::smem_u32(drain)); else ptx::umma_commit_u32_if(leader, ptx::smem_u32(drain));
            for (int i = 0; i < 4000000 && !ptx::mbar_try_wait(drain, 0); ++i) {
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue: two teams of four warps (warps 2-5 and 7-10)
        // Every tile's columns are split between the teams (team 0: the first ncol_a columns, team 1: the rest), each team
        // has its own staging buffer and running sums, and inside a team warp q owns accumulator rows [32q, 32q+32).
        // The epilogue is bound by the latency of its own instruction stream (one warp per scheduler), so a second team
        // nearly halves the time per tile.
        const int team = warp >= 7 ? 1 : 0;
        const int lane_group = warp & 3;          // TMEM lanes this warp may read: rows [32*lane_group, +32) of a sub-tile
        const int c_lo = team ? p.ncol_a : 0;     // first column (within the tile) and number of columns of this team
        const int ncol = team ? p.BN - p.ncol_a : p.ncol_a;
        const int st_ld = p.n_tiles * ncol;       // row length of this team's running sums: its columns of every n-tile
        int acc = 0, sat = 0;
        uint32_t acc_ph = 0;
        float* team_stat = wstat + (team ? (size_t)8 * p.n_tiles * p.ncol_a : 0);  // [4 warps][2][st_ld]
        float* my_stat = team_stat + (size_t)lane_group * 2 * st_ld;
        const bool tma_out = p.tma_store != 0;  // (always set for the STATS and EPI variants)
        const bool acc_out = !STATS && !EPI && p.out_accumulate != 0;
        // staging of this warp's 32 rows: padded rows for the store loop, dense rows (the TMA box) for TMA stores
        uint8_t* stg_t = stg + (size_t)team * TC_BM * pitch;
        uint8_t* const wrows = tma_out ? stg + (size_t)((team * 4 + lane_group) * 32) * (cw * 2) : stg_t + (size_t)(lane_group * 32) * pitch;
        bool store_pending = false;
        uint8_t* outb = static_cast<uint8_t*>(p.out);
        const uint32_t tempty_u32 = CG2 ? ptx::mapa_u32(ptx::smem_u32(tempty), 0u) : 0u;  // the issuer's barriers (rank 0)
        pdl_wait();
        for (int tile = worker; tile < total_tiles; tile += nworkers) {
            int cls, lt;
            igemm_tile_class<CLS4>(p, tile, nworkers, cls, lt);
            const int m_tile = lt / p.n_tiles, n_tile = lt % p.n_tiles;
            bool ok = true;
            // one poller per warp: 256 threads spinning on one mbarrier would crowd the shared-memory pipe
            if (lane == 0) ok = wait_bar(tfull + acc, acc_ph, abort_flag, p.status, 4);
            ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
            ok = epi2_bar_and(ok);
            if (!ok) break;
            ptx::tc_fence_after();
            auto release_acc = [&]() {  // this warp is done reading the tile's accumulators
                ptx::tc_fence_before();
                if (CG2) {
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive_cluster(tempty_u32 + 8u * (uint32_t)acc);
                } else {
                    ptx::mbar_arrive(tempty + acc);
                }
            };
            if (ncol == 0) {
                release_acc();
                if (++acc == nbuf) {
                    acc = 0;
                    acc_ph ^= 1u;
                }
                continue;
            }
            for (int h = 0; h < mh; ++h) {
                const long long m0 = (((CG2 ? (long long)m_tile * 2 + rank : (long long)m_tile)) * mh + h) * TC_BM;
                const uint32_t taddr = tmem_base + ((uint32_t)(lane_group * 32) << 16) + (uint32_t)((acc * mh + h) * p.acc_stride) + (uint32_t)c_lo;
                // The team's columns go through the staging buffer in passes of at most cw (<= 64) columns.
                for (int cb = 0; cb < ncol; cb += cw) {
                    const int npass = (ncol - cb < cw) ? ncol - cb : cw;  // multiple of 16
                    const bool last = h == mh - 1 && cb + cw >= ncol;    // last TMEM read of this tile: the accumulator set becomes free
                    if (tma_out) {
                        auto release = [&]() {
                            if (last) release_acc();
                        };
                        const CUtensorMap* tm = npass == p.out_w[0] ? &p.tmOut[0] : npass == p.out_w[1] ? &p.tmOut[1] : &p.tmOut[2];
                        const int col = n_tile * p.BN + c_lo + cb, grow = (int)(m0 + lane_group * 32);
                        float* ss = my_stat + n_tile * ncol + cb;
                        float* sq = ss + st_ld;
                        const uint32_t ta = taddr + (uint32_t)cb;
                        const float2* cf = reinterpret_cast<const float2*>(wstat) + col;  // read only by the EPI variant
                        if (npass == 64) epi_pass_tma<OutT, STATS, 64, EPI>(ta, wrows, lane, store_pending, sat, tm, col, grow, ss, sq, cf, p.epi_act, acc_out, release);
                        else if (npass == 48) epi_pass_tma<OutT, STATS, 48, EPI>(ta, wrows, lane, store_pending, sat, tm, col, grow, ss, sq, cf, p.epi_act, acc_out, release);
                        else if (npass == 32) epi_pass_tma<OutT, STATS, 32, EPI>(ta, wrows, lane, store_pending, sat, tm, col, grow, ss, sq, cf, p.epi_act, acc_out, release);
                        else epi_pass_tma<OutT, STATS, 16, EPI>(ta, wrows, lane, store_pending, sat, tm, col, grow, ss, sq, cf, p.epi_act, acc_out, release);
                        continue;
                    }
                    // ---- output rows that are not GEMM rows (the parity classes of a stride-2 data gradient): padded staging
                    // rows and a coalesced store loop.  TMEM -> registers -> staging (this thread's row); up to four
                    // 16-column loads are in flight before the one wait: a TMEM load has a long latency
                    uint8_t* const my_row = wrows + (size_t)lane * pitch;
                    {
                        uint32_t r[64];
                        const int nld = npass / 16;
#pragma unroll
                        for (int hh = 0; hh < 4; ++hh)
                            if (hh < nld) ptx::tmem_ld_32x32b_x16(taddr + (uint32_t)(cb + 16 * hh), r + 16 * hh);
                        ptx::tmem_ld_wait();
                        int sat_bits = 0;
#pragma unroll
                        for (int hh = 0; hh < 4; ++hh) {
                            if (hh >= nld) break;
                            uint4 v0, v1;
                            const uint32_t* q = r + 16 * hh;
                            v0.x = pack2<OutT>(__uint_as_float(q[0]), __uint_as_float(q[1]), &sat_bits);
                            v0.y = pack2<OutT>(__uint_as_float(q[2]), __uint_as_float(q[3]), &sat_bits);
                            v0.z = pack2<OutT>(__uint_as_float(q[4]), __uint_as_float(q[5]), &sat_bits);
                            v0.w = pack2<OutT>(__uint_as_float(q[6]), __uint_as_float(q[7]), &sat_bits);
                            v1.x = pack2<OutT>(__uint_as_float(q[8]), __uint_as_float(q[9]), &sat_bits);
                            v1.y = pack2<OutT>(__uint_as_float(q[10]), __uint_as_float(q[11]), &sat_bits);
                            v1.z = pack2<OutT>(__uint_as_float(q[12]), __uint_as_float(q[13]), &sat_bits);
                            v1.w = pack2<OutT>(__uint_as_float(q[14]), __uint_as_float(q[15]), &sat_bits);
                            *reinterpret_cast<uint4*>(my_row + (2 * hh) * 16) = v0;
                            *reinterpret_cast<uint4*>(my_row + (2 * hh + 1) * 16) = v1;
                        }
                        if (sat_bits & (int)0x80008000u) ++sat;  // this thread's row segment of the pass held a saturated value
                    }
                    if (last) release_acc();
                    __syncwarp();  // every warp only reads back the 32 rows it staged itself
                    // ---- coalesced stores: the warp walks its 32 staged rows as one flat sequence of 16-byte pieces
                    // (32 rows x cpr pieces = cpr iterations of 32 lanes, every lane busy); lane r first works out the
                    // output offset of row r, the others fetch it by shuffle
                    {
                        const int cpr = npass / 8;  // 16-byte pieces per staged row (<= 8)
                        long long pixrow = m0 + lane_group * 32 + lane;  // GEMM row of staged row `lane`
                        if (pixrow >= p.M) {
                            pixrow = -1;
                        } else if (p.os != 1) {
                            const int j = (int)(pixrow % p.Wq);
                            const long long t1 = pixrow / p.Wq;
                            const int i = (int)(t1 % p.Hq);
                            const long long n = t1 / p.Hq;
                            pixrow = (n * p.Hout + (long long)i * p.os + p.cls_oa[cls]) * p.Wout + (long long)j * p.os + p.cls_ob[cls];
                        }
                        // byte offset of staged row `lane` in the output (-1: not stored); pieces are handled four (or two) at
                        // a time so that their shuffle -> shared load -> global store chains overlap
                        const long long rowbyte = pixrow < 0 ? -1 : pixrow * (long long)(p.ldo * 2) + (n_tile * p.BN + c_lo + cb) * 2;
                        const int step_r = 32 / cpr, step_c = 32 - step_r * cpr;
                        int rr = lane / cpr, cc = lane - rr * cpr;
                        auto advance = [&](int& r_, int& c_) {
                            r_ += step_r;
                            c_ += step_c;
                            if (c_ >= cpr) {
                                c_ -= cpr;
                                ++r_;
                            }
                        };
                        int it = 0;
                        for (; it + 4 <= cpr; it += 4) {
                            int r0 = rr, c0 = cc, r1 = r0, c1 = c0;
                            advance(r1, c1);
                            int r2 = r1, c2 = c1;
                            advance(r2, c2);
                            int r3 = r2, c3 = c2;
                            advance(r3, c3);
                            rr = r3; cc = c3;
                            advance(rr, cc);
                            const long long o0 = __shfl_sync(0xffffffffu, rowbyte, r0), o1 = __shfl_sync(0xffffffffu, rowbyte, r1);
                            const long long o2 = __shfl_sync(0xffffffffu, rowbyte, r2), o3 = __shfl_sync(0xffffffffu, rowbyte, r3);
                            const uint4 v0 = *reinterpret_cast<const uint4*>(wrows + r0 * pitch + c0 * 16);
                            const uint4 v1 = *reinterpret_cast<const uint4*>(wrows + r1 * pitch + c1 * 16);
                            const uint4 v2 = *reinterpret_cast<const uint4*>(wrows + r2 * pitch + c2 * 16);
                            const uint4 v3 = *reinterpret_cast<const uint4*>(wrows + r3 * pitch + c3 * 16);
                            if (o0 >= 0) *reinterpret_cast<uint4*>(outb + o0 + c0 * 16) = v0;
                            if (o1 >= 0) *reinterpret_cast<uint4*>(outb + o1 + c1 * 16) = v1;
                            if (o2 >= 0) *reinterpret_cast<uint4*>(outb + o2 + c2 * 16) = v2;
                            if (o3 >= 0) *reinterpret_cast<uint4*>(outb + o3 + c3 * 16) = v3;
                        }
                        for (; it < cpr; it += 2) {  // cpr is even
                            int r0 = rr, c0 = cc, r1 = r0, c1 = c0;
                            advance(r1, c1);
                            rr = r1; cc = c1;
                            advance(rr, cc);
                            const long long o0 = __shfl_sync(0xffffffffu, rowbyte, r0), o1 = __shfl_sync(0xffffffffu, rowbyte, r1);
                            const uint4 v0 = *reinterpret_cast<const uint4*>(wrows + r0 * pitch + c0 * 16);
                            const uint4 v1 = *reinterpret_cast<const uint4*>(wrows + r1 * pitch + c1 * 16);
                            if (o0 >= 0) *reinterpret_cast<uint4*>(outb + o0 + c0 * 16) = v0;
                            if (o1 >= 0) *reinterpret_cast<uint4*>(outb + o1 + c1 * 16) = v1;
                        }
                    }
                    __syncwarp();  // staged rows consumed before the next pass overwrites them
                }
            }
            if (++acc == nbuf) {
                acc = 0;
                acc_ph ^= 1u;
            }
        }
        // the staging rows must have been read before this CTA's shared memory is released; the writes themselves are
        // complete when the grid is (a kernel boundary orders them like any other store)
        if (store_pending && lane == 0) ptx::tma_store_wait_read<0>();
        if (STATS) {
            epi2_bar_sync();  // all eight warps' running sums are final
            // channel c of the layer sits in team (c % BN >= ncol_a) at index (c / BN) * (team's columns) + its column there
            float* dst = p.partials + (size_t)blockIdx.x * 2 * p.ldo;
            const int et = (warp >= 7 ? warp - 3 : warp - 2) * 32 + lane;  // 0..255
            const int ncb = p.BN - p.ncol_a;
            for (int e = et; e < 2 * p.ldo; e += 256) {
                const int which = e >= p.ldo ? 1 : 0, c = e - which * p.ldo;
                const int nt = c / p.BN, cc = c - nt * p.BN;
                const int tm = cc >= p.ncol_a ? 1 : 0;
                const int ld = p.n_tiles * (tm ? ncb : p.ncol_a);
                const float* base = wstat + (tm ? (size_t)8 * p.n_tiles * p.ncol_a : 0) + (size_t)which * ld + nt * (tm ? ncb : p.ncol_a) + (cc - (tm ? p.ncol_a : 0));
                const float v = ((base[0] + base[2 * ld]) + base[4 * ld]) + base[6 * ld];
                if (p.acc.acc) chan_acc_add(p.acc, p.ldo, which, c, v);
                else dst[e] = v;
            }
        }
        if (sat) atomicAdd(p.status + ST_SAT, sat);
    }
    ptx::tc_fence_before();
    if (CG2) ptx::cluster_sync_all(); else __syncthreads();  // pairs: neither CTA may leave while the other still uses its memory
    if (warp == 1) {
        ptx::tc_fence_after();
        if (CG2) ptx::tmem_dealloc_cg2(tmem_base, (uint32_t)p.tmem_cols); else ptx::tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}



}  // namespace nbcbs
#include "tc_wgrad.cuh"
namespace nbcbs {

// ------------------------------------------------------------------------------------------ host side
struct IgemmCfg {
    bool ok = false;
    int Ca = 0, rowsB = 0, ntaps = 0;
    int KC = 0, BN = 0, n_tiles = 0, m_tiles = 0, stages = 0, acc_stride = 0, tmem_cols = 0, grid = 0, kpb = 1, mh = 1, acc_bufs = 2, stage_cols = 0;
    bool cg2 = false;  // CTA pairs (tcgen05 cta_group::2)
    bool tail32 = false;  // the last k-block of every tap is 32 channels wide
    uint32_t a_stage = 0, b_stage = 0, a_sub = 0, b_sub = 0;
    size_t smem_bytes = 0;
    long long M = 0;
};

struct TcGemmSlot {  // one launch: configuration plus the tensor maps encoded for the pointers last seen
    IgemmCfg cfg;
    IgemmParams prm;
    const void* a_ptr = nullptr;
    const void* b_ptr = nullptr;
    const void* out_ptr = nullptr;
    long long out_ld = 0;  // row pitch the output maps were encoded with
};

struct TcPlan {
    bool fprop = false, dgrad = false, wgrad = false;
    bool f16 = false;  // operands and 16-bit outputs are IEEE fp16 instead of bf16 (same kernels, other instruction-descriptor formats)
    long long ld_x = 0;        // row pitch (elements) of the input activation when it is a channel slice of a wider tensor (0 = dense)
    int fprop_parts = 0;
    size_t wt_bytes = 0;
    size_t wgrad_partial_bytes = 0;
    int sm_count = 0;
    long long launches = 0;  // kernels launched through this record
    TcGemmSlot fp;
    bool infer = false;  // the forward configuration also runs with the fused per-channel epilogue (its own slot: own output maps)
    TcGemmSlot inf;
    TcGemmSlot dg;  // one launch covers all output-parity classes
    WtParams wtp;
    // wgrad
    WgradParams wg;
    int wg_grid = 0;
    size_t wg_smem = 0;
    const void* wg_a_ptr = nullptr;
    const void* wg_b_ptr = nullptr;
    // 3x3 stride-1 layers with an image width that is a multiple of 16: the row-tile form (tc_wgrad_rows_kernel)
    bool wgrad_rows = false;
    WgradRowsParams wr;
    int wr_grid = 0;
    size_t wr_smem = 0;
};

namespace tcdetail {

inline std::string& err() {
    static thread_local std::string e;
    return e;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
typedef CUresult (*EncodeIm2colFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*, const int*, const int*,
                                   cuuint32_t, cuuint32_t, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                   CUtensorMapFloatOOBfill);

struct DriverFns {
    EncodeTiledFn tiled = nullptr;
    EncodeIm2colFn im2col = nullptr;
    bool tried = false;
};
inline DriverFns& driver() {
    static DriverFns d;
    if (!d.tried) {
        d.tried = true;
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            d.tiled = reinterpret_cast<EncodeTiledFn>(f);
        f = nullptr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &f, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            d.im2col = reinterpret_cast<EncodeIm2colFn>(f);
    }
    return d;
}

inline CUtensorMapSwizzle tma_swizzle_for(int KC) {
    return KC == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : KC == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
}
inline uint32_t umma_swizzle_for(int KC) { return KC == 64 ? (uint32_t)ptx::kSwizzle128 : KC == 32 ? (uint32_t)ptx::kSwizzle64 : (uint32_t)ptx::kSwizzle32; }

constexpr size_t kMaxSmem = 232448;  // 227 KB opt-in limit per CTA

// Tile configuration for a GEMM with M rows, `rowsB` output channels, `ntaps` taps of `Ca` channels each.
// Measured on B200: a tcgen05.mma of 128 x N x 16 takes max(97, N/2) cycles, so N below 192 wastes the tensor pipe;
// TMA fills shared memory at roughly 100 cycles per box plus 1.4 (256-row boxes) to 2.3 (128-row boxes) cycles per
// 128-byte row; one barrier round trip of the single-thread producer / MMA loops costs a few hundred cycles.
// The tile is [128*mh x BN]: with mh = 2 two row blocks share every B stage (fewer rows fetched per flop).
// Columns of a [128 x BN] tile that the first epilogue team takes: half of them, rounded up to a multiple of 16.
inline int igemm_team_cols(int BN) { return (BN / 16 + 1) / 2 * 16; }
// Columns per staging pass: the team's columns in the fewest passes of at most 64, balanced.
inline int igemm_stage_cw(int BN) {
    const int nc = igemm_team_cols(BN), passes = (nc + 63) / 64;
    return ((nc + passes - 1) / passes + 15) / 16 * 16;
}
inline size_t igemm_fixed_smem(int BN, int ldo) {
    return 1024 /*alignment slack*/ + (size_t)2 * TC_BM * (igemm_stage_cw(BN) * 2 + 16) + (size_t)8 * ldo * 4 + 512;
}
inline IgemmCfg igemm_configure(long long M, int Ca, int rowsB, int ntaps, int ldo, int sm_count, int nclasses) {
    IgemmCfg c;
    c.Ca = Ca; c.rowsB = rowsB; c.ntaps = ntaps; c.M = M;
    if (Ca % 16 || rowsB % 16 || M < 1) return c;
    // 64-channel k-blocks in the 128-byte swizzle (the narrower swizzles make tcgen05.mma 1.6-2.1x slower per
    // instruction); when Ca is not a multiple of 64 the last k-block of every tap reads past the channel extent and
    // TMA fills A with zeros there (whatever finite filter values B holds at those positions are multiplied by zero).
    // When at most 32 channels are left for that last k-block it is fetched 32 channels wide in the 64-byte swizzle:
    // two slower MMAs instead of four, and half the bytes written to and read from shared memory.
    c.KC = 64;
    c.tail32 = Ca % 64 != 0 && Ca % 64 <= 32 && (getenv("NB_TC_TAIL") ? atoi(getenv("NB_TC_TAIL")) != 0 : true);
    const int kblocks = ntaps * ((Ca + c.KC - 1) / c.KC);
    const int force_bn = getenv("NB_TC_BN") ? atoi(getenv("NB_TC_BN")) : 0;
    const int force_kpb = getenv("NB_TC_KPB") ? atoi(getenv("NB_TC_KPB")) : 0;
    const int force_mh = getenv("NB_TC_MH") ? atoi(getenv("NB_TC_MH")) : 0;
    // Rules distilled from sweeps over the detector's layer shapes on B200: the widest N tile that divides the channel
    // count wins everywhere (fewer shared-memory bytes written and read per flop); pairing two 128-row blocks per tile
    // (mh = 2) pays only while two accumulator sets still fit in TMEM (N <= 128) and there are enough tiles for every SM;
    // a pipeline stage should hold about 450 tensor cycles of work.
    for (int bn = std::min(256, rowsB) / 16 * 16; bn >= 16 && !c.BN; bn -= 16) {
        if (rowsB % bn) continue;
        if (force_bn && bn != force_bn && rowsB % force_bn == 0) continue;
        const int acc_stride = bn <= 32 ? 32 : bn <= 64 ? 64 : bn <= 128 ? 128 : 256;
        // CTA pairs (one tcgen05.mma over 256 rows whose B tile is split between two CTAs): a pair's MMA of 256 x N x 16
        // runs at N/2 cycles even for small N where a single CTA's 128 x N x 16 never drops below 97, and each CTA reads
        // and writes only half of B in shared memory.  Measured per layer on B200: 3x3 layers with at least 96 reduction
        // channels gain 5-15 %; 1x1 layers (one k-block group per tile, epilogue-bound) lose 5-10 % to the extra
        // cluster synchronisation, as do 3x3 layers with one k-block per tap and the stride-2 data gradients (1-4 taps
        // per parity class) below 384 channels; 1x1 layers with 960 and more input channels gain 1.5-2 us again.
        const bool pair_pays = (ntaps > 1 && Ca >= 96 && (nclasses == 1 || Ca >= 384)) || (ntaps == 1 && Ca >= 960);
        const bool cg2 = bn % 32 == 0 && (getenv("NB_TC_CG2") ? atoi(getenv("NB_TC_CG2")) != 0 : pair_pays);
        int mh = 1;
        if (4 * acc_stride <= 512) {
            const long long rows_tile = 2LL * TC_BM * (cg2 ? 2 : 1);
            const long long tiles2 = ((M + rows_tile - 1) / rows_tile) * (rowsB / bn) * nclasses;
            if (tiles2 >= (cg2 ? sm_count / 2 : sm_count)) mh = 2;
        }
        if (force_mh && force_mh * acc_stride <= 512) mh = force_mh;
        const int acc_bufs = (2 * mh * acc_stride <= 512) ? 2 : 1;
        const uint32_t a_sub = (uint32_t)(TC_BM * mh * c.KC * 2);
        const uint32_t b_sub = (uint32_t)(((cg2 ? bn / 2 : bn) * c.KC * 2 + 1023) / 1024 * 1024);
        const size_t fixed = igemm_fixed_smem(bn, ldo);
        if (fixed + 2 * (size_t)(a_sub + b_sub) > kMaxSmem) continue;
        const double mma_kb = mh * 4.0 * std::max(97.0, bn / 2.0);  // tensor cycles per k-block
        int kpb = std::max(1, std::min(kblocks, (int)((450.0 + mma_kb - 1) / mma_kb)));
        if (force_kpb) kpb = std::min(kblocks, force_kpb);
        int stages = 0;
        for (;; --kpb) {
            stages = (int)std::min<size_t>(8, (kMaxSmem - fixed) / ((size_t)kpb * (a_sub + b_sub)));
            if (stages >= 3 || kpb == 1) break;
        }
        if (stages < 2) continue;
        c.BN = bn; c.kpb = kpb; c.stages = stages; c.a_sub = a_sub; c.b_sub = b_sub; c.mh = mh; c.acc_bufs = acc_bufs;
        c.acc_stride = acc_stride;
        c.cg2 = cg2;
        c.m_tiles = (int)((M + TC_BM * mh * (cg2 ? 2 : 1) - 1) / (TC_BM * mh * (cg2 ? 2 : 1)));
    }
    if (!c.BN) return c;
    c.n_tiles = rowsB / c.BN;
    c.stage_cols = igemm_team_cols(c.BN);
    c.tmem_cols = std::max(32, c.acc_bufs * c.mh * c.acc_stride);
    c.a_stage = c.a_sub * c.kpb;
    c.b_stage = c.b_sub * c.kpb;
    c.stages = std::max(2, std::min(c.stages, std::max(2, (kblocks + c.kpb - 1) / c.kpb)));
    c.smem_bytes = std::max<size_t>(igemm_fixed_smem(c.BN, ldo) + (size_t)c.stages * (c.a_stage + c.b_stage), 120 * 1024);  // > half an SM: one CTA per SM
    c.grid = (int)std::min<long long>((long long)c.m_tiles * c.n_tiles * nclasses, c.cg2 ? sm_count / 2 : sm_count);
    if (c.cg2) c.grid *= 2;  // two CTAs per pair
    c.ok = true;
    return c;
}

inline void fill_params(IgemmParams& P, const IgemmCfg& c) {
    P.M = c.M;
    P.Ca = c.Ca; P.KC = c.KC; P.kc_per_tap = (c.Ca + c.KC - 1) / c.KC;
    P.BN = c.BN; P.n_tiles = c.n_tiles; P.m_tiles = c.m_tiles;
    P.stages = c.stages; P.acc_stride = c.acc_stride; P.tmem_cols = c.tmem_cols;
    P.umma_swizzle = umma_swizzle_for(c.KC);
    P.sbo = (uint32_t)(8 * c.KC * 2);
    P.a_stage_bytes = c.a_stage; P.b_stage_bytes = c.b_stage;
    P.kpb = c.kpb; P.a_sub_bytes = c.a_sub; P.b_sub_bytes = c.b_sub;
    P.tail32 = c.tail32 ? 1 : 0;
    P.mh = c.mh; P.acc_bufs = c.acc_bufs; P.ncol_a = c.stage_cols; P.stage_cw = igemm_stage_cw(c.BN);
    if (getenv("NB_TC_VERBOSE"))
        fprintf(stderr, "[nb_cbs] igemm M=%lld Ca=%d rowsB=%d taps=%d: mh=%d cg2=%d tail32=%d BN=%d kpb=%d stages=%d accbufs=%d tiles=%dx%d grid=%d smem=%zu\n", c.M, c.Ca,
                c.rowsB, c.ntaps, c.mh, (int)c.cg2, (int)c.tail32, c.BN, c.kpb, c.stages, c.acc_bufs, c.m_tiles, c.n_tiles, c.grid, c.smem_bytes);
    P.idesc = ptx::make_idesc_bf16(c.cg2 ? 2 * TC_BM : TC_BM, c.BN, 0, 0);
}

// im2col map over a bf16 NHWC tensor [N][H][W][C]: traversal starts at (lo, lo), steps `ts`, and ends `up` short of the far edge.
// ld = pixel pitch in elements (0: dense, = C); channels past C read as zeros whatever lies behind them in memory.
inline bool encode_im2col(CUtensorMap* m, const void* base, int N, int H, int W, int C, int lo, int up, int ts, int KC, int pixels = TC_BM, long long ld = 0) {
    DriverFns& d = driver();
    if (!d.im2col) { err() = "cuTensorMapEncodeIm2col is not available from the driver"; return false; }
    const cuuint64_t pitch = (cuuint64_t)(ld ? ld : C);
    cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N};
    cuuint64_t strides[3] = {pitch * 2, (cuuint64_t)W * pitch * 2, (cuuint64_t)H * W * pitch * 2};
    int lower[2] = {lo, lo}, upper[2] = {up, up};
    cuuint32_t estr[4] = {1, (cuuint32_t)ts, (cuuint32_t)ts, 1};
    CUresult r = d.im2col(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, lower, upper, (cuuint32_t)KC, (cuuint32_t)pixels, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, tma_swizzle_for(KC), CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { err() = "cuTensorMapEncodeIm2col failed with code " + std::to_string((int)r); return false; }
    return true;
}

// tiled map over a bf16 matrix [rows][cols] (cols contiguous), box = KC columns x box_rows rows.
inline bool encode_tiled_2d(CUtensorMap* m, const void* base, long long rows, long long cols, int KC, int box_rows, long long ld = 0) {
    DriverFns& d = driver();
    if (!d.tiled) { err() = "cuTensorMapEncodeTiled is not available from the driver"; return false; }
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)(ld ? ld : cols) * 2};
    cuuint32_t box[2] = {(cuuint32_t)KC, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = d.tiled(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         tma_swizzle_for(KC), CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { err() = "cuTensorMapEncodeTiled failed with code " + std::to_string((int)r); return false; }
    return true;
}

// tiled map over a bf16 NHWC tensor [N][H][W][C] (pixel pitch ld elements, 0 = dense): box = KC channels x box_w columns of one row.
inline bool encode_tiled_nhwc(CUtensorMap* m, const void* base, int N, int H, int W, int C, int KC, int box_w, long long ld = 0) {
    DriverFns& d = driver();
    if (!d.tiled) { err() = "cuTensorMapEncodeTiled is not available from the driver"; return false; }
    const cuuint64_t pitch = (cuuint64_t)(ld ? ld : C);
    cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N};
    cuuint64_t strides[3] = {pitch * 2, (cuuint64_t)W * pitch * 2, (cuuint64_t)H * W * pitch * 2};
    cuuint32_t box[4] = {(cuuint32_t)KC, (cuuint32_t)box_w, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = d.tiled(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         tma_swizzle_for(KC), CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { err() = "cuTensorMapEncodeTiled (NHWC) failed with code " + std::to_string((int)r); return false; }
    return true;
}

// Tiled maps over the output matrix [rows][ldo] (16-bit elements) for the epilogue's TMA stores: one per distinct pass width.
// ld = row pitch in elements when the output is a channel slice of a wider tensor (0: dense); f16: the elements are IEEE
// fp16 (it matters only for reductions: a store moves bits).
inline bool encode_out_maps(IgemmParams& P, const IgemmCfg& c, void* out, long long rows, long long ld = 0, bool f16 = false) {
    DriverFns& d = driver();
    const int na = c.stage_cols, nb = c.BN - c.stage_cols, cw = P.stage_cw;
    const int cand[3] = {cw, na % cw, nb % cw};  // full passes, team 0's last pass, team 1's last pass
    int n = 0;
    P.out_w[0] = P.out_w[1] = P.out_w[2] = 0;
    for (int i = 0; i < 3; ++i) {
        const int wv = cand[i];
        if (wv == 0 || (n > 0 && P.out_w[0] == wv) || (n > 1 && P.out_w[1] == wv)) continue;
        cuuint64_t dims[2] = {(cuuint64_t)P.ldo, (cuuint64_t)rows};
        cuuint64_t strides[1] = {(cuuint64_t)(ld ? ld : P.ldo) * 2};
        cuuint32_t box[2] = {(cuuint32_t)wv, 32};
        cuuint32_t estr[2] = {1, 1};
        CUresult r = d.tiled(&P.tmOut[n], f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, out, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                             wv == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) { err() = "cuTensorMapEncodeTiled (output) failed with code " + std::to_string((int)r); return false; }
        P.out_w[n++] = wv;
    }
    return true;
}

// Raises the dynamic shared-memory limit of one kernel instantiation once per device.
template <typename OutT, bool STATS, bool CG2, int EPI, bool CLS4> inline bool igemm_allow_smem() {
    // the attribute belongs to the (function, device) pair: one bit per device ordinal that already has it
    static std::atomic<unsigned long long> attr_set{0};
    int dev = 0;
    cudaGetDevice(&dev);
    const unsigned long long bit = 1ull << (dev & 63);
    if (!(attr_set.load(std::memory_order_acquire) & bit)) {
        if (cudaFuncSetAttribute(tc_igemm_kernel<OutT, STATS, CG2, EPI, CLS4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem) != cudaSuccess) {
            err() = "cannot raise the dynamic shared memory limit of the implicit-GEMM kernel";
            return false;
        }
        attr_set.fetch_or(bit, std::memory_order_release);
    }
    return true;
}
template <typename OutT, bool STATS, bool CG2, int EPI = 0, bool CLS4 = false> inline nb_status launch_igemm_impl(const TcGemmSlot& s, cudaStream_t st) {
    if (!igemm_allow_smem<OutT, STATS, CG2, EPI, CLS4>()) return NB_ERR_CUDA;
    // (Measured: launching a kernel only after its predecessor has completed costs 3.4 us per launch: its prologue --
    // barrier set-up, TMEM allocation, tensor-map fetch -- no longer overlaps the predecessor's tail.)
    const cudaError_t e = launch_k(tc_igemm_kernel<OutT, STATS, CG2, EPI, CLS4>, dim3((unsigned)s.cfg.grid), dim3(IG_THREADS), s.cfg.smem_bytes, st, CG2 ? 2 : 1, s.prm);
    if (e != cudaSuccess) {
        err() = std::string("launch of tc_igemm_kernel failed: ") + cudaGetErrorString(e);
        return NB_ERR_CUDA;
    }
    return NB_OK;
}
template <typename OutT, bool STATS> inline nb_status launch_igemm(const TcGemmSlot& s, cudaStream_t st) {
    if constexpr (!STATS) {  // the data gradient: the only launch with four classes
        if (s.prm.nclasses == 4) return s.cfg.cg2 ? launch_igemm_impl<OutT, false, true, 0, true>(s, st) : launch_igemm_impl<OutT, false, false, 0, true>(s, st);
    }
    return s.cfg.cg2 ? launch_igemm_impl<OutT, STATS, true>(s, st) : launch_igemm_impl<OutT, STATS, false>(s, st);
}
}  // namespace tcdetail

inline const char* tc_last_error() { return tcdetail::err().c_str(); }

// Decide which convolutions of this shape run on the tensor-core kernels and size their scratch.
inline nb_status tc_plan_init_impl(TcPlan* tc, const Geom& g, bool enable, int sm_count);
inline nb_status tc_plan_init(TcPlan* tc, const Geom& g, bool enable, int sm_count, const cudaDeviceProp&, bool f16 = false) {
    const nb_status st = tc_plan_init_impl(tc, g, enable, sm_count);
    tc->f16 = f16;
    if (st == NB_OK && f16) {  // A and B formats of the instruction descriptors: bits 7 and 10 set = bf16, clear = f16
        const uint32_t fmt = (1u << 7) | (1u << 10);
        tc->fp.prm.idesc &= ~fmt;
        tc->inf.prm.idesc &= ~fmt;
        tc->dg.prm.idesc &= ~fmt;
        tc->wg.idesc &= ~fmt;
        tc->wr.idesc &= ~fmt;
    }
    return st;
}
inline nb_status tc_plan_init_impl(TcPlan* tc, const Geom& g, bool enable, int sm_count) {
    using namespace tcdetail;
    *tc = TcPlan();
    tc->sm_count = sm_count;
    if (!enable) return NB_OK;
    DriverFns& d = driver();
    if (!d.tiled || !d.im2col) return NB_OK;  // no TMA descriptors from this driver: stay on the CUDA-core kernels
    const bool even = (g.h % 2 == 0) && (g.w % 2 == 0);
    // ---- fprop: A = x (im2col), B = w [Cout][k*k*Cin]
    if (g.c_in % 16 == 0 && g.c_out % 16 == 0) {
        const IgemmCfg c = igemm_configure(g.m, g.c_in, g.c_out, g.k * g.k, g.c_out, sm_count, 1);
        if (c.ok) {
            tc->fp.cfg = c;
            IgemmParams& P = tc->fp.prm;
            memset(&P, 0, sizeof P);
            fill_params(P, c);
            P.Hq = g.ho; P.Wq = g.wo; P.ts = g.stride; P.lo_w = -g.pad; P.lo_h = -g.pad;
            P.nclasses = 1; P.tiles_per_class = c.m_tiles * c.n_tiles;
            P.cls_ntaps[0] = g.k * g.k;
            for (int r = 0; r < g.k; ++r)
                for (int t = 0; t < g.k; ++t) {
                    P.off_h[0][r * g.k + t] = (uint16_t)r;
                    P.off_w[0][r * g.k + t] = (uint16_t)t;
                }
            P.ldo = g.c_out; P.Hout = g.ho; P.Wout = g.wo; P.os = 1;
            P.a_tiled = (g.k == 1 && g.stride == 1) ? 1 : 0;
            tc->fprop = true;
            tc->fprop_parts = c.grid;
            tc->inf = tc->fp;
            tc->infer = true;
        }
    }
    // ---- dgrad: A = dy (im2col), B = rearranged filter [Cin][taps*Cout]; stride 2 splits dx into four output-parity
    // classes, numbered heaviest (four taps) first; the order in which their tiles are visited is igemm_tile_class's
    if (g.c_in % 16 == 0 && g.c_out % 16 == 0 && (g.stride == 1 || (g.k == 3 && even))) {
        WtParams& W = tc->wtp;
        memset(&W, 0, sizeof W);
        W.c_in = g.c_in; W.c_out = g.c_out; W.k = g.k;
        IgemmParams& P = tc->dg.prm;
        memset(&P, 0, sizeof P);
        const int ncls = g.stride == 1 ? 1 : 4;
        size_t off = 0;
        int max_taps = 0;
        for (int cls = 0; cls < ncls; ++cls) {
            WtClass& C = W.cls[cls];
            C.offset = off;
            int nt = 0;
            if (g.stride == 1) {
                // dx[h][w] = sum_{r,t} dy[h+P-r][w+P-t] w[r][t]: window start runs from -(k-1-P), tap offset ro pairs with r = k-1-ro
                for (int ro = 0; ro < g.k; ++ro)
                    for (int to = 0; to < g.k; ++to) {
                        P.off_h[cls][nt] = (uint16_t)ro; P.off_w[cls][nt] = (uint16_t)to;
                        C.r[nt] = g.k - 1 - ro; C.t[nt] = g.k - 1 - to;
                        ++nt;
                    }
                P.cls_oa[cls] = 0; P.cls_ob[cls] = 0;
            } else {
                const int pa = 1 - cls / 2, pb = 1 - cls % 2;  // output row / column parity; class 0 = (odd, odd) = four taps
                // dx[2i+pa][2j+pb]: even rows see tap r=1 at dy row i; odd rows see r=0 at dy row i+1 and r=2 at dy row i
                int rs[2], ro[2], nr = 0, tsv[2], to[2], ntc = 0;
                if (pa == 0) { rs[0] = 1; ro[0] = 0; nr = 1; } else { rs[0] = 2; ro[0] = 0; rs[1] = 0; ro[1] = 1; nr = 2; }
                if (pb == 0) { tsv[0] = 1; to[0] = 0; ntc = 1; } else { tsv[0] = 2; to[0] = 0; tsv[1] = 0; to[1] = 1; ntc = 2; }
                for (int a = 0; a < nr; ++a)
                    for (int b = 0; b < ntc; ++b) {
                        P.off_h[cls][nt] = (uint16_t)ro[a]; P.off_w[cls][nt] = (uint16_t)to[b];
                        C.r[nt] = rs[a]; C.t[nt] = tsv[b];
                        ++nt;
                    }
                P.cls_oa[cls] = pa; P.cls_ob[cls] = pb;
            }
            C.ntaps = nt;
            P.cls_ntaps[cls] = nt;
            max_taps = std::max(max_taps, nt);
            off += (size_t)g.c_in * nt * g.c_out;
        }
        if (g.stride == 1) {
            P.Hq = g.h; P.Wq = g.w; P.ts = 1; P.lo_w = P.lo_h = -(g.k - 1 - g.pad);
            P.Hout = g.h; P.Wout = g.w; P.os = 1;
        } else {
            P.Hq = g.h / 2; P.Wq = g.w / 2; P.ts = 1; P.lo_w = P.lo_h = 0;
            P.Hout = g.h; P.Wout = g.w; P.os = 2;
        }
        const IgemmCfg c = igemm_configure((long long)g.n * P.Hq * P.Wq, g.c_out, g.c_in, max_taps, g.c_in, sm_count, ncls);
        if (c.ok) {
            tc->dg.cfg = c;
            fill_params(P, c);  // sets only the tiling fields; the geometry written above stays
            P.nclasses = ncls; P.tiles_per_class = c.m_tiles * c.n_tiles;
            P.cls_interleave = ncls == 4 ? 1 : 0;  // see igemm_tile_class
            P.ldo = g.c_in;
            W.nclasses = ncls;
            tc->wt_bytes = off * 2;
            tc->dgrad = true;
        }
    }
    // ---- wgrad: A = x (im2col, MN-major), B = dy (MN-major), reduction over pixels with split-K
    if (g.c_in % 16 == 0 && g.c_out % 16 == 0) {
        WgradParams& P = tc->wg;
        memset(&P, 0, sizeof P);
        P.M = g.m; P.Hq = g.ho; P.Wq = g.wo; P.ts = g.stride; P.lo_w = P.lo_h = -g.pad;
        P.c_in = g.c_in; P.c_out = g.c_out; P.kdim = g.kdim;
        for (int r = 0; r < g.k; ++r)
            for (int t = 0; t < g.k; ++t) {
                P.off_h[r * g.k + t] = (uint16_t)r;
                P.off_w[r * g.k + t] = (uint16_t)t;
            }
        P.cblk_per_tap = (g.c_in + 63) / 64;
        P.nblk_total = g.k * g.k * P.cblk_per_tap;
        P.m_tiles = (P.nblk_total + 1) / 2;
        double best = 1e30;
        for (int bn = 16; bn <= 256 && bn <= g.c_out; bn += 16) {
            if (g.c_out % bn) continue;
            const double cost = (double)(g.c_out / bn) * std::max(97.0, bn / 2.0);  // tensor cycles per K = 16 step
            if (cost < best - 1e-9 || (cost < best + 1e-9 && bn > P.BN)) {
                best = cost;
                P.BN = bn;
            }
        }
        P.n_tiles = g.c_out / P.BN;
        P.nblkB = (P.BN + 63) / 64;
        // One or two 128-row accumulator blocks per CTA.  With two, four x boxes share every dy stage (a third less
        // shared-memory traffic per MMA: measured 1.6x the time of a one-block stage for twice the work) but there are half
        // as many tiles, hence more split-K slices with fewer pixels each.  Both are planned and the cheaper one is kept;
        // cost = waves x (stage time x stages per CTA + a fixed prologue/epilogue), in units of a 128-pixel one-block stage.
        P.acc_stride = P.BN <= 32 ? 32 : P.BN <= 64 ? 64 : P.BN <= 128 ? 128 : 256;
        double best_cost = 1e30;
        WgradParams bestP = P;
        const int force_mh = getenv("NB_WG_MH") ? atoi(getenv("NB_WG_MH")) : 0;
        for (int mh = 1; mh <= 2; ++mh) {
            if (mh == 2 && (P.nblk_total < 4 || 2 * P.acc_stride > 512)) continue;
            if (force_mh && mh != force_mh && !(force_mh == 2 && (P.nblk_total < 4 || 2 * P.acc_stride > 512))) continue;
            WgradParams Q = P;
            Q.mh = mh;
            Q.m_tiles = (Q.nblk_total + 2 * mh - 1) / (2 * mh);
            // 128 pixels per stage when at least three stages fit, else 64
            Q.KP = getenv("NB_WG_KP") ? atoi(getenv("NB_WG_KP")) : 128;
            for (;;) {
                Q.blk_bytes = (uint32_t)(64 * 2 * Q.KP);
                Q.a_stage_bytes = 2 * mh * Q.blk_bytes;
                Q.b_stage_bytes = (uint32_t)Q.nblkB * Q.blk_bytes;
                Q.stages = (int)std::min<size_t>(8, (kMaxSmem - 2048) / (Q.a_stage_bytes + Q.b_stage_bytes));
                if (Q.stages >= 3 || Q.KP == 64 || getenv("NB_WG_KP")) break;
                Q.KP = 64;
            }
            if (Q.stages < 2) continue;
            Q.total_chunks = (int)((g.m + Q.KP - 1) / Q.KP);
            const int tiles = Q.m_tiles * Q.n_tiles;
            const double stage_time = (Q.KP / 128.0) * (mh == 2 ? 1.6 : 1.0), fixed = mh == 2 ? 10.0 : 6.0;
            int best_s = 1;
            double best_c = 1e30;
            const int max_s = std::max(1, std::min(64, Q.total_chunks / 4));
            for (int sp = 1; sp <= max_s; ++sp) {
                const double waves = (double)(((long long)tiles * sp + sm_count - 1) / sm_count);
                const double c = waves * (((Q.total_chunks + sp - 1) / sp) * stage_time + fixed) + 0.02 * sp;
                if (c < best_c - 1e-9) {
                    best_c = c;
                    best_s = sp;
                }
            }
            if (getenv("NB_WG_SPLITS")) best_s = std::max(1, std::min(max_s, atoi(getenv("NB_WG_SPLITS"))));
            Q.chunks_per_split = (Q.total_chunks + best_s - 1) / best_s;
            Q.splits = (Q.total_chunks + Q.chunks_per_split - 1) / Q.chunks_per_split;
            Q.stages = std::max(2, std::min(Q.stages, std::max(2, Q.chunks_per_split)));
            if (best_c < best_cost - 1e-9) {
                best_cost = best_c;
                bestP = Q;
            }
        }
        P = bestP;
        const int tiles = P.m_tiles * P.n_tiles;
        P.tmem_cols = P.mh * P.acc_stride;
        P.idesc = ptx::make_idesc_bf16(128, P.BN, 1, 1);
        tc->wg_smem = std::max<size_t>(2048 + (size_t)P.stages * (P.a_stage_bytes + P.b_stage_bytes), 120 * 1024);
        tc->wg_grid = tiles * P.splits;
        tc->wgrad_partial_bytes = P.splits > 1 ? (size_t)P.splits * g.c_out * g.kdim * 4 : 0;
        tc->wgrad = true;
        // the row-tile form: 3x3, stride 1, pad 1, image width a multiple of 16 (a stage is one output row: whole K = 16 steps)
        // (layers with more than 128 output columns per tile are not bound by x traffic in the other kernel: measured equal)
        const bool rows_wanted = getenv("NB_WG_ROWS") ? atoi(getenv("NB_WG_ROWS")) != 0 : P.acc_stride <= 128;
        if (g.k == 3 && g.stride == 1 && g.pad == 1 && g.w % 16 == 0 && g.w + 2 <= 256 && g.wo == g.w && g.ho == g.h && rows_wanted) {
            WgradRowsParams& R = tc->wr;
            memset(&R, 0, sizeof R);
            R.W = g.w; R.H = g.h; R.rows_total = g.n * g.h;
            R.c_in = g.c_in; R.c_out = g.c_out; R.kdim = g.kdim;
            R.cblk = (g.c_in + 63) / 64;
            R.ksteps = g.w / 16;
            R.blocks_total = 9 * R.cblk;
            R.BN = P.BN; R.n_tiles = P.n_tiles; R.nblkB = P.nblkB; R.acc_stride = P.acc_stride;
            const int max_acc = std::min(8, 512 / R.acc_stride);
            const int total_acc = (R.blocks_total + 1) / 2;
            R.m_tiles = (total_acc + max_acc - 1) / max_acc;
            const int acc_per_tile = (total_acc + R.m_tiles - 1) / R.m_tiles;
            R.blocks_per_tile = 2 * acc_per_tile;
            R.m_tiles = (R.blocks_total + R.blocks_per_tile - 1) / R.blocks_per_tile;
            int cols = acc_per_tile * R.acc_stride;
            R.tmem_cols = 32;
            while (R.tmem_cols < cols) R.tmem_cols *= 2;
            int max_boxes = 1;  // (r, channel block) boxes that a tile's blocks read
            for (int t = 0; t < R.m_tiles; ++t) {
                const int tb0 = t * R.blocks_per_tile, tb1 = std::min(R.blocks_total, tb0 + R.blocks_per_tile);
                max_boxes = std::max(max_boxes, (tb1 - 1) / 3 - tb0 / 3 + 1);
            }
            R.a_box_bytes = (uint32_t)((g.w + 2 + 7) / 8 * 8 * 128);
            R.b_box_bytes = (uint32_t)(g.w * 128);
            R.a_stage_bytes = (uint32_t)max_boxes * R.a_box_bytes;
            R.b_stage_bytes = (uint32_t)R.nblkB * R.b_box_bytes;
            R.stages = (int)std::min<size_t>(8, (kMaxSmem - 2048) / (R.a_stage_bytes + R.b_stage_bytes));
            const int tiles = R.m_tiles * R.n_tiles;
            int splits = std::max(1, sm_count / tiles);
            if (getenv("NB_WG_ROWS_SPLITS")) splits = std::max(1, atoi(getenv("NB_WG_ROWS_SPLITS")) / tiles);
            splits = std::min(splits, std::max(1, R.rows_total / 4));
            R.rows_per_split = (R.rows_total + splits - 1) / splits;
            R.splits = (R.rows_total + R.rows_per_split - 1) / R.rows_per_split;
            R.stages = std::max(2, std::min(R.stages, std::max(2, R.rows_per_split)));
            R.idesc = ptx::make_idesc_bf16(128, R.BN, 1, 1);
            if (R.stages >= 2 && (size_t)2 * (R.a_stage_bytes + R.b_stage_bytes) + 2048 <= kMaxSmem) {
                tc->wgrad_rows = true;
                tc->wr_smem = std::max<size_t>(2048 + (size_t)R.stages * (R.a_stage_bytes + R.b_stage_bytes), 120 * 1024);
                tc->wr_grid = tiles * R.splits;
                tc->wgrad_partial_bytes = std::max(tc->wgrad_partial_bytes, R.splits > 1 ? (size_t)R.splits * g.c_out * g.kdim * 4 : (size_t)0);
                if (getenv("NB_TC_VERBOSE"))
                    fprintf(stderr, "[nb_cbs] wgrad by rows W=%d Cin=%d Cout=%d: %d blocks, %d per tile (%d accumulators), tiles=%dx%d splits=%d (%d rows each) stages=%d smem=%zu\n",
                            g.w, g.c_in, g.c_out, R.blocks_total, R.blocks_per_tile, acc_per_tile, R.m_tiles, R.n_tiles, R.splits, R.rows_per_split, R.stages, tc->wr_smem);
            }
        }
        if (getenv("NB_TC_VERBOSE"))
            fprintf(stderr, "[nb_cbs] wgrad M=%lld Cin=%d Cout=%d k=%d: BN=%d mh=%d KP=%d stages=%d tiles=%dx%d splits=%d (chunks/split %d) grid=%d\n", (long long)g.m,
                    g.c_in, g.c_out, g.k, P.BN, P.mh, P.KP, P.stages, P.m_tiles, P.n_tiles, P.splits, P.chunks_per_split, tc->wg_grid);
    }
    return NB_OK;
}

// acc.acc != NULL: the kernel adds its channel sums to the fp64 accumulators; else it writes per-CTA partial sums.
inline nb_status tc_fprop(TcPlan* tc, const Geom& g, const void* x, const void* w, void* y, float* partials, int* status, cudaStream_t st,
                          const ChanAcc& acc) {
    using namespace tcdetail;
    TcGemmSlot& S = tc->fp;
    if (S.a_ptr != x || S.b_ptr != w) {
        const int up = g.pad - (g.k - 1);
        if (S.prm.a_tiled) {
            if (!encode_tiled_2d(&S.prm.tmA, x, g.m, g.c_in, S.cfg.KC, TC_BM * S.cfg.mh, tc->ld_x)) return NB_ERR_CUDA;
        } else if (!encode_im2col(&S.prm.tmA, x, g.n, g.h, g.w, g.c_in, -g.pad, up, g.stride, S.cfg.KC, TC_BM * S.cfg.mh, tc->ld_x)) {
            return NB_ERR_CUDA;
        }
        if (!encode_tiled_2d(&S.prm.tmB[0], w, g.c_out, (long long)g.kdim, S.cfg.KC, S.cfg.cg2 ? S.cfg.BN / 2 : S.cfg.BN)) return NB_ERR_CUDA;
        if (S.cfg.tail32) {
            if (S.prm.a_tiled) {
                if (!encode_tiled_2d(&S.prm.tmA_t, x, g.m, g.c_in, 32, TC_BM * S.cfg.mh, tc->ld_x)) return NB_ERR_CUDA;
            } else if (!encode_im2col(&S.prm.tmA_t, x, g.n, g.h, g.w, g.c_in, -g.pad, g.pad - (g.k - 1), g.stride, 32, TC_BM * S.cfg.mh, tc->ld_x)) {
                return NB_ERR_CUDA;
            }
            if (!encode_tiled_2d(&S.prm.tmB_t[0], w, g.c_out, (long long)g.kdim, 32, S.cfg.cg2 ? S.cfg.BN / 2 : S.cfg.BN)) return NB_ERR_CUDA;
        }
        S.a_ptr = x; S.b_ptr = w;
    }
    S.prm.tma_store = 1;
    if (S.out_ptr != y) {
        if (!encode_out_maps(S.prm, S.cfg, y, g.m)) return NB_ERR_CUDA;
        S.out_ptr = y;
    }
    S.prm.acc = acc;
    S.prm.out = y; S.prm.partials = partials; S.prm.status = status;
    tc->launches += 1;
    return launch_igemm<__half, true>(S, st);
}

// Forward convolution whose epilogue applies out = act(acc*scale_c + shift_c) and writes bf16: evaluation-mode BN
// (gamma, beta, running statistics) or a plain bias (gamma = rmean = rvar = NULL, beta = bias or NULL).
struct EpiAffine {
    const float *gamma, *beta, *rmean, *rvar;
    float eps;
    int act;  // 1: SiLU
};
inline nb_status tc_infer(TcPlan* tc, const Geom& g, const void* x, const void* w, void* out, const EpiAffine& e, int* status, cudaStream_t st) {
    using namespace tcdetail;
    TcGemmSlot& S = tc->inf;
    if (S.a_ptr != x || S.b_ptr != w) {
        if (S.prm.a_tiled) {
            if (!encode_tiled_2d(&S.prm.tmA, x, g.m, g.c_in, S.cfg.KC, TC_BM * S.cfg.mh)) return NB_ERR_CUDA;
        } else if (!encode_im2col(&S.prm.tmA, x, g.n, g.h, g.w, g.c_in, -g.pad, g.pad - (g.k - 1), g.stride, S.cfg.KC, TC_BM * S.cfg.mh)) {
            return NB_ERR_CUDA;
        }
        if (!encode_tiled_2d(&S.prm.tmB[0], w, g.c_out, (long long)g.kdim, S.cfg.KC, S.cfg.cg2 ? S.cfg.BN / 2 : S.cfg.BN)) return NB_ERR_CUDA;
        if (S.cfg.tail32) {
            if (S.prm.a_tiled) {
                if (!encode_tiled_2d(&S.prm.tmA_t, x, g.m, g.c_in, 32, TC_BM * S.cfg.mh, 0)) return NB_ERR_CUDA;
            } else if (!encode_im2col(&S.prm.tmA_t, x, g.n, g.h, g.w, g.c_in, -g.pad, g.pad - (g.k - 1), g.stride, 32, TC_BM * S.cfg.mh, 0)) {
                return NB_ERR_CUDA;
            }
            if (!encode_tiled_2d(&S.prm.tmB_t[0], w, g.c_out, (long long)g.kdim, 32, S.cfg.cg2 ? S.cfg.BN / 2 : S.cfg.BN)) return NB_ERR_CUDA;
        }
        S.a_ptr = x; S.b_ptr = w;
    }
    S.prm.tma_store = 1;  // the fused epilogue exists only on the TMA-store path
    if (S.out_ptr != out) {
        if (!encode_out_maps(S.prm, S.cfg, out, g.m)) return NB_ERR_CUDA;
        S.out_ptr = out;
    }
    S.prm.acc = ChanAcc{nullptr, nullptr, 1};
    S.prm.fin_gamma = e.gamma; S.prm.fin_beta = e.beta;
    S.prm.fin_rmean = e.rmean; S.prm.fin_rvar = e.rvar;
    S.prm.fin_eps = e.eps; S.prm.epi_act = e.act;
    S.prm.out = out; S.prm.partials = nullptr; S.prm.status = status;
    tc->launches += 1;
    if (tc->f16) return S.cfg.cg2 ? launch_igemm_impl<__half, false, true, 1>(S, st) : launch_igemm_impl<__half, false, false, 1>(S, st);
    return S.cfg.cg2 ? launch_igemm_impl<__nv_bfloat16, false, true, 1>(S, st) : launch_igemm_impl<__nv_bfloat16, false, false, 1>(S, st);
}

// `wt_ready`: the rearranged filter was already written by an earlier kernel of this call (the BN backward finalize kernel
// carries that work in extra blocks, where it costs nothing: the GPU is almost empty while the finalize chain runs).
// ld_dx / accumulate (stride-1 layers only, whose epilogue goes through TMA): dx is a channel slice with row pitch ld_dx
// elements (0: dense) and the result is added to what it holds instead of overwriting it.
inline nb_status tc_dgrad(TcPlan* tc, const Geom& g, const void* dy, const void* w, void* dx, void* wt, int* status, cudaStream_t st, bool wt_ready,
                          long long ld_dx = 0, bool accumulate = false) {
    using namespace tcdetail;
    if (!wt_ready) {
        const size_t total = tc->wt_bytes / 2;
        const int blocks = (int)std::min<size_t>((total + 255) / 256, (size_t)tc->sm_count * 8);
        launch_k(dgrad_weight_transform_kernel, dim3(blocks), dim3(256), 0, st, 1, static_cast<const __nv_bfloat16*>(w), static_cast<__nv_bfloat16*>(wt), tc->wtp);
        if (cudaGetLastError() != cudaSuccess) { err() = "launch of dgrad_weight_transform_kernel failed"; return NB_ERR_CUDA; }
        tc->launches += 1;
    }
    TcGemmSlot& S = tc->dg;
    if (S.a_ptr != dy || S.b_ptr != wt) {
        // stride 1: window start runs over [-(k-1-P), W-1-(k-1-P)], i.e. W positions; stride-2 classes: over [0, Wo-1]
        const int lo = g.stride == 1 ? -(g.k - 1 - g.pad) : 0;
        if (!encode_im2col(&S.prm.tmA, dy, g.n, g.ho, g.wo, g.c_out, lo, lo, 1, S.cfg.KC, TC_BM * S.cfg.mh)) return NB_ERR_CUDA;
        if (S.cfg.tail32 && !encode_im2col(&S.prm.tmA_t, dy, g.n, g.ho, g.wo, g.c_out, lo, lo, 1, 32, TC_BM * S.cfg.mh)) return NB_ERR_CUDA;
        for (int cls = 0; cls < tc->wtp.nclasses; ++cls) {
            const __nv_bfloat16* wcls = static_cast<const __nv_bfloat16*>(wt) + tc->wtp.cls[cls].offset;
            if (!encode_tiled_2d(&S.prm.tmB[cls], wcls, g.c_in, (long long)tc->wtp.cls[cls].ntaps * g.c_out, S.cfg.KC, S.cfg.cg2 ? S.cfg.BN / 2 : S.cfg.BN)) return NB_ERR_CUDA;
            if (S.cfg.tail32 && !encode_tiled_2d(&S.prm.tmB_t[cls], wcls, g.c_in, (long long)tc->wtp.cls[cls].ntaps * g.c_out, 32, S.cfg.cg2 ? S.cfg.BN / 2 : S.cfg.BN))
                return NB_ERR_CUDA;
        }
        S.a_ptr = dy; S.b_ptr = wt;
    }
    S.prm.tma_store = g.stride == 1 ? 1 : 0;  // the parity classes of a stride-2 layer write every other output pixel
    if (!S.prm.tma_store && (ld_dx || accumulate)) {
        err() = "a pitched or accumulating data gradient needs the TMA-store epilogue (stride-1 layers)";
        return NB_ERR_UNSUPPORTED;
    }
    if (S.prm.tma_store && (S.out_ptr != dx || S.out_ld != ld_dx)) {
        if (!encode_out_maps(S.prm, S.cfg, dx, (long long)g.n * g.h * g.w, ld_dx, tc->f16)) return NB_ERR_CUDA;
        S.out_ptr = dx;
        S.out_ld = ld_dx;
    }
    S.prm.out_accumulate = accumulate ? 1 : 0;
    S.prm.out = dx; S.prm.partials = nullptr; S.prm.status = status;
    nb_status r = tc->f16 ? launch_igemm<__half, false>(S, st) : launch_igemm<__nv_bfloat16, false>(S, st);
    if (r != NB_OK) return r;
    tc->launches += 1;
    return NB_OK;
}

inline nb_status tc_wgrad(TcPlan* tc, const Geom& g, const void* x, const void* dy, float* dw, float* partial, int* status, cudaStream_t st) {
    using namespace tcdetail;
    if (tc->wgrad_rows) {
        WgradRowsParams& R = tc->wr;
        if (tc->wg_a_ptr != x || tc->wg_b_ptr != dy) {
            if (!encode_tiled_nhwc(&R.tmA, x, g.n, g.h, g.w, g.c_in, 64, g.w + 2, tc->ld_x)) return NB_ERR_CUDA;
            if (!encode_tiled_2d(&R.tmB, dy, g.m, g.c_out, 64, g.w)) return NB_ERR_CUDA;
            tc->wg_a_ptr = x; tc->wg_b_ptr = dy;
        }
        R.out = R.splits > 1 ? partial : dw;
        R.status = status;
        static std::atomic<unsigned long long> rows_attr_set{0};  // one bit per device ordinal (see launch_igemm_impl)
        int dev = 0;
        cudaGetDevice(&dev);
        const unsigned long long bit = 1ull << (dev & 63);
        if (!(rows_attr_set.load(std::memory_order_acquire) & bit)) {
            if (cudaFuncSetAttribute(tc_wgrad_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem) != cudaSuccess) {
                err() = "cannot raise the dynamic shared memory limit of the row-tile wgrad kernel";
                return NB_ERR_CUDA;
            }
            rows_attr_set.fetch_or(bit, std::memory_order_release);
        }
        launch_k(tc_wgrad_rows_kernel, dim3(tc->wr_grid), dim3(TC_THREADS), tc->wr_smem, st, 1, R);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) { err() = std::string("launch of tc_wgrad_rows_kernel failed: ") + cudaGetErrorString(e); return NB_ERR_CUDA; }
        tc->launches += 1;
        if (R.splits > 1) {
            const size_t elems = (size_t)g.c_out * g.kdim;
            static const int tall_from = getenv("NB_WG_TALL") ? atoi(getenv("NB_WG_TALL")) : 96;
            if (R.splits >= tall_from) {  // many slices: 32 threads share an element's slices (same fp64 sum, fixed order)
                launch_k(splitk_reduce_tall_kernel, dim3((unsigned)((elems + 31) / 32)), dim3(1024), 0, st, 1, partial, R.splits, elems, dw);
            } else {
                const int blocks = (int)std::min<size_t>((elems / 4 + 127) / 128 + 1, (size_t)tc->sm_count * 8);
                launch_k(splitk_reduce_kernel, dim3(blocks), dim3(128), 0, st, 1, partial, R.splits, elems, dw);
            }
            if (cudaGetLastError() != cudaSuccess) { err() = "launch of splitk_reduce_kernel failed"; return NB_ERR_CUDA; }
            tc->launches += 1;
        }
        return NB_OK;
    }
    WgradParams& P = tc->wg;
    if (tc->wg_a_ptr != x || tc->wg_b_ptr != dy) {
        const int up = g.pad - (g.k - 1);
        if (!encode_im2col(&P.tmA, x, g.n, g.h, g.w, g.c_in, -g.pad, up, g.stride, 64, P.KP, tc->ld_x)) return NB_ERR_CUDA;
        if (!encode_tiled_2d(&P.tmB, dy, g.m, g.c_out, 64, P.KP)) return NB_ERR_CUDA;
        tc->wg_a_ptr = x; tc->wg_b_ptr = dy;
    }
    P.out = P.splits > 1 ? partial : dw;
    P.status = status;
    static std::atomic<unsigned long long> attr_set{0};  // one bit per device ordinal (see launch_igemm_impl)
    int dev = 0;
    cudaGetDevice(&dev);
    const unsigned long long bit = 1ull << (dev & 63);
    if (!(attr_set.load(std::memory_order_acquire) & bit)) {
        if (cudaFuncSetAttribute(tc_wgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem) != cudaSuccess) {
            err() = "cannot raise the dynamic shared memory limit of the wgrad kernel";
            return NB_ERR_CUDA;
        }
        attr_set.fetch_or(bit, std::memory_order_release);
    }
    launch_k(tc_wgrad_kernel, dim3(tc->wg_grid), dim3(TC_THREADS), tc->wg_smem, st, 1, P);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { err() = std::string("launch of tc_wgrad_kernel failed: ") + cudaGetErrorString(e); return NB_ERR_CUDA; }
    tc->launches += 1;
    if (P.splits > 1) {
        const size_t elems = (size_t)g.c_out * g.kdim;
        const int blocks = (int)std::min<size_t>((elems / 4 + 127) / 128 + 1, (size_t)tc->sm_count * 8);
        launch_k(splitk_reduce_kernel, dim3(blocks), dim3(128), 0, st, 1, partial, P.splits, elems, dw);
        if (cudaGetLastError() != cudaSuccess) { err() = "launch of splitk_reduce_kernel failed"; return NB_ERR_CUDA; }
        tc->launches += 1;
    }
    return NB_OK;
}

}  // namespace nbcbs
