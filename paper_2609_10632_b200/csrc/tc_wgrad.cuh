// Tensor-core weight gradient for sm_100a.  dw[c'][tap][c] = sum over pixels of dy[pixel][c'] * x_tap[pixel][c] is a
// GEMM whose reduction index is the pixel.  Both operands are channel-contiguous, so both are fed to tcgen05.mma
// as MN-major shared-memory tiles: A = im2col boxes of x (rows of the accumulator = positions in the flattened
// (tap, c) axis of the filter, taken in blocks of KCA channels), B = boxes of dy (columns = output channels).
// Each CTA owns one [128 x BN] tile of dw for one slice of the pixel range (split-K); slices are summed in a fixed
// order by a second kernel, so the result is bitwise reproducible.
// Included by tc_conv.cuh (uses its bounded-wait helpers).
#pragma once

namespace nbcbs {

struct WgradParams {
    CUtensorMap tmA;  // im2col map over x [N][H][W][Cin], KCA channels x KP pixels per load
    CUtensorMap tmB;  // tiled map over dy [M][Cout], KCB channels x KP pixels per load
    long long M;      // pixels (reduction length)
    int Hq, Wq, ts, lo_w, lo_h;
    int c_in, c_out, kdim;
    int KCA, KCB, nblkA, nblkB;  // channel-block widths and blocks per tile (128/KCA, BN/KCB)
    int cblk_per_tap;            // c_in / KCA
    int BN, n_tiles, m_tiles;
    int splits, chunks_per_split, total_chunks;
    int stages, tmem_cols;
    uint32_t swzA, swzB, sboA, sboB, lboA, lboB, a_stage_bytes, b_stage_bytes, idesc;
    float* out;  // [splits][c_out][kdim] (or dw itself when splits == 1)
    int* status;
    uint16_t off_w[9], off_h[9];
};

constexpr int WG_KP = 64;  // pixels per pipeline stage (four K = 16 MMA steps)

__global__ void __launch_bounds__(WG_THREADS, 1) tc_wgrad_kernel(const __grid_constant__ WgradParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* sA = smem;
    uint8_t* sB = sA + (size_t)p.stages * p.a_stage_bytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(sB + (size_t)p.stages * p.b_stage_bytes);
    uint64_t* full = bars;
    uint64_t* empty = bars + p.stages;
    uint64_t* tfull = empty + p.stages;
    uint64_t* drain = tfull + 1;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // tile = (m_tile, n_tile, split), split fastest so that CTAs sharing a pixel range run together
    const int split = blockIdx.x % p.splits;
    const int tn = blockIdx.x / p.splits;
    const int n_tile = tn % p.n_tiles, m_tile = tn / p.n_tiles;
    const int chunk0 = split * p.chunks_per_split;
    const int chunk1 = min(p.total_chunks, chunk0 + p.chunks_per_split);
    const int nchunks = chunk1 - chunk0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            ptx::mbar_init(full + s, 1);
            ptx::mbar_init(empty + s, 1);
        }
        ptx::mbar_init(tfull, 1);
        ptx::mbar_init(drain, 1);
        *abort_flag = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 1) {
        ptx::tmem_alloc(tmem_slot, (uint32_t)p.tmem_cols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0 && nchunks > 0) {
            ptx::prefetch_tmap(&p.tmA);
            ptx::prefetch_tmap(&p.tmB);
            int s = 0, issued = 0;
            uint32_t ph = 0;
            bool ok = true;
            const uint32_t blkA = (uint32_t)(WG_KP * p.KCA * 2), blkB = (uint32_t)(WG_KP * p.KCB * 2);
            const uint32_t tx_bytes = (uint32_t)p.nblkA * blkA + (uint32_t)p.nblkB * blkB;
            for (int ch = chunk0; ch < chunk1; ++ch) {
                const long long m0 = (long long)ch * WG_KP;
                const int j0 = (int)(m0 % p.Wq);
                const long long t1 = m0 / p.Wq;
                const int i0 = (int)(t1 % p.Hq), n0 = (int)(t1 / p.Hq);
                const int cw = p.lo_w + j0 * p.ts, chh = p.lo_h + i0 * p.ts;
                if (!wait_bar(empty + s, ph ^ 1u, abort_flag, p.status, 11)) {
                    ok = false;
                    break;
                }
                ptx::mbar_expect_tx(full + s, tx_bytes);
                uint8_t* a = sA + (size_t)s * p.a_stage_bytes;
                for (int b = 0; b < p.nblkA; ++b) {
                    int fb = m_tile * p.nblkA + b;             // block index along the flattened (tap, c) axis
                    if (fb * p.KCA >= p.kdim) fb = 0;           // past the end of the filter: any valid block (rows are not stored)
                    const int tap = fb / p.cblk_per_tap, c0 = (fb - tap * p.cblk_per_tap) * p.KCA;
                    ptx::tma_load_im2col_4d(a + (size_t)b * blkA, &p.tmA, full + s, c0, cw, chh, n0, p.off_w[tap], p.off_h[tap]);
                }
                uint8_t* bb = sB + (size_t)s * p.b_stage_bytes;
                for (int b = 0; b < p.nblkB; ++b)
                    ptx::tma_load_2d(bb + (size_t)b * blkB, &p.tmB, full + s, n_tile * p.BN + b * p.KCB, (int)m0);
                ++issued;
                if (++s == p.stages) {
                    s = 0;
                    ph ^= 1u;
                }
            }
            if (!ok) {
                // Gave up: wait (bounded) for the loads still in flight so that nothing lands after the CTA has exited.
                const int back = issued < p.stages ? issued : p.stages;
                for (int b = 0; b < back; ++b) {
                    s = (s == 0) ? p.stages - 1 : s - 1;
                    if (s == p.stages - 1) ph ^= 1u;
                    for (int i = 0; i < 100000 && !ptx::mbar_try_wait(full + s, ph); ++i) {
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && nchunks > 0) {
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int ch = 0; ch < nchunks; ++ch) {
                if (!wait_bar(full + s, ph, abort_flag, p.status, 12)) {
                    ok = false;
                    break;
                }
                ptx::tc_fence_after();
                const uint64_t da = ptx::make_smem_desc(ptx::smem_u32(sA + (size_t)s * p.a_stage_bytes), p.lboA, p.sboA, p.swzA);
                const uint64_t db = ptx::make_smem_desc(ptx::smem_u32(sB + (size_t)s * p.b_stage_bytes), p.lboB, p.sboB, p.swzB);
                // one K = 16 step covers two 8-pixel row groups of every block
                const uint64_t stepA = (uint64_t)((2 * p.sboA) >> 4), stepB = (uint64_t)((2 * p.sboB) >> 4);
                for (int k = 0; k < WG_KP / 16; ++k) ptx::umma_f16(tmem_base, da + k * stepA, db + k * stepB, p.idesc, (ch | k) ? 1u : 0u);
                ptx::umma_commit(empty + s);
                if (++s == p.stages) {
                    s = 0;
                    ph ^= 1u;
                }
            }
            if (ok) {
                ptx::umma_commit(tfull);
            } else {
                // tfull is never signalled (the epilogue's bounded wait sees the abort flag); make sure the MMAs already
                // issued have retired before TMEM is released
                ptx::umma_commit(drain);
                for (int i = 0; i < 4000000 && !ptx::mbar_try_wait(drain, 0); ++i) {
                }
            }
        }
    } else {
        const int lane_group = warp & 3;
        const int row = lane_group * 32 + lane;
        const int kidx = m_tile * 128 + row;  // position along the flattened (tap, c) axis
        bool ok = true;
        if (nchunks > 0) ok = wait_bar(tfull, 0, abort_flag, p.status, 13);
        ok = epi_bar_and(ok);
        if (ok) {
            ptx::tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(lane_group * 32) << 16);
            float* dst = p.out + (size_t)split * p.c_out * p.kdim;
            for (int c0 = 0; c0 < p.BN; c0 += 16) {
                uint32_t r[16];
                if (nchunks > 0) {
                    ptx::tmem_ld_32x32b_x16(taddr + (uint32_t)c0, r);
                    ptx::tmem_ld_wait();
                } else {
#pragma unroll
                    for (int j = 0; j < 16; ++j) r[j] = 0u;
                }
                if (kidx < p.kdim) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) dst[(size_t)(n_tile * p.BN + c0 + j) * p.kdim + kidx] = __uint_as_float(r[j]);
                }
            }
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}

}  // namespace nbcbs
