// Tensor-core weight gradient for sm_100a.  dw[c'][tap][c] = sum over pixels of dy[pixel][c'] * x_tap[pixel][c] is a
// GEMM whose reduction index is the pixel.  Both operands are channel-contiguous, so both are fed to tcgen05.mma
// as MN-major shared-memory tiles in the 128-byte swizzle: A = im2col boxes of x, 64 channels of one filter tap by
// KP pixels each (two boxes give the 128 accumulator rows; channels past Cin are zero-filled by TMA and never
// stored), B = boxes of dy, 64 output channels by KP pixels (columns of the accumulator).
// Each CTA owns one [128 x BN] tile of dw for one slice of the pixel range (split-K); slices are summed in a fixed
// order by a second kernel, so the result is bitwise reproducible.
// Included by tc_conv.cuh (uses its bounded-wait helpers).
#pragma once

namespace nbcbs {

struct WgradParams {
    CUtensorMap tmA;  // im2col map over x [N][H][W][Cin], 64 channels x KP pixels per load
    CUtensorMap tmB;  // tiled map over dy [M][Cout], 64 channels x KP pixels per load
    long long M;      // pixels (reduction length)
    int Hq, Wq, ts, lo_w, lo_h;
    int c_in, c_out, kdim;
    int cblk_per_tap;  // ceil(c_in / 64): 64-channel blocks per tap along the accumulator rows
    int nblk_total;    // taps * cblk_per_tap
    int nblkB;         // ceil(BN / 64)
    int KP;            // pixels per pipeline stage (64 or 128)
    int mh;            // 128-row accumulator blocks per CTA (1 or 2): with 2, four x boxes share every dy stage
    int acc_stride;    // TMEM columns between the accumulator blocks
    int BN, n_tiles, m_tiles;
    int splits, chunks_per_split, total_chunks;
    int stages, tmem_cols;
    uint32_t a_stage_bytes, b_stage_bytes, blk_bytes, idesc;
    float* out;  // [splits][c_out][kdim] (or dw itself when splits == 1)
    int* status;
    uint16_t off_w[9], off_h[9];
};

__global__ void __launch_bounds__(TC_THREADS, 1) tc_wgrad_kernel(const __grid_constant__ WgradParams p) {
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

    pdl_launch_dependents();
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    // tile = (m_tile, n_tile, split), split fastest so that CTAs sharing a pixel range run together
    const int split = blockIdx.x % p.splits;
    const int tn = blockIdx.x / p.splits;
    const int n_tile = tn % p.n_tiles, m_tile = tn / p.n_tiles;
    const int chunk0 = split * p.chunks_per_split;
    const int chunk1 = min(p.total_chunks, chunk0 + p.chunks_per_split);
    const int nchunks = chunk1 - chunk0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            ptx::mbar_init(full + s, 2);  // the x producer and the dy producer each arrive once
            ptx::mbar_init(empty + s, 1);
        }
        ptx::mbar_init(tfull, 1);
        ptx::mbar_init(drain, 1);
        *abort_flag = 0;
        ptx::fence_mbar_init();
    }
    if (lane == 0 && (warp == 0 || warp == 6)) ptx::prefetch_tmap(warp == 0 ? &p.tmA : &p.tmB);  // before the wait for the predecessor
    if (warp == 1) {
        ptx::tmem_alloc(tmem_slot, (uint32_t)p.tmem_cols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();  // everything above touched only shared memory, TMEM and kernel parameters

    if (warp == 0 || warp == 6) {
        // ------------------------------------------------------------------ TMA producers: warp 0 feeds x, warp 6 feeds dy
        // the whole warp runs the loop converged; `leader` predicates the instructions that must be issued once
        const uint32_t leader = ptx::elect_one() ? 1u : 0u;
        if (nchunks > 0) {
            const bool isA = warp == 0;
            int s = 0, issued = 0;
            uint32_t ph = 0;
            bool ok = true;
            const int stages = p.stages, KP = p.KP, Wq = p.Wq, Hq = p.Hq, ts = p.ts;
            const uint32_t blk = p.blk_bytes;
            const uint32_t stage_bytes = isA ? p.a_stage_bytes : p.b_stage_bytes;
            const uint32_t base_u32 = ptx::smem_u32(isA ? sA : sB), full_u32 = ptx::smem_u32(full);
            const CUtensorMap* tm = isA ? &p.tmA : &p.tmB;
            const int nblkA = 2 * p.mh;
            const int nblk = isA ? nblkA : p.nblkB;
            // the 64-channel blocks of x this tile owns (a block past the end of the filter is replaced by block 0:
            // its accumulator rows are never stored)
            int c0v[4];
            uint16_t owv[4], ohv[4];
            for (int b = 0; b < 4; ++b) {
                int fb = m_tile * nblkA + b;
                if (b >= nblkA || fb >= p.nblk_total) fb = 0;
                const int tap = fb / p.cblk_per_tap;
                c0v[b] = (fb - tap * p.cblk_per_tap) * 64;
                owv[b] = p.off_w[tap];
                ohv[b] = p.off_h[tap];
            }
            const int bcol = n_tile * p.BN;
            for (int ch = chunk0; ch < chunk1; ++ch) {
                const int m0 = ch * KP;
                if (!wait_bar_fast(empty + s, ph ^ 1u, abort_flag, p.status, isA ? 11 : 15)) {
                    ok = false;
                    break;
                }
                const uint32_t bar = full_u32 + 8u * (uint32_t)s;
                ptx::mbar_expect_tx_u32_if(leader, bar, blk * (uint32_t)nblk);
                const uint32_t dst = base_u32 + (uint32_t)s * stage_bytes;
                if (isA) {
                    const int j0 = m0 % Wq, t1 = m0 / Wq;
                    const int i0 = t1 % Hq, n0 = t1 / Hq;
                    const int cw = p.lo_w + j0 * ts, chh = p.lo_h + i0 * ts;
#pragma unroll
                    for (int b = 0; b < 4; ++b)
                        if (b < nblkA) ptx::tma_load_im2col_4d_u32_if(leader, dst + (uint32_t)b * blk, tm, bar, c0v[b], cw, chh, n0, owv[b], ohv[b]);
                } else {
                    for (int b = 0; b < nblk; ++b) ptx::tma_load_2d_u32_if(leader, dst + (uint32_t)b * blk, tm, bar, bcol + b * 64, m0);
                }
                ++issued;
                if (++s == stages) {
                    s = 0;
                    ph ^= 1u;
                }
            }
            if (!ok) {
                // Gave up: wait (bounded) for the loads still in flight so that nothing lands after the CTA has exited.
                const int back = issued < stages ? issued : stages;
                for (int b = 0; b < back; ++b) {
                    s = (s == 0) ? stages - 1 : s - 1;
                    if (s == stages - 1) ph ^= 1u;
                    for (int i = 0; i < 100000 && !ptx::mbar_try_wait(full + s, ph); ++i) {
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (one thread)
        const uint32_t leader = ptx::elect_one() ? 1u : 0u;
        if (nchunks > 0) {
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            const int stages = p.stages, ksteps = p.KP / 16, mh = p.mh;
            const uint32_t idesc = p.idesc, acc_stride = (uint32_t)p.acc_stride;
            const uint64_t a_half16 = (uint64_t)((2 * p.blk_bytes) >> 4);  // the second pair of x blocks inside a stage
            // MN-major, 128-byte swizzle: 8 pixel rows of 128 bytes form one 1024-byte group (SBO); the next 64 channels
            // start one block later (LBO); a K = 16 step advances by two row groups.
            const uint64_t da0 = ptx::make_smem_desc(ptx::smem_u32(sA), p.blk_bytes, 1024, ptx::kSwizzle128);
            const uint64_t db0 = ptx::make_smem_desc(ptx::smem_u32(sB), p.blk_bytes, 1024, ptx::kSwizzle128);
            const uint64_t a_stage16 = (uint64_t)(p.a_stage_bytes >> 4), b_stage16 = (uint64_t)(p.b_stage_bytes >> 4);
            const uint32_t empty_u32 = ptx::smem_u32(empty);
            uint64_t da_s = da0, db_s = db0;
            uint32_t accumulate = 0;
            for (int ch = 0; ch < nchunks; ++ch) {
                if (!wait_bar_fast(full + s, ph, abort_flag, p.status, 12)) {
                    ok = false;
                    break;
                }
                ptx::tc_fence_after();
                uint64_t da = da_s, db = db_s;
#pragma unroll 4
                for (int k = 0; k < ksteps; ++k) {
                    ptx::umma_f16_if(leader, tmem_base, da, db, idesc, accumulate);
                    if (mh == 2) ptx::umma_f16_if(leader, tmem_base + acc_stride, da + a_half16, db, idesc, accumulate);
                    accumulate = 1u;
                    da += 128;  // 2048 bytes >> 4
                    db += 128;
                }
                ptx::umma_commit_u32_if(leader, empty_u32 + 8u * (uint32_t)s);
                da_s += a_stage16;
                db_s += b_stage16;
                if (++s == stages) {
                    s = 0;
                    ph ^= 1u;
                    da_s = da0;
                    db_s = db0;
                }
            }
            if (ok) {
                ptx::umma_commit_u32_if(leader, ptx::smem_u32(tfull));
            } else {
                // tfull is never signalled (the epilogue's bounded wait sees the abort flag); make sure the MMAs already
                // issued have retired before TMEM is released
                ptx::umma_commit_u32_if(leader, ptx::smem_u32(drain));
                for (int i = 0; i < 4000000 && !ptx::mbar_try_wait(drain, 0); ++i) {
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2-5)
        const int lane_group = warp & 3;
        const int row = lane_group * 32 + lane;
        bool ok = true;
        if (nchunks > 0 && lane == 0) ok = wait_bar(tfull, 0, abort_flag, p.status, 13);
        ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
        ok = epi_bar_and(ok);
        if (ok) ptx::tc_fence_after();
        for (int h = 0; ok && h < p.mh; ++h) {
            // accumulator row -> (tap, channel): rows come in blocks of 64 channels
            const int fb = (m_tile * p.mh + h) * 2 + (row >> 6);
            const int tap = fb / p.cblk_per_tap;
            const int c = (fb - tap * p.cblk_per_tap) * 64 + (row & 63);
            const bool valid = fb < p.nblk_total && c < p.c_in;
            const int kidx = tap * p.c_in + c;  // position inside dw[c'][:]
            const uint32_t taddr = tmem_base + ((uint32_t)(lane_group * 32) << 16) + (uint32_t)(h * p.acc_stride);
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
                if (valid) {
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

// ------------------------------------------------------------------------------------------------------------------
// Weight gradient of 3x3 stride-1 layers whose image width is a multiple of 16: one stage = one output image row.
// The kernel above is bound by the bytes that travel from L2 to the SM: every filter tap fetches its own im2col box of
// x, i.e. x travels nine times.  Here a stage fetches, per filter ROW r and 64-channel block, the input row p + r - 1
// with one zero column on either side (a tiled box that starts at column -1: TMA fills what lies outside the image with
// zeros), and the three taps of that filter row read it at three different start addresses: with MN-major operands the
// pixels are the K dimension, a tap's shift is a shift of the operand's start by whole 128-byte rows, which costs
// nothing (measured: same results, same MMA rate as an aligned start).  x travels three times instead of nine.
// Accumulator rows: the blocks (r, channel block, s) in that order, two per 128-row accumulator -- the second block's
// start is simply the descriptor's leading-dimension offset behind the first (128 bytes for the next tap of the same
// box).  A CTA owns blocks [b0, b1) (as many accumulators as TMEM holds) x BN columns for a range of image rows
// (split-K); the partial tiles are summed by splitk_reduce_kernel like the other kernel's.
struct WgradRowsParams {
    CUtensorMap tmA;  // tiled map over x [N][H][W][Cin]: box = 64 channels x (W + 2) columns of one row
    CUtensorMap tmB;  // tiled map over dy [M][Cout]: box = 64 channels x W pixels
    int W, H, rows_total;  // image width, height, N * H output rows
    int c_in, c_out, kdim, cblk;
    int ksteps;            // W / 16
    int blocks_total;      // 9 * cblk
    int blocks_per_tile;   // accumulator blocks of a CTA (even, except for the last tile)
    int m_tiles, n_tiles, BN, nblkB, acc_stride, tmem_cols;
    int splits, rows_per_split;
    int stages;
    uint32_t a_box_bytes, b_box_bytes, a_stage_bytes, b_stage_bytes, idesc;
    float* out;
    int* status;
};

__global__ void __launch_bounds__(TC_THREADS, 1) tc_wgrad_rows_kernel(const __grid_constant__ WgradRowsParams p) {
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

    pdl_launch_dependents();
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    // tile = (m_tile, n_tile, split), split fastest so that CTAs sharing a range of image rows run together
    const int split = blockIdx.x % p.splits;
    const int tn = blockIdx.x / p.splits;
    const int n_tile = tn % p.n_tiles, m_tile = tn / p.n_tiles;
    const int row0 = split * p.rows_per_split;
    const int row1 = min(p.rows_total, row0 + p.rows_per_split);
    const int nrows = row1 - row0;
    const int b0 = m_tile * p.blocks_per_tile, b1 = min(p.blocks_total, b0 + p.blocks_per_tile);  // this CTA's accumulator blocks
    const int box0 = b0 / 3, nboxes = (b1 - 1) / 3 - box0 + 1;                                    // the (r, channel block) boxes they read
    const int nacc = (b1 - b0 + 1) / 2;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            ptx::mbar_init(full + s, 2);  // the x producer and the dy producer each arrive once
            ptx::mbar_init(empty + s, 1);
        }
        ptx::mbar_init(tfull, 1);
        ptx::mbar_init(drain, 1);
        *abort_flag = 0;
        ptx::fence_mbar_init();
    }
    if (lane == 0 && (warp == 0 || warp == 6)) ptx::prefetch_tmap(warp == 0 ? &p.tmA : &p.tmB);  // before the wait for the predecessor
    if (warp == 1) {
        ptx::tmem_alloc(tmem_slot, (uint32_t)p.tmem_cols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();  // everything above touched only shared memory, TMEM and kernel parameters

    if (warp == 0 || warp == 6) {
        // ------------------------------------------------------------------ TMA producers: warp 0 feeds x, warp 6 feeds dy
        const uint32_t leader = ptx::elect_one() ? 1u : 0u;
        if (nrows > 0) {
            const bool isA = warp == 0;
            int s = 0, issued = 0;
            uint32_t ph = 0;
            bool ok = true;
            const int stages = p.stages, H = p.H, W = p.W, cblk = p.cblk;
            const uint32_t stage_bytes = isA ? p.a_stage_bytes : p.b_stage_bytes;
            const uint32_t base_u32 = ptx::smem_u32(isA ? sA : sB), full_u32 = ptx::smem_u32(full);
            const uint32_t tx = isA ? (uint32_t)nboxes * (uint32_t)((W + 2) * 128) : (uint32_t)p.nblkB * (uint32_t)(W * 128);
            const int bcol = n_tile * p.BN;
            int n = row0 / H, prow = row0 - n * H;  // image and output row of the stage
            for (int row = row0; row < row1; ++row) {
                if (!wait_bar_fast(empty + s, ph ^ 1u, abort_flag, p.status, isA ? 16 : 17)) {
                    ok = false;
                    break;
                }
                const uint32_t bar = full_u32 + 8u * (uint32_t)s;
                ptx::mbar_expect_tx_u32_if(leader, bar, tx);
                const uint32_t dst = base_u32 + (uint32_t)s * stage_bytes;
                if (isA) {
                    for (int j = 0; j < nboxes; ++j) {
                        const int box = box0 + j, r = box / cblk, cb = box - r * cblk;
                        ptx::tma_load_4d_u32_if(leader, dst + (uint32_t)j * p.a_box_bytes, &p.tmA, bar, cb * 64, -1, prow + r - 1, n);
                    }
                } else {
                    for (int b = 0; b < p.nblkB; ++b) ptx::tma_load_2d_u32_if(leader, dst + (uint32_t)b * p.b_box_bytes, &p.tmB, bar, bcol + b * 64, row * W);
                }
                ++issued;
                if (++prow == H) {
                    prow = 0;
                    ++n;
                }
                if (++s == stages) {
                    s = 0;
                    ph ^= 1u;
                }
            }
            if (!ok) {
                // Gave up: wait (bounded) for the loads still in flight so that nothing lands after the CTA has exited.
                const int back = issued < stages ? issued : stages;
                for (int b = 0; b < back; ++b) {
                    s = (s == 0) ? stages - 1 : s - 1;
                    if (s == stages - 1) ph ^= 1u;
                    for (int i = 0; i < 100000 && !ptx::mbar_try_wait(full + s, ph); ++i) {
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (one thread)
        const uint32_t leader = ptx::elect_one() ? 1u : 0u;
        if (nrows > 0) {
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            const int stages = p.stages, ksteps = p.ksteps;
            const uint32_t idesc = p.idesc, acc_stride = (uint32_t)p.acc_stride;
            // accumulator a = blocks b0 + 2a and b0 + 2a + 1: block b reads box b / 3 from row b % 3 on; the second block is
            // the "next 64 rows" of the same MN-major operand, one leading-dimension offset behind the first
            uint64_t da_acc[8];
#pragma unroll
            for (int a = 0; a < 8; ++a) {
                const int g0 = b0 + 2 * a, g1 = g0 + 1;
                const uint32_t at0 = (uint32_t)(g0 / 3 - box0) * p.a_box_bytes + (uint32_t)(g0 % 3) * 128u;
                const uint32_t at1 = (uint32_t)(g1 / 3 - box0) * p.a_box_bytes + (uint32_t)(g1 % 3) * 128u;
                const bool two = g1 < b1;
                da_acc[a] = a < nacc ? ptx::make_smem_desc(ptx::smem_u32(sA) + at0, two ? at1 - at0 : 128u, 1024, ptx::kSwizzle128) : 0ull;
            }
            const uint64_t db0 = ptx::make_smem_desc(ptx::smem_u32(sB), p.b_box_bytes, 1024, ptx::kSwizzle128);
            const uint64_t a_stage16 = (uint64_t)(p.a_stage_bytes >> 4), b_stage16 = (uint64_t)(p.b_stage_bytes >> 4);
            const uint32_t empty_u32 = ptx::smem_u32(empty);
            uint64_t a_off = 0, db_s = db0;
            uint32_t accumulate = 0;
            for (int row = 0; row < nrows; ++row) {
                if (!wait_bar_fast(full + s, ph, abort_flag, p.status, 18)) {
                    ok = false;
                    break;
                }
                ptx::tc_fence_after();
                uint64_t ka = a_off, db = db_s;
                for (int k = 0; k < ksteps; ++k) {
#pragma unroll
                    for (int a = 0; a < 8; ++a)
                        if (a < nacc) ptx::umma_f16_if(leader, tmem_base + (uint32_t)a * acc_stride, da_acc[a] + ka, db, idesc, accumulate);
                    accumulate = 1u;
                    ka += 128;  // 16 pixel rows of 128 bytes, >> 4
                    db += 128;
                }
                ptx::umma_commit_u32_if(leader, empty_u32 + 8u * (uint32_t)s);
                a_off += a_stage16;
                db_s += b_stage16;
                if (++s == stages) {
                    s = 0;
                    ph ^= 1u;
                    a_off = 0;
                    db_s = db0;
                }
            }
            if (ok) {
                ptx::umma_commit_u32_if(leader, ptx::smem_u32(tfull));
            } else {
                ptx::umma_commit_u32_if(leader, ptx::smem_u32(drain));
                for (int i = 0; i < 4000000 && !ptx::mbar_try_wait(drain, 0); ++i) {
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2-5)
        const int lane_group = warp & 3;
        const int row = lane_group * 32 + lane;
        bool ok = true;
        if (nrows > 0 && lane == 0) ok = wait_bar(tfull, 0, abort_flag, p.status, 19);
        ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
        ok = epi_bar_and(ok);
        if (ok) ptx::tc_fence_after();
        for (int a = 0; ok && a < nacc; ++a) {
            // accumulator row -> block (r, channel block, s) -> position inside dw[c'][:]
            const int gb = b0 + 2 * a + (row >> 6);
            const int box = gb / 3, sft = gb - box * 3, r = box / p.cblk, cb = box - r * p.cblk;
            const int c = cb * 64 + (row & 63);
            const bool valid = gb < b1 && c < p.c_in;
            const int kidx = (r * 3 + sft) * p.c_in + c;
            const uint32_t taddr = tmem_base + ((uint32_t)(lane_group * 32) << 16) + (uint32_t)(a * p.acc_stride);
            float* dst = p.out + (size_t)split * p.c_out * p.kdim;
            for (int c0 = 0; c0 < p.BN; c0 += 16) {
                uint32_t rr[16];
                if (nrows > 0) {
                    ptx::tmem_ld_32x32b_x16(taddr + (uint32_t)c0, rr);
                    ptx::tmem_ld_wait();
                } else {
#pragma unroll
                    for (int j = 0; j < 16; ++j) rr[j] = 0u;
                }
                if (valid) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) dst[(size_t)(n_tile * p.BN + c0 + j) * p.kdim + kidx] = __uint_as_float(rr[j]);
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
