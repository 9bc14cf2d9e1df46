// C ABI of the Conv -> BN(train) -> SiLU block library (see include/nb_cbs.h): plans, validation, workspace
// carving and kernel dispatch.  No device memory is allocated here except the plan's status block.
// (The optimiser step of include/nb_sgd.h lives in nb_sgd.cu, the glue calls of include/nb_glue.h in nb_glue.cu.)
#include "../../include/nb_cbs.h"

#include <algorithm>
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <type_traits>
#include <vector>

#include "common.cuh"
#include "elementwise.cuh"
#include "simt_conv.cuh"
#include "stem_conv.cuh"
#include "tc_conv.cuh"
#include "api_common.cuh"

using namespace nbcbs;
using namespace nbapi;

namespace nbapi {  // shared with the other translation units of the library (api_common.cuh)

thread_local std::string g_err;

nb_status fail(nb_status code, const char* fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    g_err = buf;
    return code;
}

std::atomic<unsigned long long> g_launches{0};  // kernels launched by this library in this process

}  // namespace nbapi

namespace {

enum Site { SITE_FPROP = 0, SITE_STATS, SITE_FINALIZE, SITE_APPLY, SITE_BWD_REDUCE, SITE_BWD_FINALIZE, SITE_BWD_DY,
            SITE_WTRANSFORM, SITE_DGRAD, SITE_WGRAD, SITE_SPLITK_REDUCE, SITE_INFER, SITE_EVAL_COEF, SITE_FOLD, SITE_COUNT };
const char* const kSiteNames[SITE_COUNT] = {"conv_fprop", "bn_stats", "bn_finalize", "bn_silu_apply", "bn_silu_bwd_reduce",
                                            "bn_bwd_finalize", "bn_silu_bwd_dy", "dgrad_weight_transform", "conv_dgrad",
                                            "conv_wgrad", "wgrad_splitk_reduce", "conv_infer_fused", "bn_eval_coef", "bn_fold"};

struct EwCfg {  // launch geometry of the [M][C] passes
    int vec, cgs, tpb;
    long long total_vecs;
    int blocks_reduce, blocks_map;  // stats / backward-reduce grids (they size the partial buffers) and apply / dy grids
    int blocks_stats, blocks_apply, blocks_dy;
};

}  // namespace

constexpr size_t kStatusBytes = 256;  // ST_WORDS ints, padded so that what follows in the same allocation is 256-byte aligned
static_assert(ST_WORDS * sizeof(int) <= kStatusBytes, "status block");

struct nb_cbs_plan_s {
    nb_cbs_desc desc;
    Geom g;
    int device;
    int sm_count;
    int* status;  // device, ST_WORDS ints
    EwCfg ew;
    int nparts;      // rows of the partial-sum buffers
    int wg_splits;   // split-K slices of the CUDA-core wgrad
    long long wg_chunk;
    TcPlan tc;       // tensor-core kernel choices (all disabled when unsupported or forced off)
    long long ld_a = 0, ld_g = 0;  // row pitch (elements) of a_out in the forward call and of g in the backward call (set by nb_cbs_plan_set_pitches; default c_out)
    const void* fwd_res = nullptr;  // residual added to the forward call's output (nb_cbs_plan_set_fwd_residual) and its row pitch
    long long ld_res = 0;
    void* bwd_gres = nullptr;       // tensor that the data-gradient call adds (or copies) its incoming gradient to (nb_cbs_plan_set_bwd_residual)
    long long ld_gres = 0;
    bool gres_add = true;
    long long ld_dx = 0;           // row pitch of dx in the data-gradient call and whether dx is added to (nb_cbs_plan_set_dx_target)
    bool dx_accumulate = false;
    bool pitched = false;
    // Channel sums go to fp64 accumulators that the consuming pass turns into coefficients itself (ChanAcc); off
    // (NB_CBS_FLAG_SEPARATE_FINALIZE, fp32 mode): per-block partial sums and separate finalize kernels.
    bool fuse_finalize = true;
    double* acc = nullptr;      // device: [acc_copies_f][2][C] forward sums, then [acc_copies_b][2][C] backward sums; zero between calls
    int acc_copies_f = 0, acc_copies_b = 0;
    bool stem = false;       // 3-channel 3x3 stride-2 first layer: dedicated direct kernels
    int stem_blocks = 0;     // blocks (= partial slices) of the stem wgrad kernel
    bool stem_wide = false;  // the stem forward kernel takes 320-pixel strips (wide images)
    int stem_fprop_blocks = 0;  // its grid (= its partial slices)
    int stem_wgrad_blocks = 0;  // grid (= partial slices) of the stem weight-gradient kernel (128-pixel strips on wide images)
    int stem_dgrad_blocks = 0;  // grid of the stem data-gradient kernel (at most one wave of five resident blocks per SM unless the bands alone are more)
    int stem_dgrad_rows = 0;    // output row pairs per block
    bool profiling = false;  // when set, every kernel site is bracketed by events and the call waits for it
    cudaEvent_t ev0 = nullptr, ev1 = nullptr;
    double prof_ms[SITE_COUNT] = {};
    long long prof_n[SITE_COUNT] = {};
    size_t fwd_bytes, bwd_bytes;
    size_t infer_bytes, off_iy;  // evaluation-mode forward: scale and shift at the forward offsets, then the convolution output when not fused
    // workspace offsets
    size_t off_scale, off_shift, off_fpart;                  // forward
    size_t off_coef, off_bpart, off_wt, off_wgpart;          // backward
};

namespace {

bool is_f32(const nb_cbs_plan_s* p) { return p->desc.mode == NB_MODE_F32_REF; }
bool is_f16(const nb_cbs_plan_s* p) { return p->desc.mode == NB_MODE_F16_TC; }
// Run an expression with AT = the plan's 16-bit activation type (bf16, or IEEE fp16 in NB_MODE_F16_TC).
#define NB_WITH_AT(p, ...) (is_f16(p) ? ([&]() { using AT = __half; return __VA_ARGS__; })() : ([&]() { using AT = __nv_bfloat16; return __VA_ARGS__; })())
// the evaluation-mode forward is one tensor-core kernel with the per-channel epilogue fused
bool infer_fused(const nb_cbs_plan_s* p) { return !is_f32(p) && (p->stem || p->tc.infer); }

nb_status check_ptr(const void* p, const char* name, bool nullable = false) {
    if (!p) return nullable ? NB_OK : fail(NB_ERR_INVALID_ARG, "%s is NULL", name);
    if (reinterpret_cast<uintptr_t>(p) & 15u) return fail(NB_ERR_ALIGNMENT, "%s is not 16-byte aligned", name);
    return NB_OK;
}
#define NB_CHECK_PTR(p, ...)                                   \
    do {                                                       \
        nb_status s__ = check_ptr((p), #p, ##__VA_ARGS__);     \
        if (s__ != NB_OK) return s__;                          \
    } while (0)


// Brackets one kernel site with events when the plan is in profiling mode (diagnostic; synchronises the stream).
struct SiteTimer {
    nb_cbs_plan_s* p;
    int site;
    cudaStream_t st;
    SiteTimer(nb_cbs_plan_s* plan, int s, cudaStream_t stream) : p(plan), site(s), st(stream) {
        if (p->profiling) cudaEventRecord(p->ev0, st);
    }
    ~SiteTimer() {
        if (!p->profiling) return;
        cudaEventRecord(p->ev1, st);
        float ms = 0.f;
        if (cudaEventSynchronize(p->ev1) == cudaSuccess && cudaEventElapsedTime(&ms, p->ev0, p->ev1) == cudaSuccess) {
            p->prof_ms[site] += ms;
            p->prof_n[site] += 1;
        }
    }
};


// ---------------------------------------------------------------- elementwise launch helpers
template <typename YT> nb_status run_stats_partial(nb_cbs_plan_s* p, const void* y, float* partials, cudaStream_t st) {
    const EwCfg& e = p->ew;
    SiteTimer tm(p, SITE_STATS, st);
    launch_k(bn_stats_partial_kernel<YT>, dim3(e.blocks_stats), dim3(e.tpb), (size_t)e.tpb * e.vec * sizeof(float), st, 1,
        static_cast<const YT*>(y), e.total_vecs, p->g.c_out, partials);
    return launch_ok("bn_stats_partial");
}

nb_status run_finalize(nb_cbs_plan_s* p, const float* partials, int nparts, const float* gamma, const float* beta, float* mean,
                       float* invstd, float* scale, float* shift, float* rmean, float* rvar, float* sum, float* sumsq,
                       cudaStream_t st) {
    const int C = p->g.c_out;
    SiteTimer tm(p, SITE_FINALIZE, st);
    launch_k(bn_finalize_kernel, dim3((C + 7) / 8), dim3(256), 0, st, 1, partials, nparts, C, (double)p->g.m, p->desc.eps, p->desc.momentum,
                                                              gamma, beta, mean, invstd, scale, shift, rmean, rvar, sum, sumsq);
    return launch_ok("bn_finalize");
}

// res != NULL (training forward with SiLU only): a = SiLU(...) + res, res with row pitch ld_res elements.
// fin != NULL (training forward with SiLU only): scale and shift are derived inside the kernel from the plan's forward accumulators.
template <typename YT, typename AT, bool FAST, bool ACT = true>
nb_status run_apply(nb_cbs_plan_s* p, const void* y, void* a, const float* scale, const float* shift, cudaStream_t st, long long ld_a = 0,
                    const void* res = nullptr, long long ld_res = 0, const FwdFin* fin = nullptr) {
    const EwCfg& e = p->ew;
    const int C = p->g.c_out;
    SiteTimer tm(p, SITE_APPLY, st);
    const ChanAcc none{nullptr, nullptr, 1};
    const FwdFin nofin{};
    auto go = [&](auto kernel, const ChanAcc& ca, const FwdFin& f, size_t smem) {
        launch_k(kernel, dim3(e.blocks_apply), dim3(e.tpb), smem, st, 1, static_cast<const YT*>(y), static_cast<AT*>(a), e.total_vecs, C, scale, shift,
                 ld_a ? ld_a : (long long)C, static_cast<const AT*>(res), ld_res ? ld_res : (long long)C, ca, f);
    };
    if constexpr (ACT) {
        if (fin) {
            const ChanAcc ca{p->acc, p->status + ST_READERS_FWD, p->acc_copies_f};
            const size_t smem = (size_t)2 * C * sizeof(float);
            if (res) go(bn_silu_apply_kernel<YT, AT, FAST, true, true, true, true>, ca, *fin, smem);
            else if (ld_a) go(bn_silu_apply_kernel<YT, AT, FAST, true, true, false, true>, ca, *fin, smem);
            else go(bn_silu_apply_kernel<YT, AT, FAST, true, false, false, true>, ca, *fin, smem);
            return launch_ok("bn_silu_apply (statistics from the accumulators)");
        }
        if (res) {
            go(bn_silu_apply_kernel<YT, AT, FAST, true, true, true>, none, nofin, 0);
            return launch_ok("bn_silu_apply (+ residual)");
        }
    }
    if (ld_a) go(bn_silu_apply_kernel<YT, AT, FAST, ACT, true>, none, nofin, 0);
    else go(bn_silu_apply_kernel<YT, AT, FAST, ACT, false>, none, nofin, 0);
    return launch_ok("bn_silu_apply");
}

template <typename YT, typename AT, bool FAST>
nb_status run_bwd_elementwise(nb_cbs_plan_s* p, const void* g, const void* y, const float* mean, const float* invstd,
                              const float* gamma, const float* beta, float* dgamma, float* dbeta, void* dy, float* partials,
                              float* coef, cudaStream_t st, const void* w = nullptr, void* wt = nullptr, const WtParams* wtp = nullptr) {
    const EwCfg& e = p->ew;
    const int C = p->g.c_out;
    const bool fuse = p->fuse_finalize && !std::is_same<YT, float>::value;
    WtParams none;
    if (!wtp) memset(&none, 0, sizeof none);
    const ChanAcc ca{fuse ? p->acc + (size_t)p->acc_copies_f * 2 * C : nullptr, p->status + ST_READERS_BWD, p->acc_copies_b};
    {
        // sums of dz and dz*y per channel (into the accumulators, or as per-block partial sums); the blocks also rearrange the dgrad filter
        SiteTimer tm(p, SITE_BWD_REDUCE, st);
        BwdFused fb;
        memset(&fb, 0, sizeof fb);
        fb.acc = ca;
        if (fuse) {
            fb.w = static_cast<const __nv_bfloat16*>(w); fb.wt = wtp ? static_cast<__nv_bfloat16*>(wt) : nullptr;
        }
        const size_t red_smem = (size_t)e.tpb * e.vec * sizeof(float);
        auto go = [&](auto kernel, long long ld) {
            launch_k(kernel, dim3(e.blocks_reduce), dim3(e.tpb), red_smem, st, 1, static_cast<const AT*>(g), static_cast<const YT*>(y), e.total_vecs, C, mean, invstd,
                     gamma, beta, partials, fb, wtp ? *wtp : none, ld);
        };
        if (p->ld_g) go(bn_silu_bwd_reduce_kernel<YT, AT, FAST, true>, p->ld_g);
        else go(bn_silu_bwd_reduce_kernel<YT, AT, FAST, false>, (long long)C);
        NB_LAUNCH_OK("bn_silu_bwd_reduce");
    }
    if (!fuse) {
        SiteTimer tm(p, SITE_BWD_FINALIZE, st);
        const int fin_blocks = (C + 7) / 8;
        int wt_blocks = 0;
        if (wtp) {
            const size_t total = (size_t)wtp->c_in * wtp->k * wtp->k * wtp->c_out;
            wt_blocks = (int)std::min<size_t>((total + 255) / 256, (size_t)p->sm_count * 8);
        }
        launch_k(bn_bwd_finalize_kernel, dim3(fin_blocks + wt_blocks), dim3(256), 0, st, 1, partials, e.blocks_reduce, C, (double)p->g.m, mean, invstd, gamma, beta,
                 dgamma, dbeta, coef, fin_blocks, static_cast<const __nv_bfloat16*>(w), static_cast<__nv_bfloat16*>(wt), wtp ? *wtp : none);
        NB_LAUNCH_OK("bn_bwd_finalize");
    }
    SiteTimer tm(p, SITE_BWD_DY, st);
    const BwdFin bf{1.0 / (double)p->g.m, mean, invstd, gamma, beta, dgamma, dbeta};
    auto go_dy = [&](auto kernel, size_t smem) {
        launch_k(kernel, dim3(e.blocks_dy), dim3(e.tpb), smem, st, 1, static_cast<const AT*>(g), static_cast<const YT*>(y), static_cast<AT*>(dy), e.total_vecs, C, coef,
                 p->ld_g ? p->ld_g : (long long)C, ca, bf, static_cast<AT*>(p->bwd_gres), p->ld_gres ? p->ld_gres : (long long)C, p->gres_add ? 1 : 0);
    };
    const size_t coef_smem = (size_t)4 * C * sizeof(float);
    if (fuse && p->bwd_gres) {  // (the setter admits this only on plans that take this path)
        if (p->ld_g) go_dy(bn_silu_bwd_dy_kernel<YT, AT, FAST, true, true, true>, coef_smem);
        else go_dy(bn_silu_bwd_dy_kernel<YT, AT, FAST, false, true, true>, coef_smem);
    } else if (fuse) {
        if (p->ld_g) go_dy(bn_silu_bwd_dy_kernel<YT, AT, FAST, true, true>, coef_smem);
        else go_dy(bn_silu_bwd_dy_kernel<YT, AT, FAST, false, true>, coef_smem);
    } else {
        if (p->ld_g) go_dy(bn_silu_bwd_dy_kernel<YT, AT, FAST, true, false>, 0);
        else go_dy(bn_silu_bwd_dy_kernel<YT, AT, FAST, false, false>, 0);
    }
    return launch_ok("bn_silu_bwd_dy");
}

// ---------------------------------------------------------------- CUDA-core convolutions
template <typename TIN, typename TOUT>
nb_status run_simt_fprop(nb_cbs_plan_s* p, const void* x, const void* w, void* y, cudaStream_t st) {
    FpropProblem<TIN, TIN> prob{static_cast<const TIN*>(x), static_cast<const TIN*>(w), p->g};
    dim3 grid((unsigned)((p->g.m + SIMT_BM - 1) / SIMT_BM), (unsigned)((p->g.c_out + SIMT_BN - 1) / SIMT_BN), 1);
    SiteTimer tm(p, SITE_FPROP, st);
    launch_k(simt_gemm_kernel<FpropProblem<TIN, TIN>, TOUT>, grid, dim3(256), 0, st, 1, prob, static_cast<TOUT*>(y), (long long)p->g.kdim);
    return launch_ok("simt fprop");
}

template <typename TIN>
nb_status run_simt_dgrad(nb_cbs_plan_s* p, const void* dy, const void* w, void* dx, cudaStream_t st) {
    DgradProblem<TIN, TIN> prob{static_cast<const TIN*>(dy), static_cast<const TIN*>(w), p->g};
    const long long I = (long long)p->g.n * p->g.h * p->g.w;
    dim3 grid((unsigned)((I + SIMT_BM - 1) / SIMT_BM), (unsigned)((p->g.c_in + SIMT_BN - 1) / SIMT_BN), 1);
    SiteTimer tm(p, SITE_DGRAD, st);
    launch_k(simt_gemm_kernel<DgradProblem<TIN, TIN>, TIN>, grid, dim3(256), 0, st, 1, prob, static_cast<TIN*>(dx), (long long)p->g.k * p->g.k * p->g.c_out);
    return launch_ok("simt dgrad");
}

template <typename TIN>
nb_status run_simt_wgrad(nb_cbs_plan_s* p, const void* x, const void* dy, float* dw, float* partial, cudaStream_t st) {
    WgradProblem<TIN, TIN> prob{static_cast<const TIN*>(dy), static_cast<const TIN*>(x), p->g};
    dim3 grid((unsigned)((p->g.c_out + SIMT_BM - 1) / SIMT_BM), (unsigned)((p->g.kdim + SIMT_BN - 1) / SIMT_BN), (unsigned)p->wg_splits);
    if (p->wg_splits == 1) {
        SiteTimer tm(p, SITE_WGRAD, st);
        launch_k(simt_gemm_kernel<WgradProblem<TIN, TIN>, float>, grid, dim3(256), 0, st, 1, prob, dw, p->g.m);
        return launch_ok("simt wgrad");
    }
    {
        SiteTimer tm(p, SITE_WGRAD, st);
        launch_k(simt_gemm_kernel<WgradProblem<TIN, TIN>, float>, grid, dim3(256), 0, st, 1, prob, partial, p->wg_chunk);
        NB_LAUNCH_OK("simt wgrad (split-K)");
    }
    const size_t elems = (size_t)p->g.c_out * p->g.kdim;
    SiteTimer tm(p, SITE_SPLITK_REDUCE, st);
    launch_k(splitk_reduce_kernel, dim3((unsigned)((elems + 255) / 256)), dim3(256), 0, st, 1, partial, p->wg_splits, elems, dw);
    return launch_ok("splitk_reduce");
}

}  // namespace

// ====================================================================================== exported functions
extern "C" {

uint32_t nb_abi_version(void) { return NB_CBS_ABI_VERSION; }

const char* nb_last_error(void) { return g_err.c_str(); }

nb_status nb_cbs_plan_create(const nb_cbs_desc* d, int device, nb_cbs_plan* out) {
    g_err.clear();
    if (!out) return fail(NB_ERR_INVALID_ARG, "out_plan is NULL");
    *out = nullptr;
    if (!d) return fail(NB_ERR_INVALID_ARG, "desc is NULL");
    if (d->struct_size != sizeof(nb_cbs_desc))
        return fail(NB_ERR_INVALID_ARG, "desc.struct_size is %u, this library expects %zu", d->struct_size, sizeof(nb_cbs_desc));
    if (d->n <= 0 || d->h <= 0 || d->w <= 0 || d->c_in <= 0 || d->c_out <= 0)
        return fail(NB_ERR_INVALID_ARG, "extents must be positive (n=%d h=%d w=%d c_in=%d c_out=%d)", d->n, d->h, d->w, d->c_in, d->c_out);
    if (d->ksize != 1 && d->ksize != 3) return fail(NB_ERR_INVALID_ARG, "ksize must be 1 or 3, got %d", d->ksize);
    if (d->stride != 1 && d->stride != 2) return fail(NB_ERR_INVALID_ARG, "stride must be 1 or 2, got %d", d->stride);
    if (d->mode != NB_MODE_BF16_TC && d->mode != NB_MODE_F32_REF && d->mode != NB_MODE_F16_TC) return fail(NB_ERR_INVALID_ARG, "unknown mode %d", d->mode);
    if (!(d->eps > 0.f)) return fail(NB_ERR_INVALID_ARG, "eps must be positive");
    if (!(d->momentum >= 0.f && d->momentum <= 1.f)) return fail(NB_ERR_INVALID_ARG, "momentum must be in [0,1]");
    const int vec = d->mode == NB_MODE_F32_REF ? 4 : 8;
    if (d->c_out % vec) return fail(NB_ERR_UNSUPPORTED, "c_out=%d must be a multiple of %d in this mode", d->c_out, vec);
    if (d->c_out / vec > 288) return fail(NB_ERR_UNSUPPORTED, "c_out=%d is too large (at most %d channels in this mode)", d->c_out, 288 * vec);

    Geom g;
    g.n = d->n; g.h = d->h; g.w = d->w; g.c_in = d->c_in; g.c_out = d->c_out; g.k = d->ksize; g.stride = d->stride;
    g.pad = d->ksize / 2;
    g.ho = (g.h + 2 * g.pad - g.k) / g.stride + 1;
    g.wo = (g.w + 2 * g.pad - g.k) / g.stride + 1;
    g.m = (long long)g.n * g.ho * g.wo;
    g.kdim = g.k * g.k * g.c_in;
    if (g.m < 2) return fail(NB_ERR_INVALID_ARG, "batch statistics need at least 2 rows (N*Ho*Wo=%lld)", g.m);
    if ((double)g.m * g.c_out >= 9.0e18 || (long long)g.n * g.h * g.w * g.c_in < 0)
        return fail(NB_ERR_UNSUPPORTED, "tensor too large");

    int count = 0;
    NB_CUDA_CHECK(cudaGetDeviceCount(&count));
    if (device < 0 || device >= count) return fail(NB_ERR_INVALID_ARG, "device %d out of range (%d devices)", device, count);
    cudaDeviceProp prop;
    NB_CUDA_CHECK(cudaGetDeviceProperties(&prop, device));
    if (prop.major != 10) return fail(NB_ERR_ARCH, "device %d is sm_%d%d; this library is built for sm_100a only", device, prop.major, prop.minor);

    nb_cbs_plan_s* p = new (std::nothrow) nb_cbs_plan_s();
    if (!p) return fail(NB_ERR_INTERNAL, "out of host memory");
    p->desc = *d;
    p->g = g;
    p->device = device;
    p->sm_count = prop.multiProcessorCount;
    p->fuse_finalize = !(d->flags & NB_CBS_FLAG_SEPARATE_FINALIZE) && d->mode != NB_MODE_F32_REF;

    EwCfg& e = p->ew;
    e.vec = vec;
    e.cgs = g.c_out / vec;
    const int R = e.cgs >= 256 ? 1 : 256 / e.cgs;
    e.tpb = e.cgs * R;
    e.total_vecs = g.m * e.cgs;
    const long long max_blocks = (e.total_vecs + e.tpb - 1) / e.tpb;
    // enough blocks to fill the machine, but at least ~8 (reductions) / ~4 (maps) vectors per thread so that the
    // per-thread parameter loads and the block epilogue are amortised on small tensors
    // Grids are one wave of resident blocks (occupancy queried per kernel), but never so many that a thread sees fewer
    // than ~8 (reductions) / ~4 (maps) vectors: the per-thread parameter loads and block epilogues must be amortised.
    {
        auto wave = [&](const void* fn, size_t dyn_smem, int min_vecs) {
            int occ = 0;
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, fn, e.tpb, dyn_smem) != cudaSuccess || occ < 1) {
                cudaGetLastError();
                occ = 1;
            }
            const long long cap = (long long)p->sm_count * occ;
            return (int)std::max<long long>(1, std::min<long long>((max_blocks + min_vecs - 1) / min_vecs, cap));
        };
        const size_t red_smem = (size_t)e.tpb * vec * sizeof(float);
        // the passes that derive their coefficients from the accumulators keep them in dynamic shared memory
        const size_t apply_smem = p->fuse_finalize ? (size_t)2 * g.c_out * sizeof(float) : 0, dy_smem = p->fuse_finalize ? (size_t)4 * g.c_out * sizeof(float) : 0;
        if (d->mode == NB_MODE_F32_REF) {
            e.blocks_stats = wave((const void*)bn_stats_partial_kernel<float>, red_smem, 8);
            e.blocks_reduce = wave((const void*)bn_silu_bwd_reduce_kernel<float, float, false>, red_smem, 8);
            e.blocks_apply = wave((const void*)bn_silu_apply_kernel<float, float, false>, 0, 4);
            e.blocks_dy = wave((const void*)bn_silu_bwd_dy_kernel<float, float, false>, 0, 4);
        } else if (d->mode == NB_MODE_F16_TC) {
            e.blocks_stats = wave((const void*)bn_stats_partial_kernel<__half>, red_smem, 8);
            e.blocks_reduce = wave((const void*)bn_silu_bwd_reduce_kernel<__half, __half, true>, red_smem, 8);
            e.blocks_apply = wave((const void*)bn_silu_apply_kernel<__half, __half, true, true, false, false, true>, apply_smem, 4);
            e.blocks_dy = wave((const void*)bn_silu_bwd_dy_kernel<__half, __half, true, false, true>, dy_smem, 4);
        } else {
            e.blocks_stats = wave((const void*)bn_stats_partial_kernel<__half>, red_smem, 8);
            e.blocks_reduce = wave((const void*)bn_silu_bwd_reduce_kernel<__half, __nv_bfloat16, true>, red_smem, 8);
            e.blocks_apply = wave((const void*)bn_silu_apply_kernel<__half, __nv_bfloat16, true, true, false, false, true>, apply_smem, 4);
            e.blocks_dy = wave((const void*)bn_silu_bwd_dy_kernel<__half, __nv_bfloat16, true, false, true>, dy_smem, 4);
        }
        e.blocks_map = std::max(e.blocks_apply, e.blocks_dy);
    }

    // CUDA-core wgrad split-K: enough slices to fill the machine, at least 512 rows each.
    {
        const long long tiles = (long long)((g.c_out + SIMT_BM - 1) / SIMT_BM) * ((g.kdim + SIMT_BN - 1) / SIMT_BN);
        long long splits = (4LL * p->sm_count + tiles - 1) / tiles;
        const long long max_splits = std::max<long long>(1, g.m / 512);
        splits = std::max<long long>(1, std::min(splits, max_splits));
        long long chunk = (g.m + splits - 1) / splits;
        chunk = (chunk + SIMT_BK - 1) / SIMT_BK * SIMT_BK;
        splits = (g.m + chunk - 1) / chunk;
        p->wg_splits = (int)splits;
        p->wg_chunk = chunk;
    }

    int cur = 0;
    NB_CUDA_CHECK(cudaGetDevice(&cur));
    cudaError_t ce = cudaSetDevice(device);
    // one allocation: the status words, then (256-byte aligned) the fp64 channel accumulators
    {
        auto copies = [](const char* name, int dflt) {
            const char* v = getenv(name);
            const int k = v ? atoi(v) : dflt;
            return k < 1 ? 1 : k > 16 ? 16 : k;
        };
        p->acc_copies_f = p->fuse_finalize ? copies("NB_ACC_COPIES_FWD", 2) : 0;
        p->acc_copies_b = p->fuse_finalize ? copies("NB_ACC_COPIES_BWD", 4) : 0;
    }
    const size_t acc_bytes = (size_t)(p->acc_copies_f + p->acc_copies_b) * 2 * g.c_out * sizeof(double);
    if (ce == cudaSuccess) ce = cudaMalloc(&p->status, kStatusBytes + acc_bytes);
    if (ce == cudaSuccess) ce = cudaMemset(p->status, 0, kStatusBytes + acc_bytes);
    if (ce == cudaSuccess && acc_bytes) p->acc = reinterpret_cast<double*>(reinterpret_cast<char*>(p->status) + kStatusBytes);
    nb_status tcs = NB_OK;
    if (ce == cudaSuccess)
        tcs = tc_plan_init(&p->tc, g, d->mode != NB_MODE_F32_REF && !(d->flags & NB_CBS_FLAG_FORCE_SIMT), p->sm_count, prop, d->mode == NB_MODE_F16_TC);
    cudaSetDevice(cur);
    if (ce != cudaSuccess || tcs != NB_OK) {
        if (p->status) cudaFree(p->status);
        delete p;
        if (tcs != NB_OK) return fail(tcs, "tensor-core plan setup failed: %s", tc_last_error());
        return fail(NB_ERR_CUDA, "status block allocation failed: %s", cudaGetErrorString(ce));
    }

    p->stem = d->mode != NB_MODE_F32_REF && !(d->flags & NB_CBS_FLAG_FORCE_SIMT) && g.c_in == 3 && g.k == 3 && g.stride == 2 &&
              g.c_out == 48 && g.h % 2 == 0 && g.w % 2 == 0 && g.m < (1LL << 31) && (long long)g.n * g.h * g.w * 3 < (1LL << 31);
    p->stem_blocks = (int)std::min<long long>(stem_num_strips(g), (long long)p->sm_count * 4);  // grid of the three first-layer kernels: one wave of four resident blocks per SM
    p->stem_dgrad_blocks = stem_dgrad_grid(g, p->sm_count * 5, &p->stem_dgrad_rows);
    p->stem_wide = g.wo >= STEM_TQ_WIDE / 2;  // (a strip of a narrower row would leave most of its tile slots empty)
    if (const char* e2 = getenv("NB_STEM_WIDE")) p->stem_wide = atoi(e2) != 0;
    p->stem_fprop_blocks = p->stem_wide ? (int)std::min<long long>(stem_num_strips(g, STEM_TQ_WIDE), (long long)p->sm_count * 4) : p->stem_blocks;
    p->stem_wgrad_blocks = p->stem_wide ? (int)std::min<long long>(stem_num_strips(g, STEM_TQ_WGRAD), (long long)p->sm_count * 4) : p->stem_blocks;
    if (p->stem && p->stem_wide) {  // (more than the 48 KB a kernel gets without asking)
        DeviceGuard on_device(p->device);
        cudaError_t ae = cudaFuncSetAttribute(stem_wgrad_mma_kernel<48, __nv_bfloat16, STEM_TQ_WGRAD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)stem_wgrad_smem_bytes<48, __nv_bfloat16, STEM_TQ_WGRAD>());
        if (ae == cudaSuccess)
            ae = cudaFuncSetAttribute(stem_wgrad_mma_kernel<48, __half, STEM_TQ_WGRAD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)stem_wgrad_smem_bytes<48, __half, STEM_TQ_WGRAD>());
        if (ae != cudaSuccess) {
            p->stem_wide = false;
            p->stem_fprop_blocks = p->stem_wgrad_blocks = p->stem_blocks;
            (void)cudaGetLastError();
        }
    }
    p->nparts = std::max(std::max(std::max(e.blocks_reduce, e.blocks_stats), p->tc.fprop_parts), p->stem ? p->stem_blocks : 0);
    const size_t C = (size_t)g.c_out;
    size_t off = 0;
    p->off_scale = off; off = align_up(off + C * 4, 256);
    p->off_shift = off; off = align_up(off + C * 4, 256);
    p->off_fpart = off; off = align_up(off + (size_t)p->nparts * 2 * C * 4, 256);
    p->fwd_bytes = off;
    p->off_iy = p->off_fpart;
    p->infer_bytes = infer_fused(p) ? p->off_fpart : align_up(p->off_iy + (size_t)g.m * C * (is_f32(p) ? 4 : 2), 256);
    off = 0;
    p->off_coef = off; off = align_up(off + 4 * C * 4, 256);
    p->off_bpart = off; off = align_up(off + (size_t)p->nparts * 2 * C * 4, 256);
    p->off_wt = off; off = align_up(off + p->tc.wt_bytes, 256);
    p->off_wgpart = off;
    {
        size_t simt = p->wg_splits > 1 ? (size_t)p->wg_splits * C * g.kdim * 4 : 0;
        size_t stem = p->stem ? (size_t)p->stem_blocks * C * g.kdim * 4 : 0;
        off = align_up(off + std::max(std::max(simt, stem), p->tc.wgrad_partial_bytes), 256);
    }
    p->bwd_bytes = off;
    *out = p;
    return NB_OK;
}

nb_status nb_cbs_plan_destroy(nb_cbs_plan p) {
    g_err.clear();
    if (!p) return NB_OK;
    if (p->status) {
        int cur = 0;
        cudaGetDevice(&cur);
        cudaSetDevice(p->device);
        cudaFree(p->status);
        if (p->ev0) cudaEventDestroy(p->ev0);
        if (p->ev1) cudaEventDestroy(p->ev1);
        cudaSetDevice(cur);
    }
    delete p;
    return NB_OK;
}

nb_status nb_cbs_out_shape(nb_cbs_plan p, int32_t* ho, int32_t* wo) {
    g_err.clear();
    if (!p || !ho || !wo) return fail(NB_ERR_INVALID_ARG, "NULL argument");
    *ho = p->g.ho;
    *wo = p->g.wo;
    return NB_OK;
}

nb_status nb_cbs_workspace_bytes(nb_cbs_plan p, size_t* fwd, size_t* bwd) {
    g_err.clear();
    if (!p || !fwd || !bwd) return fail(NB_ERR_INVALID_ARG, "NULL argument");
    *fwd = p->fwd_bytes;
    *bwd = p->bwd_bytes;
    return NB_OK;
}

nb_status nb_cbs_plan_set_pitches(nb_cbs_plan p, int64_t ld_x, int64_t ld_a, int64_t ld_g) {
    g_err.clear();
    if (!p) return fail(NB_ERR_INVALID_ARG, "plan is NULL");
    const int vec = is_f32(p) ? 4 : 8;
    auto bad = [&](int64_t ld, int channels) { return ld != 0 && ld != channels && (ld < channels || ld % vec != 0); };  // 0 or the channel count: dense
    if (bad(ld_x, p->g.c_in) || bad(ld_a, p->g.c_out) || bad(ld_g, p->g.c_out))
        return fail(NB_ERR_INVALID_ARG, "a pitch must be 0 (dense) or at least the channel count and a multiple of %d elements", vec);
    if (ld_x != 0 && ld_x != p->g.c_in && (is_f32(p) || p->stem || !p->tc.fprop || !p->tc.wgrad))
        return fail(NB_ERR_UNSUPPORTED, "an input pitch needs the tensor-core forward and weight-gradient kernels (this plan runs them elsewhere)");
    p->tc.ld_x = (ld_x == p->g.c_in) ? 0 : ld_x;
    p->ld_a = (ld_a == p->g.c_out) ? 0 : ld_a;
    p->ld_g = (ld_g == p->g.c_out) ? 0 : ld_g;
    p->pitched = p->tc.ld_x || p->ld_a || p->ld_g;
    // tensor maps cached for the previous layout are stale
    p->tc.fp.a_ptr = nullptr;
    p->tc.inf.a_ptr = nullptr;
    p->tc.wg_a_ptr = nullptr;
    return NB_OK;
}

nb_status nb_cbs_plan_set_fwd_residual(nb_cbs_plan p, const void* res, int64_t ld_res) {
    g_err.clear();
    if (!p) return fail(NB_ERR_INVALID_ARG, "plan is NULL");
    NB_CHECK_PTR(res, true);
    const int vec = is_f32(p) ? 4 : 8;
    if (ld_res == p->g.c_out) ld_res = 0;
    if (res && ld_res != 0 && (ld_res < p->g.c_out || ld_res % vec != 0))
        return fail(NB_ERR_INVALID_ARG, "ld_res must be 0 (dense) or at least c_out and a multiple of %d elements", vec);
    p->fwd_res = res;
    p->ld_res = res ? ld_res : 0;
    return NB_OK;
}

nb_status nb_cbs_plan_set_bwd_residual(nb_cbs_plan p, void* gres, int64_t ld_gres, int32_t accumulate) {
    g_err.clear();
    if (!p) return fail(NB_ERR_INVALID_ARG, "plan is NULL");
    NB_CHECK_PTR(gres, true);
    if (accumulate != 0 && accumulate != 1) return fail(NB_ERR_INVALID_ARG, "accumulate must be 0 or 1, got %d", accumulate);
    if (ld_gres == p->g.c_out) ld_gres = 0;
    if (gres && ld_gres != 0 && (ld_gres < p->g.c_out || ld_gres % 8 != 0))
        return fail(NB_ERR_INVALID_ARG, "ld_gres must be 0 (dense) or at least c_out and a multiple of 8 elements");
    if (gres && !p->fuse_finalize)
        return fail(NB_ERR_UNSUPPORTED, "the shortcut's gradient rides in the dy pass of the default 16-bit plans only (not fp32 mode, not NB_CBS_FLAG_SEPARATE_FINALIZE)");
    p->bwd_gres = gres;
    p->ld_gres = gres ? ld_gres : 0;
    p->gres_add = accumulate != 0;
    return NB_OK;
}

nb_status nb_cbs_plan_set_dx_target(nb_cbs_plan p, int64_t ld_dx, int32_t accumulate) {
    g_err.clear();
    if (!p) return fail(NB_ERR_INVALID_ARG, "plan is NULL");
    if (accumulate != 0 && accumulate != 1) return fail(NB_ERR_INVALID_ARG, "accumulate must be 0 or 1, got %d", accumulate);
    if (ld_dx == p->g.c_in) ld_dx = 0;
    if (ld_dx != 0 && (ld_dx < p->g.c_in || ld_dx % 8 != 0)) return fail(NB_ERR_INVALID_ARG, "ld_dx must be 0 (dense) or at least c_in and a multiple of 8 elements");
    if ((ld_dx != 0 || accumulate) && (is_f32(p) || p->stem || !p->tc.dgrad || p->g.stride != 1))
        return fail(NB_ERR_UNSUPPORTED, "a pitched or accumulating dx needs the tensor-core data gradient of a stride-1 layer (its epilogue stores through TMA)");
    p->ld_dx = ld_dx;
    p->dx_accumulate = accumulate != 0;
    return NB_OK;
}

nb_status nb_cbs_plan_paths(nb_cbs_plan p, int32_t* paths3) {
    g_err.clear();
    if (!p || !paths3) return fail(NB_ERR_INVALID_ARG, "NULL argument");
    paths3[0] = p->tc.fprop ? 1 : 0;
    paths3[1] = p->tc.dgrad ? 1 : 0;
    paths3[2] = p->tc.wgrad ? 1 : 0;
    return NB_OK;
}

unsigned long long nb_cbs_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

nb_status nb_cbs_profile_enable(nb_cbs_plan p, int32_t enable) {
    g_err.clear();
    if (!p) return fail(NB_ERR_INVALID_ARG, "plan is NULL");
    if (enable && !p->ev0) {
        NB_CUDA_CHECK(cudaEventCreate(&p->ev0));
        NB_CUDA_CHECK(cudaEventCreate(&p->ev1));
    }
    p->profiling = enable != 0;
    for (int i = 0; i < SITE_COUNT; ++i) {
        p->prof_ms[i] = 0.0;
        p->prof_n[i] = 0;
    }
    return NB_OK;
}

const char* nb_cbs_profile_site_name(int32_t site) { return (site >= 0 && site < SITE_COUNT) ? kSiteNames[site] : nullptr; }

nb_status nb_cbs_profile_read(nb_cbs_plan p, int32_t site, double* total_ms, int64_t* launches) {
    g_err.clear();
    if (!p || !total_ms || !launches) return fail(NB_ERR_INVALID_ARG, "NULL argument");
    if (site < 0 || site >= SITE_COUNT) return fail(NB_ERR_INVALID_ARG, "site %d out of range", site);
    *total_ms = p->prof_ms[site];
    *launches = p->prof_n[site];
    return NB_OK;
}

nb_status nb_cbs_poll_status(nb_cbs_plan p, void* stream) {
    g_err.clear();
    if (!p) return fail(NB_ERR_INVALID_ARG, "plan is NULL");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int host[ST_WORDS];
    NB_CUDA_CHECK(cudaStreamSynchronize(st));
    NB_CUDA_CHECK(cudaMemcpy(host, p->status, sizeof host, cudaMemcpyDeviceToHost));
    NB_CUDA_CHECK(cudaMemset(p->status, 0, sizeof host));
    if (host[ST_ERR] != 0 && p->acc)  // a kernel that gave up may have left sums behind: the next call must find zeros
        NB_CUDA_CHECK(cudaMemset(p->acc, 0, (size_t)(p->acc_copies_f + p->acc_copies_b) * 2 * p->g.c_out * sizeof(double)));
    if (host[ST_ERR] != 0)
        return fail((nb_status)host[ST_ERR], "device status: error %d at site %d (detail %d)", host[ST_ERR], host[ST_WHERE], host[ST_DETAIL]);
    if (host[ST_SAT] != 0) {
        char buf[96];
        snprintf(buf, sizeof buf, "%d fp16 stores of the saved convolution output saturated", host[ST_SAT]);
        g_err = buf;
    }
    return NB_OK;
}

nb_status nb_conv_bn_silu_fwd(nb_cbs_plan p, const void* x, const void* w, const float* gamma, const float* beta,
                              float* running_mean, float* running_var, void* y_saved, float* save_mean, float* save_invstd,
                              void* a_out, void* workspace, size_t workspace_bytes, void* stream) {
    g_err.clear();
    if (!p) return fail(NB_ERR_INVALID_ARG, "plan is NULL");
    NB_CHECK_PTR(x); NB_CHECK_PTR(w); NB_CHECK_PTR(gamma); NB_CHECK_PTR(beta);
    NB_CHECK_PTR(y_saved); NB_CHECK_PTR(save_mean); NB_CHECK_PTR(save_invstd); NB_CHECK_PTR(a_out);
    if ((running_mean == nullptr) != (running_var == nullptr))
        return fail(NB_ERR_INVALID_ARG, "running_mean and running_var must both be given or both be NULL");
    NB_TRY(check_ws(workspace, workspace_bytes, p->fwd_bytes));
    DeviceGuard on_device(p->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char* ws = static_cast<char*>(workspace);
    float* scale = reinterpret_cast<float*>(ws + p->off_scale);
    float* shift = reinterpret_cast<float*>(ws + p->off_shift);
    float* part = reinterpret_cast<float*>(ws + p->off_fpart);
    int nparts = p->ew.blocks_stats;
    bool finalized = false;
    if (is_f32(p)) {
        NB_TRY((run_simt_fprop<float, float>(p, x, w, y_saved, st)));
        NB_TRY(run_stats_partial<float>(p, y_saved, part, st));
    } else if (p->stem) {
        // the first layer's kernel sums the statistics of the values it stores itself (one partial slice per block)
        SiteTimer tm(p, SITE_FPROP, st);
        const bool fuse = p->fuse_finalize;  // sums into the plan's accumulators; the normalise + SiLU pass finalizes
        if (p->stem_wide) {
            NB_WITH_AT(p, launch_k(stem_fprop_mma_kernel<48, __half, false, AT, STEM_TQ_WIDE>, dim3(p->stem_fprop_blocks), dim3(128), 0, st, 1,
                                   static_cast<const AT*>(x), static_cast<const AT*>(w), static_cast<__half*>(y_saved), p->g, StemEpi{},
                                   fuse ? static_cast<float*>(nullptr) : part, fuse ? p->acc : static_cast<double*>(nullptr), fuse ? p->acc_copies_f : 1));
        } else {
            NB_WITH_AT(p, launch_k(stem_fprop_mma_kernel<48, __half, false, AT, STEM_TQ>, dim3(p->stem_fprop_blocks), dim3(128), 0, st, 1,
                                   static_cast<const AT*>(x), static_cast<const AT*>(w), static_cast<__half*>(y_saved), p->g, StemEpi{},
                                   fuse ? static_cast<float*>(nullptr) : part, fuse ? p->acc : static_cast<double*>(nullptr), fuse ? p->acc_copies_f : 1));
        }
        NB_LAUNCH_OK("stem_fprop");
        nparts = p->stem_fprop_blocks;
        finalized = fuse;
    } else if (p->tc.fprop) {
        SiteTimer tm(p, SITE_FPROP, st);
        const long long l0 = p->tc.launches;
        // writes y (fp16) and adds its channel sums to the accumulators (or writes them as per-CTA partial sums)
        const bool fuse = p->fuse_finalize;
        const ChanAcc ca{fuse ? p->acc : nullptr, nullptr, fuse ? p->acc_copies_f : 1};
        const nb_status ts = tc_fprop(&p->tc, p->g, x, w, y_saved, part, p->status, st, ca);
        g_launches.fetch_add((unsigned long long)(p->tc.launches - l0), std::memory_order_relaxed);
        if (ts != NB_OK) return fail(ts, "%s", tc_last_error());
        nparts = p->tc.fprop_parts;
        finalized = fuse;
    } else {
        NB_TRY(NB_WITH_AT(p, run_simt_fprop<AT, __half>(p, x, w, y_saved, st)));
        NB_TRY(run_stats_partial<__half>(p, y_saved, part, st));
    }
    if (!finalized)
        NB_TRY(run_finalize(p, part, nparts, gamma, beta, save_mean, save_invstd, scale, shift, running_mean, running_var, nullptr, nullptr, st));
    if (is_f32(p)) return run_apply<float, float, false>(p, y_saved, a_out, scale, shift, st, p->ld_a, p->fwd_res, p->ld_res);
    // after the tensor-core kernel the pass derives mean, invstd, scale and shift from the accumulators itself
    const double M = (double)p->g.m;
    const FwdFin fin{1.0 / M, M / (M - 1.0), p->desc.eps, p->desc.momentum, gamma, beta, save_mean, save_invstd, running_mean, running_var};
    return NB_WITH_AT(p, run_apply<__half, AT, true>(p, y_saved, a_out, scale, shift, st, p->ld_a, p->fwd_res, p->ld_res, finalized ? &fin : nullptr));
}

namespace {
// conv -> out = act(conv*scale_c + shift_c) with (scale, shift) from evaluation-mode BN or a bias (see bn_eval_coef)
nb_status run_infer(nb_cbs_plan_s* p, const void* x, const void* w, const float* gamma, const float* beta, const float* rmean, const float* rvar,
                    int act, void* out, char* ws, cudaStream_t st) {
    if (infer_fused(p) && !p->stem) {
        SiteTimer tm(p, SITE_INFER, st);
        const long long l0 = p->tc.launches;
        const EpiAffine e{gamma, beta, rmean, rvar, p->desc.eps, act};
        const nb_status ts = tc_infer(&p->tc, p->g, x, w, out, e, p->status, st);
        g_launches.fetch_add((unsigned long long)(p->tc.launches - l0), std::memory_order_relaxed);
        if (ts != NB_OK) return fail(ts, "%s", tc_last_error());
        return NB_OK;
    }
    if (!is_f32(p) && p->stem) {  // the first layer's own kernel applies the coefficients and the activation itself
        SiteTimer tm(p, SITE_INFER, st);
        if (p->stem_wide) {
            NB_WITH_AT(p, launch_k(stem_fprop_mma_kernel<48, AT, true, AT, STEM_TQ_WIDE>, dim3(p->stem_fprop_blocks), dim3(128), 0, st, 1, static_cast<const AT*>(x),
                                   static_cast<const AT*>(w), static_cast<AT*>(out), p->g, StemEpi{gamma, beta, rmean, rvar, p->desc.eps, act},
                                   static_cast<float*>(nullptr), static_cast<double*>(nullptr), 1));
        } else {
            NB_WITH_AT(p, launch_k(stem_fprop_mma_kernel<48, AT, true, AT, STEM_TQ>, dim3(p->stem_fprop_blocks), dim3(128), 0, st, 1, static_cast<const AT*>(x),
                                   static_cast<const AT*>(w), static_cast<AT*>(out), p->g, StemEpi{gamma, beta, rmean, rvar, p->desc.eps, act},
                                   static_cast<float*>(nullptr), static_cast<double*>(nullptr), 1));
        }
        return launch_ok("stem_fprop (fused epilogue)");
    }
    float* scale = reinterpret_cast<float*>(ws + p->off_scale);
    float* shift = reinterpret_cast<float*>(ws + p->off_shift);
    void* y = ws + p->off_iy;
    if (is_f32(p)) {
        NB_TRY((run_simt_fprop<float, float>(p, x, w, y, st)));
    } else {
        NB_TRY(NB_WITH_AT(p, run_simt_fprop<AT, __half>(p, x, w, y, st)));
    }
    {
        SiteTimer tm(p, SITE_EVAL_COEF, st);
        launch_k(bn_eval_coef_kernel, dim3((unsigned)((p->g.c_out + 255) / 256)), dim3(256), 0, st, 1, gamma, beta, rmean, rvar, p->desc.eps, p->g.c_out, scale, shift);
        NB_LAUNCH_OK("bn_eval_coef");
    }
    if (is_f32(p)) return act ? run_apply<float, float, false, true>(p, y, out, scale, shift, st) : run_apply<float, float, false, false>(p, y, out, scale, shift, st);
    return NB_WITH_AT(p, act ? run_apply<__half, AT, true, true>(p, y, out, scale, shift, st) : run_apply<__half, AT, true, false>(p, y, out, scale, shift, st));
}
}  // namespace

nb_status nb_cbs_infer_workspace_bytes(nb_cbs_plan p, size_t* bytes, int32_t* fused) {
    g_err.clear();
    if (!p || !bytes) return fail(NB_ERR_INVALID_ARG, "NULL argument");
    *bytes = p->infer_bytes;
    if (fused) *fused = infer_fused(p) ? 1 : 0;
    return NB_OK;
}

nb_status nb_conv_bn_silu_infer(nb_cbs_plan p, const void* x, const void* w, const float* gamma, const float* beta, const float* running_mean,
                                const float* running_var, void* a_out, void* workspace, size_t workspace_bytes, void* stream) {
    g_err.clear();
    if (!p) return fail(NB_ERR_INVALID_ARG, "plan is NULL");
    NB_CHECK_PTR(x); NB_CHECK_PTR(w); NB_CHECK_PTR(gamma); NB_CHECK_PTR(beta); NB_CHECK_PTR(running_mean); NB_CHECK_PTR(running_var);
    NB_CHECK_PTR(a_out);
    if (p->pitched || p->fwd_res) return fail(NB_ERR_UNSUPPORTED, "the plan has row pitches or a residual set: only the three training calls honour them");
    NB_TRY(check_ws(workspace, workspace_bytes, p->infer_bytes));
    DeviceGuard on_device(p->device);
    return run_infer(p, x, w, gamma, beta, running_mean, running_var, 1, a_out, static_cast<char*>(workspace), static_cast<cudaStream_t>(stream));
}

nb_status nb_conv_bias_act(nb_cbs_plan p, const void* x, const void* w, const float* bias, int32_t act, void* out, void* workspace,
                           size_t workspace_bytes, void* stream) {
    g_err.clear();
    if (!p) return fail(NB_ERR_INVALID_ARG, "plan is NULL");
    NB_CHECK_PTR(x); NB_CHECK_PTR(w); NB_CHECK_PTR(bias, true); NB_CHECK_PTR(out);
    if (act != 0 && act != 1) return fail(NB_ERR_INVALID_ARG, "act must be 0 (none) or 1 (SiLU), got %d", act);
    if (p->pitched || p->fwd_res) return fail(NB_ERR_UNSUPPORTED, "the plan has row pitches or a residual set: only the three training calls honour them");
    NB_TRY(check_ws(workspace, workspace_bytes, p->infer_bytes));
    DeviceGuard on_device(p->device);
    return run_infer(p, x, w, nullptr, bias, nullptr, nullptr, act, out, static_cast<char*>(workspace), static_cast<cudaStream_t>(stream));
}

nb_status nb_bn_fold(nb_cbs_plan p, const void* w, const float* gamma, const float* beta, const float* running_mean, const float* running_var,
                     void* w_folded, float* bias_folded, void* stream) {
    g_err.clear();
    if (!p) return fail(NB_ERR_INVALID_ARG, "plan is NULL");
    NB_CHECK_PTR(w); NB_CHECK_PTR(gamma); NB_CHECK_PTR(beta); NB_CHECK_PTR(running_mean); NB_CHECK_PTR(running_var);
    NB_CHECK_PTR(w_folded); NB_CHECK_PTR(bias_folded);
    DeviceGuard on_device(p->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const long long K = p->g.kdim, total = K * p->g.c_out;
    const unsigned blocks = (unsigned)std::min<long long>((total + 255) / 256, (long long)p->sm_count * 8);
    SiteTimer tm(p, SITE_FOLD, st);
    if (is_f32(p))
        launch_k(bn_fold_kernel<float>, dim3(blocks), dim3(256), 0, st, 1, static_cast<const float*>(w), K, p->g.c_out, gamma, beta, running_mean, running_var,
                 p->desc.eps, static_cast<float*>(w_folded), bias_folded);
    else if (is_f16(p))
        launch_k(bn_fold_kernel<__half>, dim3(blocks), dim3(256), 0, st, 1, static_cast<const __half*>(w), K, p->g.c_out, gamma, beta, running_mean, running_var,
                 p->desc.eps, static_cast<__half*>(w_folded), bias_folded);
    else
        launch_k(bn_fold_kernel<__nv_bfloat16>, dim3(blocks), dim3(256), 0, st, 1, static_cast<const __nv_bfloat16*>(w), K, p->g.c_out, gamma, beta, running_mean,
                 running_var, p->desc.eps, static_cast<__nv_bfloat16*>(w_folded), bias_folded);
    return launch_ok("bn_fold");
}

nb_status nb_bn_stats(nb_cbs_plan p, const void* y, int32_t y_dtype, float* mean, float* invstd, float* sum, float* sumsq,
                      void* workspace, size_t workspace_bytes, void* stream) {
    g_err.clear();
    if (!p) return fail(NB_ERR_INVALID_ARG, "plan is NULL");
    NB_CHECK_PTR(y); NB_CHECK_PTR(mean); NB_CHECK_PTR(invstd);
    NB_CHECK_PTR(sum, true); NB_CHECK_PTR(sumsq, true);
    const int want = is_f32(p) ? NB_DTYPE_F32 : NB_DTYPE_F16;
    if (y_dtype != want) return fail(NB_ERR_UNSUPPORTED, "y_dtype %d does not match the plan's mode (expected %d)", y_dtype, want);
    NB_TRY(check_ws(workspace, workspace_bytes, p->fwd_bytes));
    DeviceGuard on_device(p->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float* part = reinterpret_cast<float*>(static_cast<char*>(workspace) + p->off_fpart);
    if (is_f32(p)) NB_TRY(run_stats_partial<float>(p, y, part, st));
    else NB_TRY(run_stats_partial<__half>(p, y, part, st));
    return run_finalize(p, part, p->ew.blocks_stats, nullptr, nullptr, mean, invstd, nullptr, nullptr, nullptr, nullptr, sum, sumsq, st);
}

nb_status nb_conv_bn_silu_bwd_data(nb_cbs_plan p, const void* g, const void* y_saved, const float* save_mean,
                                   const float* save_invstd, const float* gamma, const float* beta, const void* w, void* dx,
                                   float* dgamma, float* dbeta, void* dy_out, void* workspace, size_t workspace_bytes, void* stream) {
    g_err.clear();
    if (!p) return fail(NB_ERR_INVALID_ARG, "plan is NULL");
    NB_CHECK_PTR(g); NB_CHECK_PTR(y_saved); NB_CHECK_PTR(save_mean); NB_CHECK_PTR(save_invstd);
    NB_CHECK_PTR(gamma); NB_CHECK_PTR(beta); NB_CHECK_PTR(dgamma); NB_CHECK_PTR(dbeta); NB_CHECK_PTR(dy_out);
    NB_CHECK_PTR(dx, true);
    if (dx) NB_CHECK_PTR(w);
    NB_TRY(check_ws(workspace, workspace_bytes, p->bwd_bytes));
    DeviceGuard on_device(p->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char* ws = static_cast<char*>(workspace);
    float* coef = reinterpret_cast<float*>(ws + p->off_coef);
    float* part = reinterpret_cast<float*>(ws + p->off_bpart);
    if (is_f32(p)) {
        NB_TRY((run_bwd_elementwise<float, float, false>(p, g, y_saved, save_mean, save_invstd, gamma, beta, dgamma, dbeta, dy_out, part, coef, st)));
        if (dx) NB_TRY(run_simt_dgrad<float>(p, dy_out, w, dx, st));
        return NB_OK;
    }
    const bool tc_dg = dx && !p->stem && p->tc.dgrad;  // the finalize kernel also rearranges the filter for the tensor-core dgrad
    NB_TRY(NB_WITH_AT(p, run_bwd_elementwise<__half, AT, true>(p, g, y_saved, save_mean, save_invstd, gamma, beta, dgamma, dbeta, dy_out, part, coef, st,
                                                               tc_dg ? w : nullptr, tc_dg ? ws + p->off_wt : nullptr, tc_dg ? &p->tc.wtp : nullptr)));
    if (!dx) return NB_OK;
    if (p->stem) {
        SiteTimer tm(p, SITE_DGRAD, st);
        NB_WITH_AT(p, launch_k(stem_dgrad_mma_kernel<48, AT>, dim3(p->stem_dgrad_blocks), dim3(128), 0, st, 1, static_cast<const AT*>(dy_out), static_cast<const AT*>(w),
                               static_cast<AT*>(dx), p->g, p->stem_dgrad_rows));
        return launch_ok("stem_dgrad");
    }
    if (p->tc.dgrad) {
        SiteTimer tm(p, SITE_DGRAD, st);
        const long long l0 = p->tc.launches;
        const nb_status ts = tc_dgrad(&p->tc, p->g, dy_out, w, dx, ws + p->off_wt, p->status, st, true, p->ld_dx, p->dx_accumulate);
        g_launches.fetch_add((unsigned long long)(p->tc.launches - l0), std::memory_order_relaxed);
        if (ts != NB_OK) return fail(ts, "%s", tc_last_error());
        return NB_OK;
    }
    return NB_WITH_AT(p, run_simt_dgrad<AT>(p, dy_out, w, dx, st));
}

nb_status nb_conv_bias_bwd(nb_cbs_plan p, const void* x, const void* w, const void* dout, void* dx, float* dw, float* dbias, void* workspace,
                           size_t workspace_bytes, void* stream) {
    g_err.clear();
    if (!p) return fail(NB_ERR_INVALID_ARG, "plan is NULL");
    NB_CHECK_PTR(x); NB_CHECK_PTR(dout); NB_CHECK_PTR(dw); NB_CHECK_PTR(dx, true); NB_CHECK_PTR(dbias, true);
    if (dx) NB_CHECK_PTR(w);
    if (p->pitched || p->ld_dx || p->dx_accumulate || p->fwd_res || p->bwd_gres) return fail(NB_ERR_UNSUPPORTED, "the plan has row pitches, a dx target or a residual set: only the three training calls honour them");
    NB_TRY(check_ws(workspace, workspace_bytes, p->bwd_bytes));
    {
        DeviceGuard on_device(p->device);
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        char* ws = static_cast<char*>(workspace);
        if (dbias) {  // column sums of dout: the statistics kernels with only the raw sum requested
            float* part = reinterpret_cast<float*>(ws + p->off_bpart);
            if (is_f32(p)) NB_TRY(run_stats_partial<float>(p, dout, part, st));
            else NB_TRY(NB_WITH_AT(p, run_stats_partial<AT>(p, dout, part, st)));
            NB_TRY(run_finalize(p, part, p->ew.blocks_stats, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, dbias, nullptr, st));
        }
        if (dx) {
            if (is_f32(p)) {
                NB_TRY(run_simt_dgrad<float>(p, dout, w, dx, st));
            } else if (p->stem) {
                SiteTimer tm(p, SITE_DGRAD, st);
                NB_WITH_AT(p, launch_k(stem_dgrad_mma_kernel<48, AT>, dim3(p->stem_dgrad_blocks), dim3(128), 0, st, 1, static_cast<const AT*>(dout), static_cast<const AT*>(w),
                                       static_cast<AT*>(dx), p->g, p->stem_dgrad_rows));
                NB_LAUNCH_OK("stem_dgrad");
            } else if (p->tc.dgrad) {
                SiteTimer tm(p, SITE_DGRAD, st);
                const long long l0 = p->tc.launches;
                const nb_status ts = tc_dgrad(&p->tc, p->g, dout, w, dx, ws + p->off_wt, p->status, st, false);  // rearranges the filter itself
                g_launches.fetch_add((unsigned long long)(p->tc.launches - l0), std::memory_order_relaxed);
                if (ts != NB_OK) return fail(ts, "%s", tc_last_error());
            } else {
                NB_TRY(NB_WITH_AT(p, run_simt_dgrad<AT>(p, dout, w, dx, st)));
            }
        }
    }
    return nb_conv_bn_silu_bwd_weight(p, x, dout, dw, workspace, workspace_bytes, stream);
}

nb_status nb_conv_bn_silu_bwd_weight(nb_cbs_plan p, const void* x, const void* dy, float* dw, void* workspace,
                                     size_t workspace_bytes, void* stream) {
    g_err.clear();
    if (!p) return fail(NB_ERR_INVALID_ARG, "plan is NULL");
    NB_CHECK_PTR(x); NB_CHECK_PTR(dy); NB_CHECK_PTR(dw);
    NB_TRY(check_ws(workspace, workspace_bytes, p->bwd_bytes));
    DeviceGuard on_device(p->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float* partial = reinterpret_cast<float*>(static_cast<char*>(workspace) + p->off_wgpart);
    if (is_f32(p)) return run_simt_wgrad<float>(p, x, dy, dw, partial, st);
    if (p->stem) {
        {
            SiteTimer tm(p, SITE_WGRAD, st);
            if (p->stem_wide) {
                NB_WITH_AT(p, launch_k(stem_wgrad_mma_kernel<48, AT, STEM_TQ_WGRAD>, dim3(p->stem_wgrad_blocks), dim3(128),
                                       stem_wgrad_smem_bytes<48, AT, STEM_TQ_WGRAD>(), st, 1, static_cast<const AT*>(x), static_cast<const AT*>(dy), partial, p->g));
            } else {
                NB_WITH_AT(p, launch_k(stem_wgrad_mma_kernel<48, AT, STEM_TQ>, dim3(p->stem_wgrad_blocks), dim3(128), stem_wgrad_smem_bytes<48, AT, STEM_TQ>(), st, 1,
                                       static_cast<const AT*>(x), static_cast<const AT*>(dy), partial, p->g));
            }
            NB_LAUNCH_OK("stem_wgrad");
        }
        const size_t elems = (size_t)p->g.c_out * p->g.kdim;
        SiteTimer tm(p, SITE_SPLITK_REDUCE, st);
        launch_k(splitk_reduce_tall_kernel, dim3((unsigned)((elems + 31) / 32)), dim3(1024), 0, st, 1, partial, p->stem_wgrad_blocks, elems, dw);
        return launch_ok("splitk_reduce");
    }
    if (p->tc.wgrad) {
        SiteTimer tm(p, SITE_WGRAD, st);
        const long long l0 = p->tc.launches;
        const nb_status ts = tc_wgrad(&p->tc, p->g, x, dy, dw, partial, p->status, st);
        g_launches.fetch_add((unsigned long long)(p->tc.launches - l0), std::memory_order_relaxed);
        if (ts != NB_OK) return fail(ts, "%s", tc_last_error());
        return NB_OK;
    }
    return NB_WITH_AT(p, run_simt_wgrad<AT>(p, x, dy, dw, partial, st));
}

}  // extern "C"

// ---------------------------------------------------------------- batch statistics without any allocation
// Scratch for nb_bn_stats_static: partial sums [kStaticParts][2][kStaticMaxC] floats = 2 MiB, resident on every
// GPU that loads this library until the process exits.  In host code the name `g_static_partials` is only a
// handle for the symbol, never a device address: the address comes from cudaGetSymbolAddress below.
namespace {
constexpr int kStaticParts = 256;
constexpr int kStaticMaxC = 1024;
constexpr int kStaticMaxDevices = 64;
}  // namespace
static __device__ __align__(256) float g_static_partials[(size_t)kStaticParts * 2 * kStaticMaxC];

namespace {
std::mutex g_static_mu;
float* g_static_ptr[kStaticMaxDevices] = {};
int g_static_sms[kStaticMaxDevices] = {};

// Once per device, with that device current: resolve the device address of the static scratch array.
nb_status static_scratch_for_current_device(float** out, int* sms) {
    int dev = -1;
    NB_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kStaticMaxDevices) return fail(NB_ERR_UNSUPPORTED, "device ordinal %d is beyond %d", dev, kStaticMaxDevices);
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[dev]) {
        int major = 0, count = 0;
        NB_CUDA_CHECK(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
        if (major != 10) return fail(NB_ERR_ARCH, "device %d is not compute capability 10.x", dev);
        NB_CUDA_CHECK(cudaDeviceGetAttribute(&count, cudaDevAttrMultiProcessorCount, dev));
        void* ptr = nullptr;
        NB_CUDA_CHECK(cudaGetSymbolAddress(&ptr, g_static_partials));
        if (!ptr) return fail(NB_ERR_CUDA, "cudaGetSymbolAddress returned a null address");
        g_static_sms[dev] = count;
        g_static_ptr[dev] = static_cast<float*>(ptr);
    }
    *out = g_static_ptr[dev];
    *sms = g_static_sms[dev];
    return NB_OK;
}
}  // namespace

extern "C" nb_status nb_bn_stats_static(const void* y, int32_t y_dtype, int64_t m, int32_t c, float eps, float* mean, float* invstd,
                                        float* sum, float* sumsq, void* stream) {
    g_err.clear();
    NB_CHECK_PTR(y); NB_CHECK_PTR(mean); NB_CHECK_PTR(invstd);
    NB_CHECK_PTR(sum, true); NB_CHECK_PTR(sumsq, true);
    if (y_dtype != NB_DTYPE_F16 && y_dtype != NB_DTYPE_F32) return fail(NB_ERR_UNSUPPORTED, "y_dtype %d: only F16 and F32 are supported", y_dtype);
    if (m < 2 || c <= 0) return fail(NB_ERR_INVALID_ARG, "need m >= 2 rows and c > 0 channels (m=%lld c=%d)", (long long)m, c);
    if (!(eps > 0.f)) return fail(NB_ERR_INVALID_ARG, "eps must be positive");
    const int vec = y_dtype == NB_DTYPE_F32 ? 4 : 8;
    if (c % vec) return fail(NB_ERR_UNSUPPORTED, "c=%d must be a multiple of %d for this dtype", c, vec);
    if (c > kStaticMaxC)
        return fail(NB_ERR_UNSUPPORTED, "c=%d exceeds the %d channels the built-in scratch array holds; use nb_bn_stats with a workspace", c, kStaticMaxC);
    if ((double)m * c >= 9.0e18) return fail(NB_ERR_UNSUPPORTED, "tensor too large");
    float* part = nullptr;
    int sms = 0;
    NB_TRY(static_scratch_for_current_device(&part, &sms));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int cgs = c / vec;
    const int R = cgs >= 256 ? 1 : 256 / cgs;
    const int tpb = cgs * R;
    const long long total_vecs = (long long)m * cgs;
    const long long max_blocks = (total_vecs + tpb - 1) / tpb;
    const int blocks = (int)std::min<long long>(max_blocks, std::min(kStaticParts, std::max(1, sms)));
    // Every partial that the second kernel reads is written by the first one in this same call, so nothing in the
    // array has to start at zero and the previous call's contents do not matter.
    if (y_dtype == NB_DTYPE_F32)
        launch_k(bn_stats_partial_kernel<float>, dim3(blocks), dim3(tpb), (size_t)tpb * vec * sizeof(float), st, 1, static_cast<const float*>(y), total_vecs, c, part);
    else
        launch_k(bn_stats_partial_kernel<__half>, dim3(blocks), dim3(tpb), (size_t)tpb * vec * sizeof(float), st, 1, static_cast<const __half*>(y), total_vecs, c, part);
    NB_LAUNCH_OK("bn_stats_partial (static scratch)");
    launch_k(bn_finalize_kernel, dim3((c + 7) / 8), dim3(256), 0, st, 1, part, blocks, c, (double)m, eps, 0.f, nullptr, nullptr, mean, invstd, nullptr,
                                                              nullptr, nullptr, nullptr, sum, sumsq);
    return launch_ok("bn_finalize (static scratch)");
}

extern "C" {

// ---------------------------------------------------------------- host-buffer step
namespace {
struct StepLayout {
    size_t x, w, gamma, beta, g, y, mean, invstd, a, dy, dx, dw, dgamma, dbeta, ws_fwd, ws_bwd, total;
    size_t nx, nw, ny_act, ny_saved, ndw;  // byte counts
};
StepLayout step_layout(const nb_cbs_plan_s* p) {
    StepLayout L;
    const size_t act = is_f32(p) ? 4 : 2, ysz = is_f32(p) ? 4 : 2;
    const Geom& g = p->g;
    L.nx = (size_t)g.n * g.h * g.w * g.c_in * act;
    L.nw = (size_t)g.c_out * g.kdim * act;
    L.ny_act = (size_t)g.m * g.c_out * act;
    L.ny_saved = (size_t)g.m * g.c_out * ysz;
    L.ndw = (size_t)g.c_out * g.kdim * 4;
    const size_t cb = (size_t)g.c_out * 4;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    L.x = take(L.nx); L.w = take(L.nw); L.gamma = take(cb); L.beta = take(cb); L.g = take(L.ny_act);
    L.y = take(L.ny_saved); L.mean = take(cb); L.invstd = take(cb); L.a = take(L.ny_act); L.dy = take(L.ny_act);
    L.dx = take(L.nx); L.dw = take(L.ndw); L.dgamma = take(cb); L.dbeta = take(cb);
    L.ws_fwd = take(p->fwd_bytes); L.ws_bwd = take(p->bwd_bytes);
    L.total = off;
    return L;
}
}  // namespace

nb_status nb_cbs_step_host_scratch_bytes(nb_cbs_plan p, size_t* bytes) {
    g_err.clear();
    if (!p || !bytes) return fail(NB_ERR_INVALID_ARG, "NULL argument");
    *bytes = step_layout(p).total;
    return NB_OK;
}

nb_status nb_conv_bn_silu_step_host(nb_cbs_plan p, const void* host_x, const void* host_w, const float* host_gamma,
                                    const float* host_beta, const void* host_g, void* host_a, void* host_dx, float* host_dw,
                                    float* host_dgamma, float* host_dbeta, void* device_scratch, size_t scratch_bytes, void* stream) {
    g_err.clear();
    if (!p) return fail(NB_ERR_INVALID_ARG, "plan is NULL");
    if (!host_x || !host_w || !host_gamma || !host_beta || !host_g || !host_a || !host_dw || !host_dgamma || !host_dbeta)
        return fail(NB_ERR_INVALID_ARG, "a required host pointer is NULL");
    if (p->pitched || p->ld_dx || p->dx_accumulate || p->fwd_res || p->bwd_gres) return fail(NB_ERR_UNSUPPORTED, "the plan has row pitches, a dx target or a residual set: the host-buffer step works on dense tensors");
    const StepLayout L = step_layout(p);
    NB_TRY(check_ws(device_scratch, scratch_bytes, L.total));
    DeviceGuard on_device(p->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char* d = static_cast<char*>(device_scratch);
    const size_t cb = (size_t)p->g.c_out * 4;
    NB_CUDA_CHECK(cudaMemcpyAsync(d + L.x, host_x, L.nx, cudaMemcpyHostToDevice, st));
    NB_CUDA_CHECK(cudaMemcpyAsync(d + L.w, host_w, L.nw, cudaMemcpyHostToDevice, st));
    NB_CUDA_CHECK(cudaMemcpyAsync(d + L.gamma, host_gamma, cb, cudaMemcpyHostToDevice, st));
    NB_CUDA_CHECK(cudaMemcpyAsync(d + L.beta, host_beta, cb, cudaMemcpyHostToDevice, st));
    NB_CUDA_CHECK(cudaMemcpyAsync(d + L.g, host_g, L.ny_act, cudaMemcpyHostToDevice, st));
    float* gam = reinterpret_cast<float*>(d + L.gamma);
    float* bet = reinterpret_cast<float*>(d + L.beta);
    float* mean = reinterpret_cast<float*>(d + L.mean);
    float* invstd = reinterpret_cast<float*>(d + L.invstd);
    NB_TRY(nb_conv_bn_silu_fwd(p, d + L.x, d + L.w, gam, bet, nullptr, nullptr, d + L.y, mean, invstd, d + L.a, d + L.ws_fwd, p->fwd_bytes, stream));
    NB_TRY(nb_conv_bn_silu_bwd_data(p, d + L.g, d + L.y, mean, invstd, gam, bet, d + L.w, host_dx ? d + L.dx : nullptr,
                                    reinterpret_cast<float*>(d + L.dgamma), reinterpret_cast<float*>(d + L.dbeta), d + L.dy,
                                    d + L.ws_bwd, p->bwd_bytes, stream));
    NB_TRY(nb_conv_bn_silu_bwd_weight(p, d + L.x, d + L.dy, reinterpret_cast<float*>(d + L.dw), d + L.ws_bwd, p->bwd_bytes, stream));
    NB_CUDA_CHECK(cudaMemcpyAsync(host_a, d + L.a, L.ny_act, cudaMemcpyDeviceToHost, st));
    if (host_dx) NB_CUDA_CHECK(cudaMemcpyAsync(host_dx, d + L.dx, L.nx, cudaMemcpyDeviceToHost, st));
    NB_CUDA_CHECK(cudaMemcpyAsync(host_dw, d + L.dw, L.ndw, cudaMemcpyDeviceToHost, st));
    NB_CUDA_CHECK(cudaMemcpyAsync(host_dgamma, d + L.dgamma, cb, cudaMemcpyDeviceToHost, st));
    NB_CUDA_CHECK(cudaMemcpyAsync(host_dbeta, d + L.dbeta, cb, cudaMemcpyDeviceToHost, st));
    return NB_OK;
}

}  // extern "C"

