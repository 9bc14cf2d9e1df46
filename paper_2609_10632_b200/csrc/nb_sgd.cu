// C ABI of the fused optimiser step (see include/nb_sgd.h): tensor-list plans, the clip + SGD-Nesterov step and its
// loss-scaled form.  Host memory only; the workspace is the caller's.
#include <algorithm>
#include <cstring>
#include <new>
#include <vector>

#include "api_common.cuh"
#include "common.cuh"
#include "sgd.cuh"

using namespace nbcbs;
using namespace nbapi;

// ---------------------------------------------------------------- fused optimiser step (include/nb_sgd.h)
struct nb_sgd_plan_s {
    int device = 0;
    SgdHeader h;
    std::vector<uint8_t> image;  // header + tensor list + chunk table, as they sit at the start of the workspace
};

extern "C" {

nb_status nb_sgd_plan_create(const nb_sgd_tensor* t, int32_t count, int device, nb_sgd_plan* out) {
    g_err.clear();
    if (!out) return fail(NB_ERR_INVALID_ARG, "out_plan is NULL");
    *out = nullptr;
    if (!t) return fail(NB_ERR_INVALID_ARG, "host_tensors is NULL");
    if (count <= 0) return fail(NB_ERR_INVALID_ARG, "count must be positive, got %d", count);
    long long nchunks = 0;
    for (int i = 0; i < count; ++i) {
        if (t[i].numel <= 0) return fail(NB_ERR_INVALID_ARG, "tensor %d: numel must be positive", i);
        if (t[i].group < 0 || t[i].group >= NB_SGD_GROUPS) return fail(NB_ERR_INVALID_ARG, "tensor %d: group %d out of range", i, t[i].group);
        if (!t[i].grad || !t[i].param || !t[i].momentum) return fail(NB_ERR_INVALID_ARG, "tensor %d: grad, param and momentum must not be NULL", i);
        if (t[i].copy_dtype != 0 && t[i].copy_dtype != NB_DTYPE_BF16 && t[i].copy_dtype != NB_DTYPE_F16)
            return fail(NB_ERR_INVALID_ARG, "tensor %d: copy_dtype %d is neither bf16 nor fp16", i, t[i].copy_dtype);
        const uintptr_t bits = reinterpret_cast<uintptr_t>(t[i].grad) | reinterpret_cast<uintptr_t>(t[i].param) |
                               reinterpret_cast<uintptr_t>(t[i].momentum) | reinterpret_cast<uintptr_t>(t[i].param_bf16);
        if (bits & 15u) return fail(NB_ERR_ALIGNMENT, "tensor %d: a pointer is not 16-byte aligned", i);
        nchunks += (t[i].numel + SGD_CHUNK - 1) / SGD_CHUNK;
    }
    if (nchunks > 0x7fffffffLL) return fail(NB_ERR_UNSUPPORTED, "too many elements for one tensor list");
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
        cudaGetLastError();
        return fail(NB_ERR_CUDA, "cannot query device %d", device);
    }
    nb_sgd_plan_s* p = new (std::nothrow) nb_sgd_plan_s;
    if (!p) return fail(NB_ERR_INTERNAL, "out of host memory");
    p->device = device;
    SgdHeader& h = p->h;
    memset(&h, 0, sizeof h);
    h.magic = SGD_MAGIC;
    h.count = count;
    h.nchunks = (int32_t)nchunks;
    h.grid = (int32_t)std::min<long long>(nchunks, std::min<long long>(SGD_MAX_BLOCKS, (long long)std::max(sms, 1) * 8));
    size_t off = 256;
    h.off_tensors = off; off = align_up(off + (size_t)count * sizeof(nb_sgd_tensor), 256);
    h.off_chunks = off; off = align_up(off + (size_t)nchunks * sizeof(SgdChunk), 256);
    h.off_partials = off; off = align_up(off + (size_t)SGD_MAX_BLOCKS * sizeof(double), 256);
    h.total_bytes = off;
    p->image.assign((size_t)h.off_partials, 0);
    memcpy(p->image.data(), &h, sizeof h);
    memcpy(p->image.data() + h.off_tensors, t, (size_t)count * sizeof(nb_sgd_tensor));
    SgdChunk* c = reinterpret_cast<SgdChunk*>(p->image.data() + h.off_chunks);  // chunk i goes to block i % grid
    for (int i = 0; i < count; ++i)
        for (int64_t s = 0; s < t[i].numel; s += SGD_CHUNK, ++c) {
            c->tensor = i;
            c->start = s;
            c->len = (int32_t)std::min<int64_t>(SGD_CHUNK, t[i].numel - s);
        }
    *out = p;
    return NB_OK;
}

nb_status nb_sgd_plan_destroy(nb_sgd_plan p) {
    g_err.clear();
    delete p;
    return NB_OK;
}

nb_status nb_sgd_workspace_bytes(nb_sgd_plan p, size_t* bytes) {
    g_err.clear();
    if (!p || !bytes) return fail(NB_ERR_INVALID_ARG, "NULL argument");
    *bytes = (size_t)p->h.total_bytes;
    return NB_OK;
}

nb_status nb_sgd_upload(nb_sgd_plan p, void* workspace, size_t workspace_bytes, void* stream) {
    g_err.clear();
    if (!p) return fail(NB_ERR_INVALID_ARG, "plan is NULL");
    NB_TRY(check_ws(workspace, workspace_bytes, (size_t)p->h.total_bytes));
    DeviceGuard on_device(p->device);
    // the source is the plan's own host image, which lives as long as the plan
    NB_CUDA_CHECK(cudaMemcpyAsync(workspace, p->image.data(), p->image.size(), cudaMemcpyHostToDevice, static_cast<cudaStream_t>(stream)));
    return NB_OK;
}

namespace {
nb_status sgd_step_impl(nb_sgd_plan p, void* workspace, size_t workspace_bytes, const nb_sgd_hyper* hyper, const nb_scaler_hyper* sc, nb_loss_scaler* state,
                        float* total_norm, void* stream);
}
nb_status nb_sgd_clip_nesterov_step(nb_sgd_plan p, void* workspace, size_t workspace_bytes, const nb_sgd_hyper* hyper, float* total_norm,
                                    void* stream) {
    g_err.clear();
    return sgd_step_impl(p, workspace, workspace_bytes, hyper, nullptr, nullptr, total_norm, stream);
}

nb_status nb_sgd_clip_nesterov_step_scaled(nb_sgd_plan p, void* workspace, size_t workspace_bytes, const nb_sgd_hyper* hyper, const nb_scaler_hyper* sc,
                                           nb_loss_scaler* state, float* total_norm, void* stream) {
    g_err.clear();
    if (!sc || !state) return fail(NB_ERR_INVALID_ARG, "scaler and state must not be NULL");
    if (sc->struct_size != sizeof(nb_scaler_hyper)) return fail(NB_ERR_INVALID_ARG, "nb_scaler_hyper.struct_size is %u, expected %zu", sc->struct_size, sizeof(nb_scaler_hyper));
    if (reinterpret_cast<uintptr_t>(state) & 15u) return fail(NB_ERR_ALIGNMENT, "state is not 16-byte aligned");
    if (!(sc->growth_factor > 0.f) || !(sc->backoff_factor > 0.f) || sc->growth_interval < 1) return fail(NB_ERR_INVALID_ARG, "scaler factors must be positive, growth_interval >= 1");
    return sgd_step_impl(p, workspace, workspace_bytes, hyper, sc, state, total_norm, stream);
}

}  // extern "C"

namespace {
nb_status sgd_step_impl(nb_sgd_plan p, void* workspace, size_t workspace_bytes, const nb_sgd_hyper* hyper, const nb_scaler_hyper* sc, nb_loss_scaler* state,
                        float* total_norm, void* stream) {
    if (!p) return fail(NB_ERR_INVALID_ARG, "plan is NULL");
    if (!hyper) return fail(NB_ERR_INVALID_ARG, "hyper is NULL");
    if (hyper->struct_size != sizeof(nb_sgd_hyper))
        return fail(NB_ERR_INVALID_ARG, "nb_sgd_hyper.struct_size is %u, expected %zu", hyper->struct_size, sizeof(nb_sgd_hyper));
    NB_TRY(check_ws(workspace, workspace_bytes, (size_t)p->h.total_bytes));
    if (reinterpret_cast<uintptr_t>(total_norm) & 3u) return fail(NB_ERR_ALIGNMENT, "total_norm is not 4-byte aligned");
    DeviceGuard on_device(p->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    SgdScalars s;
    s.momentum = hyper->momentum; s.max_norm = hyper->max_norm; s.first_step = hyper->first_step;
    s.scaler = state;
    for (int i = 0; i < NB_SGD_GROUPS; ++i) { s.lr[i] = hyper->lr[i]; s.wd[i] = hyper->weight_decay[i]; }
    const uint8_t* ws = static_cast<const uint8_t*>(workspace);
    launch_k(sgd_sqnorm_kernel, dim3((unsigned)p->h.grid), dim3(SGD_THREADS), 0, st, 1, ws);
    NB_LAUNCH_OK("sgd_sqnorm");
    launch_k(sgd_update_kernel, dim3((unsigned)p->h.grid), dim3(SGD_THREADS), 0, st, 1, ws, s, total_norm);
    NB_LAUNCH_OK("sgd_update");
    if (state) {
        launch_k(sgd_scaler_kernel, dim3(1), dim3(32), 0, st, 1, ws, state, sc->growth_factor, sc->backoff_factor, sc->floor_scale, (int)sc->growth_interval);
        NB_LAUNCH_OK("sgd_scaler");
    }
    return NB_OK;
}
}  // namespace

