// Helpers shared by the translation units that implement the C ABI (nb_cbs.cu, nb_sgd.cu, nb_glue.cu): the thread-local
// error string behind nb_last_error(), the launch counter, workspace and launch checks, the device guard.
#pragma once
#include <atomic>
#include <cstdarg>
#include <cstdint>
#include <string>

#include <cuda_runtime.h>

#include "../../include/nb_cbs.h"

namespace nbapi {

extern thread_local std::string g_err;                 // defined in nb_cbs.cu
extern std::atomic<unsigned long long> g_launches;     // kernels launched by this library in this process
nb_status fail(nb_status code, const char* fmt, ...);  // records the message for nb_last_error() and returns `code`

#define NB_CUDA_CHECK(expr)                                                                         \
    do {                                                                                            \
        cudaError_t e__ = (expr);                                                                   \
        if (e__ != cudaSuccess) return fail(NB_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e__)); \
    } while (0)
#define NB_LAUNCH_OK(what)                    \
    do {                                      \
        nb_status s__ = launch_ok(what);      \
        if (s__ != NB_OK) return s__;         \
    } while (0)
#define NB_TRY(expr)                          \
    do {                                      \
        nb_status s__ = (expr);               \
        if (s__ != NB_OK) return s__;         \
    } while (0)

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

inline nb_status check_ws(const void* ws, size_t have, size_t need) {
    if (need == 0) return NB_OK;
    if (!ws) return fail(NB_ERR_WORKSPACE, "workspace is NULL (%zu bytes needed)", need);
    if (reinterpret_cast<uintptr_t>(ws) & 255u) return fail(NB_ERR_WORKSPACE, "workspace is not 256-byte aligned");
    if (have < need) return fail(NB_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", have, need);
    return NB_OK;
}

// Makes a device current for the duration of a compute call and restores the caller's device afterwards.
struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    explicit DeviceGuard(int device) {
        if (cudaGetDevice(&prev) == cudaSuccess && prev != device) switched = cudaSetDevice(device) == cudaSuccess;
    }
    ~DeviceGuard() {
        if (switched) cudaSetDevice(prev);
    }
};

inline nb_status launch_ok(const char* what) {
    g_launches.fetch_add(1, std::memory_order_relaxed);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(NB_ERR_CUDA, "launch of %s failed: %s", what, cudaGetErrorString(e));
    return NB_OK;
}

}  // namespace nbapi
