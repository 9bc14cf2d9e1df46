// Tensor-core (tcgen05 / TMEM / TMA) convolution kernels: plan record and entry points.
#pragma once
#include "common.cuh"
#include "../../include/nb_cbs.h"

namespace nbcbs {

struct TcPlan {
    bool fprop = false, dgrad = false, wgrad = false;
    int fprop_parts = 0;             // rows of the [parts][2][Cout] partial-sum buffer the fprop epilogue writes
    size_t wt_bytes = 0;             // rearranged filter for dgrad
    size_t wgrad_partial_bytes = 0;  // split-K partial buffer of the wgrad kernel
};

inline const char* tc_last_error() { return ""; }

inline nb_status tc_plan_init(TcPlan* tc, const Geom&, bool, int, const cudaDeviceProp&) {
    *tc = TcPlan();
    return NB_OK;
}
inline nb_status tc_fprop(TcPlan*, const Geom&, const void*, const void*, void*, float*, int*, cudaStream_t) { return NB_ERR_INTERNAL; }
inline nb_status tc_dgrad(TcPlan*, const Geom&, const void*, const void*, void*, void*, int*, cudaStream_t) { return NB_ERR_INTERNAL; }
inline nb_status tc_wgrad(TcPlan*, const Geom&, const void*, const void*, float*, float*, int*, cudaStream_t) { return NB_ERR_INTERNAL; }

}  // namespace nbcbs
