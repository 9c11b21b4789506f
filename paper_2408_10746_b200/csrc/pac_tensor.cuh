// Tensor-core path (tcgen05 + TMA) for bf16 caches: interface used by the host runtime.
#pragma once
#include "pac_common.cuh"

namespace pac {

struct TensorPlan {
    bool ready = false;
};

inline const char* tensor_last_error() { return "tensor path not built"; }
inline bool tensor_shape_supported(const Dims&) { return false; }
inline pac_status tensor_plan_create(TensorPlan&, int, const bf16*, const Dims&, int, const bf16*, const bf16*, long long*) {
    return PAC_ERR_UNSUPPORTED;
}
inline void tensor_plan_destroy(TensorPlan&) {}
inline pac_status tensor_down_projection(TensorPlan&, cudaStream_t, const int*, int, float*, unsigned*, long long*) {
    return PAC_ERR_UNSUPPORTED;
}
inline pac_status tensor_dw_down(TensorPlan&, cudaStream_t, const int*, int, const bf16*, float*, float*, unsigned*, long long*) {
    return PAC_ERR_UNSUPPORTED;
}

}  // namespace pac
