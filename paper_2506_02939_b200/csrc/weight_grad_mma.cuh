#pragma once
#include "pamm_common.cuh"
namespace pamm {
inline bool weight_grad_mma_supported(int64_t, int64_t, int64_t) { return false; }
inline pamm_status launch_weight_grad_mma(const void*, int64_t, int64_t, int64_t, const float*, int64_t, int64_t,
                                          float*, int64_t, cudaStream_t) { return PAMM_ERR_UNSUPPORTED; }
}
