#pragma once
#include "pamm_common.cuh"
namespace pamm {
inline bool compress_umma_supported(int64_t, int64_t, int64_t) { return false; }
inline pamm_status launch_compress_umma(const void*, int64_t, int64_t, int64_t, const void*, int64_t, int64_t,
                                        const float*, int32_t*, float*, cudaStream_t) { return PAMM_ERR_UNSUPPORTED; }
}
