// Pieces shared by the tensor-core weight-gradient kernels (dW = C^T B~): both operands
// are "MN-major" for the tensor core -- C is k x n row-major, so for a fixed generator j
// the hidden index is contiguous, and likewise the columns of B~ (k x m).  B~ is fp32 and
// is split on the fly into bf16 hi + lo halves (hi = rn(x), lo = rn(x - hi); the pair
// carries about 16 mantissa bits), multiplied by two accumulating MMAs.
#pragma once
#include "pamm_common.cuh"
#include "sm100_ptx.cuh"

namespace pamm {

// Shared-memory operand descriptor, MN-major, 128-byte swizzle: blocks of 64
// elements along M/N (128 bytes) x 8 along K are 1024 bytes; successive 8-deep K
// groups are `sbo` bytes apart, successive 64-wide M/N blocks `lbo` bytes apart.
__device__ __forceinline__ uint64_t umma_desc_mn_sw128(uint32_t smem_addr, uint32_t lbo, uint32_t sbo) {
    return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo >> 4) & 0x3FFFu) << 32) | ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo_elem, float hi_elem) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo_elem, hi_elem);   // .x = first argument = low 16 bits
    return *reinterpret_cast<uint32_t*>(&t);
}

}  // namespace pamm
