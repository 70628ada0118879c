// Pieces shared by the tensor-core weight-gradient kernels (dW = C^T B~): both operands
// are "MN-major" for the tensor core -- C is k x n row-major, so for a fixed generator j
// the hidden index is contiguous, and likewise the columns of B~ (k x m).  B~ is fp32 and
// is split on the fly into bf16 hi + lo halves (hi = rn(x), lo = rn(x - hi); the pair
// carries about 16 mantissa bits), multiplied by two accumulating MMAs.
//
// Because the two operand tiles have the same shared-memory layout, either can play the
// M side: with C as the M operand the accumulator tile is a piece of dW in the paper's
// n x m layout, with B~ as the M operand it is a piece of dW^T (m x n, what a linear
// layer that keeps its weight as out x in wants).  The epilogue below is the same for
// both; only the tile's coordinates in the output differ.
#pragma once
#include "pamm_common.cuh"
#include "sm100_ptx.cuh"

namespace pamm {

constexpr int WG_TILE = 128;                 // output tile: 128 x 128
constexpr int WG_EPI_GROUP_THREADS = 128;    // the four epilogue warps
constexpr uint32_t WG_EPI_BARRIER0 = 1;      // named barriers 1 and 2: one per column half

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

// Splits eight consecutive fp32 values of one generator's B~ row into bf16 hi / lo and
// stores both as one 16-byte chunk of the swizzled MN-major operand layout.
//   jr  generator (row of the operand block, 128 bytes each)     cg  8-column group, 0..15
__device__ __forceinline__ void split_store_hi_lo(uint8_t* sBhi, uint8_t* sBlo, uint32_t blk_bytes, int jr, int cg,
                                                  const float4& a, const float4& b) {
    const float x[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    float h[8], l[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        h[e] = __bfloat162float(__float2bfloat16_rn(x[e]));
        l[e] = x[e] - h[e];
    }
    const uint32_t off = (uint32_t)(cg >> 3) * blk_bytes + (uint32_t)jr * 128u + (uint32_t)(((cg & 7) ^ (jr & 7)) << 4);
    *reinterpret_cast<uint4*>(sBhi + off) = make_uint4(pack_bf16(h[0], h[1]), pack_bf16(h[2], h[3]),
                                                       pack_bf16(h[4], h[5]), pack_bf16(h[6], h[7]));
    *reinterpret_cast<uint4*>(sBlo + off) = make_uint4(pack_bf16(l[0], l[1]), pack_bf16(l[2], l[3]),
                                                       pack_bf16(l[4], l[5]), pack_bf16(l[6], l[7]));
}

// Eight fp32 values of row j of B~ starting at column `col` (zeros past column m).
__device__ __forceinline__ void load_bt8(const float* __restrict__ Bt, int64_t ldb, int64_t j, int64_t col, int64_t m,
                                         bool full_cols, float4& a, float4& b) {
    const float* src = Bt + j * ldb + col;
    if (full_cols) {
        a = *reinterpret_cast<const float4*>(src);
        b = *reinterpret_cast<const float4*>(src + 4);
    } else {
        float x[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) x[e] = col + e < m ? src[e] : 0.f;
        a = make_float4(x[0], x[1], x[2], x[3]);
        b = make_float4(x[4], x[5], x[6], x[7]);
    }
}

// Staging of the output tile in shared memory: TMA boxes of 128 rows x 128 bytes
// (32 fp32 or 64 bf16 columns) in the 128-byte swizzle.  A column half of the tile
// (64 columns) is two fp32 boxes or one bf16 box.
template <typename OutT> struct WgOut;
template <> struct WgOut<float> {
    static constexpr int BOX_COLS = 32;
    static constexpr int HALF_BYTES = 2 * WG_TILE * 128;
};
template <> struct WgOut<__nv_bfloat16> {
    static constexpr int BOX_COLS = 64;
    static constexpr int HALF_BYTES = WG_TILE * 128;
};

// Epilogue of one column half of an output tile for one warp: the warp owns TMEM lanes
// [32 quad, 32 quad + 32) (= 32 rows of the tile) and handles the 64 columns of half `h`.  Accumulators go
// TMEM -> registers (scaled by beta) -> the half's staging area; the four warps of the half
// then meet and one thread hands the area to the TMA engine (store, or reduce-add for
// gradient accumulation).  `x0`, `y0` are the tile's column / row in the output matrix.
// The accumulator is handed back (`tempty`) as soon as it sits in registers.
// `ok == false` keeps only the barrier sequence going.  The two halves have a staging area
// each and alternate, so the store of one half is still reading shared memory while the other
// is staged: the leader waits until at most one of its earlier stores is still reading.
template <typename OutT>
__device__ __forceinline__ void wg_epilogue_half(const CUtensorMap* tm_w, uint32_t tmem_acc, uint64_t* tempty,
                                                 uint8_t* half_stage, int quad, int lane, int h, bool leader, int x0, int y0,
                                                 float beta, bool accumulate, bool ok) {
    const int row = quad * 32 + lane;
    const uint32_t lane_base = ((uint32_t)(quad * 32)) << 16;
    uint32_t v0[32], v1[32];
    if (ok) {
        ptx::tmem_ld_32x32(tmem_acc + lane_base + (uint32_t)(h * 64), v0);
        ptx::tmem_ld_32x32(tmem_acc + lane_base + (uint32_t)(h * 64 + 32), v1);
        ptx::tmem_ld_wait();
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(tempty);
        if (beta != 1.f) {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                v0[i] = __float_as_uint(beta * __uint_as_float(v0[i]));
                v1[i] = __float_as_uint(beta * __uint_as_float(v1[i]));
            }
        }
    }
    // the store that last used this staging area must have read it before it is overwritten
    if (leader) ptx::bulk_wait_group_read<1>();
    ptx::named_barrier(WG_EPI_BARRIER0 + (uint32_t)h, WG_EPI_GROUP_THREADS);
    if (ok) {
        if constexpr (sizeof(OutT) == 4) {
            uint8_t* d0 = half_stage + row * 128;
            uint8_t* d1 = d0 + WG_TILE * 128;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                *reinterpret_cast<uint4*>(d0 + ((c ^ (row & 7)) << 4)) = make_uint4(v0[4 * c], v0[4 * c + 1], v0[4 * c + 2], v0[4 * c + 3]);
                *reinterpret_cast<uint4*>(d1 + ((c ^ (row & 7)) << 4)) = make_uint4(v1[4 * c], v1[4 * c + 1], v1[4 * c + 2], v1[4 * c + 3]);
            }
        } else {
            uint8_t* d0 = half_stage + row * 128;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                *reinterpret_cast<uint4*>(d0 + ((c ^ (row & 7)) << 4)) =
                    make_uint4(pack_bf16(__uint_as_float(v0[8 * c]), __uint_as_float(v0[8 * c + 1])),
                               pack_bf16(__uint_as_float(v0[8 * c + 2]), __uint_as_float(v0[8 * c + 3])),
                               pack_bf16(__uint_as_float(v0[8 * c + 4]), __uint_as_float(v0[8 * c + 5])),
                               pack_bf16(__uint_as_float(v0[8 * c + 6]), __uint_as_float(v0[8 * c + 7])));
                *reinterpret_cast<uint4*>(d0 + (((c + 4) ^ (row & 7)) << 4)) =
                    make_uint4(pack_bf16(__uint_as_float(v1[8 * c]), __uint_as_float(v1[8 * c + 1])),
                               pack_bf16(__uint_as_float(v1[8 * c + 2]), __uint_as_float(v1[8 * c + 3])),
                               pack_bf16(__uint_as_float(v1[8 * c + 4]), __uint_as_float(v1[8 * c + 5])),
                               pack_bf16(__uint_as_float(v1[8 * c + 6]), __uint_as_float(v1[8 * c + 7])));
            }
        }
    }
    ptx::fence_proxy_async();
    ptx::named_barrier(WG_EPI_BARRIER0 + (uint32_t)h, WG_EPI_GROUP_THREADS);
    if (leader) {
        if (ok) {
            constexpr int BOXES = WgOut<OutT>::HALF_BYTES / (WG_TILE * 128);
#pragma unroll
            for (int q = 0; q < BOXES; ++q) {
                const int x = x0 + h * 64 + q * WgOut<OutT>::BOX_COLS;
                if (accumulate) ptx::tma_reduce_add_2d(tm_w, half_stage + q * (WG_TILE * 128), x, y0);
                else            ptx::tma_store_2d(tm_w, half_stage + q * (WG_TILE * 128), x, y0);
            }
        }
        ptx::bulk_commit_group();
    }
}

}  // namespace pamm
