// Step 4 on tensor cores (bf16 generators): dW = C^T B~ (Algorithm 1 ApproxMM,
// "O~ <- C^T B~") with tcgen05.mma, one CTA per 128 x 128 tile of dW.
//
// Both operands are "MN-major" for the tensor core: C is k x n row-major, so for
// a fixed generator j the n-index is contiguous, and likewise B~ (k x m).  The C
// tile arrives by TMA (boxes of 64 columns x KC generators, 128-byte swizzle).
// B~ is fp32: the CTA splits it on the fly into bf16 hi + lo halves
// (hi = rn(x), lo = rn(x - hi); the pair carries ~16 mantissa bits) and writes
// them into shared memory in the same swizzled layout, so the product is two
// accumulating MMAs per 16 generators.  The contraction length k is tiny, so
// the kernel is bound by writing dW (fp32) and two CTAs per SM overlap one
// tile's loads with the other's stores.
#pragma once
#include "pamm_common.cuh"
#include "sm100_ptx.cuh"

namespace pamm {

constexpr int WU_THREADS = 256;
constexpr int WU_TILE = 128;          // output tile is WU_TILE x WU_TILE
constexpr int WU_KC_MAX = 128;        // generators per shared-memory chunk

inline bool weight_grad_mma_supported(int64_t k, int64_t n, int64_t m) {
    return k >= 8 && n >= 8 && m >= 4 && n < (1ll << 31) && m < (1ll << 31) && k < (1ll << 24);
}

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

__global__ void __launch_bounds__(WU_THREADS, 2)
weight_grad_umma_kernel(const __grid_constant__ CUtensorMap tm_c, const float* __restrict__ Bt, int64_t ldb,
                        int k, int n, int m, int kc, int nchunks, float* __restrict__ dW, int64_t ldw,
                        int64_t b_rows, const int32_t* __restrict__ dropped, int accumulate) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_tma, s_mma;
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t blk_bytes = (uint32_t)kc * 128u;       // one 64-wide block: kc rows of 128 bytes
    uint8_t* sA = base;                                    // 2 blocks (128 rows of dW)
    uint8_t* sBhi = sA + 2 * blk_bytes;                    // 2 blocks (128 columns of dW)
    uint8_t* sBlo = sBhi + 2 * blk_bytes;
    const int n0 = blockIdx.y * WU_TILE, m0 = blockIdx.x * WU_TILE;

    if (tid == 0) {
        ptx::mbar_init(&s_tma, 1);
        ptx::mbar_init(&s_mma, 1);
        s_abort = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async();
    }
    if (warp == 0) {
        ptx::tmem_alloc(&s_tmem_base, WU_TILE);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = s_tmem_base;
    volatile int* abort_flag = &s_abort;
    grid_dependency_wait();     // B~ (and C) may come from the kernel before
    grid_launch_dependents();
    // kind::f16, D fp32, A/B bf16, both MN-major (bits 15 and 16), M = N = 128
    const uint32_t idesc = ptx::umma_idesc_bf16(WU_TILE, WU_TILE) | (1u << 15) | (1u << 16);
    bool ok = true;

    for (int c = 0; c < nchunks; ++c) {
        if (c > 0) {   // the previous chunk's MMAs must have read shared memory before it is overwritten
            ok = ptx::mbar_wait(&s_mma, (uint32_t)(c - 1) & 1u, abort_flag);
            ok = __syncthreads_and(ok);
            if (!ok) break;
        }
        const int j0 = c * kc;
        if (tid == 0) {
            ptx::mbar_arrive_expect_tx(&s_tma, 2 * blk_bytes);
            ptx::tma_load_2d(sA, &tm_c, n0, j0, &s_tma);
            ptx::tma_load_2d(sA + blk_bytes, &tm_c, n0 + 64, j0, &s_tma);
        }
        // B~ chunk: kc rows x 128 columns fp32 -> bf16 hi / lo, swizzled MN-major blocks
        for (int g = tid; g < kc * 16; g += WU_THREADS) {
            const int jr = g >> 4;                 // row inside the chunk
            const int cg = g & 15;                 // group of 8 columns
            const int j = j0 + jr;
            const int64_t col = (int64_t)m0 + cg * 8;
            float x[8];
            if (j < k && col + 8 <= m) {
                const float4 a = __ldg(reinterpret_cast<const float4*>(Bt + (int64_t)j * ldb + col));
                const float4 b4 = __ldg(reinterpret_cast<const float4*>(Bt + (int64_t)j * ldb + col + 4));
                x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b4.x; x[5] = b4.y; x[6] = b4.z; x[7] = b4.w;
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) x[e] = (j < k && col + e < m) ? __ldg(Bt + (int64_t)j * ldb + col + e) : 0.f;
            }
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
        ptx::fence_proxy_async();    // generic-proxy stores -> visible to the tensor core's async proxy
        __syncthreads();
        if (tid == 0) {
            if (ptx::mbar_wait(&s_tma, (uint32_t)c & 1u, abort_flag)) {
                ptx::tc_fence_after_sync();
                const uint32_t a_addr = ptx::smem_u32(sA), bh_addr = ptx::smem_u32(sBhi), bl_addr = ptx::smem_u32(sBlo);
                for (int kk = 0; kk < kc / 16; ++kk) {   // 16 generators = two 8-deep K groups = 2048 bytes
                    const uint64_t da = umma_desc_mn_sw128(a_addr + kk * 2048, blk_bytes, 1024);
                    const uint64_t dh = umma_desc_mn_sw128(bh_addr + kk * 2048, blk_bytes, 1024);
                    const uint64_t dl = umma_desc_mn_sw128(bl_addr + kk * 2048, blk_bytes, 1024);
                    ptx::umma_bf16(tmem_base, da, dh, idesc, (c | kk) != 0);
                    ptx::umma_bf16(tmem_base, da, dl, idesc, true);
                }
            } else {
                raise_status(DEV_TIMEOUT);
            }
            ptx::umma_commit(&s_mma);
        }
    }
    if (ok) ok = ptx::mbar_wait(&s_mma, (uint32_t)(nchunks - 1) & 1u, abort_flag);
    ok = __syncthreads_and(ok);
    if (ok) {
        ptx::tc_fence_after_sync();
        // epilogue: thread = one row of the tile; warps 0-3 take columns [0,64), warps 4-7 [64,128)
        const int quad = warp & 3, half = warp >> 2;
        const int64_t row = (int64_t)n0 + quad * 32 + lane;
        const float beta = beta_factor(dropped, b_rows);
#pragma unroll
        for (int c0 = 0; c0 < 64; c0 += 32) {
            uint32_t v[32];
            ptx::tmem_ld_32x32(tmem_base + (((uint32_t)(quad * 32)) << 16) + (uint32_t)(half * 64 + c0), v);
            ptx::tmem_ld_wait();
            const int64_t col = (int64_t)m0 + half * 64 + c0;
            if (row < n) {
                float* out = dW + row * ldw + col;
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                    if (col + i + 4 <= m) {
                        float4 o = make_float4(beta * __uint_as_float(v[i]), beta * __uint_as_float(v[i + 1]),
                                               beta * __uint_as_float(v[i + 2]), beta * __uint_as_float(v[i + 3]));
                        if (accumulate) {
                            const float4 old = *reinterpret_cast<const float4*>(out + i);
                            o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
                        }
                        *reinterpret_cast<float4*>(out + i) = o;
                    } else {
                        for (int e = 0; e < 4; ++e)
                            if (col + i + e < m) out[i + e] = beta * __uint_as_float(v[i + e]) + (accumulate ? out[i + e] : 0.f);
                    }
                }
            }
        }
    } else if (tid == 0) {
        raise_status(DEV_TIMEOUT);
        int never = 0;
        volatile int* no_abort = &never;
        ptx::mbar_wait(&s_tma, 0, no_abort);   // at most one pair of copies can still be in flight
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, WU_TILE);
    }
}

inline pamm_status launch_weight_grad_mma(const void* C, int64_t ldc, int64_t k, int64_t n, const float* Bt, int64_t ldb,
                                          int64_t m, float* dW, int64_t ldw, cudaStream_t st, int64_t b_rows = 0,
                                          const int32_t* dropped = nullptr, bool accumulate = false) {
    const int kpad = (int)round_up(k, 16);
    const int kc = std::min(kpad, WU_KC_MAX);
    const int nchunks = (kpad + kc - 1) / kc;
    CUtensorMap tm_c;
    if (!make_tmap_bf16_sw128(&tm_c, C, (uint64_t)k, (uint64_t)n, (uint64_t)ldc, (uint32_t)kc)) return PAMM_ERR_CUDA;
    const size_t smem = 1024 + (size_t)6 * kc * 128;
    if (cudaFuncSetAttribute(weight_grad_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return PAMM_ERR_CUDA;
    dim3 grid((unsigned)((m + WU_TILE - 1) / WU_TILE), (unsigned)((n + WU_TILE - 1) / WU_TILE));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(WU_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // set up while the kernel before drains
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, weight_grad_umma_kernel, tm_c, Bt, ldb, (int)k, (int)n, (int)m, kc, nchunks, dW, ldw, b_rows,
                       dropped, accumulate ? 1 : 0);
    return cudaGetLastError() == cudaSuccess ? PAMM_OK : PAMM_ERR_CUDA;
}

}  // namespace pamm
