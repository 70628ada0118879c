// Step 4 on tensor cores for k > 128 (bf16 generators): dW = C^T B~ (Algorithm 1
// ApproxMM, the final product), persistent and pipelined over chunks of 64 generators.
//
// One CTA per SM takes a contiguous run of 128 x 128 output tiles (numbered column
// block by column block, so neighbours share their B~ columns in L2).  Every tile
// walks the generators in chunks of 64 through a ring of three shared-memory stages;
// a stage holds the C chunk (A operand, by TMA) and the B~ chunk split into bf16
// hi + lo (B operands):
//   warp 0       TMA producer of the C chunks
//   warp 1       issues tcgen05.mma: D (+)= A Bhi + A Blo, two TMEM accumulators
//   warps 2-5    epilogue: TMEM -> registers -> swizzled shared memory -> TMA store
//                (or reduce-add), two halves of 64 columns in flight
//   warps 6-17   three groups of four warps; group q owns stage q and converts the
//                fp32 B~ chunk that goes there (hi = rn(x), lo = rn(x - hi)), all of a
//                thread's sixteen 16-byte loads in flight at once, so three chunks
//                are being fetched from L2 at any time
// Operand layouts, descriptors and the epilogue are those of the k <= 128 kernel.
#pragma once
#include "pamm_common.cuh"
#include "sm100_ptx.cuh"
#include "weight_grad_persist.cuh"

namespace pamm {

constexpr int WC_THREADS = 576;
constexpr int WC_KC = 64;                                 // generators per chunk
constexpr int WC_STAGES = 3;
constexpr int WC_GROUP_THREADS = 128;                     // converter threads per stage
constexpr uint32_t WC_BLK_BYTES = WC_KC * 128;            // one 64-wide block of a chunk
constexpr uint32_t WC_STAGE_BYTES = 6 * WC_BLK_BYTES;     // A, Bhi, Blo: two blocks each

inline bool weight_grad_chunked_supported(int64_t k, int64_t n, int64_t m) {
    return k >= 8 && n >= 8 && m >= 4 && n < (1ll << 31) && m < (1ll << 31) && k < (1ll << 24);
}

__global__ void __launch_bounds__(WC_THREADS, 1)
weight_grad_chunked_kernel(const __grid_constant__ CUtensorMap tm_c, const __grid_constant__ CUtensorMap tm_w,
                           const float* __restrict__ Bt, int64_t ldb, int k, int m, int nch, int n_tiles,
                           int total_tiles, int64_t b_rows, const int32_t* __restrict__ dropped, int accumulate) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_full[WC_STAGES], s_empty[WC_STAGES], s_tfull[2], s_tempty[2];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* sStages = base;
    uint8_t* sOut = base + WC_STAGES * WC_STAGE_BYTES;     // two halves

    const int t0 = (int)((int64_t)blockIdx.x * total_tiles / gridDim.x);
    const int t1 = (int)((int64_t)(blockIdx.x + 1) * total_tiles / gridDim.x);
    const uint32_t total_chunks = (uint32_t)(t1 - t0) * (uint32_t)nch;

    if (tid == 0) {
        for (int s = 0; s < WC_STAGES; ++s) {
            ptx::mbar_init(&s_full[s], 1 + WC_GROUP_THREADS / 32);   // the producer's arrive + one per converter warp
            ptx::mbar_init(&s_empty[s], 1);
        }
        for (int u = 0; u < 2; ++u) {
            ptx::mbar_init(&s_tfull[u], 1);
            ptx::mbar_init(&s_tempty[u], 4);
        }
        s_abort = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async();
    }
    if (warp == 1) {
        ptx::tmem_alloc(&s_tmem_base, 2 * WP_TILE);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = s_tmem_base;
    volatile int* abort_flag = &s_abort;
    grid_dependency_wait();     // B~ (and C) may come from the kernel before
    grid_launch_dependents();

    if (warp == 0) {
        // ---------------- TMA producer: C chunks ----------------
        if (ptx::elect_one()) {
            ptx::prefetch_tensormap(&tm_c);
            uint32_t g = 0;
            bool ok = true;
            for (; g < total_chunks; ++g) {
                const int s = g % WC_STAGES;
                if (!ptx::mbar_wait(&s_empty[s], ((g / WC_STAGES) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                const int t = t0 + (int)(g / (uint32_t)nch), c = (int)(g % (uint32_t)nch);
                const int n0 = (t % n_tiles) * WP_TILE;
                uint8_t* dst = sStages + (size_t)s * WC_STAGE_BYTES;
                ptx::mbar_arrive_expect_tx(&s_full[s], 2 * WC_BLK_BYTES);
                ptx::tma_load_2d(dst, &tm_c, n0, c * WC_KC, &s_full[s]);
                ptx::tma_load_2d(dst + WC_BLK_BYTES, &tm_c, n0 + 64, c * WC_KC, &s_full[s]);
            }
            if (!ok) {
                raise_status(DEV_TIMEOUT);
                // A stage completes only together with its converters' arrivals, which may never come now,
                // so the copies already issued cannot be waited for on their barrier: give them time to land
                // (they take microseconds) before this warp lets the CTA go.
                for (int i = 0; i < 64; ++i) __nanosleep(1000);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (ptx::elect_one()) {
            // kind::f16, D fp32, A/B bf16, both MN-major (bits 15 and 16), M = N = 128
            const uint32_t idesc = ptx::umma_idesc_bf16(WP_TILE, WP_TILE) | (1u << 15) | (1u << 16);
            bool ok = true;
            for (uint32_t g = 0; g < total_chunks && ok; ++g) {
                const int s = g % WC_STAGES;
                const uint32_t it = g / (uint32_t)nch, c = g % (uint32_t)nch;
                const uint32_t buf = it & 1u;
                if (c == 0 && !ptx::mbar_wait(&s_tempty[buf], ((it >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                if (!ptx::mbar_wait(&s_full[s], (g / WC_STAGES) & 1u, abort_flag)) { ok = false; break; }
                ptx::tc_fence_after_sync();
                const uint32_t a_addr = ptx::smem_u32(sStages + (size_t)s * WC_STAGE_BYTES);
                const uint32_t bh_addr = a_addr + 2 * WC_BLK_BYTES, bl_addr = a_addr + 4 * WC_BLK_BYTES;
                const uint32_t d_addr = tmem_base + buf * (uint32_t)WP_TILE;
#pragma unroll
                for (int kk = 0; kk < WC_KC / 16; ++kk) {   // 16 generators = two 8-deep K groups = 2048 bytes
                    const uint64_t da = umma_desc_mn_sw128(a_addr + kk * 2048, WC_BLK_BYTES, 1024);
                    const uint64_t dh = umma_desc_mn_sw128(bh_addr + kk * 2048, WC_BLK_BYTES, 1024);
                    const uint64_t dl = umma_desc_mn_sw128(bl_addr + kk * 2048, WC_BLK_BYTES, 1024);
                    ptx::umma_bf16(d_addr, da, dh, idesc, (c | (uint32_t)kk) != 0);
                    ptx::umma_bf16(d_addr, da, dl, idesc, true);
                }
                ptx::umma_commit(&s_empty[s]);
                if (c + 1 == (uint32_t)nch) ptx::umma_commit(&s_tfull[buf]);
            }
            if (!ok) raise_status(DEV_TIMEOUT);
        }
    } else if (warp < 6) {
        // ---------------- epilogue: one row of the tile per thread ----------------
        const int etid = tid - 64;
        const int quad = warp & 3;                       // TMEM lanes [32*quad, 32*quad+32)
        const int row = quad * 32 + lane;
        const uint32_t lane_base = ((uint32_t)(quad * 32)) << 16;
        const float beta = beta_factor(dropped, b_rows);     // Eq. 4-5; 1 unless rows were dropped
        uint32_t it = 0;
        bool ok = true;   // once false this warp only keeps the barrier sequence going
        for (int t = t0; t < t1; ++t, ++it) {
            const int s = it & 1;
            const int n0 = (t % n_tiles) * WP_TILE, m0 = (t / n_tiles) * WP_TILE;
            if (ok) ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_tfull[s], (it >> 1) & 1u, abort_flag));
            ptx::tc_fence_after_sync();
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                if (etid == 0) ptx::bulk_wait_group_read<1>();   // the store that last used this half has read it
                ptx::named_barrier(WP_EPI_BARRIER, WP_EPI_THREADS);
                uint8_t* half = sOut + h * WP_OUT_HALF_BYTES;
                if (ok) {
#pragma unroll
                    for (int gg = 0; gg < 2; ++gg) {
                        uint32_t v[32];
                        ptx::tmem_ld_32x32(tmem_base + lane_base + (uint32_t)(s * WP_TILE + (h * 2 + gg) * 32), v);
                        ptx::tmem_ld_wait();
                        if (beta != 1.f) {
#pragma unroll
                            for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(beta * __uint_as_float(v[i]));
                        }
                        uint8_t* dst = half + gg * (WP_TILE * 128) + row * 128;
#pragma unroll
                        for (int c = 0; c < 8; ++c)
                            *reinterpret_cast<uint4*>(dst + ((c ^ (row & 7)) << 4)) =
                                make_uint4(v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3]);
                    }
                }
                if (h == 1) {   // every TMEM read of this tile is done: hand the accumulator back
                    ptx::tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0 && ok) ptx::mbar_arrive(&s_tempty[s]);
                }
                ptx::fence_proxy_async();
                ptx::named_barrier(WP_EPI_BARRIER, WP_EPI_THREADS);
                if (etid == 0) {
                    if (ok && !accumulate) {
                        ptx::tma_store_2d(&tm_w, half, m0 + h * 64, n0);
                        ptx::tma_store_2d(&tm_w, half + WP_TILE * 128, m0 + h * 64 + 32, n0);
                    } else if (ok) {     // dW += tile (gradient accumulation)
                        ptx::tma_reduce_add_2d(&tm_w, half, m0 + h * 64, n0);
                        ptx::tma_reduce_add_2d(&tm_w, half + WP_TILE * 128, m0 + h * 64 + 32, n0);
                    }
                    ptx::bulk_commit_group();
                }
            }
        }
        if (etid == 0) ptx::bulk_wait_group<0>();
        if (!ok && lane == 0) raise_status(DEV_TIMEOUT);
    } else {
        // ---------------- B~ chunks: fp32 -> bf16 hi / lo, swizzled MN-major; group q feeds stage q ----------------
        const int q = (warp - 6) >> 2;                       // stage this group owns
        const int gt = tid - 192 - q * WC_GROUP_THREADS;     // thread inside the group
        bool ok = true;
        for (uint32_t g = (uint32_t)q; g < total_chunks && ok; g += WC_STAGES) {
            ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_empty[q], ((g / WC_STAGES) & 1u) ^ 1u, abort_flag));
            if (!ok) break;
            const int t = t0 + (int)(g / (uint32_t)nch), c = (int)(g % (uint32_t)nch);
            const int64_t m0 = (int64_t)(t / n_tiles) * WP_TILE;
            const int j0 = c * WC_KC;
            const bool full_cols = m0 + WP_TILE <= m;
            uint8_t* sBhi = sStages + (size_t)q * WC_STAGE_BYTES + 2 * WC_BLK_BYTES;
            uint8_t* sBlo = sBhi + 2 * WC_BLK_BYTES;
            constexpr int ITEMS = WC_KC * 16 / WC_GROUP_THREADS;     // 8-column groups per thread: 8
            float4 lo4[ITEMS], hi4[ITEMS];
#pragma unroll
            for (int u = 0; u < ITEMS; ++u) {     // all loads first
                const int idx = gt + u * WC_GROUP_THREADS;
                const int j = j0 + (idx >> 4);
                const int64_t col = m0 + (idx & 15) * 8;
                lo4[u] = hi4[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (j < k) {
                    const float* src = Bt + (int64_t)j * ldb + col;
                    if (full_cols) {
                        lo4[u] = *reinterpret_cast<const float4*>(src);
                        hi4[u] = *reinterpret_cast<const float4*>(src + 4);
                    } else {
                        float x[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) x[e] = col + e < m ? src[e] : 0.f;
                        lo4[u] = make_float4(x[0], x[1], x[2], x[3]);
                        hi4[u] = make_float4(x[4], x[5], x[6], x[7]);
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < ITEMS; ++u) {
                const int idx = gt + u * WC_GROUP_THREADS;
                const int jr = idx >> 4, cg = idx & 15;
                const float x[8] = {lo4[u].x, lo4[u].y, lo4[u].z, lo4[u].w, hi4[u].x, hi4[u].y, hi4[u].z, hi4[u].w};
                float h[8], l[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    h[e] = __bfloat162float(__float2bfloat16_rn(x[e]));
                    l[e] = x[e] - h[e];
                }
                const uint32_t off = (uint32_t)(cg >> 3) * WC_BLK_BYTES + (uint32_t)jr * 128u + (uint32_t)(((cg & 7) ^ (jr & 7)) << 4);
                *reinterpret_cast<uint4*>(sBhi + off) = make_uint4(pack_bf16(h[0], h[1]), pack_bf16(h[2], h[3]),
                                                                   pack_bf16(h[4], h[5]), pack_bf16(h[6], h[7]));
                *reinterpret_cast<uint4*>(sBlo + off) = make_uint4(pack_bf16(l[0], l[1]), pack_bf16(l[2], l[3]),
                                                                   pack_bf16(l[4], l[5]), pack_bf16(l[6], l[7]));
            }
            ptx::fence_proxy_async();    // generic-proxy stores -> visible to the tensor core's async proxy
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&s_full[q]);
        }
        if (!ok && lane == 0) raise_status(DEV_TIMEOUT);
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, 2 * WP_TILE);
    }
}

inline pamm_status launch_weight_grad_chunked(const void* C, int64_t ldc, int64_t k, int64_t n, const float* Bt,
                                              int64_t ldb, int64_t m, float* dW, int64_t ldw, int sms, cudaStream_t st,
                                              int64_t b_rows = 0, const int32_t* dropped = nullptr, bool accumulate = false) {
    const int kpad = (int)round_up(k, 16);
    const int nch = (kpad + WC_KC - 1) / WC_KC;
    CUtensorMap tm_c, tm_w;
    if (!make_tmap_bf16_sw128(&tm_c, C, (uint64_t)k, (uint64_t)n, (uint64_t)ldc, (uint32_t)WC_KC) ||
        !make_tmap_f32_sw128(&tm_w, dW, (uint64_t)n, (uint64_t)m, (uint64_t)ldw, WP_TILE))
        return PAMM_ERR_CUDA;
    const int n_tiles = (int)((n + WP_TILE - 1) / WP_TILE), m_tiles = (int)((m + WP_TILE - 1) / WP_TILE);
    const int64_t total = (int64_t)n_tiles * m_tiles;
    if (total * nch >= (1ll << 31)) return PAMM_ERR_UNSUPPORTED;
    const size_t smem = 1024 + (size_t)WC_STAGES * WC_STAGE_BYTES + 2 * WP_OUT_HALF_BYTES;
    if (!ensure_dynamic_smem((const void*)weight_grad_chunked_kernel, smem)) return PAMM_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)std::min<int64_t>(total, sms));
    cfg.blockDim = dim3(WC_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // set up while the kernel before drains
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, weight_grad_chunked_kernel, tm_c, tm_w, Bt, ldb, (int)k, (int)m, nch, n_tiles, (int)total,
                       b_rows, dropped, accumulate ? 1 : 0);
    return cudaGetLastError() == cudaSuccess ? PAMM_OK : PAMM_ERR_CUDA;
}

}  // namespace pamm
