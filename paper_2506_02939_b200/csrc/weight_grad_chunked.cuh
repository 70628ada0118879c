// Step 4 on tensor cores for k > 128 (bf16 generators): dW = C^T B~ (Algorithm 1
// ApproxMM, the final product), persistent and pipelined over chunks of 64 generators.
//
// One CTA per SM takes a contiguous run of 128 x 128 output tiles (numbered column
// block by column block, so neighbours share their B~ columns in L2).  Every tile
// walks the generators in chunks of 64 through a ring of three shared-memory stages;
// a stage holds the C chunk (A operand, by TMA) and the B~ chunk split into bf16
// hi + lo (B operands):
//   warp 0       TMA producer of the C chunks (its own transaction barrier per stage, so that
//                it can drain exactly what it issued if a wait ever runs out)
//   warp 1       issues tcgen05.mma: D (+)= P Qhi + P Qlo, two TMEM accumulators
//   warps 2-5    epilogue: TMEM -> registers -> swizzled shared memory -> TMA store
//                (or reduce-add), the two column halves of a tile one after the other,
//                each with its own staging area so that its store stays in flight
//   warps 6-17   three groups of four warps; group q owns stage q and converts the
//                fp32 B~ chunk that goes there (hi = rn(x), lo = rn(x - hi)), all of a
//                thread's sixteen 16-byte loads in flight at once, so three chunks
//                are being fetched from L2 at any time
// Operand layouts, descriptors and the epilogue are those of the k <= 128 kernel, and so
// is `swap` (dW^T, m x n, instead of dW).
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

template <typename OutT>
__global__ void __launch_bounds__(WC_THREADS, 1)
weight_grad_chunked_kernel(const __grid_constant__ CUtensorMap tm_c, const __grid_constant__ CUtensorMap tm_w,
                           const float* __restrict__ Bt, int64_t ldb, int k, int m, int nch, int n_tiles,
                           int total_tiles, int64_t b_rows, const int32_t* __restrict__ dropped, int accumulate,
                           int swap) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_cfull[WC_STAGES], s_bfull[WC_STAGES], s_empty[WC_STAGES], s_tfull[2], s_tempty[2];
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
            ptx::mbar_init(&s_cfull[s], 1);                        // the producer's arrive + its bytes
            ptx::mbar_init(&s_bfull[s], WC_GROUP_THREADS / 32);    // one arrival per converter warp
            ptx::mbar_init(&s_empty[s], 1);
        }
        for (int u = 0; u < 2; ++u) {
            ptx::mbar_init(&s_tfull[u], 1);
            ptx::mbar_init(&s_tempty[u], 8);     // four epilogue warps x two column halves
        }
        s_abort = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async();
    }
    if (warp == 1) {
        ptx::tmem_alloc(&s_tmem_base, 2 * WG_TILE);
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
                const int n0 = (t % n_tiles) * WG_TILE;
                uint8_t* dst = sStages + (size_t)s * WC_STAGE_BYTES;
                ptx::mbar_arrive_expect_tx(&s_cfull[s], 2 * WC_BLK_BYTES);
                ptx::tma_load_2d(dst, &tm_c, n0, c * WC_KC, &s_cfull[s]);
                ptx::tma_load_2d(dst + WC_BLK_BYTES, &tm_c, n0 + 64, c * WC_KC, &s_cfull[s]);
            }
            if (!ok) {
                raise_status(DEV_TIMEOUT);
                int never = 0;
                volatile int* no_abort = &never;   // let the copies already issued land before the CTA leaves
                const uint32_t back = g < (uint32_t)WC_STAGES ? g : (uint32_t)WC_STAGES;
                for (uint32_t d = 1; d <= back; ++d)
                    ptx::mbar_wait(&s_cfull[(g - d) % WC_STAGES], ((g - d) / WC_STAGES) & 1u, no_abort);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (ptx::elect_one()) {
            // kind::f16, D fp32, A/B bf16, both MN-major (bits 15 and 16), M = N = 128
            const uint32_t idesc = ptx::umma_idesc_bf16(WG_TILE, WG_TILE) | (1u << 15) | (1u << 16);
            bool ok = true;
            for (uint32_t g = 0; g < total_chunks && ok; ++g) {
                const int s = g % WC_STAGES;
                const uint32_t it = g / (uint32_t)nch, c = g % (uint32_t)nch;
                const uint32_t buf = it & 1u;
                if (c == 0 && !ptx::mbar_wait(&s_tempty[buf], ((it >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                if (!ptx::mbar_wait(&s_cfull[s], (g / WC_STAGES) & 1u, abort_flag) ||
                    !ptx::mbar_wait(&s_bfull[s], (g / WC_STAGES) & 1u, abort_flag)) { ok = false; break; }
                ptx::tc_fence_after_sync();
                const uint32_t a_addr = ptx::smem_u32(sStages + (size_t)s * WC_STAGE_BYTES);
                const uint32_t bh_addr = a_addr + 2 * WC_BLK_BYTES, bl_addr = a_addr + 4 * WC_BLK_BYTES;
                const uint32_t d_addr = tmem_base + buf * (uint32_t)WG_TILE;
#pragma unroll
                for (int kk = 0; kk < WC_KC / 16; ++kk) {   // 16 generators = two 8-deep K groups = 2048 bytes
                    const uint64_t da = umma_desc_mn_sw128(a_addr + kk * 2048, WC_BLK_BYTES, 1024);
                    const uint64_t dh = umma_desc_mn_sw128(bh_addr + kk * 2048, WC_BLK_BYTES, 1024);
                    const uint64_t dl = umma_desc_mn_sw128(bl_addr + kk * 2048, WC_BLK_BYTES, 1024);
                    if (!swap) {
                        ptx::umma_bf16(d_addr, da, dh, idesc, (c | (uint32_t)kk) != 0);
                        ptx::umma_bf16(d_addr, da, dl, idesc, true);
                    } else {
                        ptx::umma_bf16(d_addr, dh, da, idesc, (c | (uint32_t)kk) != 0);
                        ptx::umma_bf16(d_addr, dl, da, idesc, true);
                    }
                }
                ptx::umma_commit(&s_empty[s]);
                if (c + 1 == (uint32_t)nch) ptx::umma_commit(&s_tfull[buf]);
            }
            if (!ok) raise_status(DEV_TIMEOUT);
        }
    } else if (warp < 6) {
        // ---------------- epilogue: 32 rows of the tile per warp, one column half after the other ----------------
        const int quad = warp & 3;                       // TMEM lanes [32*quad, 32*quad+32)
        const bool leader = warp == 2 && lane == 0;
        const float beta = beta_factor(dropped, b_rows);     // Eq. 4-5; 1 unless rows were dropped
        uint32_t it = 0;
        bool ok = true;   // once false this warp only keeps the barrier sequence going
        for (int t = t0; t < t1; ++t, ++it) {
            const int s = it & 1;
            const int n0 = (t % n_tiles) * WG_TILE, m0 = (t / n_tiles) * WG_TILE;
            if (ok) ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_tfull[s], (it >> 1) & 1u, abort_flag));
            ptx::tc_fence_after_sync();
#pragma unroll
            for (int h = 0; h < 2; ++h)
                wg_epilogue_half<OutT>(&tm_w, tmem_base + (uint32_t)(s * WG_TILE), &s_tempty[s],
                                       sOut + h * WgOut<OutT>::HALF_BYTES, quad, lane, h, leader, swap ? n0 : m0,
                                       swap ? m0 : n0, beta, accumulate != 0, ok);
        }
        if (leader) ptx::bulk_wait_group<0>();
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
            const int64_t m0 = (int64_t)(t / n_tiles) * WG_TILE;
            const int j0 = c * WC_KC;
            const bool full_cols = m0 + WG_TILE <= m;
            uint8_t* sBhi = sStages + (size_t)q * WC_STAGE_BYTES + 2 * WC_BLK_BYTES;
            uint8_t* sBlo = sBhi + 2 * WC_BLK_BYTES;
            constexpr int ITEMS = WC_KC * 16 / WC_GROUP_THREADS;     // 8-column groups per thread: 8
            float4 lo4[ITEMS], hi4[ITEMS];
#pragma unroll
            for (int u = 0; u < ITEMS; ++u) {     // all loads first
                const int idx = gt + u * WC_GROUP_THREADS;
                const int j = j0 + (idx >> 4);
                lo4[u] = hi4[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (j < k) load_bt8(Bt, ldb, j, m0 + (idx & 15) * 8, m, full_cols, lo4[u], hi4[u]);
            }
#pragma unroll
            for (int u = 0; u < ITEMS; ++u) {
                const int idx = gt + u * WC_GROUP_THREADS;
                split_store_hi_lo(sBhi, sBlo, WC_BLK_BYTES, idx >> 4, idx & 15, lo4[u], hi4[u]);
            }
            ptx::fence_proxy_async();    // generic-proxy stores -> visible to the tensor core's async proxy
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&s_bfull[q]);
        }
        if (!ok && lane == 0) raise_status(DEV_TIMEOUT);
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, 2 * WG_TILE);
    }
}

// dw_bf16: dW stored as bf16 instead of fp32.  swap: dW^T (m x n) instead of dW (n x m).
inline pamm_status launch_weight_grad_chunked(const void* C, int64_t ldc, int64_t k, int64_t n, const float* Bt,
                                              int64_t ldb, int64_t m, void* dW, int64_t ldw, bool dw_bf16, bool swap,
                                              int sms, cudaStream_t st, int64_t b_rows = 0,
                                              const int32_t* dropped = nullptr, bool accumulate = false) {
    const int kpad = (int)round_up(k, 16);
    const int nch = (kpad + WC_KC - 1) / WC_KC;
    CUtensorMap tm_c, tm_w;
    const uint64_t out_rows = swap ? (uint64_t)m : (uint64_t)n, out_cols = swap ? (uint64_t)n : (uint64_t)m;
    if (!make_tmap_bf16_sw128(&tm_c, C, (uint64_t)k, (uint64_t)n, (uint64_t)ldc, (uint32_t)WC_KC) ||
        !(dw_bf16 ? make_tmap_bf16_sw128(&tm_w, dW, out_rows, out_cols, (uint64_t)ldw, WG_TILE)
                  : make_tmap_f32_sw128(&tm_w, dW, out_rows, out_cols, (uint64_t)ldw, WG_TILE)))
        return tensor_map_failed();
    const int n_tiles = (int)((n + WG_TILE - 1) / WG_TILE), m_tiles = (int)((m + WG_TILE - 1) / WG_TILE);
    const int64_t total = (int64_t)n_tiles * m_tiles;
    if (total * nch >= (1ll << 31)) return PAMM_ERR_UNSUPPORTED;
    const size_t smem = 1024 + (size_t)WC_STAGES * WC_STAGE_BYTES +
                        2 * (dw_bf16 ? WgOut<__nv_bfloat16>::HALF_BYTES : WgOut<float>::HALF_BYTES);
    auto kern = dw_bf16 ? weight_grad_chunked_kernel<__nv_bfloat16> : weight_grad_chunked_kernel<float>;
    if (!ensure_dynamic_smem((const void*)kern, smem)) return PAMM_ERR_CUDA;
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
    cudaLaunchKernelEx(&cfg, kern, tm_c, tm_w, Bt, ldb, (int)k, (int)m, nch, n_tiles, (int)total, b_rows, dropped,
                       accumulate ? 1 : 0, swap ? 1 : 0);
    return launch_result("weight_grad_chunked_kernel launch");
}

}  // namespace pamm
