// Step 4 on tensor cores for k > 128 inside the fused backward call: dW = C^T B~ (Algorithm 1,
// ApproxMM, the final product) with B~ already split into bf16 hi and lo planes by the
// reduction kernel of the contraction.  All three operands of a chunk of 64 generators -- the C
// chunk, the hi chunk, the lo chunk -- come by TMA, so no CTA converts anything: the kernel of
// weight_grad_chunked.cuh re-splits the same fp32 chunk in every CTA that needs it (once per
// 128-row tile of dW: n / 128 times), which bounds it at about 1.3 us per chunk.
//
// One CTA per SM takes a contiguous run of 128 x 128 output tiles (column block by column
// block, so neighbours share their B~ columns in L2); a tile walks the generators in chunks
// of 64 through a ring of three 48 KB stages:
//   warp 0     TMA producer: two 64-column boxes each of C, hi and lo per chunk
//   warp 1     issues tcgen05.mma: D (+)= P Qhi + P Qlo, two TMEM accumulators
//   warps 2-5  epilogue: TMEM -> registers -> swizzled shared memory -> TMA store (or
//              reduce-add), the two column halves of a tile one after the other
// Operand layouts, descriptors, the order of the MMAs and the epilogue are those of the
// chunked kernel, so the two give the same bits; `swap` (dW^T, m x n) likewise.
#pragma once
#include "weight_grad_chunked.cuh"

namespace pamm {

constexpr int WPL_THREADS = 192;

template <typename OutT>
__global__ void __launch_bounds__(WPL_THREADS, 1)
weight_grad_planes_kernel(const __grid_constant__ CUtensorMap tm_c, const __grid_constant__ CUtensorMap tm_hi,
                          const __grid_constant__ CUtensorMap tm_lo, const __grid_constant__ CUtensorMap tm_w,
                          int nch, int n_tiles, int total_tiles, int64_t b_rows, const int32_t* __restrict__ dropped,
                          int accumulate, int swap) {
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
        for (int s = 0; s < WC_STAGES; ++s) { ptx::mbar_init(&s_full[s], 1); ptx::mbar_init(&s_empty[s], 1); }
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
    grid_dependency_wait();     // the planes come from the kernel before
    grid_launch_dependents();

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (ptx::elect_one()) {
            ptx::prefetch_tensormap(&tm_c);
            ptx::prefetch_tensormap(&tm_hi);
            ptx::prefetch_tensormap(&tm_lo);
            uint32_t g = 0, sph = 0;
            int s = 0, c = 0, t = t0;
            bool ok = true;
            for (; g < total_chunks; ++g) {
                if (!ptx::mbar_wait(&s_empty[s], sph ^ 1u, abort_flag)) { ok = false; break; }
                const int n0 = (t % n_tiles) * WG_TILE, m0 = (t / n_tiles) * WG_TILE;
                uint8_t* dst = sStages + (size_t)s * WC_STAGE_BYTES;
                ptx::mbar_arrive_expect_tx(&s_full[s], WC_STAGE_BYTES);
                ptx::tma_load_2d(dst, &tm_c, n0, c * WC_KC, &s_full[s]);
                ptx::tma_load_2d(dst + WC_BLK_BYTES, &tm_c, n0 + 64, c * WC_KC, &s_full[s]);
                ptx::tma_load_2d(dst + 2 * WC_BLK_BYTES, &tm_hi, m0, c * WC_KC, &s_full[s]);
                ptx::tma_load_2d(dst + 3 * WC_BLK_BYTES, &tm_hi, m0 + 64, c * WC_KC, &s_full[s]);
                ptx::tma_load_2d(dst + 4 * WC_BLK_BYTES, &tm_lo, m0, c * WC_KC, &s_full[s]);
                ptx::tma_load_2d(dst + 5 * WC_BLK_BYTES, &tm_lo, m0 + 64, c * WC_KC, &s_full[s]);
                if (++s == WC_STAGES) { s = 0; sph ^= 1u; }
                if (++c == nch) { c = 0; ++t; }
            }
            if (!ok) {
                raise_status(DEV_TIMEOUT);
                int never = 0;
                volatile int* no_abort = &never;   // let the copies already issued land before the CTA leaves
                const uint32_t back = g < (uint32_t)WC_STAGES ? g : (uint32_t)WC_STAGES;
                for (uint32_t d = 1; d <= back; ++d)
                    ptx::mbar_wait(&s_full[(g - d) % WC_STAGES], ((g - d) / WC_STAGES) & 1u, no_abort);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (ptx::elect_one()) {
            // kind::f16, D fp32, A/B bf16, both MN-major (bits 15 and 16), M = N = 128
            const uint32_t idesc = ptx::umma_idesc_bf16(WG_TILE, WG_TILE) | (1u << 15) | (1u << 16);
            uint32_t sph = 0, it = 0;
            int s = 0, c = 0;
            bool ok = true;
            for (uint32_t g = 0; g < total_chunks && ok; ++g) {
                const uint32_t buf = it & 1u;
                if (c == 0 && !ptx::mbar_wait(&s_tempty[buf], ((it >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                if (!ptx::mbar_wait(&s_full[s], sph, abort_flag)) { ok = false; break; }
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
                        ptx::umma_bf16(d_addr, da, dh, idesc, (c | kk) != 0);
                        ptx::umma_bf16(d_addr, da, dl, idesc, true);
                    } else {
                        ptx::umma_bf16(d_addr, dh, da, idesc, (c | kk) != 0);
                        ptx::umma_bf16(d_addr, dl, da, idesc, true);
                    }
                }
                ptx::umma_commit(&s_empty[s]);
                if (++s == WC_STAGES) { s = 0; sph ^= 1u; }
                if (++c == nch) {
                    ptx::umma_commit(&s_tfull[buf]);
                    c = 0;
                    ++it;
                }
            }
            if (!ok) raise_status(DEV_TIMEOUT);
        }
    } else {
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
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, 2 * WG_TILE);
    }
}

// planes: bf16 hi plane (k x plane_ld) followed by the lo plane, as the contraction's reduction leaves them.
inline pamm_status launch_weight_grad_planes(const void* C, int64_t ldc, int64_t k, int64_t n, const uint16_t* planes,
                                             int64_t plane_ld, int64_t m, void* dW, int64_t ldw, bool dw_bf16, bool swap,
                                             int sms, cudaStream_t st, int64_t b_rows = 0,
                                             const int32_t* dropped = nullptr, bool accumulate = false) {
    const int kpad = (int)round_up(k, 16);
    const int nch = (kpad + WC_KC - 1) / WC_KC;
    CUtensorMap tm_c, tm_hi, tm_lo, tm_w;
    const uint64_t out_rows = swap ? (uint64_t)m : (uint64_t)n, out_cols = swap ? (uint64_t)n : (uint64_t)m;
    if (!make_tmap_bf16_sw128(&tm_c, C, (uint64_t)k, (uint64_t)n, (uint64_t)ldc, (uint32_t)WC_KC) ||
        !make_tmap_bf16_sw128(&tm_hi, planes, (uint64_t)k, (uint64_t)m, (uint64_t)plane_ld, (uint32_t)WC_KC) ||
        !make_tmap_bf16_sw128(&tm_lo, planes + (size_t)k * plane_ld, (uint64_t)k, (uint64_t)m, (uint64_t)plane_ld, (uint32_t)WC_KC) ||
        !(dw_bf16 ? make_tmap_bf16_sw128(&tm_w, dW, out_rows, out_cols, (uint64_t)ldw, WG_TILE)
                  : make_tmap_f32_sw128(&tm_w, dW, out_rows, out_cols, (uint64_t)ldw, WG_TILE)))
        return tensor_map_failed();
    const int n_tiles = (int)((n + WG_TILE - 1) / WG_TILE), m_tiles = (int)((m + WG_TILE - 1) / WG_TILE);
    const int64_t total = (int64_t)n_tiles * m_tiles;
    if (total * nch >= (1ll << 31)) return PAMM_ERR_UNSUPPORTED;
    const size_t smem = 1024 + (size_t)WC_STAGES * WC_STAGE_BYTES +
                        2 * (dw_bf16 ? WgOut<__nv_bfloat16>::HALF_BYTES : WgOut<float>::HALF_BYTES);
    auto kern = dw_bf16 ? weight_grad_planes_kernel<__nv_bfloat16> : weight_grad_planes_kernel<float>;
    if (!ensure_dynamic_smem((const void*)kern, smem)) return PAMM_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)std::min<int64_t>(total, sms));
    cfg.blockDim = dim3(WPL_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // set up while the kernel before drains
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kern, tm_c, tm_hi, tm_lo, tm_w, nch, n_tiles, (int)total, b_rows, dropped, accumulate ? 1 : 0,
                       swap ? 1 : 0);
    return launch_result("weight_grad_planes_kernel launch");
}

}  // namespace pamm
