// Step 4 on tensor cores for k <= 128 (bf16 generators): dW = C^T B~ (Algorithm 1
// ApproxMM, the final product) as a persistent, pipelined kernel.
//
// The product is bound by writing dW (2k flops per output element), so the
// kernel is built around keeping stores in flight.  One CTA per SM takes a
// contiguous run of 128 x 128 output tiles, ordered so that consecutive tiles
// share their 128 columns of B~:
//   warp 0       TMA producer: the C tile of the next output tile (two boxes of
//                64 hidden columns x kc generators, 128-byte swizzle), two stages
//   warp 1       issues tcgen05.mma into one of two TMEM accumulators:
//                D = P Qhi + P Qlo; the first tile of a B~ block starts generator group
//                by generator group, as soon as the converters have delivered each
//   warps 2-9    epilogue: TMEM -> registers -> swizzled shared memory -> TMA store; a warp
//                owns 32 rows (its TMEM lane quadrant) x 64 columns, the four warps of a
//                column half share one staging area and one store stream
//   warps 10-13  split the fp32 B~ column block into bf16 hi + lo (hi = rn(x),
//                lo = rn(x - hi), about 16 mantissa bits together) in the MN-major
//                swizzled operand layout, once per column block; every group of 16
//                generators is announced on its own barrier.  The CTA's FIRST block is
//                converted by these warps and the eight epilogue warps together: nothing
//                can be stored before it exists, so they would only wait
// (fourteen warps: four per scheduler at most, which leaves each thread 128 registers)
// When there are at least as many SMs as column blocks, every column block is
// shared by a fixed number of CTAs that split its row tiles, so no CTA ever
// converts a second block.
// Both operands are MN-major: for a fixed generator j, the hidden index of C and
// the column index of B~ are contiguous.  `swap` exchanges their roles and yields
// dW^T (m x n) instead of dW (n x m).
#pragma once
#include "pamm_common.cuh"
#include "sm100_ptx.cuh"
#include "weight_grad_common.cuh"

namespace pamm {

constexpr int WP_CVT_THREADS = 128;
constexpr int WP_THREADS = 64 + 32 * WG_EPI_WARPS + WP_CVT_THREADS;  // 448
constexpr int WP_CVT_TID0 = 64 + 32 * WG_EPI_WARPS;       // first converter thread
constexpr int WP_MAX_GROUPS = 8;                          // groups of 16 generators in a block (k <= 128)

inline bool weight_grad_persist_supported(int64_t k, int64_t n, int64_t m) {
    return k >= 8 && round_up(k, 16) <= 128 && n >= 8 && m >= 4 && n < (1ll << 31) && m < (1ll << 31);
}

template <typename OutT>
__global__ void __launch_bounds__(WP_THREADS, 1)
weight_grad_persist_kernel(const __grid_constant__ CUtensorMap tm_c, const __grid_constant__ CUtensorMap tm_w,
                           const float* __restrict__ Bt, int64_t ldb, int k, int m, int kc, int n_tiles,
                           int total_tiles, int parts, int64_t b_rows, const int32_t* __restrict__ dropped,
                           int accumulate, int swap) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_afull[2], s_aempty[2], s_tfull[2], s_tempty[2], s_bfull[WP_MAX_GROUPS], s_bempty;
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t blk_bytes = (uint32_t)kc * 128u;       // one 64-wide block: kc rows of 128 bytes
    uint8_t* sBhi = base;
    uint8_t* sBlo = sBhi + 2 * blk_bytes;
    uint8_t* sA = sBlo + 2 * blk_bytes;                    // two stages of 2 blocks
    uint8_t* sOut = sA + 4 * blk_bytes;                    // one staging area per column half
    const int groups = kc / 16;

    // tiles are numbered column block by column block; this CTA takes [t0, t1)
    int t0, t1;
    if (parts > 0) {          // `parts` CTAs per column block
        const int cb = blockIdx.x / parts, part = blockIdx.x % parts;
        t0 = cb * n_tiles + (int)((int64_t)part * n_tiles / parts);
        t1 = cb * n_tiles + (int)((int64_t)(part + 1) * n_tiles / parts);
    } else {
        t0 = (int)((int64_t)blockIdx.x * total_tiles / gridDim.x);
        t1 = (int)((int64_t)(blockIdx.x + 1) * total_tiles / gridDim.x);
    }

    if (tid == 0) {
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(&s_afull[s], 1);
            ptx::mbar_init(&s_aempty[s], 1);
            ptx::mbar_init(&s_tfull[s], 1);
            ptx::mbar_init(&s_tempty[s], WG_EPI_WARPS);
        }
        for (int g = 0; g < WP_MAX_GROUPS; ++g) ptx::mbar_init(&s_bfull[g], 8);   // 256 items of 32 per warp-arrival
        ptx::mbar_init(&s_bempty, 1);
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
        // ---------------- TMA producer: C tiles ----------------
        if (ptx::elect_one()) {
            ptx::prefetch_tensormap(&tm_c);
            uint32_t it = 0;
            bool ok = true;
            for (int t = t0; t < t1; ++t, ++it) {
                const int s = it & 1;
                if (!ptx::mbar_wait(&s_aempty[s], ((it >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                const int n0 = (t % n_tiles) * WG_TILE;
                uint8_t* dst = sA + (size_t)s * 2 * blk_bytes;
                ptx::mbar_arrive_expect_tx(&s_afull[s], 2 * blk_bytes);
                ptx::tma_load_2d(dst, &tm_c, n0, 0, &s_afull[s]);
                ptx::tma_load_2d(dst + blk_bytes, &tm_c, n0 + 64, 0, &s_afull[s]);
            }
            if (!ok) {
                raise_status(DEV_TIMEOUT);
                int never = 0;
                volatile int* no_abort = &never;   // let the copies already issued land before the CTA leaves
                const uint32_t back = it < 2u ? it : 2u;
                for (uint32_t d = 1; d <= back; ++d) ptx::mbar_wait(&s_afull[(it - d) & 1], ((it - d) >> 1) & 1u, no_abort);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (ptx::elect_one()) {
            // kind::f16, D fp32, A/B bf16, both MN-major (bits 15 and 16), M = N = 128
            const uint32_t idesc = ptx::umma_idesc_bf16(WG_TILE, WG_TILE) | (1u << 15) | (1u << 16);
            const uint32_t bh_addr = ptx::smem_u32(sBhi), bl_addr = ptx::smem_u32(sBlo);
            uint32_t it = 0, g = 0;
            int prev_cb = -1;
            bool ok = true;
            for (int t = t0; t < t1 && ok; ++t, ++it) {
                const int cb = t / n_tiles;
                const bool fresh = cb != prev_cb;      // first tile on this B~ block: its generator groups arrive one by one
                const int s = it & 1;
                if (!ptx::mbar_wait(&s_afull[s], (it >> 1) & 1u, abort_flag) ||
                    !ptx::mbar_wait(&s_tempty[s], ((it >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                ptx::tc_fence_after_sync();
                const uint32_t a_addr = ptx::smem_u32(sA + (size_t)s * 2 * blk_bytes);
                const uint32_t d_addr = tmem_base + (uint32_t)(s * WG_TILE);
                for (int kk = 0; kk < groups; ++kk) {   // 16 generators = two 8-deep K groups = 2048 bytes
                    if (fresh) {
                        if (!ptx::mbar_wait(&s_bfull[kk], g & 1u, abort_flag)) { ok = false; break; }
                        ptx::tc_fence_after_sync();
                    }
                    const uint64_t dc = umma_desc_mn_sw128(a_addr + kk * 2048, blk_bytes, 1024);
                    const uint64_t dh = umma_desc_mn_sw128(bh_addr + kk * 2048, blk_bytes, 1024);
                    const uint64_t dl = umma_desc_mn_sw128(bl_addr + kk * 2048, blk_bytes, 1024);
                    if (!swap) {      // rows of the tile = hidden index (C), columns = B~ columns
                        ptx::umma_bf16(d_addr, dc, dh, idesc, kk != 0);
                        ptx::umma_bf16(d_addr, dc, dl, idesc, true);
                    } else {          // rows = B~ columns, columns = hidden index: the tile of dW^T
                        ptx::umma_bf16(d_addr, dh, dc, idesc, kk != 0);
                        ptx::umma_bf16(d_addr, dl, dc, idesc, true);
                    }
                }
                if (!ok) break;
                if (fresh) { prev_cb = cb; ++g; }
                ptx::umma_commit(&s_aempty[s]);
                ptx::umma_commit(&s_tfull[s]);
                if (t + 1 < t1 && (t + 1) / n_tiles != cb) ptx::umma_commit(&s_bempty);   // B~ block may be replaced
            }
            if (!ok) raise_status(DEV_TIMEOUT);
        }
    } else if (warp < 2 + WG_EPI_WARPS) {
        // ---------------- epilogue: 32 rows x 64 columns of the tile per warp ----------------
        if (t0 < t1)      // lend a hand with the first B~ block
            convert_bt_block<6>(Bt, ldb, k, m, kc, (int64_t)(t0 / n_tiles) * WG_TILE, sBhi, sBlo, blk_bytes, s_bfull, tid - 64,
                                WP_THREADS - 64);
        const int quad = warp & 3;                       // TMEM lanes [32*quad, 32*quad+32)
        const int h = (warp - 2) >> 2;                   // column half
        const bool leader = ((warp - 2) & 3) == 0 && lane == 0;
        uint8_t* half_stage = sOut + h * WgOut<OutT>::HALF_BYTES;
        const float beta = beta_factor(dropped, b_rows);     // Eq. 4-5; 1 unless rows were dropped
        uint32_t it = 0;
        bool ok = true;   // once false this warp only keeps the barrier sequence going
        for (int t = t0; t < t1; ++t, ++it) {
            const int s = it & 1;
            const int n0 = (t % n_tiles) * WG_TILE, m0 = (t / n_tiles) * WG_TILE;
            if (ok) ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_tfull[s], (it >> 1) & 1u, abort_flag));
            ptx::tc_fence_after_sync();
            wg_epilogue_half<OutT, 0>(&tm_w, tmem_base + (uint32_t)(s * WG_TILE), &s_tempty[s], half_stage, quad, lane, h,
                                   leader, swap ? n0 : m0, swap ? m0 : n0, beta, accumulate != 0, ok);
        }
        if (leader) ptx::bulk_wait_group<0>();
        if (!ok && lane == 0) raise_status(DEV_TIMEOUT);
    } else {
        // ---------------- B~ column block: fp32 -> bf16 hi / lo, swizzled MN-major ----------------
        uint32_t g = 0;
        int prev_cb = -1;
        bool ok = true;
        for (int t = t0; t < t1 && ok; ++t) {
            const int cb = t / n_tiles;
            if (cb == prev_cb) continue;
            prev_cb = cb;
            if (g == 0) {     // the first block, together with the epilogue warps
                convert_bt_block<6>(Bt, ldb, k, m, kc, (int64_t)cb * WG_TILE, sBhi, sBlo, blk_bytes, s_bfull, tid - 64,
                                    WP_THREADS - 64);
            } else {
                ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_bempty, (g - 1) & 1u, abort_flag));
                if (!ok) break;
                convert_bt_block<4>(Bt, ldb, k, m, kc, (int64_t)cb * WG_TILE, sBhi, sBlo, blk_bytes, s_bfull,
                                    tid - WP_CVT_TID0, WP_CVT_THREADS);
            }
            ++g;
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
inline pamm_status launch_weight_grad_persist(const void* C, int64_t ldc, int64_t k, int64_t n, const float* Bt,
                                              int64_t ldb, int64_t m, void* dW, int64_t ldw, bool dw_bf16, bool swap,
                                              int sms, cudaStream_t st, int64_t b_rows = 0,
                                              const int32_t* dropped = nullptr, bool accumulate = false) {
    const int kc = (int)round_up(k, 16);
    CUtensorMap tm_c, tm_w;
    const uint64_t out_rows = swap ? (uint64_t)m : (uint64_t)n, out_cols = swap ? (uint64_t)n : (uint64_t)m;
    if (!make_tmap_bf16_sw128(&tm_c, C, (uint64_t)k, (uint64_t)n, (uint64_t)ldc, (uint32_t)kc) ||
        !(dw_bf16 ? make_tmap_bf16_sw128(&tm_w, dW, out_rows, out_cols, (uint64_t)ldw, WG_TILE)
                  : make_tmap_f32_sw128(&tm_w, dW, out_rows, out_cols, (uint64_t)ldw, WG_TILE)))
        return tensor_map_failed();
    const int n_tiles = (int)((n + WG_TILE - 1) / WG_TILE), m_tiles = (int)((m + WG_TILE - 1) / WG_TILE);
    const int64_t total = (int64_t)n_tiles * m_tiles;
    if (total >= (1ll << 31)) return PAMM_ERR_UNSUPPORTED;
    const size_t smem = 1024 + (size_t)8 * kc * 128 + 2 * (dw_bf16 ? WgOut<__nv_bfloat16>::HALF_BYTES : WgOut<float>::HALF_BYTES);
    // one column block per group of `parts` CTAs when the SMs allow it, else a plain linear split
    int parts = 0;
    int64_t grid = std::min<int64_t>(total, sms);
    if (m_tiles <= sms) {
        parts = std::max(1, std::min(n_tiles, sms / m_tiles));
        grid = (int64_t)m_tiles * parts;
    }
    auto kern = dw_bf16 ? weight_grad_persist_kernel<__nv_bfloat16> : weight_grad_persist_kernel<float>;
    if (!ensure_dynamic_smem((const void*)kern, smem)) return PAMM_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(WP_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // set up while the kernel before drains
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kern, tm_c, tm_w, Bt, ldb, (int)k, (int)m, kc, n_tiles, (int)total, parts, b_rows, dropped,
                       accumulate ? 1 : 0, swap ? 1 : 0);
    return launch_result("weight_grad_persist_kernel launch");
}

}  // namespace pamm
