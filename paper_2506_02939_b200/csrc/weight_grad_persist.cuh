// Step 4 on tensor cores for k <= 128 (bf16 generators): dW = C^T B~ (Algorithm 1
// ApproxMM, the final product) as a persistent, pipelined kernel.
//
// The product is bound by writing dW (2k flops per 4 bytes written), so the
// kernel is built around keeping stores in flight.  One CTA per SM takes a
// contiguous run of 128 x 128 output tiles, ordered so that consecutive tiles
// share their 128 columns of B~:
//   warp 0      TMA producer: the C tile of the next output tile (two boxes of
//               64 hidden columns x kc generators, 128-byte swizzle), two stages
//   warp 1      issues tcgen05.mma into one of two TMEM accumulators: D = A Bhi + A Blo
//   warps 2-5   epilogue: TMEM -> registers -> swizzled shared memory -> TMA store,
//               in two halves of 64 columns so the store of one half overlaps the
//               staging of the other
//   warps 6-13  split the fp32 B~ column block into bf16 hi + lo (hi = rn(x),
//               lo = rn(x - hi), about 16 mantissa bits together) in the MN-major
//               swizzled operand layout, once per column block
// When there are at least as many SMs as column blocks, every column block is
// shared by a fixed number of CTAs that split its row tiles, so no CTA ever
// converts a second block.
// Both operands are MN-major: for a fixed generator j, the hidden index of C and
// the column index of B~ are contiguous.  `swap` exchanges their roles and yields
// dW^T (m x n) instead of dW (n x m); OutT is the storage type of dW (fp32, or bf16:
// the fp32 accumulator rounded to nearest even on its way to shared memory).
#pragma once
#include "pamm_common.cuh"
#include "sm100_ptx.cuh"
#include "weight_grad_common.cuh"

namespace pamm {

constexpr int WP_THREADS = 448;
constexpr int WP_CVT_THREADS = 256;
constexpr int WP_CVT_BATCH = 4;                          // 8-column groups loaded before any is converted
constexpr int WP_TILE = WG_TILE;
constexpr int WP_EPI_THREADS = 128;
constexpr uint32_t WP_EPI_BARRIER = 1;

inline bool weight_grad_persist_supported(int64_t k, int64_t n, int64_t m) {
    return k >= 8 && round_up(k, 16) <= 128 && n >= 8 && m >= 4 && n < (1ll << 31) && m < (1ll << 31);
}

template <typename OutT>
__global__ void __launch_bounds__(WP_THREADS, 1)
weight_grad_persist_kernel(const __grid_constant__ CUtensorMap tm_c, const __grid_constant__ CUtensorMap tm_w,
                           const float* __restrict__ Bt, int64_t ldb, int k, int m, int kc, int n_tiles,
                           int total_tiles, int parts, int64_t b_rows, const int32_t* __restrict__ dropped,
                           int accumulate, int swap) {
    constexpr int WP_OUT_HALF_BYTES = WgOut<OutT>::HALF_BYTES;     // staging of 64 columns x 128 rows
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_afull[2], s_aempty[2], s_tfull[2], s_tempty[2], s_bfull, s_bempty;
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t blk_bytes = (uint32_t)kc * 128u;       // one 64-wide block: kc rows of 128 bytes
    uint8_t* sBhi = base;
    uint8_t* sBlo = sBhi + 2 * blk_bytes;
    uint8_t* sA = sBlo + 2 * blk_bytes;                    // two stages of 2 blocks
    uint8_t* sOut = sA + 4 * blk_bytes;                    // two halves

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
            ptx::mbar_init(&s_tempty[s], 4);
        }
        ptx::mbar_init(&s_bfull, WP_CVT_THREADS);
        ptx::mbar_init(&s_bempty, 1);
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
        // ---------------- TMA producer: C tiles ----------------
        if (ptx::elect_one()) {
            ptx::prefetch_tensormap(&tm_c);
            uint32_t it = 0;
            bool ok = true;
            for (int t = t0; t < t1; ++t, ++it) {
                const int s = it & 1;
                if (!ptx::mbar_wait(&s_aempty[s], ((it >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                const int n0 = (t % n_tiles) * WP_TILE;
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
            const uint32_t idesc = ptx::umma_idesc_bf16(WP_TILE, WP_TILE) | (1u << 15) | (1u << 16);
            const uint32_t bh_addr = ptx::smem_u32(sBhi), bl_addr = ptx::smem_u32(sBlo);
            uint32_t it = 0, g = 0;
            int prev_cb = -1;
            bool ok = true;
            for (int t = t0; t < t1 && ok; ++t, ++it) {
                const int cb = t / n_tiles;
                if (cb != prev_cb) {
                    if (!ptx::mbar_wait(&s_bfull, g & 1u, abort_flag)) { ok = false; break; }
                    prev_cb = cb;
                    ++g;
                }
                const int s = it & 1;
                if (!ptx::mbar_wait(&s_afull[s], (it >> 1) & 1u, abort_flag) ||
                    !ptx::mbar_wait(&s_tempty[s], ((it >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                ptx::tc_fence_after_sync();
                const uint32_t a_addr = ptx::smem_u32(sA + (size_t)s * 2 * blk_bytes);
                const uint32_t d_addr = tmem_base + (uint32_t)(s * WP_TILE);
                for (int kk = 0; kk < kc / 16; ++kk) {   // 16 generators = two 8-deep K groups = 2048 bytes
                    const uint64_t da = umma_desc_mn_sw128(a_addr + kk * 2048, blk_bytes, 1024);
                    const uint64_t dh = umma_desc_mn_sw128(bh_addr + kk * 2048, blk_bytes, 1024);
                    const uint64_t dl = umma_desc_mn_sw128(bl_addr + kk * 2048, blk_bytes, 1024);
                    if (!swap) {      // rows of the tile = hidden index (C), columns = B~ columns
                        ptx::umma_bf16(d_addr, da, dh, idesc, kk != 0);
                        ptx::umma_bf16(d_addr, da, dl, idesc, true);
                    } else {          // rows = B~ columns, columns = hidden index: the tile of dW^T
                        ptx::umma_bf16(d_addr, dh, da, idesc, kk != 0);
                        ptx::umma_bf16(d_addr, dl, da, idesc, true);
                    }
                }
                ptx::umma_commit(&s_aempty[s]);
                ptx::umma_commit(&s_tfull[s]);
                if (t + 1 < t1 && (t + 1) / n_tiles != cb) ptx::umma_commit(&s_bempty);   // B~ block may be replaced
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
                        if constexpr (sizeof(OutT) == 4) {     // a box of 32 fp32 columns per 32 accumulator columns
                            uint8_t* dst = half + gg * (WP_TILE * 128) + row * 128;
#pragma unroll
                            for (int c = 0; c < 8; ++c)
                                *reinterpret_cast<uint4*>(dst + ((c ^ (row & 7)) << 4)) =
                                    make_uint4(v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3]);
                        } else {                               // one box of 64 bf16 columns: this load fills half of each row
                            uint8_t* dst = half + row * 128;
#pragma unroll
                            for (int c = 0; c < 4; ++c)
                                *reinterpret_cast<uint4*>(dst + (((gg * 4 + c) ^ (row & 7)) << 4)) =
                                    make_uint4(pack_bf16(__uint_as_float(v[8 * c]), __uint_as_float(v[8 * c + 1])),
                                               pack_bf16(__uint_as_float(v[8 * c + 2]), __uint_as_float(v[8 * c + 3])),
                                               pack_bf16(__uint_as_float(v[8 * c + 4]), __uint_as_float(v[8 * c + 5])),
                                               pack_bf16(__uint_as_float(v[8 * c + 6]), __uint_as_float(v[8 * c + 7])));
                        }
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
                    if (ok) {
                        const int x0 = (swap ? n0 : m0) + h * 64, y0 = swap ? m0 : n0;     // the tile's place in dW or dW^T
                        constexpr int BOXES = WP_OUT_HALF_BYTES / (WP_TILE * 128);
#pragma unroll
                        for (int q = 0; q < BOXES; ++q) {
                            if (accumulate) ptx::tma_reduce_add_2d(&tm_w, half + q * (WP_TILE * 128), x0 + q * WgOut<OutT>::BOX_COLS, y0);
                            else            ptx::tma_store_2d(&tm_w, half + q * (WP_TILE * 128), x0 + q * WgOut<OutT>::BOX_COLS, y0);
                        }
                    }
                    ptx::bulk_commit_group();
                }
            }
        }
        if (etid == 0) ptx::bulk_wait_group<0>();
        if (!ok && lane == 0) raise_status(DEV_TIMEOUT);
    } else {
        // ---------------- B~ column block: fp32 -> bf16 hi / lo, swizzled MN-major ----------------
        const int ctid = tid - 192;
        uint32_t g = 0;
        int prev_cb = -1;
        bool ok = true;
        for (int t = t0; t < t1 && ok; ++t) {
            const int cb = t / n_tiles;
            if (cb == prev_cb) continue;
            prev_cb = cb;
            if (g > 0 && !ptx::mbar_wait(&s_bempty, (g - 1) & 1u, abort_flag)) { ok = false; break; }
            const int64_t m0 = (int64_t)cb * WP_TILE;
            const bool full_cols = m0 + WP_TILE <= m;
            for (int i0 = ctid; i0 < kc * 16; i0 += WP_CVT_THREADS * WP_CVT_BATCH) {
                float4 lo4[WP_CVT_BATCH], hi4[WP_CVT_BATCH];
#pragma unroll
                for (int u = 0; u < WP_CVT_BATCH; ++u) {     // all loads of the batch first
                    const int idx = i0 + u * WP_CVT_THREADS;
                    const int jr = idx >> 4;               // generator
                    const int64_t col = m0 + (idx & 15) * 8;
                    lo4[u] = hi4[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (idx < kc * 16 && jr < k) {
                        const float* src = Bt + (int64_t)jr * ldb + col;
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
                for (int u = 0; u < WP_CVT_BATCH; ++u) {
                    const int idx = i0 + u * WP_CVT_THREADS;
                    if (idx >= kc * 16) break;
                    const int jr = idx >> 4, cg = idx & 15;
                    const float x[8] = {lo4[u].x, lo4[u].y, lo4[u].z, lo4[u].w, hi4[u].x, hi4[u].y, hi4[u].z, hi4[u].w};
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
            }
            ptx::fence_proxy_async();    // generic-proxy stores -> visible to the tensor core's async proxy
            ptx::mbar_arrive(&s_bfull);
            ++g;
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
    const int n_tiles = (int)((n + WP_TILE - 1) / WP_TILE), m_tiles = (int)((m + WP_TILE - 1) / WP_TILE);
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
