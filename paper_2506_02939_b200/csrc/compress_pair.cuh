// Step 2 on tensor cores for MANY generators (more than 128 per chunk, where the pass is bound by
// the tensor pipe, not by HBM): the kernel of compress_umma.cuh on PAIRS of CTAs.  A cluster of
// two CTAs (the two SMs of a TPC) issues `tcgen05.mma.cta_group::2` with M = 256: 128 rows of X
// from each CTA's own row range, and each CTA holding HALF of the chunk's generators.  Per 64
// hidden indices a CTA then moves 16 KB of X and at most 16 KB of C through its shared memory
// (one CTA with two row tiles: 32 + 32 KB), and a chunk of 256 generators leaves room for TWO
// accumulator sets in tensor memory (128 lanes x 256 columns each), so the argmax epilogue of
// one pass overlaps the MMAs of the next -- with two row tiles per CTA the accumulators of
// one pass fill tensor memory.
//
// Rows, results and the per-CTA histograms of f are cut exactly as in the one-CTA kernel (every
// CTA owns the same contiguous row range), so the sort products of either kernel feed the same
// backward pass.  The two CTAs of a pair walk the same number of 128-row tiles (rows beyond the
// range or beyond b are zero-filled by TMA and never stored); an odd last CTA without rows
// still feeds its half of the generators.
//   rank 0 (leader)  warp 0 loads its tiles, warp 1 issues every MMA of the pair
//   rank 1           warp 0 loads its tiles, warp 1 only allocates and frees tensor memory
//   both             warps 2-5: epilogue, one thread per row of the CTA's tile
// Barriers as in linear_forward_pair.cuh: `full` in the leader counts both CTAs' bytes, one
// multicast commit arrives on `empty` / `tfull` in both, `tempty` in the leader takes the eight
// epilogue warps.  No load uses multicast.  Every wait is bounded; both CTAs meet at a cluster
// barrier before tensor memory is freed.
#pragma once
#include "compress_umma.cuh"

namespace pamm {

constexpr int CP_THREADS = 192;
constexpr int CP_MIN_CHUNK = 160;      // generators per chunk from which pairs pay (below: HBM-bound, one CTA does as well)

struct CompressPairPlan {
    int n_chunk, num_chunks, stages, stage_bytes, rows_per_cta, tiles_per_cta, grid;
    size_t smem_bytes;
};

inline CompressPairPlan compress_pair_plan(int64_t b, int64_t k, int groups, int sms, size_t static_smem) {
    CompressPairPlan p;
    const int npad = (int)round_up(k, 32);
    p.num_chunks = (npad + 255) / 256;
    p.n_chunk = (int)round_up((npad + p.num_chunks - 1) / p.num_chunks, 32);     // each CTA holds half, in groups of 16
    p.stage_bytes = CU_X_TILE_BYTES + (p.n_chunk / 2) * 128;
    const size_t fixed = 1024 + (size_t)groups * (p.num_chunks * p.n_chunk + 2 * k) * 4 + 256;
    const size_t budget = CU_SMEM_LIMIT > fixed + static_smem ? CU_SMEM_LIMIT - fixed - static_smem : 0;
    p.stages = (int)std::min<size_t>(8, std::min<size_t>(CU_SMEM_BUDGET, budget) / p.stage_bytes);
    if (p.stages < 2) p.stages = 0;
    p.rows_per_cta = compress_rows_per_cta(b, sms);       // the partition of the one-CTA kernel and of the sort
    p.tiles_per_cta = (p.rows_per_cta + CU_TILE_M - 1) / CU_TILE_M;
    const int ctas = (int)((b + p.rows_per_cta - 1) / p.rows_per_cta);
    p.grid = (ctas + 1) & ~1;
    p.smem_bytes = fixed + (size_t)p.stages * p.stage_bytes;
    return p;
}

__global__ void __launch_bounds__(CP_THREADS, 1)
compress_pair_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_c,
                     int64_t b, int n, int k, int groups, int n_chunk, int num_chunks, int stages, int stage_bytes,
                     int rows_per_cta, int tiles_per_cta, int x_is_ready, const float* __restrict__ c_invnorm,
                     CompressOut out) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_full[8], s_empty[8], s_tfull[2], s_tempty[2];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();            // 0 = leader
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int kpad = n_chunk * num_chunks;
    float* s_inv = reinterpret_cast<float*>(tiles + (size_t)stages * stage_bytes);
    float* s_inv2 = s_inv + groups * kpad;
    int32_t* s_hist = reinterpret_cast<int32_t*>(s_inv2 + groups * k);

    const int64_t r0 = (int64_t)blockIdx.x * rows_per_cta;
    const int64_t r1 = min(b, r0 + (int64_t)rows_per_cta);     // r1 <= r0: this CTA has no rows of its own
    const int ksteps = (n + CU_BLOCK_K - 1) / CU_BLOCK_K;
    const int passes = groups * num_chunks;          // passes over a tile of X: one per (group, chunk)
    const int half = n_chunk / 2;                    // this CTA's generators of a chunk

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) { ptx::mbar_init(&s_full[s], 1); ptx::mbar_init(&s_empty[s], 1); }
        for (int u = 0; u < 2; ++u) { ptx::mbar_init(&s_tfull[u], 1); ptx::mbar_init(&s_tempty[u], 8); }
        s_abort = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async();
    }
    if (warp == 1) {
        ptx::tmem_alloc_pair(&s_tmem_base, 512);
        ptx::tmem_relinquish_pair();
    }
    grid_launch_dependents();     // released early; see the rule beside grid_dependency_wait
    if (!x_is_ready) grid_dependency_wait();
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync_all();      // the partner's barriers and tensor memory exist before anything is sent there
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = s_tmem_base;
    volatile int* abort_flag = &s_abort;

    if (warp == 0) {
        // ---------------- TMA producer (both CTAs) ----------------
        if (ptx::elect_one()) {
            ptx::prefetch_tensormap(&tm_x);
            ptx::prefetch_tensormap(&tm_c);
            // pipeline step = (row tile, pass = (group, chunk), 64-column step), walked with additions only
            struct Cursor {
                int tile, g, ch, ks, s;
                uint32_t phase;
            };
            auto advance = [&](Cursor& c) {
                if (++c.s == stages) { c.s = 0; c.phase ^= 1u; }
                if (++c.ks < ksteps) return;
                c.ks = 0;
                if (++c.ch == num_chunks) { c.ch = 0; ++c.g; }
                if (c.g < groups) return;
                c.g = 0;
                ++c.tile;
            };
            const uint32_t step_bytes = 2u * (uint32_t)stage_bytes;      // both CTAs' tiles, counted in the leader
            auto issue = [&](const Cursor& c, bool with_x, bool with_c, bool arm) {
                uint8_t* stage = tiles + (size_t)c.s * stage_bytes;
                if (arm && rank == 0) ptx::mbar_arrive_expect_tx(&s_full[c.s], step_bytes);
                const uint32_t full = ptx::map_to_rank(&s_full[c.s], 0);
                if (with_x) {
                    const int64_t y = r0 + (int64_t)c.tile * CU_TILE_M;      // rows beyond b read as zeros
#pragma unroll
                    for (int q = 0; q < CU_TILE_M / CU_BOX_ROWS; ++q)
                        ptx::tma_load_2d_pair(stage + q * (CU_BOX_ROWS * 128), &tm_x, c.ks * CU_BLOCK_K,
                                              (int32_t)min(y + q * CU_BOX_ROWS, (int64_t)0x7fffffff), full);
                }
                if (with_c)
                    ptx::tma_load_2d_pair(stage + CU_X_TILE_BYTES, &tm_c, c.ks * CU_BLOCK_K,
                                          c.g * k + c.ch * n_chunk + (int)rank * half, full);
            };
            const uint32_t total = (uint32_t)tiles_per_cta * (uint32_t)(passes * ksteps);
            Cursor cur = {0, 0, 0, 0, 0, 0u};
            uint32_t it = 0;
            bool ok = true;
            if (x_is_ready) {     // fill the ring with X, then wait for the kernel before, then add the C tiles
                const uint32_t ahead = total < (uint32_t)stages ? total : (uint32_t)stages;
                Cursor pre = cur;
                for (uint32_t a = 0; a < ahead; ++a, advance(pre)) issue(pre, true, false, true);
                grid_dependency_wait();
                for (uint32_t a = 0; a < ahead; ++a, advance(cur)) issue(cur, false, true, false);
                it = ahead;
            }
            for (; it < total; ++it, advance(cur)) {
                if (!ptx::mbar_wait(&s_empty[cur.s], cur.phase ^ 1u, abort_flag)) { ok = false; break; }
                issue(cur, true, true, true);
            }
            if (!ok) {
                raise_status(DEV_TIMEOUT);
                // the leader can wait for the copies already issued (their bytes are counted there); the partner
                // waits a fixed time, and the cluster barrier below keeps both CTAs until the other has come
                if (rank == 0) {
                    const uint32_t back = it < (uint32_t)stages ? it : (uint32_t)stages;
                    int never = 0;
                    volatile int* no_abort = &never;
                    for (uint32_t d = 1; d <= back; ++d) {
                        const uint32_t jt = it - d;
                        ptx::mbar_wait(&s_full[jt % stages], (jt / stages) & 1u, no_abort);
                    }
                } else {
                    for (int w = 0; w < 64; ++w) __nanosleep(1000);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader only) ----------------
        if (rank == 0 && ptx::elect_one()) {
            const uint32_t idesc = ptx::umma_idesc_bf16(2 * CU_TILE_M, (uint32_t)n_chunk);
            uint32_t unit = 0, sph = 0;
            int s = 0;
            bool ok = true;
            for (int tile = 0; tile < tiles_per_cta && ok; ++tile) {
                for (int pass = 0; pass < passes && ok; ++pass, ++unit) {
                    const uint32_t buf = unit & 1u, uph = (unit >> 1) & 1u;
                    if (!ptx::mbar_wait(&s_tempty[buf], uph ^ 1u, abort_flag)) { ok = false; break; }
                    ptx::tc_fence_after_sync();
                    const uint32_t d_base = tmem_base + buf * 256u;
                    for (int ks = 0; ks < ksteps; ++ks) {
                        if (!ptx::mbar_wait(&s_full[s], sph, abort_flag)) { ok = false; break; }
                        ptx::tc_fence_after_sync();
                        const uint32_t stage_addr = ptx::smem_u32(tiles + (size_t)s * stage_bytes);
                        const uint64_t desc_a = ptx::umma_desc_k_sw128(stage_addr);
                        const uint64_t desc_b = ptx::umma_desc_k_sw128(stage_addr + CU_X_TILE_BYTES);
#pragma unroll
                        for (int kk = 0; kk < CU_BLOCK_K / 16; ++kk)   // +32 bytes along K = +2 in the address field
                            ptx::umma_bf16_pair(d_base, desc_a + 2 * kk, desc_b + 2 * kk, idesc, (ks | kk) != 0);
                        ptx::umma_commit_pair(&s_empty[s]);   // frees the stage in both CTAs once these MMAs have read it
                        if (++s == stages) { s = 0; sph ^= 1u; }
                    }
                    if (ok) ptx::umma_commit_pair(&s_tfull[buf]);
                }
            }
            if (!ok) raise_status(DEV_TIMEOUT);
        }
    } else {
        // ---------------- epilogue: one row of this CTA's tile per thread ----------------
        const int et = threadIdx.x - 64;
        const int quad = warp & 3;                       // TMEM lanes [32*quad, 32*quad+32)
        const uint32_t lane_base = ((uint32_t)(quad * 32)) << 16;
        const uint32_t tempty0 = ptx::map_to_rank(&s_tempty[0], 0), tempty1 = ptx::map_to_rank(&s_tempty[1], 0);
        for (int j = et; j < groups * k; j += 128) s_hist[j] = 0;
        if (x_is_ready) grid_dependency_wait();
        for (int j = et; j < groups * kpad; j += 128) {
            const int g = j / kpad, jj = j % kpad;
            s_inv[j] = jj < k ? c_invnorm[(size_t)g * 2 * k + jj] : 0.f;
        }
        for (int j = et; j < groups * k; j += 128) s_inv2[j] = c_invnorm[(size_t)(j / k) * 2 * k + k + j % k];
        ptx::named_barrier(1, 128);                      // the epilogue warps share the norms
        uint32_t unit = 0;
        bool ok = true;
        for (int tile = 0; tile < tiles_per_cta && ok; ++tile) {
            const int64_t row = r0 + (int64_t)tile * CU_TILE_M + quad * 32 + lane;
            const bool live = r0 + (int64_t)tile * CU_TILE_M < r1;
            for (int g = 0; g < groups && ok; ++g) {
                float best = -1.f, s_best = 0.f;
                int j_best = 0;
                for (int ch = 0; ch < num_chunks && ok; ++ch, ++unit) {
                    const uint32_t buf = unit & 1u, uph = (unit >> 1) & 1u;
                    ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_tfull[buf], uph, abort_flag));   // warp-uniform
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    if (live) {
                        const uint32_t t_base = tmem_base + buf * 256u + lane_base;
                        const int jb = ch * n_chunk;
                        const float* inv = s_inv + g * kpad + jb;
                        uint32_t va[16], vb[16];
                        ptx::tmem_ld_16cols(t_base, va);
                        for (int c0 = 0; c0 < n_chunk; c0 += 32) {
                            ptx::tmem_ld_wait(va);
                            const bool second = c0 + 16 < n_chunk;
                            if (second) ptx::tmem_ld_16cols(t_base + (uint32_t)(c0 + 16), vb);
                            argmax16(va, inv + c0, jb + c0, best, s_best, j_best);
                            if (second) {
                                ptx::tmem_ld_wait(vb);
                                if (c0 + 32 < n_chunk) ptx::tmem_ld_16cols(t_base + (uint32_t)(c0 + 32), va);
                                argmax16(vb, inv + c0 + 16, jb + c0 + 16, best, s_best, j_best);
                            }
                        }
                    }
                    ptx::tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive_cluster(buf ? tempty1 : tempty0);
                }
                if (!ok) break;
                if (row < r1) {
                    store_index(out.f, out.f_type, (int64_t)g * out.out_stride + row, j_best);
                    const float a = s_best * s_inv2[g * k + j_best];
                    out.alpha[(int64_t)g * out.out_stride + row] = a;
                    if (a != 0.f) atomicAdd(&s_hist[g * k + j_best], 1);     // a row with alpha = 0 takes no part in the backward pass
                }
            }
        }
        if (!ok && lane == 0) raise_status(DEV_TIMEOUT);
        // this CTA's histograms of f, one row of the per-block table per group
        ptx::named_barrier(1, 128);
        if (out.hist && r0 < b) {
            for (int j = et; j < groups * k; j += 128) {
                const int g = j / k, jj = j % k;
                out.hist[(int64_t)g * out.hist_stride + (int64_t)blockIdx.x * k + jj] = s_hist[j];
            }
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync_all();      // neither CTA frees tensor memory or leaves while the other may still use it
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc_pair(tmem_base, 512);
    }
}

inline CompressPairPlan compress_pair_plan_for(int64_t b, int64_t k, int groups, int sms) {
    static size_t static_smem = 0;
    if (!static_smem) {
        cudaFuncAttributes fa;
        static_smem = cudaFuncGetAttributes(&fa, compress_pair_kernel) == cudaSuccess ? fa.sharedSizeBytes : 1024;
    }
    return compress_pair_plan(b, k, groups, sms, static_smem);
}

// Pairs pay where the chunks are wide enough for the pass to be bound by the tensor pipe.
inline bool compress_pair_usable(int64_t b, int64_t n, int64_t k, int groups, int sms) {
    if (!compress_umma_supported(b, n, k) || (int64_t)groups * k > (1 << 20) || sms < 2) return false;
    const CompressPairPlan p = compress_pair_plan_for(b, k, groups, sms);
    return p.stages >= 2 && p.n_chunk >= CP_MIN_CHUNK && cta_pairs_can_launch((const void*)compress_pair_kernel, CP_THREADS, p.smem_bytes);
}

inline pamm_status launch_compress_pair(const void* X, int64_t ldx, int64_t b, int64_t n, const void* C, int64_t ldc,
                                        int64_t k, int groups, const float* c_invnorm, const CompressOut& out, int sms,
                                        bool x_is_ready, cudaStream_t st) {
    const CompressPairPlan p = compress_pair_plan_for(b, k, groups, sms);
    if (p.stages < 2) return PAMM_ERR_UNSUPPORTED;
    CUtensorMap tm_x, tm_c;
    if (!make_tmap_bf16_sw128(&tm_x, X, (uint64_t)b, (uint64_t)n, (uint64_t)ldx, CU_BOX_ROWS) ||
        !make_tmap_bf16_sw128(&tm_c, C, (uint64_t)groups * (uint64_t)k, (uint64_t)n, (uint64_t)ldc, (uint32_t)(p.n_chunk / 2)))
        return tensor_map_failed();
    if (!ensure_dynamic_smem((const void*)compress_pair_kernel, p.smem_bytes)) return PAMM_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.grid);
    cfg.blockDim = dim3(CP_THREADS);
    cfg.dynamicSmemBytes = p.smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // set up while the select kernel runs
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    cudaLaunchKernelEx(&cfg, compress_pair_kernel, tm_x, tm_c, b, (int)n, (int)k, groups, p.n_chunk, p.num_chunks, p.stages,
                       p.stage_bytes, p.rows_per_cta, p.tiles_per_cta, x_is_ready ? 1 : 0, c_invnorm, out);
    return launch_result("compress_pair_kernel launch");
}

}  // namespace pamm
