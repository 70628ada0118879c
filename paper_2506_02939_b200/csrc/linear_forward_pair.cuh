// The fused forward pass (Algorithm 2: Z = X W and Compress(X) from one tensor-core kernel)
// on PAIRS of CTAs: a cluster of two CTAs on the two SMs of a TPC computes one 256 x 256
// tile with `tcgen05.mma.cta_group::2`.  Each CTA brings 128 rows of X and HALF of the B
// operand (128 of the tile's 256 columns of W, or half of the chunk's generators), so a CTA
// moves 32 KB through its shared memory per 64 hidden indices instead of the 48 KB of the
// one-CTA kernel (linear_forward.cuh) -- that kernel keeps the tensor pipe busy 84% of the
// time because operand reads and TMA writes together saturate shared memory.
//
// Work items are those of the one-CTA kernel with row-block PAIRS (256 rows) in place of row
// blocks; the epilogue (one thread per row, each CTA its own 128 rows) is the same code.
//   rank 0 (leader)  warp 0 loads its tiles, warp 1 issues every MMA of the pair
//   rank 1           warp 0 loads its tiles, warp 1 only allocates and frees tensor memory
// Barriers: `full` lives in the leader and counts the bytes of both CTAs' loads (the
// loads name it by its cluster address); `empty` and `tfull` exist in both CTAs at the same
// offset and are arrived on by one multicast `tcgen05.commit`; `tempty` lives in the leader
// and takes the arrivals of the eight epilogue warps of the pair.  No load uses multicast.
// Every wait is bounded; all threads of both CTAs meet at a cluster barrier before the tensor
// memory is freed, whatever happened before.
#pragma once
#include "linear_forward.cuh"

namespace pamm {

constexpr int LP_PAIR_M = 2 * LF_TILE_M;                 // rows of a pair's tile
constexpr int LP_GROUP = LF_GROUP / 2;                   // row-block pairs whose items are interleaved
constexpr int LP_B_BYTES = (LF_TILE_N / 2) * 128;        // 16 KiB: this CTA's half of the B operand
constexpr int LP_STAGE_BYTES = LF_A_BYTES + LP_B_BYTES;

// n_chunk is a multiple of 32 here: each CTA holds half of a chunk's generators, in groups of 16.
inline LinearForwardPlan linear_forward_pair_plan(int64_t b, int64_t m, int64_t k, int sms, size_t static_smem) {
    LinearForwardPlan p;
    const int npad = (int)round_up(std::max<int64_t>(k, 32), 32);
    p.num_chunks = (npad + 255) / 256;
    p.n_chunk = (int)round_up((npad + p.num_chunks - 1) / p.num_chunks, 32);
    p.row_blocks = (b + LP_PAIR_M - 1) / LP_PAIR_M;          // pairs of row blocks
    p.col_tiles = (m + LF_TILE_N - 1) / LF_TILE_N;
    p.items = p.row_blocks * (p.col_tiles + (k > 0 ? 1 : 0));
    const size_t fixed = 1024 + LF_SLAB_BYTES + (size_t)(p.num_chunks * p.n_chunk + 3 * k) * 4 + 256;
    const size_t room = LF_SMEM_LIMIT > fixed + static_smem ? LF_SMEM_LIMIT - fixed - static_smem : 0;
    p.stages = (int)std::min<size_t>(8, room / LP_STAGE_BYTES);
    if (p.stages < 2) p.stages = 0;
    p.smem_bytes = fixed + (size_t)p.stages * LP_STAGE_BYTES;
    p.grid = 2 * (int)std::max<int64_t>(1, std::min<int64_t>(p.items, sms / 2));
    return p;
}

__global__ void __launch_bounds__(LF_THREADS, 1)
linear_forward_pair_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
                           const __grid_constant__ CUtensorMap tm_c, const __grid_constant__ CUtensorMap tm_z,
                           int64_t b, int n, int m, int k, int n_chunk, int num_chunks, int stages,
                           int64_t row_pairs, int64_t col_tiles, int64_t items,
                           const float* __restrict__ c_invnorm, LinearForwardOut out, int w_kmajor) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_full[8], s_empty[8], s_tfull[2], s_tempty[2];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();            // 0 = leader
    const int64_t pair = blockIdx.x >> 1, pairs_in_grid = gridDim.x >> 1;
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* slab = tiles + (size_t)stages * LP_STAGE_BYTES;
    const int kpad = n_chunk * num_chunks;
    float* s_inv = reinterpret_cast<float*>(slab + LF_SLAB_BYTES);
    float* s_inv2 = s_inv + kpad;
    int32_t* s_hist = reinterpret_cast<int32_t*>(s_inv2 + k);      // two tables of k
    const int ksteps = (n + LF_BLOCK_K - 1) / LF_BLOCK_K;
    const int64_t per_pair = col_tiles + (k > 0 ? 1 : 0);

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
    if (k == 0) grid_dependency_wait();
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
            ptx::prefetch_tensormap(&tm_w);
            ptx::prefetch_tensormap(&tm_c);
            bool c_ready = false;
            uint32_t it = 0, sph = 0;
            int s = 0;               // ring stage and the parity of its use
            bool ok = true;
            for (int64_t t = pair; t < items && ok; t += pairs_in_grid) {
                int64_t rp, ct;
                lf_decode(t, row_pairs, per_pair, rp, ct, LP_GROUP);
                const bool score = k > 0 && ct == col_tiles;
                if (score && !c_ready) { grid_dependency_wait(); c_ready = true; }
                const int units = score ? num_chunks : 1;
                const int32_t row0 = (int32_t)(rp * LP_PAIR_M + rank * LF_TILE_M);
                for (int u = 0; u < units && ok; ++u) {
                    for (int ks = 0; ks < ksteps; ++ks, ++it) {
                        if (!ptx::mbar_wait(&s_empty[s], sph ^ 1u, abort_flag)) { ok = false; break; }
                        uint8_t* stage = tiles + (size_t)s * LP_STAGE_BYTES;
                        const uint32_t b_bytes = score ? (uint32_t)(n_chunk / 2) * 128u : (uint32_t)LP_B_BYTES;
                        // the leader's barrier counts the bytes of both CTAs
                        if (rank == 0) ptx::mbar_arrive_expect_tx(&s_full[s], 2u * (LF_A_BYTES + b_bytes));
                        const uint32_t full = ptx::map_to_rank(&s_full[s], 0);
                        ptx::tma_load_2d_pair(stage, &tm_x, ks * LF_BLOCK_K, row0, full);
                        if (score) {
                            ptx::tma_load_2d_pair(stage + LF_A_BYTES, &tm_c, ks * LF_BLOCK_K,
                                                  u * n_chunk + (int32_t)rank * (n_chunk / 2), full);
                        } else if (w_kmajor) {      // W given as columns x hidden: this CTA's 128 columns are 128 rows of it
                            ptx::tma_load_2d_pair(stage + LF_A_BYTES, &tm_w, ks * LF_BLOCK_K,
                                                  (int32_t)(ct * LF_TILE_N + rank * (LF_TILE_N / 2)), full);
                        } else {
#pragma unroll
                            for (int q = 0; q < 2; ++q)
                                ptx::tma_load_2d_pair(stage + LF_A_BYTES + q * 8192, &tm_w,
                                                      (int32_t)(ct * LF_TILE_N + rank * (LF_TILE_N / 2) + q * 64), ks * LF_BLOCK_K, full);
                        }
                        if (++s == stages) { s = 0; sph ^= 1u; }
                    }
                }
            }
            if (!ok) {
                raise_status(DEV_TIMEOUT);
                // Copies already issued land in this CTA's shared memory; their completion is counted in the
                // leader, which can wait for it.  The partner waits a fixed time instead (the cluster barrier
                // below then keeps both CTAs, and their shared memory, alive until the other has come too).
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
            const uint32_t idesc_z = ptx::umma_idesc_bf16(LP_PAIR_M, LF_TILE_N) | (w_kmajor ? 0u : 1u << 16);   // bit 16: B (W) MN-major
            const uint32_t idesc_s = ptx::umma_idesc_bf16(LP_PAIR_M, (uint32_t)n_chunk);          // B (C) is K-major
            uint32_t unit = 0, sph = 0;
            int s = 0;
            bool ok = true;
            for (int64_t t = pair; t < items && ok; t += pairs_in_grid) {
                int64_t rp, ct;
                lf_decode(t, row_pairs, per_pair, rp, ct, LP_GROUP);
                const bool score = k > 0 && ct == col_tiles;
                const int units = score ? num_chunks : 1;
                for (int u = 0; u < units && ok; ++u, ++unit) {
                    const uint32_t buf = unit & 1u, uph = (unit >> 1) & 1u;
                    if (!ptx::mbar_wait(&s_tempty[buf], uph ^ 1u, abort_flag)) { ok = false; break; }
                    ptx::tc_fence_after_sync();
                    const uint32_t d_addr = tmem_base + buf * (uint32_t)LF_TILE_N;
                    for (int ks = 0; ks < ksteps; ++ks) {
                        if (!ptx::mbar_wait(&s_full[s], sph, abort_flag)) { ok = false; break; }
                        ptx::tc_fence_after_sync();
                        const uint32_t a_addr = ptx::smem_u32(tiles + (size_t)s * LP_STAGE_BYTES);
                        const uint32_t b_addr = a_addr + LF_A_BYTES;
                        const uint64_t desc_a = ptx::umma_desc_k_sw128(a_addr);
                        if (score || w_kmajor) {
                            const uint64_t desc_b = ptx::umma_desc_k_sw128(b_addr);
                            const uint32_t idesc = score ? idesc_s : idesc_z;
#pragma unroll
                            for (int kk = 0; kk < LF_BLOCK_K / 16; ++kk)
                                ptx::umma_bf16_pair(d_addr, desc_a + 2 * kk, desc_b + 2 * kk, idesc, (ks | kk) != 0);
                        } else {
#pragma unroll
                            for (int kk = 0; kk < LF_BLOCK_K / 16; ++kk)   // 16 hidden indices = two 8-deep groups = 2048 bytes
                                ptx::umma_bf16_pair(d_addr, desc_a + 2 * kk, umma_desc_mn_sw128(b_addr + kk * 2048, 8192, 1024),
                                                    idesc_z, (ks | kk) != 0);
                        }
                        ptx::umma_commit_pair(&s_empty[s]);      // frees the stage in both CTAs
                        if (++s == stages) { s = 0; sph ^= 1u; }
                    }
                    if (ok) ptx::umma_commit_pair(&s_tfull[buf]);
                }
            }
            if (!ok) raise_status(DEV_TIMEOUT);
        }
    } else {
        // ---------------- epilogue: one row of this CTA's half of the tile per thread ----------------
        const int et = threadIdx.x - 64;
        const int quad = warp & 3;                       // TMEM lanes [32*quad, 32*quad+32)
        const int row_in_tile = quad * 32 + lane;
        const uint32_t lane_base = ((uint32_t)(quad * 32)) << 16;
        const bool leader = et == 0;
        const uint32_t tempty0 = ptx::map_to_rank(&s_tempty[0], 0), tempty1 = ptx::map_to_rank(&s_tempty[1], 0);
        bool norms_loaded = false;
        uint32_t unit = 0;
        bool ok = true;
        for (int64_t t = pair; t < items && ok; t += pairs_in_grid) {
            int64_t rp, ct;
            lf_decode(t, row_pairs, per_pair, rp, ct, LP_GROUP);
            const bool score = k > 0 && ct == col_tiles;
            const int64_t rb = rp * 2 + rank;             // this CTA's row block
            const int64_t row = rb * LF_TILE_M + row_in_tile;
            if (!score) {
                const uint32_t buf = unit & 1u, uph = (unit >> 1) & 1u;
                ++unit;
                ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_tfull[buf], uph, abort_flag));   // warp-uniform
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t t_base = tmem_base + buf * (uint32_t)LF_TILE_N + lane_base;
                lf_store_z_tile(t_base, slab, row_in_tile, leader, &tm_z, (int32_t)(ct * LF_TILE_N), (int32_t)(rb * LF_TILE_M),
                                [&] { if (lane == 0) ptx::mbar_arrive_cluster(buf ? tempty1 : tempty0); });
            } else {
                if (!norms_loaded) {      // C's norms come from the kernel in front
                    grid_dependency_wait();
                    for (int j = et; j < kpad; j += 128) s_inv[j] = j < k ? c_invnorm[j] : 0.f;
                    for (int j = et; j < k; j += 128) s_inv2[j] = c_invnorm[k + j];
                    norms_loaded = true;
                }
                for (int j = et; j < 2 * k; j += 128) s_hist[j] = 0;
                ptx::named_barrier(1, 128);
                float best = -1.f, s_best = 0.f;
                int j_best = 0;
                for (int ch = 0; ch < num_chunks && ok; ++ch, ++unit) {
                    const uint32_t buf = unit & 1u, uph = (unit >> 1) & 1u;
                    ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_tfull[buf], uph, abort_flag));
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    const uint32_t t_base = tmem_base + buf * (uint32_t)LF_TILE_N + lane_base;
                    lf_score_chunk(t_base, n_chunk, s_inv + ch * n_chunk, ch * n_chunk, best, s_best, j_best);
                    ptx::tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive_cluster(buf ? tempty1 : tempty0);
                }
                if (!ok) break;
                lf_finish_scores(out, b, k, rb, row, et, j_best, s_best, s_inv2, s_hist);
            }
        }
        if (leader) ptx::bulk_wait_group<0>();
        if (!ok && lane == 0) raise_status(DEV_TIMEOUT);
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync_all();      // neither CTA frees tensor memory or leaves while the other may still use it
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc_pair(tmem_base, 512);
    }
}

// Needs at least one pair of SMs; k a multiple of 32 per chunk is arranged by padding.
inline LinearForwardPlan linear_forward_pair_plan_for(int64_t b, int64_t m, int64_t k, int sms) {
    static size_t static_smem = 0;
    if (!static_smem) {
        cudaFuncAttributes fa;
        static_smem = cudaFuncGetAttributes(&fa, linear_forward_pair_kernel) == cudaSuccess ? fa.sharedSizeBytes : 1024;
    }
    return linear_forward_pair_plan(b, m, k, sms, static_smem);
}

inline pamm_status launch_linear_forward_pair(const void* X, int64_t ldx, int64_t b, int64_t n, const void* W, int64_t ldw,
                                              int64_t m, const void* C, int64_t ldc, int64_t k, const float* c_invnorm,
                                              void* Z, int64_t ldz, const LinearForwardOut& out, int sms, cudaStream_t st,
                                              bool w_kmajor = false) {
    const LinearForwardPlan p = linear_forward_pair_plan_for(b, m, k, sms);
    if (p.stages < 2 || sms < 2) return PAMM_ERR_UNSUPPORTED;
    CUtensorMap tm_x, tm_w, tm_c, tm_z;
    if (!make_tmap_bf16_sw128(&tm_x, X, (uint64_t)b, (uint64_t)n, (uint64_t)ldx, LF_TILE_M) ||
        !(w_kmajor ? make_tmap_bf16_sw128(&tm_w, W, (uint64_t)m, (uint64_t)n, (uint64_t)ldw, LF_TILE_N / 2)      // m x n: columns x hidden
                   : make_tmap_bf16_sw128(&tm_w, W, (uint64_t)n, (uint64_t)m, (uint64_t)ldw, LF_BLOCK_K)) ||
        !(k > 0 ? make_tmap_bf16_sw128(&tm_c, C, (uint64_t)k, (uint64_t)n, (uint64_t)ldc, (uint32_t)(p.n_chunk / 2))
                : make_tmap_bf16_sw128(&tm_c, X, (uint64_t)b, (uint64_t)n, (uint64_t)ldx, LF_TILE_M)) ||     // unused without generators
        !make_tmap_bf16_sw128(&tm_z, Z, (uint64_t)b, (uint64_t)m, (uint64_t)ldz, LF_TILE_M))
        return tensor_map_failed();
    if (!ensure_dynamic_smem((const void*)linear_forward_pair_kernel, p.smem_bytes)) return PAMM_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.grid);
    cfg.blockDim = dim3(LF_THREADS);
    cfg.dynamicSmemBytes = p.smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // starts on X and W while the selection still runs
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    cudaLaunchKernelEx(&cfg, linear_forward_pair_kernel, tm_x, tm_w, tm_c, tm_z, b, (int)n, (int)m, (int)k, p.n_chunk,
                       p.num_chunks, p.stages, p.row_blocks, p.col_tiles, p.items, c_invnorm, out, w_kmajor ? 1 : 0);
    return launch_result("linear_forward_pair_kernel launch");
}

}  // namespace pamm
