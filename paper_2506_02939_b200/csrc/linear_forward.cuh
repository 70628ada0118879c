// Forward pass of the linear layer with the compression fused into it (Algorithm 2):
//   Z = X W   and   (alpha, f) = Compress(X) against the generators C,
// in ONE tensor-core kernel.  The scores S = X C^T are k more output columns of the
// product X [W | C^T]: a row block of X that is in flight for the tiles of Z is also
// multiplied by the generators, so the compression costs no pass over X of its own.
//
// bf16 operands, fp32 accumulation in tensor memory, Z stored as bf16.
//
// Work items: the rows are cut into blocks of 128; a row block has one item per
// 256 columns of W (a 128 x 256 tile of Z) plus one "score" item, which walks the
// generators in chunks of up to 256 with a running (best score, argmax, dot product)
// per row, exactly as the stand-alone compress kernel does (Lemma 1, Eq. 1, lowest index
// on ties).  Items are numbered so that the CTAs that run at the same time share
// operands in L2: groups of LF_GROUP row blocks, inside a group column tile by column
// tile.  One persistent CTA per SM takes items blockIdx.x, blockIdx.x + gridDim.x, ...
//   warp 0      TMA producer: the X tile (128 rows x 64 of the hidden dimension) and the
//               matching tile of W (64 x 256, four boxes) or of C, 128-byte swizzle;
//               every CTA fetches its own tiles
//   warp 1      issues tcgen05.mma (M = 128, N = 256 or the chunk's generators, K = 16);
//               two TMEM accumulators, so the epilogue of one item overlaps the MMAs
//               of the next
//   warps 2-5   epilogue, one thread per row of the tile: TMEM -> registers -> bf16 ->
//               swizzled shared memory -> TMA store in slabs of 64 columns; for a score
//               item the tournament argmax of the compress kernel, then f, alpha and
//               the row's count in the histogram of f
// W is n x m row-major, i.e. for a fixed hidden index the output columns are contiguous:
// an "MN-major" B operand.  C is k x n row-major: a K-major B operand.
#pragma once
#include "pamm_common.cuh"
#include "sm100_ptx.cuh"
#include "weight_grad_common.cuh"
#include "compress_umma.cuh"

namespace pamm {

constexpr int LF_THREADS = 192;
constexpr int LF_TILE_M = 128;
constexpr int LF_TILE_N = 256;
constexpr int LF_BLOCK_K = 64;
constexpr int LF_GROUP = 6;                              // row blocks whose items are interleaved
constexpr int LF_A_BYTES = LF_TILE_M * 128;              // 16 KiB
constexpr int LF_B_BYTES = LF_TILE_N * 128;              // 32 KiB (four 64-column boxes of 64 rows)
constexpr int LF_STAGE_BYTES = LF_A_BYTES + LF_B_BYTES;
constexpr int LF_SLAB_BYTES = LF_TILE_M * 128;           // staging of 128 rows x 64 bf16 columns
constexpr size_t LF_SMEM_LIMIT = 227 * 1024;

struct LinearForwardPlan {
    int n_chunk, num_chunks, stages, grid;
    int64_t row_blocks, col_tiles, items;
    size_t smem_bytes;
};

// k == 0: no compression, the plain product Z = X W (no score items).
inline LinearForwardPlan linear_forward_plan(int64_t b, int64_t m, int64_t k, int sms, size_t static_smem) {
    LinearForwardPlan p;
    const int npad = (int)round_up(std::max<int64_t>(k, 16), 16);
    p.num_chunks = (npad + 255) / 256;
    p.n_chunk = (int)round_up((npad + p.num_chunks - 1) / p.num_chunks, 16);
    p.row_blocks = (b + LF_TILE_M - 1) / LF_TILE_M;
    p.col_tiles = (m + LF_TILE_N - 1) / LF_TILE_N;
    p.items = p.row_blocks * (p.col_tiles + (k > 0 ? 1 : 0));
    // 1/||C||, 1/||C||^2, two histograms (a row block may straddle two blocks of the sort's partition)
    const size_t fixed = 1024 + LF_SLAB_BYTES + (size_t)(p.num_chunks * p.n_chunk + 3 * k) * 4 + 256;
    const size_t room = LF_SMEM_LIMIT > fixed + static_smem ? LF_SMEM_LIMIT - fixed - static_smem : 0;
    p.stages = (int)std::min<size_t>(8, room / LF_STAGE_BYTES);
    if (p.stages < 2) p.stages = 0;
    p.smem_bytes = fixed + (size_t)p.stages * LF_STAGE_BYTES;
    p.grid = (int)std::min<int64_t>(p.items, sms);
    return p;
}

// Item t -> (row block, column tile); `per_block` items per row block: the column tiles of W and,
// if there is one, the score item (column tile == col_tiles).
__device__ __forceinline__ void lf_decode(int64_t t, int64_t row_blocks, int64_t per_block, int64_t& rb, int64_t& ct,
                                          int group = LF_GROUP) {
    const int64_t per_group = (int64_t)group * per_block;
    const int64_t grp = t / per_group;
    const int64_t first = grp * group;
    const int64_t in_group = min((int64_t)group, row_blocks - first);     // the last group may be short
    const int64_t r = t - grp * per_group;
    ct = r / in_group;
    rb = first + r % in_group;
}

struct LinearForwardOut {
    void* f;
    float* alpha;
    int32_t* hist;           // per-block counts of f in the sort's row partition (zeroed beforehand), or nullptr
    int rows_per_block;      // that partition
    int f_type;
};

// Epilogue of a 128 x 256 tile of Z for one thread (one row): TMEM -> registers -> bf16 -> swizzled
// staging area -> TMA store, 64 columns at a time.  `release()` hands the accumulator back once its
// last columns are in registers (called by every thread of the warp, converged).
template <typename Release>
__device__ __forceinline__ void lf_store_z_tile(uint32_t t_base, uint8_t* slab, int row_in_tile, bool leader,
                                                const CUtensorMap* tm_z, int32_t col0, int32_t row0, Release release) {
#pragma unroll 1
    for (int sl = 0; sl < LF_TILE_N / 64; ++sl) {
        uint32_t v0[32], v1[32];
        ptx::tmem_ld_32x32(t_base + (uint32_t)(sl * 64), v0);
        ptx::tmem_ld_32x32(t_base + (uint32_t)(sl * 64 + 32), v1);
        ptx::tmem_ld_wait();
        if (sl == LF_TILE_N / 64 - 1) {          // the accumulator is in registers: hand it back
            ptx::tc_fence_before_sync();
            __syncwarp();
            release();
        }
        if (leader) ptx::bulk_wait_group_read<0>();     // the previous store has read the staging area
        ptx::named_barrier(1, 128);
        uint8_t* d0 = slab + row_in_tile * 128;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            *reinterpret_cast<uint4*>(d0 + ((c ^ (row_in_tile & 7)) << 4)) =
                make_uint4(pack_bf16(__uint_as_float(v0[8 * c]), __uint_as_float(v0[8 * c + 1])),
                           pack_bf16(__uint_as_float(v0[8 * c + 2]), __uint_as_float(v0[8 * c + 3])),
                           pack_bf16(__uint_as_float(v0[8 * c + 4]), __uint_as_float(v0[8 * c + 5])),
                           pack_bf16(__uint_as_float(v0[8 * c + 6]), __uint_as_float(v0[8 * c + 7])));
            *reinterpret_cast<uint4*>(d0 + (((c + 4) ^ (row_in_tile & 7)) << 4)) =
                make_uint4(pack_bf16(__uint_as_float(v1[8 * c]), __uint_as_float(v1[8 * c + 1])),
                           pack_bf16(__uint_as_float(v1[8 * c + 2]), __uint_as_float(v1[8 * c + 3])),
                           pack_bf16(__uint_as_float(v1[8 * c + 4]), __uint_as_float(v1[8 * c + 5])),
                           pack_bf16(__uint_as_float(v1[8 * c + 6]), __uint_as_float(v1[8 * c + 7])));
        }
        ptx::fence_proxy_async();
        ptx::named_barrier(1, 128);
        if (leader) {
            ptx::tma_store_2d(tm_z, slab, col0 + sl * 64, row0);
            ptx::bulk_commit_group();
        }
    }
}

// One chunk of generators for one row: the running (best score, dot product, argmax) over the
// chunk's n_chunk accumulator columns, the next 16 columns in flight while 16 are compared.
__device__ __forceinline__ void lf_score_chunk(uint32_t t_base, int n_chunk, const float* inv, int jb,
                                               float& best, float& s_best, int& j_best) {
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

// What a score item leaves behind for one row: f, alpha and the row's count in the histograms of
// the sort's row partition (a row block lies in block p0 of it and possibly p0 + 1).
__device__ __forceinline__ void lf_finish_scores(const LinearForwardOut& out, int64_t b, int k, int64_t rb, int64_t row, int et,
                                                 int j_best, float s_best, const float* s_inv2, int32_t* s_hist) {
    const int64_t p0 = out.hist ? (rb * LF_TILE_M) / out.rows_per_block : 0;
    if (row < b) {
        store_index(out.f, out.f_type, row, j_best);
        const float a = s_best * s_inv2[j_best];
        out.alpha[row] = a;
        if (out.hist && a != 0.f) atomicAdd(&s_hist[(int)(row / out.rows_per_block - p0) * k + j_best], 1);
    }
    ptx::named_barrier(1, 128);
    if (out.hist) {
        for (int j = et; j < 2 * k; j += 128) {
            const int32_t c = s_hist[j];
            if (c) atomicAdd(&out.hist[(p0 + j / k) * k + j % k], c);     // integers: exact in any order
        }
    }
    ptx::named_barrier(1, 128);
}

__global__ void __launch_bounds__(LF_THREADS, 1)
linear_forward_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
                      const __grid_constant__ CUtensorMap tm_c, const __grid_constant__ CUtensorMap tm_z,
                      int64_t b, int n, int m, int k, int n_chunk, int num_chunks, int stages,
                      int64_t row_blocks, int64_t col_tiles, int64_t items,
                      const float* __restrict__ c_invnorm, LinearForwardOut out, int w_kmajor) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_full[8], s_empty[8], s_tfull[2], s_tempty[2];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* slab = tiles + (size_t)stages * LF_STAGE_BYTES;
    const int kpad = n_chunk * num_chunks;
    float* s_inv = reinterpret_cast<float*>(slab + LF_SLAB_BYTES);
    float* s_inv2 = s_inv + kpad;
    int32_t* s_hist = reinterpret_cast<int32_t*>(s_inv2 + k);      // two tables of k
    const int ksteps = (n + LF_BLOCK_K - 1) / LF_BLOCK_K;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) { ptx::mbar_init(&s_full[s], 1); ptx::mbar_init(&s_empty[s], 1); }
        for (int u = 0; u < 2; ++u) { ptx::mbar_init(&s_tfull[u], 1); ptx::mbar_init(&s_tempty[u], 4); }
        s_abort = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async();
    }
    if (warp == 1) {
        ptx::tmem_alloc(&s_tmem_base, 512);
        ptx::tmem_relinquish();
    }
    grid_launch_dependents();     // released early; see the rule beside grid_dependency_wait
    // With generators, the kernel in front is the library's own selection, and X and W were complete
    // before it started.  Without, anything may be in front: wait for it before touching X or W.
    if (k == 0) grid_dependency_wait();
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = s_tmem_base;
    volatile int* abort_flag = &s_abort;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (ptx::elect_one()) {
            ptx::prefetch_tensormap(&tm_x);
            ptx::prefetch_tensormap(&tm_w);
            ptx::prefetch_tensormap(&tm_c);
            // X and W were complete before the kernel in front of this one (the generator selection)
            // started; C comes from it and is waited for where the first score item begins
            bool c_ready = false;
            uint32_t it = 0, sph = 0;
            int s = 0;               // ring stage and the parity of its use
            bool ok = true;
            for (int64_t t = blockIdx.x; t < items && ok; t += gridDim.x) {
                int64_t rb, ct;
                lf_decode(t, row_blocks, col_tiles + (k > 0 ? 1 : 0), rb, ct);
                const bool score = k > 0 && ct == col_tiles;
                if (score && !c_ready) { grid_dependency_wait(); c_ready = true; }
                const int units = score ? num_chunks : 1;
                for (int u = 0; u < units && ok; ++u) {
                    for (int ks = 0; ks < ksteps; ++ks, ++it) {
                        if (!ptx::mbar_wait(&s_empty[s], sph ^ 1u, abort_flag)) { ok = false; break; }
                        uint8_t* stage = tiles + (size_t)s * LF_STAGE_BYTES;
                        const uint32_t b_bytes = score ? (uint32_t)n_chunk * 128u : (uint32_t)LF_B_BYTES;
                        ptx::mbar_arrive_expect_tx(&s_full[s], LF_A_BYTES + b_bytes);
                        ptx::tma_load_2d(stage, &tm_x, ks * LF_BLOCK_K, (int32_t)(rb * LF_TILE_M), &s_full[s]);
                        if (score) {
                            ptx::tma_load_2d(stage + LF_A_BYTES, &tm_c, ks * LF_BLOCK_K, u * n_chunk, &s_full[s]);
                        } else if (w_kmajor) {      // W given as columns x hidden: the tile's 256 columns are 256 rows of it
                            ptx::tma_load_2d(stage + LF_A_BYTES, &tm_w, ks * LF_BLOCK_K, (int32_t)(ct * LF_TILE_N), &s_full[s]);
                        } else {
#pragma unroll
                            for (int q = 0; q < 4; ++q)
                                ptx::tma_load_2d(stage + LF_A_BYTES + q * 8192, &tm_w, (int32_t)(ct * LF_TILE_N + q * 64),
                                                 ks * LF_BLOCK_K, &s_full[s]);
                        }
                        if (++s == stages) { s = 0; sph ^= 1u; }
                    }
                }
            }
            if (!ok) {
                raise_status(DEV_TIMEOUT);
                const uint32_t back = it < (uint32_t)stages ? it : (uint32_t)stages;
                int never = 0;
                volatile int* no_abort = &never;     // let the copies already issued land before the CTA leaves
                for (uint32_t d = 1; d <= back; ++d) {
                    const uint32_t jt = it - d;
                    ptx::mbar_wait(&s_full[jt % stages], (jt / stages) & 1u, no_abort);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (ptx::elect_one()) {
            const uint32_t idesc_z = ptx::umma_idesc_bf16(LF_TILE_M, LF_TILE_N) | (w_kmajor ? 0u : 1u << 16);   // bit 16: B (W) MN-major
            const uint32_t idesc_s = ptx::umma_idesc_bf16(LF_TILE_M, (uint32_t)n_chunk);          // B (C) is K-major
            uint32_t unit = 0, sph = 0;
            int s = 0;               // ring stage and the parity of its use
            bool ok = true;
            for (int64_t t = blockIdx.x; t < items && ok; t += gridDim.x) {
                int64_t rb, ct;
                lf_decode(t, row_blocks, col_tiles + (k > 0 ? 1 : 0), rb, ct);
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
                        const uint32_t a_addr = ptx::smem_u32(tiles + (size_t)s * LF_STAGE_BYTES);
                        const uint32_t b_addr = a_addr + LF_A_BYTES;
                        const uint64_t desc_a = ptx::umma_desc_k_sw128(a_addr);
                        if (score || w_kmajor) {
                            const uint64_t desc_b = ptx::umma_desc_k_sw128(b_addr);
                            const uint32_t idesc = score ? idesc_s : idesc_z;
#pragma unroll
                            for (int kk = 0; kk < LF_BLOCK_K / 16; ++kk)
                                ptx::umma_bf16(d_addr, desc_a + 2 * kk, desc_b + 2 * kk, idesc, (ks | kk) != 0);
                        } else {
#pragma unroll
                            for (int kk = 0; kk < LF_BLOCK_K / 16; ++kk)   // 16 hidden indices = two 8-deep groups = 2048 bytes
                                ptx::umma_bf16(d_addr, desc_a + 2 * kk, umma_desc_mn_sw128(b_addr + kk * 2048, 8192, 1024),
                                               idesc_z, (ks | kk) != 0);
                        }
                        ptx::umma_commit(&s_empty[s]);
                        if (++s == stages) { s = 0; sph ^= 1u; }
                    }
                    if (ok) ptx::umma_commit(&s_tfull[buf]);
                }
            }
            if (!ok) raise_status(DEV_TIMEOUT);
        }
    } else {
        // ---------------- epilogue: one row of the tile per thread ----------------
        const int et = threadIdx.x - 64;
        const int quad = warp & 3;                       // TMEM lanes [32*quad, 32*quad+32)
        const int row_in_tile = quad * 32 + lane;
        const uint32_t lane_base = ((uint32_t)(quad * 32)) << 16;
        const bool leader = et == 0;
        bool norms_loaded = false;
        uint32_t unit = 0;
        bool ok = true;
        for (int64_t t = blockIdx.x; t < items && ok; t += gridDim.x) {
            int64_t rb, ct;
            lf_decode(t, row_blocks, col_tiles + (k > 0 ? 1 : 0), rb, ct);
            const bool score = k > 0 && ct == col_tiles;
            const int64_t row = rb * LF_TILE_M + row_in_tile;
            if (!score) {
                const uint32_t buf = unit & 1u, uph = (unit >> 1) & 1u;
                ++unit;
                ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_tfull[buf], uph, abort_flag));   // warp-uniform
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t t_base = tmem_base + buf * (uint32_t)LF_TILE_N + lane_base;
                lf_store_z_tile(t_base, slab, row_in_tile, leader, &tm_z, (int32_t)(ct * LF_TILE_N), (int32_t)(rb * LF_TILE_M),
                                [&] { if (lane == 0) ptx::mbar_arrive(&s_tempty[buf]); });
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
                    if (lane == 0) ptx::mbar_arrive(&s_tempty[buf]);
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
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, 512);
    }
}

inline bool linear_forward_supported(int64_t b, int64_t n, int64_t m, int64_t k) {
    return (k == 0 || compress_umma_supported(b, n, k)) && b >= 1 && n >= 8 && n < (1ll << 31) && m >= 8 && m < (1ll << 31);
}

inline LinearForwardPlan linear_forward_plan_for(int64_t b, int64_t m, int64_t k, int sms) {
    static size_t static_smem = 0;
    if (!static_smem) {
        cudaFuncAttributes fa;
        static_smem = cudaFuncGetAttributes(&fa, linear_forward_kernel) == cudaSuccess ? fa.sharedSizeBytes : 1024;
    }
    return linear_forward_plan(b, m, k, sms, static_smem);
}

inline pamm_status launch_linear_forward(const void* X, int64_t ldx, int64_t b, int64_t n, const void* W, int64_t ldw,
                                         int64_t m, const void* C, int64_t ldc, int64_t k, const float* c_invnorm,
                                         void* Z, int64_t ldz, const LinearForwardOut& out, int sms, cudaStream_t st,
                                         bool w_kmajor = false) {
    const LinearForwardPlan p = linear_forward_plan_for(b, m, k, sms);
    if (p.stages < 2) return PAMM_ERR_UNSUPPORTED;
    CUtensorMap tm_x, tm_w, tm_c, tm_z;
    if (!make_tmap_bf16_sw128(&tm_x, X, (uint64_t)b, (uint64_t)n, (uint64_t)ldx, LF_TILE_M) ||
        !(w_kmajor ? make_tmap_bf16_sw128(&tm_w, W, (uint64_t)m, (uint64_t)n, (uint64_t)ldw, LF_TILE_N)      // m x n: columns x hidden
                   : make_tmap_bf16_sw128(&tm_w, W, (uint64_t)n, (uint64_t)m, (uint64_t)ldw, LF_BLOCK_K)) ||
        !(k > 0 ? make_tmap_bf16_sw128(&tm_c, C, (uint64_t)k, (uint64_t)n, (uint64_t)ldc, (uint32_t)p.n_chunk)
                : make_tmap_bf16_sw128(&tm_c, X, (uint64_t)b, (uint64_t)n, (uint64_t)ldx, LF_TILE_M)) ||     // unused without generators
        !make_tmap_bf16_sw128(&tm_z, Z, (uint64_t)b, (uint64_t)m, (uint64_t)ldz, LF_TILE_M))
        return tensor_map_failed();
    if (!ensure_dynamic_smem((const void*)linear_forward_kernel, p.smem_bytes)) return PAMM_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.grid);
    cfg.blockDim = dim3(LF_THREADS);
    cfg.dynamicSmemBytes = p.smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // starts on X and W while the selection still runs
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, linear_forward_kernel, tm_x, tm_w, tm_c, tm_z, b, (int)n, (int)m, (int)k, p.n_chunk, p.num_chunks,
                       p.stages, p.row_blocks, p.col_tiles, p.items, c_invnorm, out, w_kmajor ? 1 : 0);
    return launch_result("linear_forward_kernel launch");
}

}  // namespace pamm
