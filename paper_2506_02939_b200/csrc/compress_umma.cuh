// Step 2 on tensor cores (bf16 inputs): S = X C^T with tcgen05.mma into tensor
// memory, then per-row argmax of |S_ij| / ||C_j|| (Lemma 1) and alpha (Eq. 1).
//
// One streaming pass over X.  The rows are cut into equal contiguous ranges, one
// per CTA (one CTA per SM, a single balanced wave).  Inside a CTA:
//   warp 0     TMA producer: X tiles (64-row boxes, so a ragged last tile costs
//              only the boxes it needs) and the matching C tile, 64 columns of
//              the hidden dimension per pipeline stage, 128-byte swizzle
//   warp 1     issues tcgen05.mma (M = 128 rows, N = generators of the chunk,
//              K = 16 per instruction), fp32 accumulators in TMEM, two buffers
//   warps 2-   epilogue, four warps per row tile of the super tile: each thread owns one
//              row (TMEM lane) of one tile, reads its scores
//              with tcgen05.ld and scans them in ascending j with a strict '>'
//              so the lowest index wins ties; the epilogue of one tile overlaps
//              the MMAs of the next
//   warps 6-   (neighbourhood variant only, Eq. 2; four warps per row tile of the
//              super tile) squared row norms ||X_i||^2: each thread re-reads its
//              row's 128 bytes of every X tile from shared memory
//              while the tile waits for / feeds the tensor core, so X is still read
//              from HBM once; the epilogue then drops a row when
//              ||X_i||^2 - S^2/||C_f||^2 > eps^2 ||X_i||^2 (+ a rounding allowance)
// C is small (k x n) and is re-read per row tile from L2; with MT = 2 two row
// tiles share every C tile.  For k > 256 the generators are processed in chunks
// with a running (best score, argmax, dot product) per row; X is then fetched once
// per chunk, from HBM the first time and from L2 afterwards (only the last pass
// over a tile carries the evict-first hint).
//
// Several independent generator sets ("groups": one compression per projection,
// Section 4) are served by the same pass: the chunks of all groups follow one
// another, the running argmax restarts at every group, and every group gets its
// own f and alpha.  The epilogue also counts, per CTA and group, how many rows with
// alpha != 0 chose each generator (integer atomics in shared memory): the per-block
// histograms the backward pass's counting sort starts from.
#pragma once
#include "pamm_common.cuh"
#include "sm100_ptx.cuh"

namespace pamm {

__host__ __device__ constexpr int CU_THREADS(int mt) { return 64 + mt * 128; }         // producer, MMA issuer, one epilogue thread per row of the super tile
__host__ __device__ constexpr int CU_THREADS_EPS(int mt) { return 64 + mt * 256; }     // + one thread per row for ||X_i||^2
constexpr int CU_BLOCK_K = 64;                 // bf16 columns per stage = one 128-byte swizzle row
constexpr int CU_TILE_M = 128;
constexpr int CU_BOX_ROWS = 64;                // rows per TMA box of X (a ragged last tile fetches only the boxes it needs)
constexpr int CU_X_TILE_BYTES = CU_TILE_M * 128;   // 16 KiB
constexpr int CU_MAX_K = 4096;                 // 1/||C_j|| and 1/||C_j||^2 live in shared memory
constexpr int CU_SMEM_BUDGET = 200 * 1024;     // pipeline stages: more than this buys nothing
constexpr size_t CU_SMEM_LIMIT = 227 * 1024;   // dynamic + static shared memory a CTA may have

struct CompressUmmaPlan {
    int mt;            // row tiles (of 128) per super tile
    int n_chunk;       // generators per chunk, padded to a multiple of 16 (<= 256)
    int num_chunks;    // chunks per group
    int stages;        // 0 when the shared memory does not allow two stages
    int stage_bytes;
    int tmem_cols;
    int tmem_bufs;
    int rows_per_cta;
    int grid;
    size_t smem_bytes;
};

inline bool compress_umma_supported(int64_t b, int64_t n, int64_t k) {
    return k >= 16 && k <= CU_MAX_K && n >= 8 && b >= 1 && n < (1ll << 31);
}

// Rows per CTA of the streaming pass: equal contiguous ranges, a multiple of the TMA box.
// The same partition is used for the per-block histograms of f.
inline int compress_rows_per_cta(int64_t b, int sms) {
    const int64_t per = (b + sms - 1) / sms;
    return (int)std::min<int64_t>(std::max<int64_t>(CU_BOX_ROWS, round_up(per, CU_BOX_ROWS)), 1ll << 30);
}

// static_smem: the kernel's statically declared shared memory (barriers, row norms).
inline CompressUmmaPlan compress_umma_plan(int64_t b, int64_t k, int groups, int sms, size_t static_smem) {
    CompressUmmaPlan p;
    const int npad = (int)round_up(k, 16);
    p.num_chunks = (npad + 255) / 256;
    p.n_chunk = (int)round_up((npad + p.num_chunks - 1) / p.num_chunks, 16);
    p.mt = 2;      // two row tiles share every C tile; beyond 128 generators per chunk they fill TMEM (one buffer)
    p.stage_bytes = p.mt * CU_X_TILE_BYTES + p.n_chunk * 128;
    // 1/||C||, 1/||C||^2 and the histogram of every group, the 1024-byte alignment slack
    const size_t fixed = 1024 + (size_t)groups * (p.num_chunks * p.n_chunk + 2 * k) * 4 + 256;
    const size_t budget = CU_SMEM_LIMIT > fixed + static_smem ? CU_SMEM_LIMIT - fixed - static_smem : 0;
    p.stages = (int)std::min<size_t>(8, std::min<size_t>(CU_SMEM_BUDGET, budget) / p.stage_bytes);
    if (p.stages < 2) p.stages = 0;
    p.tmem_bufs = 2 * p.mt * p.n_chunk <= 512 ? 2 : 1;     // accumulator sets: the epilogue overlaps the next MMAs only with two
    int cols = p.tmem_bufs * p.mt * p.n_chunk;
    p.tmem_cols = 32;
    while (p.tmem_cols < cols) p.tmem_cols *= 2;
    p.rows_per_cta = compress_rows_per_cta(b, sms);
    p.grid = (int)((b + p.rows_per_cta - 1) / p.rows_per_cta);
    p.smem_bytes = fixed + (size_t)p.stages * p.stage_bytes;
    return p;
}

// Folds 16 consecutive scores |s_i| * inv_i into the running (best score, its dot
// product, its index).  A left-biased tournament: at every node the right entry
// wins only if strictly larger, so the lowest index keeps a tie, exactly as an
// ascending scan with '>' would -- but four levels deep instead of sixteen.
__device__ __forceinline__ void argmax16(const uint32_t (&v)[16], const float* __restrict__ inv, int j0,
                                         float& best, float& s_best, int& j_best) {
    float sc[16], sv[16];
    int ji[16];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const float4 w = *reinterpret_cast<const float4*>(inv + 4 * q);
        sv[4 * q] = __uint_as_float(v[4 * q]);         sc[4 * q] = fabsf(sv[4 * q]) * w.x;
        sv[4 * q + 1] = __uint_as_float(v[4 * q + 1]); sc[4 * q + 1] = fabsf(sv[4 * q + 1]) * w.y;
        sv[4 * q + 2] = __uint_as_float(v[4 * q + 2]); sc[4 * q + 2] = fabsf(sv[4 * q + 2]) * w.z;
        sv[4 * q + 3] = __uint_as_float(v[4 * q + 3]); sc[4 * q + 3] = fabsf(sv[4 * q + 3]) * w.w;
    }
#pragma unroll
    for (int i = 0; i < 16; ++i) ji[i] = i;
#pragma unroll
    for (int width = 1; width < 16; width <<= 1) {
#pragma unroll
        for (int i = 0; i < 16; i += 2 * width) {
            const bool right = sc[i + width] > sc[i];
            sc[i] = right ? sc[i + width] : sc[i];
            sv[i] = right ? sv[i + width] : sv[i];
            ji[i] = right ? ji[i + width] : ji[i];
        }
    }
    if (sc[0] > best) { best = sc[0]; s_best = sv[0]; j_best = j0 + ji[0]; }
}

// Rounding allowance of the neighbourhood test, relative to ||X_i||^2: both
// ||X_i||^2 and S^2/||C_f||^2 are fp32 sums of n terms, so their difference is
// only known to about 2 n 2^-24 ||X_i||^2.  With it, a row that lies exactly on
// its generator's line (distance 0) is kept for every eps >= 0.
__host__ __device__ inline float neighbourhood_slack(int64_t n) { return 2.f * (float)n * 5.9604645e-8f; }

// What the compress kernel writes besides alpha.
struct CompressOut {
    void* f;                 // groups x out_stride entries of `f_type` (a pamm_index_type)
    float* alpha;            // groups x out_stride
    int64_t out_stride;      // distance between two groups' vectors, in entries
    int32_t* hist;           // per group, gridDim.x x k counts of f per CTA; or nullptr
    int64_t hist_stride;     // distance between two groups' tables, in counts
    int f_type;
};

// EPS = false: the paper's setting (epsilon = infinity), nothing is dropped.
// EPS = true : eps2 = epsilon^2 and slack as above; *dropped counts the dropped rows (one group only).
// C holds the generators of all groups, group g in rows [g k, (g+1) k); c_invnorm holds 2k
// entries per group (1/||C_j||, then 1/||C_j||^2).
template <int MT, bool EPS>
__global__ void __launch_bounds__(EPS ? CU_THREADS_EPS(MT) : CU_THREADS(MT), 1)
compress_umma_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_c,
                     int64_t b, int n, int k, int groups, int n_chunk, int num_chunks, int stages, int stage_bytes,
                     int tmem_cols, int tmem_bufs, int rows_per_cta, int x_is_ready, const float* __restrict__ c_invnorm,
                     CompressOut out, float eps2, float slack, int32_t* __restrict__ dropped) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_full[8], s_empty[8], s_tfull[2], s_tempty[2], s_nfull[2], s_nempty[2];
    __shared__ float s_norm[EPS ? 2 : 1][EPS ? MT * CU_TILE_M : 1];     // ||X_i||^2 of the rows of a super tile (EPS only)
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    // per group: 1/||C_j|| for every column the chunks cover, zero beyond k (a padded column
    // scores 0 and never beats a real one); then 1/||C_j||^2; then the histogram of f
    const int kpad = n_chunk * num_chunks;
    float* s_inv = reinterpret_cast<float*>(tiles + (size_t)stages * stage_bytes);
    float* s_inv2 = s_inv + groups * kpad;
    int32_t* s_hist = reinterpret_cast<int32_t*>(s_inv2 + groups * k);

    const int64_t r0 = (int64_t)blockIdx.x * rows_per_cta;
    const int64_t r1 = min(b, r0 + (int64_t)rows_per_cta);
    const int ksteps = (n + CU_BLOCK_K - 1) / CU_BLOCK_K;
    const int super_rows = MT * CU_TILE_M;
    const int passes = groups * num_chunks;          // passes over a super tile of X: one per (group, chunk)

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) { ptx::mbar_init(&s_full[s], 1); ptx::mbar_init(&s_empty[s], EPS ? 1 + 4 * MT : 1); }
        for (int u = 0; u < 2; ++u) {
            ptx::mbar_init(&s_tfull[u], 1);
            ptx::mbar_init(&s_tempty[u], 4 * MT);
            ptx::mbar_init(&s_nfull[u], 4 * MT);
            ptx::mbar_init(&s_nempty[u], 4 * MT);
        }
        s_abort = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async();
    }
    if (warp == 1) {
        ptx::tmem_alloc(&s_tmem_base, (uint32_t)tmem_cols);
        ptx::tmem_relinquish();
    }
    // The next kernel of the stream may set itself up meanwhile.  It is released before this
    // kernel's own wait: its grid_dependency_wait() still covers everything older (see the
    // rule beside grid_dependency_wait), and it must not touch f, alpha or the histograms
    // before that wait.
    grid_launch_dependents();
    // C and the norms come from the kernel before.  When the caller vouches that X was
    // complete before that kernel started, the producer streams the first X tiles while
    // it still runs and everybody else waits for it only where C or the norms are read.
    if (!x_is_ready) grid_dependency_wait();
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = s_tmem_base;
    volatile int* abort_flag = &s_abort;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (ptx::elect_one()) {
            ptx::prefetch_tensormap(&tm_x);
            ptx::prefetch_tensormap(&tm_c);
            const uint64_t stream_policy = ptx::l2_policy_evict_first();   // X is read once; C stays in L2
            // pipeline step = (row super tile, pass = (group, chunk), 64-column step).  The cursor walks the steps with
            // additions only: what happens between a stage falling free and its copies being issued is on the critical
            // path of a pipeline that is bound by the bytes it keeps in flight
            struct Cursor {
                int64_t st;          // first row of the super tile
                int g, ch, ks, s;    // group, chunk, column step, ring stage
                uint32_t phase;      // parity of the stage's use
                int boxes[MT];
                uint32_t x_bytes;
            };
            auto set_tile = [&](Cursor& c) {
                c.x_bytes = 0;
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    const int64_t rows = min((int64_t)CU_TILE_M, r1 - (c.st + (int64_t)mt * CU_TILE_M));
                    c.boxes[mt] = rows > 0 ? (int)((rows + CU_BOX_ROWS - 1) / CU_BOX_ROWS) : 0;
                    c.x_bytes += (uint32_t)c.boxes[mt] * (CU_BOX_ROWS * 128u);
                }
            };
            auto advance = [&](Cursor& c) {
                if (++c.s == stages) { c.s = 0; c.phase ^= 1u; }
                if (++c.ks < ksteps) return;
                c.ks = 0;
                if (++c.ch == num_chunks) { c.ch = 0; ++c.g; }
                if (c.g < groups) return;
                c.g = 0;
                c.st += super_rows;
                set_tile(c);
            };
            auto issue = [&](const Cursor& c, bool with_x, bool with_c, bool arm) {
                uint8_t* stage = tiles + (size_t)c.s * stage_bytes;
                if (arm) ptx::mbar_arrive_expect_tx(&s_full[c.s], c.x_bytes + (uint32_t)n_chunk * 128u);
                if (with_x) {
                    // the tile comes back once per pass: only its last visit may push it out of L2 early
                    const bool last_pass = c.g + 1 == groups && c.ch + 1 == num_chunks;
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt)
                        for (int q = 0; q < c.boxes[mt]; ++q) {
                            uint8_t* dst = stage + mt * CU_X_TILE_BYTES + q * (CU_BOX_ROWS * 128);
                            const int32_t y = (int32_t)(c.st + mt * CU_TILE_M + q * CU_BOX_ROWS);
                            if (last_pass) ptx::tma_load_2d_hint(dst, &tm_x, c.ks * CU_BLOCK_K, y, &s_full[c.s], stream_policy);
                            else           ptx::tma_load_2d(dst, &tm_x, c.ks * CU_BLOCK_K, y, &s_full[c.s]);
                        }
                }
                if (with_c)
                    ptx::tma_load_2d(stage + MT * CU_X_TILE_BYTES, &tm_c, c.ks * CU_BLOCK_K, c.g * k + c.ch * n_chunk, &s_full[c.s]);
            };
            const uint32_t total = (uint32_t)((r1 - r0 + super_rows - 1) / super_rows) * (uint32_t)(passes * ksteps);
            Cursor cur;
            cur.st = r0; cur.g = 0; cur.ch = 0; cur.ks = 0; cur.s = 0; cur.phase = 0;
            set_tile(cur);
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
                // let the copies already issued land before the CTA leaves
                const uint32_t back = it < (uint32_t)stages ? it : (uint32_t)stages;
                int never = 0;
                volatile int* no_abort = &never;
                for (uint32_t d = 1; d <= back; ++d) {
                    const uint32_t jt = it - d;
                    ptx::mbar_wait(&s_full[jt % stages], (jt / stages) & 1u, no_abort);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (ptx::elect_one()) {
            const uint32_t idesc = ptx::umma_idesc_bf16(CU_TILE_M, (uint32_t)n_chunk);
            uint32_t unit = 0, sph = 0;
            int s = 0;               // ring stage and the parity of its use, advanced without divisions
            bool ok = true;
            for (int64_t st = r0; st < r1 && ok; st += super_rows) {
                for (int pass = 0; pass < passes && ok; ++pass, ++unit) {
                    const uint32_t buf = unit % (uint32_t)tmem_bufs, uph = (unit / (uint32_t)tmem_bufs) & 1u;
                    if (!ptx::mbar_wait(&s_tempty[buf], uph ^ 1u, abort_flag)) { ok = false; break; }
                    ptx::tc_fence_after_sync();
                    const uint32_t d_base = tmem_base + buf * (uint32_t)(MT * n_chunk);
                    for (int ks = 0; ks < ksteps; ++ks) {
                        if (!ptx::mbar_wait(&s_full[s], sph, abort_flag)) { ok = false; break; }
                        ptx::tc_fence_after_sync();
                        const uint32_t stage_addr = ptx::smem_u32(tiles + (size_t)s * stage_bytes);
                        const uint64_t desc_b = ptx::umma_desc_k_sw128(stage_addr + MT * CU_X_TILE_BYTES);
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt) {
                            if (st + (int64_t)mt * CU_TILE_M >= r1) continue;
                            const uint64_t desc_a = ptx::umma_desc_k_sw128(stage_addr + mt * CU_X_TILE_BYTES);
#pragma unroll
                            for (int kk = 0; kk < CU_BLOCK_K / 16; ++kk)   // +32 bytes along K = +2 in the address field
                                ptx::umma_bf16(d_base + (uint32_t)(mt * n_chunk), desc_a + 2 * kk, desc_b + 2 * kk, idesc,
                                               (ks | kk) != 0);
                        }
                        ptx::umma_commit(&s_empty[s]);   // frees the stage once these MMAs have read it
                        if (++s == stages) { s = 0; sph ^= 1u; }
                    }
                    if (ok) ptx::umma_commit(&s_tfull[buf]);
                }
            }
            if (!ok) raise_status(DEV_TIMEOUT);
        }
    } else if (EPS && warp >= 2 + 4 * MT) {
        // ---------------- squared row norms: one row of the super tile per thread ----------------
        const int nt = threadIdx.x - CU_THREADS(MT);
        const int my_mt = nt / CU_TILE_M, row_in_tile = nt % CU_TILE_M;
        const int ksteps_all = passes * ksteps;
        uint32_t it = 0, sup = 0;
        bool ok = true;
        for (int64_t st = r0; st < r1 && ok; st += super_rows, ++sup) {
            float nrm[4] = {0.f, 0.f, 0.f, 0.f};     // four chains, added at the end in a fixed order
            const bool live = st + (int64_t)my_mt * CU_TILE_M < r1;
            for (int q = 0; q < ksteps_all; ++q, ++it) {
                const int s = it % stages;
                ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_full[s], (it / stages) & 1u, abort_flag));   // warp-uniform
                if (!ok) break;
                if (q < ksteps && live) {     // the first pass sees every column of X once
                    const uint8_t* rowp = tiles + (size_t)s * stage_bytes + my_mt * CU_X_TILE_BYTES + row_in_tile * 128;
                    uint4 w[8];
#pragma unroll
                    for (int c = 0; c < 8; ++c)     // chunk c sits at position c ^ (row & 7): conflict-free across the lanes
                        w[c] = *reinterpret_cast<const uint4*>(rowp + ((c ^ (row_in_tile & 7)) << 4));
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const uint32_t ws[4] = {w[c].x, w[c].y, w[c].z, w[c].w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float lo = bf16_lo(ws[e]), hi = bf16_hi(ws[e]);
                            nrm[e] = fmaf(lo, lo, nrm[e]);
                            nrm[e] = fmaf(hi, hi, nrm[e]);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&s_empty[s]);     // ordered after this warp's reads of the stage
            }
            if (!ok) break;
            const uint32_t nb = sup & 1u;
            ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_nempty[nb], ((sup >> 1) & 1u) ^ 1u, abort_flag));
            if (!ok) break;
            s_norm[nb][my_mt * CU_TILE_M + row_in_tile] = (nrm[0] + nrm[1]) + (nrm[2] + nrm[3]);
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&s_nfull[nb]);
        }
        if (!ok && lane == 0) raise_status(DEV_TIMEOUT);
    } else {
        // ---------------- epilogue: one row of one tile per thread ----------------
        const int quad = warp & 3;                       // TMEM lanes [32*quad, 32*quad+32)
        const int mt = (warp - 2) >> 2;                  // my row tile of the super tile
        const uint32_t lane_base = ((uint32_t)(quad * 32)) << 16;
        for (int j = threadIdx.x - 64; j < groups * k; j += 128 * MT) s_hist[j] = 0;
        if (x_is_ready) grid_dependency_wait();
        for (int j = threadIdx.x - 64; j < groups * kpad; j += 128 * MT) {
            const int g = j / kpad, jj = j % kpad;
            s_inv[j] = jj < k ? c_invnorm[(size_t)g * 2 * k + jj] : 0.f;
        }
        for (int j = threadIdx.x - 64; j < groups * k; j += 128 * MT) s_inv2[j] = c_invnorm[(size_t)(j / k) * 2 * k + k + j % k];
        ptx::named_barrier(1, 128 * MT);                 // the epilogue warps share the norms
        uint32_t unit = 0, sup = 0;
        bool ok = true;
        for (int64_t st = r0; st < r1 && ok; st += super_rows, ++sup) {
            const bool live = st + (int64_t)mt * CU_TILE_M < r1;
            const int64_t row = st + (int64_t)mt * CU_TILE_M + quad * 32 + lane;
            for (int g = 0; g < groups && ok; ++g) {
                float best = -1.f, s_best = 0.f;
                int j_best = 0;
                for (int ch = 0; ch < num_chunks && ok; ++ch, ++unit) {
                    const uint32_t buf = unit % (uint32_t)tmem_bufs, uph = (unit / (uint32_t)tmem_bufs) & 1u;
                    ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_tfull[buf], uph, abort_flag));   // warp-uniform
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    if (live) {
                        // two register buffers: the TMEM load of the next 16 columns is in flight
                        // while the current 16 go through the tournament
                        const uint32_t t_base = tmem_base + buf * (uint32_t)(MT * n_chunk) + lane_base + (uint32_t)(mt * n_chunk);
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
                    if (lane == 0) ptx::mbar_arrive(&s_tempty[buf]);
                }
                if (ok && EPS) ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_nfull[sup & 1u], (sup >> 1) & 1u, abort_flag));
                if (!ok) break;
                int ndrop = 0;
                if (row < r1) {
                    float a = s_best * s_inv2[g * k + j_best];
                    if (EPS) {     // Eq. 2: ||X_i - alpha C_f||^2 = ||X_i||^2 - S^2/||C_f||^2 against eps^2 ||X_i||^2
                        const float nx = s_norm[sup & 1u][mt * CU_TILE_M + quad * 32 + lane];
                        const float dist2 = nx - s_best * a;
                        if (dist2 > (eps2 + slack) * nx) { a = 0.f; ++ndrop; }
                    }
                    store_index(out.f, out.f_type, (int64_t)g * out.out_stride + row, j_best);
                    out.alpha[(int64_t)g * out.out_stride + row] = a;
                    if (a != 0.f) atomicAdd(&s_hist[g * k + j_best], 1);     // a row with alpha = 0 takes no part in the backward pass
                }
                if (EPS) {
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(&s_nempty[sup & 1u]);
#pragma unroll
                    for (int off = 16; off > 0; off >>= 1) ndrop += __shfl_xor_sync(0xffffffffu, ndrop, off);
                    if (lane == 0 && ndrop) atomicAdd(dropped, ndrop);
                }
            }
        }
        if (!ok && lane == 0) raise_status(DEV_TIMEOUT);
        // this CTA's histograms of f, one row of the per-block table per group
        ptx::named_barrier(1, 128 * MT);
        if (out.hist) {
            for (int j = threadIdx.x - 64; j < groups * k; j += 128 * MT) {
                const int g = j / k, jj = j % k;
                out.hist[(int64_t)g * out.hist_stride + (int64_t)blockIdx.x * k + jj] = s_hist[j];
            }
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, (uint32_t)tmem_cols);
    }
}

template <int MT, bool EPS>
inline size_t compress_umma_static_smem() {
    cudaFuncAttributes fa;
    if (cudaFuncGetAttributes(&fa, compress_umma_kernel<MT, EPS>) != cudaSuccess) return 4096;
    return fa.sharedSizeBytes;
}

// The plan for these sizes, with the kernel's own static shared memory taken into account.
inline CompressUmmaPlan compress_umma_plan_for(int64_t b, int64_t k, int groups, int sms, bool with_eps) {
    static size_t st_plain = 0, st_eps = 0;     // the same on every device
    if (!st_plain) st_plain = compress_umma_static_smem<2, false>();
    if (!st_eps) st_eps = compress_umma_static_smem<2, true>();
    return compress_umma_plan(b, k, groups, sms, with_eps ? st_eps : st_plain);
}

// Whether the tensor-core kernel serves these sizes (else the CUDA-core kernel does).
inline bool compress_umma_usable(int64_t b, int64_t n, int64_t k, int groups, int sms, bool with_eps) {
    return compress_umma_supported(b, n, k) && (int64_t)groups * k <= (1 << 20) &&
           compress_umma_plan_for(b, k, groups, sms, with_eps).stages >= 2;
}

inline pamm_status launch_compress_umma(const void* X, int64_t ldx, int64_t b, int64_t n, const void* C, int64_t ldc,
                                        int64_t k, int groups, const float* c_invnorm, const CompressOut& out, int sms,
                                        bool x_is_ready, cudaStream_t st, bool with_eps = false, float eps = 0.f,
                                        int32_t* dropped = nullptr) {
    const CompressUmmaPlan p = compress_umma_plan_for(b, k, groups, sms, with_eps);
    if (p.stages < 2) return PAMM_ERR_UNSUPPORTED;
    CUtensorMap tm_x, tm_c;
    if (!make_tmap_bf16_sw128(&tm_x, X, (uint64_t)b, (uint64_t)n, (uint64_t)ldx, CU_BOX_ROWS) ||
        !make_tmap_bf16_sw128(&tm_c, C, (uint64_t)groups * (uint64_t)k, (uint64_t)n, (uint64_t)ldc, (uint32_t)p.n_chunk))
        return tensor_map_failed();
    auto kern = with_eps ? compress_umma_kernel<2, true> : compress_umma_kernel<2, false>;
    if (!ensure_dynamic_smem((const void*)kern, p.smem_bytes)) return PAMM_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.grid);
    cfg.blockDim = dim3(with_eps ? CU_THREADS_EPS(p.mt) : CU_THREADS(p.mt));
    cfg.dynamicSmemBytes = p.smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // set up while the select kernel runs
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kern, tm_x, tm_c, b, (int)n, (int)k, groups, p.n_chunk, p.num_chunks, p.stages, p.stage_bytes,
                       p.tmem_cols, p.tmem_bufs, p.rows_per_cta, x_is_ready ? 1 : 0, c_invnorm, out, eps * eps,
                       neighbourhood_slack(n), dropped);
    return launch_result("compress_umma_kernel launch");
}

}  // namespace pamm
