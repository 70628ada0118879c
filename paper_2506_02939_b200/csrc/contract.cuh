// Step 3: B~[j,:] = sum_{i: f_i = j} alpha_i * dY[i,:]  (Algorithm 1 ApproxMM,
// the alpha-scaling of B and the index_add), as a deterministic segmented reduction.
//
//   hist    : per block of rows, a histogram of f (integers).  The blocks are the row
//             ranges of the compress pass, whose epilogue already counted f: when the
//             caller hands those counts over, this launch is skipped
//   scan    : exclusive scans -> segment starts and per-block offsets
//   scatter : stable counting sort of row ids by f  -> perm
//   main    : the sorted rows are cut into equal contiguous ranges, one per CTA
//             (a single balanced wave).  Each thread owns 16 bytes of the dY row
//             (coalesced 128-bit loads) and sums alpha_i * dY_i over its range in
//             ascending sorted order in fp32 registers, flushing at every segment
//             boundary: a segment that lies wholly inside the range goes straight
//             to B~, a segment cut by a range boundary goes to a partial row
//   reduce  : B~[j] for the cut segments = sum of their partial rows, ascending
//
// dY is read exactly once; the extra traffic is at most (#CTAs + k) partial
// rows.  No floating-point atomics anywhere, so results are bit-reproducible.
#pragma once
#include "pamm_common.cuh"

namespace pamm {

constexpr int SORT_BLK = 1024;         // threads of a histogram / scatter block: it walks its rows 1024 at a time
constexpr int CT_TILE = 256;           // rows of (perm, alpha) staged in shared memory at a time
constexpr int64_t CT_MAX_K = 49152;    // k * 4 bytes of dynamic shared memory in hist / scatter
constexpr int CT_MAX_THREADS = 768;
constexpr int CT_UNROLL = 8;           // rows in flight per thread
constexpr int CT_MAX_CTAS = 148 * 8;   // upper bound on row ranges (sizes the partial buffer)

struct ContractWs {
    int32_t* hist;        // NB x k   (counts; the three-launch sort turns them into exclusive per-block offsets)
    int32_t* seg_start;   // k + 1
    int32_t* perm;        // b
    float* partials;      // (CT_MAX_CTAS + k) x m_pad
    float* btilde;        // k x m_pad (used when the caller passes no B~)
    uint16_t* planes;     // optional, behind everything else: B~ split into bf16 hi and lo, 2 x k x plane_ld
    int64_t nb, rows_per_block, m_pad, plane_ld;
    size_t bytes;         // without the planes
    size_t bytes_with_planes;
};

// rows_per_block: the row partition of the histograms (compress_rows_per_cta).
inline ContractWs contract_ws_layout(void* base, int64_t b, int64_t m, int64_t k, int64_t rows_per_block) {
    ContractWs w;
    w.rows_per_block = rows_per_block;
    w.nb = (b + rows_per_block - 1) / rows_per_block;
    w.m_pad = round_up(m, 4);
    char* p = (char*)base;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = (size_t)round_up((int64_t)(off + bytes), 256); return p ? p + o : (char*)0; };
    w.hist = (int32_t*)take((size_t)w.nb * k * 4);
    w.seg_start = (int32_t*)take((size_t)(k + 1) * 4);
    w.perm = (int32_t*)take((size_t)b * 4);
    w.partials = (float*)take((size_t)(CT_MAX_CTAS + k) * w.m_pad * 4);
    w.btilde = (float*)take((size_t)k * w.m_pad * 4);
    w.bytes = off;
    w.plane_ld = round_up(m, 8);
    w.planes = (uint16_t*)take((size_t)2 * k * w.plane_ld * 2);
    w.bytes_with_planes = off;
    return w;
}

// The key a row is sorted by: its generator f_i, or -1 for a row that takes no part -- one whose
// alpha_i is zero (dropped by the neighbourhood condition, an all-zero row, a row orthogonal to its
// generator: it adds nothing to B~ and is not read at all) or whose f_i is out of range (reported).
// Every producer of the per-block counts uses the same rule.
__device__ __forceinline__ int32_t sort_key(const void* f, int f_type, const float* alpha, int64_t i, int k) {
    const int32_t j = load_index(f, f_type, i);
    const float a = alpha[i];            // both loads travel together
    if (j < 0 || j >= k) {
        raise_status(DEV_BAD_INDEX);
        return -1;
    }
    return a != 0.f ? j : -1;
}

// The rows of the sorted order are cut into `ranges` equal contiguous ranges (one CTA of the main
// pass each); how many rows there are is known on the device only (rows with alpha = 0 are left out).
__device__ __forceinline__ int range_rows(int32_t total, int ranges) { return max(1, (total + ranges - 1) / ranges); }

__global__ void __launch_bounds__(SORT_BLK)
contract_hist_kernel(const void* __restrict__ f, int f_type, const float* __restrict__ alpha, int64_t b, int k,
                     int rows_per_block, int32_t* __restrict__ hist) {
    extern __shared__ int32_t s_hist[];
    for (int j = threadIdx.x; j < k; j += SORT_BLK) s_hist[j] = 0;
    grid_dependency_wait();     // f may come from the kernel before
    grid_launch_dependents();
    __syncthreads();
    const int64_t i0 = (int64_t)blockIdx.x * rows_per_block;
    const int64_t i1 = min(b, i0 + (int64_t)rows_per_block);
    for (int64_t i = i0 + threadIdx.x; i < i1; i += SORT_BLK) {
        const int32_t j = sort_key(f, f_type, alpha, i, k);
        if (j >= 0) atomicAdd(&s_hist[j], 1);
    }
    __syncthreads();
    int32_t* out = hist + (int64_t)blockIdx.x * k;
    for (int j = threadIdx.x; j < k; j += SORT_BLK) out[j] = s_hist[j];
}

constexpr int SCAN_THREADS = 1024;

// Single CTA.  Turns the per-block counts into exclusive per-block offsets and
// scans the segment sizes into seg_start[0..k].
__global__ void __launch_bounds__(SCAN_THREADS)
contract_scan_kernel(int32_t* __restrict__ hist, int nb, int k, int32_t* __restrict__ seg_start) {
    __shared__ int32_t s_warp[32];
    __shared__ int32_t s_carry;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    grid_dependency_wait();
    grid_launch_dependents();
    if (tid == 0) s_carry = 0;
    __syncthreads();
    for (int j0 = 0; j0 < k; j0 += SCAN_THREADS) {
        const int j = j0 + tid;
        int32_t cnt = 0;
        if (j < k) {
            int32_t run = 0;
            for (int blk = 0; blk < nb; ++blk) {
                const int32_t c = hist[(int64_t)blk * k + j];
                hist[(int64_t)blk * k + j] = run;
                run += c;
            }
            cnt = run;
        }
        int32_t a = cnt;   // inclusive scan across the CTA
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int32_t t = __shfl_up_sync(0xffffffffu, a, off);
            if (lane >= off) a += t;
        }
        if (lane == 31) s_warp[warp] = a;
        __syncthreads();
        if (warp == 0) {
            int32_t wa = s_warp[lane];
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int32_t t = __shfl_up_sync(0xffffffffu, wa, off);
                if (lane >= off) wa += t;
            }
            s_warp[lane] = wa;
        }
        __syncthreads();
        const int32_t base = s_carry + (warp ? s_warp[warp - 1] : 0);
        if (j < k) seg_start[j] = base + a - cnt;
        __syncthreads();
        if (tid == SCAN_THREADS - 1) s_carry = base + a;
        __syncthreads();
    }
    if (tid == 0) seg_start[k] = s_carry;
}

// Stable ranking of up to SORT_BLK rows of one block in ascending row order.  Inside a
// warp, match_any groups equal keys (rank = position inside the group, the lowest lane
// leads).  Across the warps of the block either
//   - a table of per-warp counts (s_tbl != nullptr: warps x k words of shared memory):
//     the leaders post their group sizes, one thread per key turns the column of its key
//     into running slot numbers (continuing s_next), and every row reads its slot; or
//   - warp by warp, each leader reserving its group's slots in s_next in turn
//     (no extra shared memory, as many block-wide barriers as there are warps).
// A slot outside [0, b) can only come from counts that do not belong to this f (a caller's
// mistake): it is skipped and reported.
__device__ __forceinline__ void scatter_chunk(int32_t key, int64_t i, int nrows, int k, int32_t* s_next, int32_t* s_tbl,
                                              int32_t* __restrict__ perm, int64_t b) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned peers = __match_any_sync(0xffffffffu, key);
    const int rank = __popc(peers & ((1u << lane) - 1u));
    const int leader = __ffs(peers) - 1;
    const int count = __popc(peers);
    const int warps = (nrows + 31) >> 5;
    if (s_tbl) {
        for (int t = threadIdx.x; t < warps * k; t += SORT_BLK) s_tbl[t] = 0;
        __syncthreads();
        if (lane == leader && key >= 0) s_tbl[warp * k + key] = count;
        __syncthreads();
        for (int j = threadIdx.x; j < k; j += SORT_BLK) {
            int32_t run = s_next[j];
            for (int w = 0; w < warps; ++w) {
                const int32_t c = s_tbl[w * k + j];
                s_tbl[w * k + j] = run;
                run += c;
            }
            s_next[j] = run;
        }
        __syncthreads();
        if (key >= 0) {
            const int64_t pos = (int64_t)s_tbl[warp * k + key] + rank;
            if (pos >= 0 && pos < b) perm[pos] = (int32_t)i;
            else raise_status(DEV_BAD_INDEX);
        }
        __syncthreads();
        return;
    }
    for (int w = 0; w < warps; ++w) {
        __syncthreads();
        if (warp == w) {
            int32_t base = 0;
            if (lane == leader && key >= 0) {
                base = s_next[key];
                s_next[key] = base + count;
            }
            base = __shfl_sync(0xffffffffu, base, leader);
            if (key >= 0) {
                const int64_t pos = (int64_t)base + rank;
                if (pos >= 0 && pos < b) perm[pos] = (int32_t)i;
                else raise_status(DEV_BAD_INDEX);
            }
        }
    }
    __syncthreads();
}

// Warps of a block's largest chunk, and whether their count table fits beside s_next.
inline int scatter_table_warps(int64_t rows_per_block, int64_t k) {
    const int warps = (int)((std::min<int64_t>(rows_per_block, SORT_BLK) + 31) / 32);
    return (int64_t)(1 + warps) * k * 4 <= 96 * 1024 ? warps : 0;
}

// Stable scatter of one block's rows, given the scanned tables.
__global__ void __launch_bounds__(SORT_BLK)
contract_scatter_kernel(const void* __restrict__ f, int f_type, const float* __restrict__ alpha, int64_t b, int k,
                        int rows_per_block, int tbl_warps, const int32_t* __restrict__ hist,
                        const int32_t* __restrict__ seg_start, int32_t* __restrict__ perm) {
    extern __shared__ int32_t s_next[];    // next free slot of every segment for this block, then the count table
    int32_t* s_tbl = tbl_warps ? s_next + k : nullptr;
    const int tid = threadIdx.x;
    const int32_t* my_hist = hist + (int64_t)blockIdx.x * k;
    grid_dependency_wait();
    grid_launch_dependents();
    for (int j = tid; j < k; j += SORT_BLK) s_next[j] = seg_start[j] + my_hist[j];
    const int64_t i0 = (int64_t)blockIdx.x * rows_per_block;
    const int64_t i1 = min(b, i0 + (int64_t)rows_per_block);
    for (int64_t c0 = i0; c0 < i1; c0 += SORT_BLK) {
        const int64_t i = c0 + tid;
        int32_t key = -1;
        if (i < i1) key = sort_key(f, f_type, alpha, i, k);
        scatter_chunk(key, i, (int)min((int64_t)SORT_BLK, i1 - c0), k, s_next, s_tbl, perm, b);
    }
}

// Scan and scatter in one launch, for the common case of a small histogram
// matrix: every block derives what it needs from the raw per-block counts --
// the segment starts (an exclusive scan over j of the column totals) and its own
// offset inside every segment (the counts of the blocks before it) -- and then
// scatters its rows exactly as contract_scatter_kernel does.  Block 0 also
// publishes seg_start.  Costs nb * k reads per block instead of a serial
// single-CTA pass between two launches.  The column sums are spread over all
// threads: with W = the chunk's width rounded up to a power of two, the SORT_BLK
// / W thread groups each take every (SORT_BLK / W)-th histogram row.
__global__ void __launch_bounds__(SORT_BLK)
contract_scan_scatter_kernel(const void* __restrict__ f, int f_type, const float* __restrict__ alpha, int64_t b, int k,
                             int rows_per_block, int tbl_warps, const int32_t* __restrict__ hist, int nb,
                             int32_t* __restrict__ seg_start, int32_t* __restrict__ perm) {
    extern __shared__ int32_t s_next[];    // next free slot of every segment for this block, then the count table
    int32_t* s_tbl = tbl_warps ? s_next + k : nullptr;
    __shared__ int32_t s_part[2][SORT_BLK];   // per-thread partial (total, before) of the column sums
    __shared__ int32_t s_warp[32];
    __shared__ int32_t s_carry;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int me = blockIdx.x;
    grid_dependency_wait();     // f and the histograms come from kernels before
    grid_launch_dependents();
    const int64_t i0 = (int64_t)me * rows_per_block;
    const int64_t i1 = min(b, i0 + (int64_t)rows_per_block);
    // the keys of the first chunk travel while the column sums are formed
    const int32_t first_key = i0 + tid < i1 ? sort_key(f, f_type, alpha, i0 + tid, k) : -1;
    if (tid == 0) s_carry = 0;
    __syncthreads();
    for (int j0 = 0; j0 < k; j0 += SORT_BLK) {
        const int width = min(SORT_BLK, k - j0);
        int W = 32;
        while (W < width) W <<= 1;
        const int groups = SORT_BLK / W;
        const int grp = tid / W, jj = tid % W;
        int32_t total = 0, before = 0;
        if (jj < width) {
            const int32_t* col = hist + j0 + jj;
            int blk = grp;
            for (; blk + 7 * groups < nb; blk += 8 * groups) {   // eight independent loads in flight
                int32_t c[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) c[u] = __ldg(col + (int64_t)(blk + u * groups) * k);
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    total += c[u];
                    before += blk + u * groups < me ? c[u] : 0;
                }
            }
            for (; blk < nb; blk += groups) {
                const int32_t c = __ldg(col + (int64_t)blk * k);
                total += c;
                before += blk < me ? c : 0;
            }
        }
        s_part[0][tid] = total;
        s_part[1][tid] = before;
        __syncthreads();
        total = 0;
        before = 0;
        if (tid < width) {
            for (int g = 0; g < groups; ++g) {
                total += s_part[0][g * W + tid];
                before += s_part[1][g * W + tid];
            }
        }
        const int j = j0 + tid;
        int32_t a = total;   // inclusive scan across the CTA (threads beyond the chunk hold 0)
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int32_t t = __shfl_up_sync(0xffffffffu, a, off);
            if (lane >= off) a += t;
        }
        if (lane == 31) s_warp[warp] = a;
        __syncthreads();
        if (warp == 0) {
            int32_t wa = s_warp[lane];
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int32_t t = __shfl_up_sync(0xffffffffu, wa, off);
                if (lane >= off) wa += t;
            }
            s_warp[lane] = wa;
        }
        __syncthreads();
        const int32_t base = s_carry + (warp ? s_warp[warp - 1] : 0);
        if (tid < width) {
            const int32_t start = base + a - total;
            s_next[j] = start + before;
            if (me == 0) seg_start[j] = start;
        }
        __syncthreads();
        if (tid == SORT_BLK - 1) s_carry = base + a;
        __syncthreads();
    }
    if (me == 0 && tid == 0) seg_start[k] = s_carry;

    for (int64_t c0 = i0; c0 < i1; c0 += SORT_BLK) {
        const int64_t i = c0 + tid;
        int32_t key = -1;
        if (i < i1) key = c0 == i0 ? first_key : sort_key(f, f_type, alpha, i, k);
        scatter_chunk(key, i, (int)min((int64_t)SORT_BLK, i1 - c0), k, s_next, s_tbl, perm, b);
    }
}

// First index j in [0,k) with seg_start[j] <= r < seg_start[j+1].
__device__ __forceinline__ int segment_of(const int32_t* __restrict__ seg_start, int k, int32_t r) {
    int lo = 0, hi = k;   // invariant: seg_start[lo] <= r < seg_start[hi]
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (seg_start[mid] <= r) lo = mid; else hi = mid;
    }
    return lo;
}

// acc += a * (16 bytes of T held in raw)
template <typename T>
__device__ __forceinline__ void fma_raw(float (&acc)[Vec16<T>::N], float a, const uint4& raw);
template <>
__device__ __forceinline__ void fma_raw<float>(float (&acc)[4], float a, const uint4& raw) {
    acc[0] = fmaf(a, __uint_as_float(raw.x), acc[0]); acc[1] = fmaf(a, __uint_as_float(raw.y), acc[1]);
    acc[2] = fmaf(a, __uint_as_float(raw.z), acc[2]); acc[3] = fmaf(a, __uint_as_float(raw.w), acc[3]);
}
template <>
__device__ __forceinline__ void fma_raw<__nv_bfloat16>(float (&acc)[8], float a, const uint4& raw) {
    acc[0] = fmaf(a, bf16_lo(raw.x), acc[0]); acc[1] = fmaf(a, bf16_hi(raw.x), acc[1]);
    acc[2] = fmaf(a, bf16_lo(raw.y), acc[2]); acc[3] = fmaf(a, bf16_hi(raw.y), acc[3]);
    acc[4] = fmaf(a, bf16_lo(raw.z), acc[4]); acc[5] = fmaf(a, bf16_hi(raw.z), acc[5]);
    acc[6] = fmaf(a, bf16_lo(raw.w), acc[6]); acc[7] = fmaf(a, bf16_hi(raw.w), acc[7]);
}

template <typename T>
__global__ void __launch_bounds__(CT_MAX_THREADS)
contract_main_kernel(const float* __restrict__ alpha, const T* __restrict__ dY, int64_t ldy, int64_t b, int64_t m,
                     int k, const int32_t* __restrict__ seg_start, const int32_t* __restrict__ perm,
                     int ranges, float* __restrict__ partials, int64_t m_pad,
                     float* __restrict__ Bt, int64_t ldb) {
    constexpr int V = Vec16<T>::N;
    __shared__ int32_t s_row[CT_TILE];
    __shared__ float s_alpha[CT_TILE];
    const int c = blockIdx.x;
    grid_dependency_wait();
    grid_launch_dependents();
    const int32_t total = (int32_t)min((int64_t)max(seg_start[k], 0), b);
    const int rows_per_cta = range_rows(total, ranges);
    const int32_t r_begin = (int32_t)min((int64_t)c * rows_per_cta, (int64_t)total);
    const int32_t r_end = (int32_t)min((int64_t)r_begin + rows_per_cta, (int64_t)total);
    if (r_begin >= r_end) return;
    const int64_t col = ((int64_t)blockIdx.y * blockDim.x + threadIdx.x) * V;
    const bool active = col < m;
    const bool full_vec = col + V <= m;
    int j = segment_of(seg_start, k, r_begin);
    int32_t j_end = seg_start[j + 1];

    float acc[V];
#pragma unroll
    for (int e = 0; e < V; ++e) acc[e] = 0.f;

    auto flush = [&](int seg) {
        if (!active) return;
        const bool inside = seg_start[seg] >= r_begin && seg_start[seg + 1] <= r_end;
        if (inside) {
            float* out = Bt + (int64_t)seg * ldb + col;
#pragma unroll
            for (int e = 0; e < V; e += 4) {
                if (col + e + 4 <= m) {
                    *reinterpret_cast<float4*>(out + e) = make_float4(acc[e], acc[e + 1], acc[e + 2], acc[e + 3]);
                } else {
                    for (int t = 0; t < 4 && col + e + t < m; ++t) out[e + t] = acc[e + t];
                }
            }
        } else {
            float* out = partials + (int64_t)(c + seg) * m_pad + col;   // m_pad % 4 == 0, col % V == 0
#pragma unroll
            for (int e = 0; e < V; e += 4)
                if (col + e < m_pad) *reinterpret_cast<float4*>(out + e) = make_float4(acc[e], acc[e + 1], acc[e + 2], acc[e + 3]);
        }
    };

    for (int32_t t0 = r_begin; t0 < r_end; t0 += CT_TILE) {
        const int tcnt = min(CT_TILE, r_end - t0);
        __syncthreads();
        for (int t = threadIdx.x; t < tcnt; t += blockDim.x) {
            int32_t i = perm[t0 + t];
            const bool bad = (uint32_t)i >= (uint32_t)b;     // only if the sort was fed counts of another f
            if (bad) { raise_status(DEV_BAD_INDEX); i = 0; }
            s_row[t] = i;
            s_alpha[t] = bad ? 0.f : alpha[i];
        }
        __syncthreads();
        int pos = 0;
        while (pos < tcnt) {
            const int lim = min(tcnt, j_end - t0);
            if (active && full_vec) {
                int t = pos;
                for (; t + CT_UNROLL <= lim; t += CT_UNROLL) {
                    uint4 raw[CT_UNROLL];
#pragma unroll
                    for (int u = 0; u < CT_UNROLL; ++u)
                        raw[u] = __ldg(reinterpret_cast<const uint4*>(dY + (int64_t)s_row[t + u] * ldy + col));
#pragma unroll
                    for (int u = 0; u < CT_UNROLL; ++u) fma_raw<T>(acc, s_alpha[t + u], raw[u]);
                }
                for (; t < lim; ++t)
                    fma_raw<T>(acc, s_alpha[t], __ldg(reinterpret_cast<const uint4*>(dY + (int64_t)s_row[t] * ldy + col)));
            } else if (active) {   // ragged last vector of the row
                for (int t = pos; t < lim; ++t) {
                    float x[V];
                    load_vec<T>(dY + (int64_t)s_row[t] * ldy, col, m, x);
                    const float a = s_alpha[t];
#pragma unroll
                    for (int e = 0; e < V; ++e) acc[e] = fmaf(a, x[e], acc[e]);
                }
            }
            pos = lim;
            if (t0 + pos == j_end) {          // segment j is complete
                flush(j);
#pragma unroll
                for (int e = 0; e < V; ++e) acc[e] = 0.f;
                if (j_end >= r_end) { j = -1; break; }
                do { ++j; j_end = seg_start[j + 1]; } while (j_end <= t0 + pos && j + 1 < k);   // skip empty segments
            }
        }
        if (j < 0) break;
    }
    if (j >= 0) flush(j);   // the range ended inside segment j
}

constexpr int RED_THREADS = 256;

// Finishes B~: zero rows for empty segments, sums of partial rows for segments
// that were cut by a range boundary; rows written directly by main are left alone.
// With `planes` it also leaves every element of B~ split into two bf16 values,
// hi = rn(x) and lo = rn(x - hi), in two k x plane_ld planes (hi first): the operands
// of the product over many generators, which then come by TMA instead of being
// converted by every CTA that needs them.
__global__ void __launch_bounds__(RED_THREADS)
contract_reduce_kernel(const float* __restrict__ partials, int64_t m_pad, int64_t m, int k, int64_t b,
                       const int32_t* __restrict__ seg_start, int ranges,
                       float* __restrict__ Bt, int64_t ldb, uint16_t* __restrict__ planes, int64_t plane_ld) {
    // grid: x over groups of four columns, y over the generators (no divisions; a CTA's threads share the segment's bounds)
    const int64_t col = ((int64_t)blockIdx.x * RED_THREADS + threadIdx.x) * 4;
    grid_dependency_wait();
    grid_launch_dependents();
    if (col >= m_pad) return;
    for (int j = blockIdx.y; j < k; j += gridDim.y) {
        const int32_t s0 = (int32_t)min((int64_t)max(seg_start[j], 0), b), s1 = (int32_t)min((int64_t)max(seg_start[j + 1], 0), b);
        float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
        float* out = Bt + (int64_t)j * ldb + col;
        bool written = false;      // the main pass wrote this row itself
        if (s1 > s0) {
            const int rows_per_cta = range_rows((int32_t)min((int64_t)max(seg_start[k], 0), b), ranges);
            const int c_lo = s0 / rows_per_cta, c_hi = (s1 - 1) / rows_per_cta;
            if (c_lo == c_hi) {
                if (!planes) continue;
                written = true;
                if (col + 4 <= m) {
                    s = *reinterpret_cast<const float4*>(out);
                } else {
                    float v[4] = {0.f, 0.f, 0.f, 0.f};
                    for (int e = 0; e < 4 && col + e < m; ++e) v[e] = out[e];
                    s = make_float4(v[0], v[1], v[2], v[3]);
                }
            } else {
                for (int c = c_lo; c <= c_hi; ++c) {
                    const float4 p = *reinterpret_cast<const float4*>(partials + (int64_t)(c + j) * m_pad + col);
                    s.x += p.x; s.y += p.y; s.z += p.z; s.w += p.w;
                }
            }
        }
        if (!written) {
            if (col + 4 <= m) {
                *reinterpret_cast<float4*>(out) = s;
            } else {
                const float v[4] = {s.x, s.y, s.z, s.w};
                for (int e = 0; e < 4 && col + e < m; ++e) out[e] = v[e];
            }
        }
        if (planes) {
            const float x[4] = {s.x, s.y, s.z, s.w};
            float h[4], l[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const bool in = col + e < m;
                h[e] = in ? __bfloat162float(__float2bfloat16_rn(x[e])) : 0.f;
                l[e] = in ? x[e] - h[e] : 0.f;
            }
            auto pack2 = [](float a, float c) {
                __nv_bfloat162 t = __floats2bfloat162_rn(a, c);     // .x = first argument = low 16 bits
                return *reinterpret_cast<uint32_t*>(&t);
            };
            uint16_t* hi = planes + (int64_t)j * plane_ld + col;      // col % 4 == 0 and plane_ld % 8 == 0: 8-byte aligned
            uint16_t* lo = hi + (int64_t)k * plane_ld;
            if (col + 4 <= plane_ld) {
                *reinterpret_cast<uint2*>(hi) = make_uint2(pack2(h[0], h[1]), pack2(h[2], h[3]));
                *reinterpret_cast<uint2*>(lo) = make_uint2(pack2(l[0], l[1]), pack2(l[2], l[3]));
            }
        }
    }
}

}  // namespace pamm
