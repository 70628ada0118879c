// Step 3: B~[j,:] = sum_{i: f_i = j} alpha_i * dY[i,:]  (Algorithm 1 ApproxMM,
// "B' <- alpha (.) B" and "index_add"), as a deterministic segmented reduction.
//
//   hist    : per block of SORT_BLK rows, a histogram of f            (integers)
//   scan    : exclusive scans -> segment starts, per-block offsets, chunk list
//   scatter : stable counting sort of row ids by f  -> perm
//   main    : one CTA per chunk of <= CH sorted rows (all of one segment); each
//             thread owns 16 bytes of the dY row (coalesced 128-bit loads), sums
//             alpha_i * dY_i over the chunk's rows in ascending row order in
//             fp32 registers, and writes one partial row
//   reduce  : B~[j] = sum of segment j's partial rows, ascending chunk order
//
// dY is read exactly once; the extra traffic is the partial rows
// (<= (b/CH + k) * m * 4 bytes written and read back).  No floating-point
// atomics anywhere, so results are bit-reproducible.
#pragma once
#include "pamm_common.cuh"

namespace pamm {

constexpr int SORT_BLK = 256;          // rows per histogram / scatter block
constexpr int CH = 128;                // rows per chunk of the main pass
constexpr int64_t CT_MAX_K = 49152;    // k * 4 bytes of dynamic shared memory in hist
constexpr int CT_MAX_THREADS = 768;
constexpr int CT_UNROLL = 4;

struct ContractWs {
    int32_t* hist;        // NB x k   (counts, then exclusive per-block offsets)
    int32_t* seg_start;   // k + 1
    int32_t* chunk_base;  // k + 1
    int32_t* chunk_seg;   // max_chunks
    int32_t* perm;        // b
    float* partials;      // max_chunks x m_pad
    float* btilde;        // k x m_pad (used when the caller passes no B~)
    int64_t nb, max_chunks, m_pad;
    size_t bytes;
};

inline ContractWs contract_ws_layout(void* base, int64_t b, int64_t m, int64_t k) {
    ContractWs w;
    w.nb = (b + SORT_BLK - 1) / SORT_BLK;
    w.max_chunks = (b + CH - 1) / CH + k;
    w.m_pad = round_up(m, 4);
    char* p = (char*)base;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = (size_t)round_up((int64_t)(off + bytes), 256); return p ? p + o : (char*)0; };
    w.hist = (int32_t*)take((size_t)w.nb * k * 4);
    w.seg_start = (int32_t*)take((size_t)(k + 1) * 4);
    w.chunk_base = (int32_t*)take((size_t)(k + 1) * 4);
    w.chunk_seg = (int32_t*)take((size_t)w.max_chunks * 4);
    w.perm = (int32_t*)take((size_t)b * 4);
    w.partials = (float*)take((size_t)w.max_chunks * w.m_pad * 4);
    w.btilde = (float*)take((size_t)k * w.m_pad * 4);
    w.bytes = off;
    return w;
}

__global__ void __launch_bounds__(SORT_BLK)
contract_hist_kernel(const int32_t* __restrict__ f, int64_t b, int k, int32_t* __restrict__ hist) {
    extern __shared__ int32_t s_hist[];
    for (int j = threadIdx.x; j < k; j += SORT_BLK) s_hist[j] = 0;
    __syncthreads();
    const int64_t i = (int64_t)blockIdx.x * SORT_BLK + threadIdx.x;
    if (i < b) {
        const int32_t j = f[i];
        if (j >= 0 && j < k) atomicAdd(&s_hist[j], 1);
        else raise_status(DEV_BAD_INDEX);
    }
    __syncthreads();
    int32_t* out = hist + (int64_t)blockIdx.x * k;
    for (int j = threadIdx.x; j < k; j += SORT_BLK) out[j] = s_hist[j];
}

constexpr int SCAN_THREADS = 1024;

// Single CTA.  Turns the per-block counts into exclusive per-block offsets,
// scans segment sizes into seg_start and chunk counts into chunk_base, and
// lists the owning segment of every chunk.
__global__ void __launch_bounds__(SCAN_THREADS)
contract_scan_kernel(int32_t* __restrict__ hist, int nb, int k, int32_t* __restrict__ seg_start,
                     int32_t* __restrict__ chunk_base, int32_t* __restrict__ chunk_seg) {
    __shared__ int32_t s_warp_a[32], s_warp_b[32];
    __shared__ int32_t s_carry_a, s_carry_b;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) { s_carry_a = 0; s_carry_b = 0; }
    __syncthreads();
    for (int j0 = 0; j0 < k; j0 += SCAN_THREADS) {
        const int j = j0 + tid;
        int32_t cnt = 0;
        if (j < k) {
            int32_t run = 0;
            for (int blk = 0; blk < nb; ++blk) {
                int32_t c = hist[(int64_t)blk * k + j];
                hist[(int64_t)blk * k + j] = run;
                run += c;
            }
            cnt = run;
        }
        const int32_t nch = (cnt + CH - 1) / CH;
        // inclusive scan of (cnt, nch) across the CTA
        int32_t a = cnt, c = nch;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            int32_t ta = __shfl_up_sync(0xffffffffu, a, off), tc = __shfl_up_sync(0xffffffffu, c, off);
            if (lane >= off) { a += ta; c += tc; }
        }
        if (lane == 31) { s_warp_a[warp] = a; s_warp_b[warp] = c; }
        __syncthreads();
        if (warp == 0) {
            int32_t wa = s_warp_a[lane], wc = s_warp_b[lane];
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                int32_t ta = __shfl_up_sync(0xffffffffu, wa, off), tc = __shfl_up_sync(0xffffffffu, wc, off);
                if (lane >= off) { wa += ta; wc += tc; }
            }
            s_warp_a[lane] = wa;
            s_warp_b[lane] = wc;
        }
        __syncthreads();
        const int32_t base_a = s_carry_a + (warp ? s_warp_a[warp - 1] : 0);
        const int32_t base_b = s_carry_b + (warp ? s_warp_b[warp - 1] : 0);
        const int32_t excl_a = base_a + a - cnt, excl_b = base_b + c - nch;
        if (j < k) {
            seg_start[j] = excl_a;
            chunk_base[j] = excl_b;
            for (int32_t w = 0; w < nch; ++w) chunk_seg[excl_b + w] = j;
        }
        __syncthreads();
        if (tid == SCAN_THREADS - 1) { s_carry_a = base_a + a; s_carry_b = base_b + c; }
        __syncthreads();
    }
    if (tid == 0) { seg_start[k] = s_carry_a; chunk_base[k] = s_carry_b; }
}

__global__ void __launch_bounds__(SORT_BLK)
contract_scatter_kernel(const int32_t* __restrict__ f, int64_t b, int k, const int32_t* __restrict__ hist,
                        const int32_t* __restrict__ seg_start, int32_t* __restrict__ perm) {
    __shared__ int32_t s_f[SORT_BLK];
    const int tid = threadIdx.x;
    const int64_t i = (int64_t)blockIdx.x * SORT_BLK + tid;
    int32_t j = -1;
    if (i < b) {
        j = f[i];
        if (j < 0 || j >= k) j = -1;
    }
    s_f[tid] = j;
    __syncthreads();
    if (j < 0) return;
    int rank = 0;
    for (int t = 0; t < tid; ++t) rank += (s_f[t] == j);
    perm[seg_start[j] + hist[(int64_t)blockIdx.x * k + j] + rank] = (int32_t)i;
}

template <typename T>
__global__ void __launch_bounds__(CT_MAX_THREADS)
contract_main_kernel(const float* __restrict__ alpha, const T* __restrict__ dY, int64_t ldy, int64_t m,
                     int k, const int32_t* __restrict__ seg_start, const int32_t* __restrict__ chunk_base,
                     const int32_t* __restrict__ chunk_seg, const int32_t* __restrict__ perm,
                     float* __restrict__ partials, int64_t m_pad) {
    constexpr int V = Vec16<T>::N;
    __shared__ int32_t s_row[CH];
    __shared__ float s_alpha[CH];
    const int w = blockIdx.x;
    if (w >= chunk_base[k]) return;
    const int j = chunk_seg[w];
    const int r0 = seg_start[j] + (w - chunk_base[j]) * CH;
    const int cnt = min(CH, seg_start[j + 1] - r0);
    for (int t = threadIdx.x; t < cnt; t += blockDim.x) {
        const int32_t i = perm[r0 + t];
        s_row[t] = i;
        s_alpha[t] = alpha[i];
    }
    __syncthreads();
    const int64_t col = ((int64_t)blockIdx.y * blockDim.x + threadIdx.x) * V;
    if (col >= m) return;
    float acc[V];
#pragma unroll
    for (int e = 0; e < V; ++e) acc[e] = 0.f;
    int t = 0;
    for (; t + CT_UNROLL <= cnt; t += CT_UNROLL) {
        float x[CT_UNROLL][V];
#pragma unroll
        for (int u = 0; u < CT_UNROLL; ++u) load_vec<T>(dY + (int64_t)s_row[t + u] * ldy, col, m, x[u]);
#pragma unroll
        for (int u = 0; u < CT_UNROLL; ++u) {
            const float a = s_alpha[t + u];
#pragma unroll
            for (int e = 0; e < V; ++e) acc[e] = fmaf(a, x[u][e], acc[e]);
        }
    }
    for (; t < cnt; ++t) {
        float x[V];
        load_vec<T>(dY + (int64_t)s_row[t] * ldy, col, m, x);
        const float a = s_alpha[t];
#pragma unroll
        for (int e = 0; e < V; ++e) acc[e] = fmaf(a, x[e], acc[e]);
    }
    float* out = partials + (int64_t)w * m_pad + col;   // m_pad is a multiple of 4, col of V
#pragma unroll
    for (int e = 0; e < V; e += 4)
        if (col + e < m_pad) *reinterpret_cast<float4*>(out + e) = make_float4(acc[e], acc[e + 1], acc[e + 2], acc[e + 3]);
}

constexpr int RED_THREADS = 256;

__global__ void __launch_bounds__(RED_THREADS)
contract_reduce_kernel(const float* __restrict__ partials, int64_t m_pad, int64_t m, int k,
                       const int32_t* __restrict__ chunk_base, float* __restrict__ Bt, int64_t ldb) {
    const int64_t mv = m_pad / 4;
    const int64_t idx = (int64_t)blockIdx.x * RED_THREADS + threadIdx.x;
    if (idx >= (int64_t)k * mv) return;
    const int j = (int)(idx / mv);
    const int64_t col = (idx % mv) * 4;
    const int w0 = chunk_base[j], w1 = chunk_base[j + 1];
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int w = w0; w < w1; ++w) {
        const float4 p = *reinterpret_cast<const float4*>(partials + (int64_t)w * m_pad + col);
        s.x += p.x; s.y += p.y; s.z += p.z; s.w += p.w;
    }
    float* out = Bt + (int64_t)j * ldb + col;
    if (col + 4 <= m) {
        *reinterpret_cast<float4*>(out) = s;
    } else {
        const float v[4] = {s.x, s.y, s.z, s.w};
        for (int e = 0; e < 4 && col + e < m; ++e) out[e] = v[e];
    }
}

}  // namespace pamm
