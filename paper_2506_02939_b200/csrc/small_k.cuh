// The whole path for a handful of generators (k <= 8) in three launches instead of seven.
//
// With so few generators the problem is small (the paper's ratio r = k / b puts b at a few
// thousand tokens) and the cost of a step is the number of launches, not bytes.  So:
//   compress_small   selects the generators AND compresses (Algorithm 1, Compress): every
//                    CTA recomputes the k indices, keeps the k generator rows in shared
//                    memory (read straight from X) and their norms, then scores its rows,
//                    one warp per row; CTA 0 also writes C, the indices and the norms
//   contract_small   B~ without sorting (Algorithm 1, ApproxMM: alpha-scaling and
//                    index_add): a thread owns 16 bytes of the dY row and k accumulator
//                    sets in registers, walks its CTA's rows in ascending order and adds
//                    alpha_i dY_i to the set f_i names; one partial B~ per row range
//   wgrad_small      adds the partial B~ in ascending range order (fixed order, no
//                    floating-point atomics) and multiplies by C^T (ApproxMM, the product)
// Results are bit-reproducible; the order of the fp32 sums differs from the large-k
// kernels', which is within the same rounding bounds.
#pragma once
#include "pamm_common.cuh"
#include "select.cuh"
#include "contract.cuh"
#include "weight_grad_simt.cuh"

namespace pamm {

constexpr int SK_MAX_K = 8;
constexpr int SK_THREADS = 256;
constexpr int SK_WARPS = SK_THREADS / 32;
constexpr int SK_MAX_C_BYTES = 96 * 1024;        // the generator rows a CTA keeps in shared memory
constexpr int SK_CT_THREADS = 384;               // contract: 16-byte column chunks per CTA
constexpr int SK_BATCH = 64;                     // rows whose (f, alpha) are staged together
constexpr int SK_ROWS_IN_FLIGHT = 8;             // 16-byte loads of dY a contract thread keeps in flight
constexpr int SK_WG_COLS = 128;                  // columns of B~ per product CTA

template <typename T>
inline bool small_k_compress_supported(int64_t n, int64_t k) {
    constexpr int V = Vec16<T>::N;
    return k <= SK_MAX_K && k * round_up(n, V) * (int64_t)sizeof(T) <= SK_MAX_C_BYTES;
}

template <typename T>
__global__ void __launch_bounds__(SK_THREADS)
compress_small_kernel(const T* __restrict__ X, int64_t ldx, int64_t b, int64_t n, int k, PermKey pk,
                      const int32_t* __restrict__ idx_in, int32_t* __restrict__ idx_out, T* __restrict__ C, int64_t ldc,
                      float* __restrict__ c_invnorm, void* __restrict__ f, int f_type, float* __restrict__ alpha,
                      int rows_per_cta) {
    constexpr int V = Vec16<T>::N;
    extern __shared__ uint4 s_c_raw[];                      // k generator rows of n_pad elements
    __shared__ int32_t s_val[SK_MAX_K], s_idx[SK_MAX_K];
    __shared__ float s_inv[SK_MAX_K], s_inv2[SK_MAX_K];
    T* sC = reinterpret_cast<T*>(s_c_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t n_pad = (n + V - 1) / V * V;

    // drawn indices need no memory: they are ready before the kernel in front has finished
    if (!idx_in && tid < k) s_val[tid] = (int32_t)perm_apply(pk, (uint32_t)tid);
    grid_dependency_wait();
    grid_launch_dependents();
    if (idx_in && tid < k) {
        int32_t v = idx_in[tid];
        bool bad = false;
        if (v < 0) { v = 0; bad = true; }
        if ((int64_t)v >= b) { v = (int32_t)(b - 1); bad = true; }
        for (int t = 0; t < k; ++t) bad = bad || (t != tid && idx_in[t] == idx_in[tid]);
        if (bad && blockIdx.x == 0) raise_status(DEV_BAD_INDEX);
        s_idx[tid] = v;                                    // the caller's order
    }
    __syncthreads();
    if (!idx_in && tid < k) {
        int smaller = 0;
        for (int t = 0; t < k; ++t) smaller += s_val[t] < s_val[tid];
        s_idx[smaller] = s_val[tid];                       // distinct by construction: rank = ascending position
    }
    __syncthreads();

    // the generator rows, straight from X, zero beyond column n
    const int64_t vec_per_row = n_pad / V;
    for (int64_t it = tid; it < (int64_t)k * vec_per_row; it += SK_THREADS) {
        const int j = (int)(it / vec_per_row);
        const int64_t col = (it % vec_per_row) * V;
        const T* src = X + (int64_t)s_idx[j] * ldx;
        float x[V];
        load_vec<T>(src, col, n, x);                       // zero beyond column n
        s_c_raw[it] = pack_vec<T>(x);
    }
    __syncthreads();

    // ||C_j||^2 by warp j, as an unevaluated fp32 pair with error-free additions (as the selection kernel does)
    if (warp < k) {
        const T* row = sC + (int64_t)warp * n_pad;
        float q_hi = 0.f, q_lo = 0.f;
        for (int64_t col = lane; col < n; col += 32) {
            const float x = load_scalar_generic(row + col);
            const float p = __fmul_rn(x, x);
            const float pe = fmaf(x, x, -p);
            q_lo += two_sum(q_hi, p) + pe;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float o_hi = __shfl_xor_sync(0xffffffffu, q_hi, off);
            const float o_lo = __shfl_xor_sync(0xffffffffu, q_lo, off);
            q_lo = (q_lo + o_lo) + two_sum(q_hi, o_hi);
        }
        if (lane == 0) {
            const double q = (double)q_hi + (double)q_lo;
            s_inv[warp] = q > 0.0 ? (float)(1.0 / sqrt(q)) : 0.f;
            s_inv2[warp] = q > 0.0 ? (float)(1.0 / q) : 0.f;
        }
    }
    __syncthreads();

    if (blockIdx.x == 0) {      // what the selection step hands to the caller
        for (int64_t it = tid; it < (int64_t)k * vec_per_row; it += SK_THREADS) {
            const int j = (int)(it / vec_per_row);
            const int64_t col = (it % vec_per_row) * V;
            T* dst = C + (int64_t)j * ldc;
            if (col + V <= n) {
                *reinterpret_cast<uint4*>(dst + col) = s_c_raw[it];
            } else {
                const T* srow = sC + (int64_t)j * n_pad;
                for (int e = 0; e < V && col + e < n; ++e) dst[col + e] = srow[col + e];
            }
        }
        if (tid < k) {
            idx_out[tid] = s_idx[tid];
            c_invnorm[tid] = s_inv[tid];
            c_invnorm[k + tid] = s_inv2[tid];
        }
    }

    // scores, argmax and alpha: one warp per row of this CTA's range (Lemma 1, Eq. 1; lowest index on ties)
    const int64_t r0 = (int64_t)blockIdx.x * rows_per_cta;
    const int64_t r1 = min(b, r0 + (int64_t)rows_per_cta);
    for (int64_t i = r0 + warp; i < r1; i += SK_WARPS) {
        const T* xrow = X + i * ldx;
        float acc[SK_MAX_K];
#pragma unroll
        for (int jj = 0; jj < SK_MAX_K; ++jj) acc[jj] = 0.f;
        for (int64_t col0 = (int64_t)lane * V; col0 < n; col0 += 4 * 32 * V) {
            float x[4][V];
#pragma unroll
            for (int u = 0; u < 4; ++u)            // four 16-byte loads of the row in flight
                if (col0 + u * 32 * V < n) load_vec<T>(xrow, col0 + u * 32 * V, n, x[u]);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int64_t col = col0 + u * 32 * V;
                if (col < n) {
#pragma unroll
                    for (int jj = 0; jj < SK_MAX_K; ++jj) {
                        if (jj < k) {
                            float c[V];
                            unpack_vec<T>(*reinterpret_cast<const uint4*>(sC + (int64_t)jj * n_pad + col), c);
#pragma unroll
                            for (int e = 0; e < V; ++e) acc[jj] = fmaf(x[u][e], c[e], acc[jj]);
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int jj = 0; jj < SK_MAX_K; ++jj) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) acc[jj] += __shfl_xor_sync(0xffffffffu, acc[jj], off);
        }
        float best = -1.f, s_best = 0.f;
        int j_best = 0;
#pragma unroll
        for (int jj = 0; jj < SK_MAX_K; ++jj) {
            if (jj < k) {
                const float score = fabsf(acc[jj]) * s_inv[jj];
                if (score > best) { best = score; s_best = acc[jj]; j_best = jj; }
            }
        }
        if (lane == 0) {
            store_index(f, f_type, i, j_best);
            alpha[i] = s_best * s_inv2[j_best];
        }
    }
}

// B~ per row range, without sorting.  grid = (row ranges, column slabs of blockDim.x 16-byte chunks).
template <typename T>
__global__ void __launch_bounds__(SK_CT_THREADS)
contract_small_kernel(const void* __restrict__ f, int f_type, const float* __restrict__ alpha, const T* __restrict__ dY,
                      int64_t ldy, int64_t b, int64_t m, int k, int rows_per_range, float* __restrict__ partials,
                      int64_t m_pad) {
    constexpr int V = Vec16<T>::N;
    __shared__ int32_t s_f[SK_BATCH];
    __shared__ float s_a[SK_BATCH];
    const int tid = threadIdx.x;
    const int64_t col = ((int64_t)blockIdx.y * blockDim.x + tid) * V;
    const bool active = col < m, full_vec = col + V <= m;
    const int64_t r0 = (int64_t)blockIdx.x * rows_per_range;
    const int64_t r1 = min(b, r0 + (int64_t)rows_per_range);
    float acc[SK_MAX_K][V];
#pragma unroll
    for (int jj = 0; jj < SK_MAX_K; ++jj)
#pragma unroll
        for (int e = 0; e < V; ++e) acc[jj][e] = 0.f;
    grid_dependency_wait();     // f and alpha come from the kernel before
    grid_launch_dependents();

    for (int64_t t0 = r0; t0 < r1; t0 += SK_BATCH) {
        const int cnt = (int)min((int64_t)SK_BATCH, r1 - t0);
        __syncthreads();
        if (tid < cnt) {
            int32_t j = load_index(f, f_type, t0 + tid);
            if (j < 0 || j >= k) {          // skipped and reported, as the sorting path does
                if (blockIdx.y == 0) raise_status(DEV_BAD_INDEX);
                j = -1;
            }
            const float a = alpha[t0 + tid];
            s_f[tid] = a != 0.f ? j : -1;       // a row with alpha = 0 adds nothing: it matches no generator below
            s_a[tid] = a;
        }
        __syncthreads();
        if (!active) continue;
        for (int t = 0; t < cnt; t += SK_ROWS_IN_FLIGHT) {
            uint4 raw[SK_ROWS_IN_FLIGHT];
            float x[SK_ROWS_IN_FLIGHT][V];
#pragma unroll
            for (int u = 0; u < SK_ROWS_IN_FLIGHT; ++u) {
                if (t + u < cnt) {
                    const T* row = dY + (t0 + t + u) * ldy;
                    if (full_vec) raw[u] = __ldg(reinterpret_cast<const uint4*>(row + col));
                    else load_vec<T>(row, col, m, x[u]);
                }
            }
#pragma unroll
            for (int u = 0; u < SK_ROWS_IN_FLIGHT; ++u) {
                if (t + u < cnt) {
                    if (full_vec) unpack_vec<T>(raw[u], x[u]);
                    const int32_t j = s_f[t + u];
                    const float a = s_a[t + u];
#pragma unroll
                    for (int jj = 0; jj < SK_MAX_K; ++jj) {
                        if (jj == j) {
#pragma unroll
                            for (int e = 0; e < V; ++e) acc[jj][e] = fmaf(a, x[u][e], acc[jj][e]);
                        }
                    }
                }
            }
        }
    }
    if (!active) return;
#pragma unroll
    for (int jj = 0; jj < SK_MAX_K; ++jj) {
        if (jj < k) {
            float* out = partials + ((int64_t)blockIdx.x * k + jj) * m_pad + col;      // m_pad % 4 == 0, col % V == 0
#pragma unroll
            for (int e = 0; e < V; e += 4)
                if (col + e < m_pad) *reinterpret_cast<float4*>(out + e) = make_float4(acc[jj][e], acc[jj][e + 1], acc[jj][e + 2], acc[jj][e + 3]);
        }
    }
}

// Adds the partial B~ of all ranges (ascending) for a slab of 128 columns, then dW = C^T B~ for
// this CTA's SK_WG_ROWS hidden indices.  grid = (column slabs, blocks of the hidden index).  The
// CTA's slice of C is fetched into shared memory while the partial sums are on their way.
constexpr int SK_WG_ROWS = 64;

template <typename T, typename OutT, bool SWAP>
__global__ void __launch_bounds__(SK_THREADS)
wgrad_small_kernel(const T* __restrict__ C, int64_t ldc, int k, int64_t n, const float* __restrict__ partials, int ranges,
                   int64_t m_pad, int64_t m, float* __restrict__ Bt, int64_t ldb, OutT* __restrict__ dW, int64_t ldw,
                   int accumulate) {
    __shared__ float s_b[SK_MAX_K][SK_WG_COLS];
    __shared__ float s_c[SK_MAX_K][SK_WG_ROWS];
    const int tid = threadIdx.x;
    const int64_t c0 = (int64_t)blockIdx.x * SK_WG_COLS;
    const int64_t h0 = (int64_t)blockIdx.y * SK_WG_ROWS;
    grid_dependency_wait();
    grid_launch_dependents();
    for (int it = tid; it < k * SK_WG_ROWS; it += SK_THREADS) {
        const int jj = it / SK_WG_ROWS, r = it % SK_WG_ROWS;
        s_c[jj][r] = h0 + r < n ? load_scalar<T>(C + (int64_t)jj * ldc + h0 + r) : 0.f;
    }
    for (int it = tid; it < k * SK_WG_COLS; it += SK_THREADS) {
        const int jj = it / SK_WG_COLS, c = it % SK_WG_COLS;
        float s = 0.f;
        if (c0 + c < m) {
            const float* p = partials + (int64_t)jj * m_pad + c0 + c;
            const int64_t stride = (int64_t)k * m_pad;
            int r = 0;
            for (; r + 16 <= ranges; r += 16) {      // sixteen loads in flight, added in ascending order
                float v[16];
#pragma unroll
                for (int u = 0; u < 16; ++u) v[u] = p[(int64_t)(r + u) * stride];
#pragma unroll
                for (int u = 0; u < 16; ++u) s += v[u];
            }
            for (; r < ranges; ++r) s += p[(int64_t)r * stride];
            if (Bt && blockIdx.y == 0) Bt[(int64_t)jj * ldb + c0 + c] = s;
        }
        s_b[jj][c] = s;
    }
    __syncthreads();

    if (!SWAP) {
        // rows of dW = hidden index; a thread owns four consecutive columns of the slab
        const int cg = tid % 32, rl = tid / 32;
        const int64_t col = c0 + cg * 4;
        if (col >= m) return;
        for (int r = rl; r < SK_WG_ROWS && h0 + r < n; r += SK_THREADS / 32) {
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int jj = 0; jj < SK_MAX_K; ++jj) {
                if (jj < k) {
                    const float p = s_c[jj][r];
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[e] = fmaf(p, s_b[jj][cg * 4 + e], acc[e]);
                }
            }
            OutT* out = dW + (h0 + r) * ldw + col;
            if constexpr (sizeof(OutT) == 4) {
                if (col + 4 <= m) {      // rows start 16-byte aligned and col is a multiple of four
                    float4 o = make_float4(acc[0], acc[1], acc[2], acc[3]);
                    float4* o4 = reinterpret_cast<float4*>(out);
                    if (accumulate) { const float4 old = *o4; o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w; }
                    *o4 = o;
                    continue;
                }
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if (col + e < m) {
                    float v = acc[e];
                    if (accumulate) v += out_to_float(out[e]);
                    out[e] = float_to_out<OutT>(v);
                }
            }
        }
    } else {
        // rows of dW^T = columns of B~; a thread owns four consecutive hidden indices
        const int rg = tid % (SK_WG_ROWS / 4), cl = tid / (SK_WG_ROWS / 4);
        const int r = rg * 4;
        if (h0 + r >= n) return;
        for (int c = cl; c < SK_WG_COLS && c0 + c < m; c += SK_THREADS / (SK_WG_ROWS / 4)) {
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int jj = 0; jj < SK_MAX_K; ++jj) {
                if (jj < k) {
                    const float q = s_b[jj][c];
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[e] = fmaf(s_c[jj][r + e], q, acc[e]);
                }
            }
            OutT* out = dW + (c0 + c) * ldw + h0 + r;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if (h0 + r + e < n) {
                    float v = acc[e];
                    if (accumulate) v += out_to_float(out[e]);
                    out[e] = float_to_out<OutT>(v);
                }
            }
        }
    }
}

}  // namespace pamm
