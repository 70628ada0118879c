// Step 2 on CUDA cores: scoring S = X C^T, per-row argmax of |S_ij| / ||C_j||
// (Lemma 1) and alpha (Eq. 1).  One warp streams one row of X with 16-byte
// loads and keeps KC dot products per lane; a shuffle tree finishes each dot
// product and every lane then holds the same totals, so the argmax needs no
// further exchange.  This is the path for fp32 inputs and for small k, where
// the contraction is too thin for tensor cores.
#pragma once
#include "pamm_common.cuh"

namespace pamm {

constexpr int CS_THREADS = 256;
constexpr int CS_WARPS = CS_THREADS / 32;

// EPS = true adds the neighbourhood condition (Eq. 2): ||X_i||^2 is summed in the same
// pass and a row with ||X_i||^2 - S^2/||C_f||^2 > (eps^2 + slack) ||X_i||^2 gets alpha = 0;
// *dropped counts such rows.
template <typename T, int KC, bool EPS>
__global__ void __launch_bounds__(CS_THREADS)
compress_simt_kernel(const T* __restrict__ X, int64_t ldx, int64_t b, int64_t n,
                     const T* __restrict__ C, int64_t ldc, int k,
                     const float* __restrict__ c_invnorm,
                     void* __restrict__ f, int f_type, float* __restrict__ alpha, float eps2, float slack,
                     int32_t* __restrict__ dropped) {
    constexpr int V = Vec16<T>::N;
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = (int64_t)blockIdx.x * CS_WARPS + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * CS_WARPS;
    grid_dependency_wait();     // C and the norms come from the kernel before
    grid_launch_dependents();

    for (int64_t i = warp0; i < b; i += nwarps) {
        const T* xrow = X + i * ldx;
        float best = -1.f, s_best = 0.f, xx = 0.f;
        int j_best = 0;
        for (int j0 = 0; j0 < k; j0 += KC) {
            float acc[KC];
#pragma unroll
            for (int jj = 0; jj < KC; ++jj) acc[jj] = 0.f;
            for (int64_t col = (int64_t)lane * V; col < n; col += 32 * V) {
                float x[V];
                load_vec<T>(xrow, col, n, x);
                if (EPS && j0 == 0) {
#pragma unroll
                    for (int e = 0; e < V; ++e) xx = fmaf(x[e], x[e], xx);
                }
#pragma unroll
                for (int jj = 0; jj < KC; ++jj) {
                    if (j0 + jj < k) {
                        float c[V];
                        load_vec<T>(C + (int64_t)(j0 + jj) * ldc, col, n, c);
#pragma unroll
                        for (int e = 0; e < V; ++e) acc[jj] = fmaf(x[e], c[e], acc[jj]);
                    }
                }
            }
#pragma unroll
            for (int jj = 0; jj < KC; ++jj) {
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) acc[jj] += __shfl_xor_sync(0xffffffffu, acc[jj], off);
            }
#pragma unroll
            for (int jj = 0; jj < KC; ++jj) {
                if (j0 + jj < k) {
                    float score = fabsf(acc[jj]) * __ldg(c_invnorm + j0 + jj);
                    if (score > best) {   // strict: the lowest index keeps a tie
                        best = score;
                        s_best = acc[jj];
                        j_best = j0 + jj;
                    }
                }
            }
        }
        if (EPS) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) xx += __shfl_xor_sync(0xffffffffu, xx, off);
        }
        if (lane == 0) {
            float a = s_best * __ldg(c_invnorm + k + j_best);
            if (EPS && xx - s_best * a > (eps2 + slack) * xx) {
                a = 0.f;
                atomicAdd(dropped, 1);
            }
            store_index(f, f_type, i, j_best);
            alpha[i] = a;
        }
    }
}

}  // namespace pamm
