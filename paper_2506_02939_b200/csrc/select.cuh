// Step 1: generator selection (Algorithm 1, Compress: index sampling, the gather of C,
// and the norms of the generator rows).  One launch, no cross-CTA dependency:
// every CTA recomputes the k candidate indices in shared memory, ranks its own
// candidate (rank = sorted position), copies that row of X into C with one
// 16-byte load per thread and accumulates its squared norm as an unevaluated fp32 pair (hi, lo)
// with error-free additions, which carries about 48 bits: the stored 1/||C_j||
// then has fp32 rounding only, at a fraction of the cost of fp64 arithmetic.
#pragma once
#include "pamm_common.cuh"

namespace pamm {

constexpr int SEL_THREADS = 256;
constexpr int SEL_WARPS = SEL_THREADS / 32;
constexpr int64_t SEL_MAX_K = 49152;   // k * 4 bytes of dynamic shared memory

// a <- fl(a + b); returns the rounding error of that addition (Knuth's branch-free form).
__device__ __forceinline__ float two_sum(float& a, float b) {
    const float s = __fadd_rn(a, b);
    const float bb = __fsub_rn(s, a);
    const float err = __fadd_rn(__fsub_rn(a, __fsub_rn(s, bb)), __fsub_rn(b, bb));
    a = s;
    return err;
}

template <typename T>
__global__ void __launch_bounds__(SEL_THREADS)
select_kernel(const T* __restrict__ X, int64_t ldx, int64_t b, int64_t n, int k, PermKey pk,
              const int32_t* __restrict__ idx_in, int32_t* __restrict__ idx_out,
              T* __restrict__ C, int64_t ldc, float* __restrict__ c_invnorm,
              int32_t* __restrict__ zero_words, int64_t zero_count) {
    extern __shared__ int32_t s_vals[];
    __shared__ int s_cnt[2][SEL_WARPS];
    __shared__ float s_q[2][SEL_WARPS];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // Drawn indices need no memory, so they are computed while the kernel before may
    // still be running; everything read from memory comes after the wait.  Only then
    // is the compress kernel let in: it may read X as soon as it starts.
    if (!idx_in)
        for (int j = tid; j < k; j += SEL_THREADS) s_vals[j] = (int32_t)perm_apply(pk, (uint32_t)j);
    grid_dependency_wait();
    grid_launch_dependents();
    if (idx_in)
        for (int j = tid; j < k; j += SEL_THREADS) s_vals[j] = idx_in[j];
    // counters the next kernel adds to (the histograms of f of the fused forward pass) start at zero
    for (int64_t z = (int64_t)blockIdx.x * SEL_THREADS + tid; z < zero_count; z += (int64_t)gridDim.x * SEL_THREADS)
        zero_words[z] = 0;
    __syncthreads();

    const int j = blockIdx.x;          // one CTA per generator
    int32_t val = s_vals[j];

    // rank among all candidates, and a duplicate count
    int smaller = 0, dup = 0;
    for (int t = tid; t < k; t += SEL_THREADS) {
        const int32_t o = s_vals[t];
        smaller += (o < val);
        dup += (o == val && t != j);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        smaller += __shfl_xor_sync(0xffffffffu, smaller, off);
        dup += __shfl_xor_sync(0xffffffffu, dup, off);
    }
    if (lane == 0) { s_cnt[0][warp] = smaller; s_cnt[1][warp] = dup; }
    __syncthreads();
    smaller = 0;
    dup = 0;
#pragma unroll
    for (int w = 0; w < SEL_WARPS; ++w) { smaller += s_cnt[0][w]; dup += s_cnt[1][w]; }

    int slot;
    if (idx_in) {
        slot = j;   // caller's order
        bool bad = dup > 0;
        if (val < 0) { val = 0; bad = true; }
        if ((int64_t)val >= b) { val = (int32_t)(b - 1); bad = true; }
        if (bad && tid == 0) raise_status(DEV_BAD_INDEX);
    } else {
        slot = smaller;   // distinct by construction: rank = ascending position
    }

    constexpr int V = Vec16<T>::N;
    const T* src = X + (int64_t)val * ldx;
    T* dst = C + (int64_t)slot * ldc;
    float q_hi = 0.f, q_lo = 0.f;
    for (int64_t col = (int64_t)tid * V; col < n; col += SEL_THREADS * V) {
        float x[V];
        load_vec<T>(src, col, n, x);
        if (col + V <= n) {
            *reinterpret_cast<uint4*>(dst + col) = __ldg(reinterpret_cast<const uint4*>(src + col));
        } else {
            for (int e = 0; e < V && col + e < n; ++e) dst[col + e] = src[col + e];
        }
#pragma unroll
        for (int e = 0; e < V; ++e) {
            const float p = __fmul_rn(x[e], x[e]);
            const float pe = fmaf(x[e], x[e], -p);      // x^2 = p + pe exactly
            q_lo += two_sum(q_hi, p) + pe;
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float o_hi = __shfl_xor_sync(0xffffffffu, q_hi, off);
        const float o_lo = __shfl_xor_sync(0xffffffffu, q_lo, off);
        q_lo = (q_lo + o_lo) + two_sum(q_hi, o_hi);
    }
    if (lane == 0) { s_q[0][warp] = q_hi; s_q[1][warp] = q_lo; }
    __syncthreads();
    if (tid == 0) {
        double q = 0.0;     // eight pairs, added in warp order
#pragma unroll
        for (int w = 0; w < SEL_WARPS; ++w) q += (double)s_q[0][w] + (double)s_q[1][w];
        idx_out[slot] = val;
        c_invnorm[slot] = (q > 0.0) ? (float)(1.0 / sqrt(q)) : 0.f;
        c_invnorm[k + slot] = (q > 0.0) ? (float)(1.0 / q) : 0.f;
    }
}

}  // namespace pamm
