// Step 4 on CUDA cores: dW[r,c] = sum_j C[j,r] * B~[j,c]  (Algorithm 1 ApproxMM,
// the final product).  Each thread owns four consecutive columns of one output
// row and walks the k generators in ascending order with fp32 FMAs.  Used for
// fp32 generators and whenever the tensor-core path does not apply.
// With SWAP the output is dW^T (m x n): rows run over the columns of B~, the four
// consecutive columns over the hidden index.
#pragma once
#include "pamm_common.cuh"

namespace pamm {

constexpr int WG_THREADS = 256;

template <typename T>
__device__ __forceinline__ float load_scalar(const T* p);
template <> __device__ __forceinline__ float load_scalar<float>(const float* p) { return __ldg(p); }
template <> __device__ __forceinline__ float load_scalar<__nv_bfloat16>(const __nv_bfloat16* p) {
    return __uint_as_float(((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p))) << 16);
}

__device__ __forceinline__ float out_to_float(float v) { return v; }
__device__ __forceinline__ float out_to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename OutT> __device__ __forceinline__ OutT float_to_out(float v);
template <> __device__ __forceinline__ float float_to_out<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 float_to_out<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// T: type of C.  OutT: type of dW.  SWAP: dW^T (m x n) instead of dW (n x m).
template <typename T, typename OutT, bool SWAP>
__global__ void __launch_bounds__(WG_THREADS)
weight_grad_simt_kernel(const T* __restrict__ C, int64_t ldc, int k, int64_t n,
                        const float* __restrict__ Bt, int64_t ldb, int64_t m,
                        OutT* __restrict__ dW, int64_t ldw, int64_t b_rows, const int32_t* __restrict__ dropped,
                        int accumulate) {
    const int64_t rows = SWAP ? m : n, cols = SWAP ? n : m;
    const int64_t cv = (cols + 3) / 4;
    const int64_t idx = (int64_t)blockIdx.x * WG_THREADS + threadIdx.x;
    grid_dependency_wait();     // B~ (and C) may come from the kernel before
    grid_launch_dependents();
    if (idx >= rows * cv) return;
    const int64_t r = idx / cv, col = (idx % cv) * 4;
    const float beta = beta_factor(dropped, b_rows);
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    const bool full = col + 4 <= cols;
    for (int j = 0; j < k; ++j) {
        // the row's factor, then the four column factors; every product is C[j,.] * B~[j,.] in that order
        const float p = SWAP ? __ldg(Bt + (int64_t)j * ldb + r) : load_scalar<T>(C + (int64_t)j * ldc + r);
        if (!SWAP && full) {
            const float4 v = __ldg(reinterpret_cast<const float4*>(Bt + (int64_t)j * ldb + col));
            acc[0] = fmaf(p, v.x, acc[0]); acc[1] = fmaf(p, v.y, acc[1]);
            acc[2] = fmaf(p, v.z, acc[2]); acc[3] = fmaf(p, v.w, acc[3]);
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if (col + e < cols) {
                    const float q = SWAP ? load_scalar<T>(C + (int64_t)j * ldc + col + e) : __ldg(Bt + (int64_t)j * ldb + col + e);
                    acc[e] = SWAP ? fmaf(q, p, acc[e]) : fmaf(p, q, acc[e]);
                }
            }
        }
    }
    OutT* out = dW + r * ldw + col;
    if constexpr (sizeof(OutT) == 4) {
        if (full) {     // rows start 16-byte aligned and col is a multiple of four
            float4 o = make_float4(beta * acc[0], beta * acc[1], beta * acc[2], beta * acc[3]);
            float4* o4 = reinterpret_cast<float4*>(out);
            if (accumulate) { const float4 old = *o4; o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w; }
            *o4 = o;
            return;
        }
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        if (col + e < cols) {
            float v = beta * acc[e];
            if (accumulate) v += out_to_float(out[e]);
            out[e] = float_to_out<OutT>(v);
        }
    }
}

}  // namespace pamm
