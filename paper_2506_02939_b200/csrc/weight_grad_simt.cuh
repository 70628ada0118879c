// Step 4 on CUDA cores: dW[r,c] = sum_j C[j,r] * B~[j,c]  (Algorithm 1 ApproxMM,
// the final product).  Each thread owns four consecutive columns of one output
// row and walks the k generators in ascending order with fp32 FMAs.  Used for
// fp32 generators and whenever the tensor-core path does not apply.
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

template <typename T>
__global__ void __launch_bounds__(WG_THREADS)
weight_grad_simt_kernel(const T* __restrict__ C, int64_t ldc, int k, int64_t n,
                        const float* __restrict__ Bt, int64_t ldb, int64_t m,
                        float* __restrict__ dW, int64_t ldw, int64_t b_rows, const int32_t* __restrict__ dropped,
                        int accumulate) {
    const int64_t mv = (m + 3) / 4;
    const int64_t idx = (int64_t)blockIdx.x * WG_THREADS + threadIdx.x;
    grid_dependency_wait();     // B~ (and C) may come from the kernel before
    grid_launch_dependents();
    if (idx >= n * mv) return;
    const int64_t r = idx / mv, col = (idx % mv) * 4;
    const float beta = beta_factor(dropped, b_rows);
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    if (col + 4 <= m) {
        for (int j = 0; j < k; ++j) {
            const float c = load_scalar<T>(C + (int64_t)j * ldc + r);
            const float4 v = __ldg(reinterpret_cast<const float4*>(Bt + (int64_t)j * ldb + col));
            acc[0] = fmaf(c, v.x, acc[0]); acc[1] = fmaf(c, v.y, acc[1]);
            acc[2] = fmaf(c, v.z, acc[2]); acc[3] = fmaf(c, v.w, acc[3]);
        }
        float4 o = make_float4(beta * acc[0], beta * acc[1], beta * acc[2], beta * acc[3]);
        if (accumulate) {
            const float4 old = *reinterpret_cast<const float4*>(dW + r * ldw + col);
            o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
        }
        *reinterpret_cast<float4*>(dW + r * ldw + col) = o;
    } else {
        for (int j = 0; j < k; ++j) {
            const float c = load_scalar<T>(C + (int64_t)j * ldc + r);
            for (int e = 0; e < 4 && col + e < m; ++e) acc[e] = fmaf(c, __ldg(Bt + (int64_t)j * ldb + col + e), acc[e]);
        }
        for (int e = 0; e < 4 && col + e < m; ++e)
            dW[r * ldw + col + e] = beta * acc[e] + (accumulate ? dW[r * ldw + col + e] : 0.f);
    }
}

}  // namespace pamm
