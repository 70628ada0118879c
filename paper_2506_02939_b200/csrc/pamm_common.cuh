// Shared device/host helpers of the PAMM sm_100a library: status word, storage
// types, 16-byte vector access, the keyed permutation used for sampling.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/pamm.h"

namespace pamm {

// Bits ORed into the per-device status word by kernels (never a trap).
enum : int { DEV_TIMEOUT = 1, DEV_BAD_INDEX = 2 };

__device__ int g_status_word;

__device__ __forceinline__ void raise_status(int bit) { atomicOr(&g_status_word, bit); }

// ---- programmatic dependent launch ---------------------------------------------
// A kernel launched with the programmatic-serialization attribute may start
// while its predecessor in the stream is still running.  It must call
// grid_dependency_wait() before it touches anything the predecessor writes (or
// anything the predecessor still reads and this kernel overwrites); the call
// returns once the predecessor has finished and its writes are visible, and is
// a no-op for an ordinary launch.  grid_launch_dependents() lets the successor's
// CTAs be scheduled as soon as every CTA of this grid has issued it.
//
// RULE for every kernel of this library: call grid_dependency_wait() before the first
// access to global memory that a predecessor may write (or may still read, if this kernel
// overwrites it).  Kernels rely on it transitively: a kernel may release its dependents
// before its own wait has returned (the tensor-core compress kernel does, so that its
// successor's set-up overlaps the whole pass), and the successor's wait then still covers
// everything older, because it returns only when the predecessor grid -- which itself
// waited for its own predecessor -- has completed.  A kernel that reads anything before its
// wait may read only what was complete before its predecessor was LAUNCHED.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---- the assignment f in its storage type ------------------------------------------
// `type` is a pamm_index_type: 32-bit signed, or unsigned 16 / 8 bits for k <= 65536 / 256.
__device__ __forceinline__ void store_index(void* f, int type, int64_t i, int32_t j) {
    if (type == PAMM_IDX_I32) static_cast<int32_t*>(f)[i] = j;
    else if (type == PAMM_IDX_U16) static_cast<uint16_t*>(f)[i] = (uint16_t)j;
    else static_cast<uint8_t*>(f)[i] = (uint8_t)j;
}
__device__ __forceinline__ int32_t load_index(const void* f, int type, int64_t i) {
    if (type == PAMM_IDX_I32) return static_cast<const int32_t*>(f)[i];
    if (type == PAMM_IDX_U16) return (int32_t)static_cast<const uint16_t*>(f)[i];
    return (int32_t)static_cast<const uint8_t*>(f)[i];
}

// Normalisation factor of Section 3.2 ("Normalization factor beta", Eq. 4-5):
// beta = b / (b - eta) with eta dropped rows, read from device memory; 1 when no
// counter is given, 0 when every row was dropped (the estimate is the zero matrix).
__device__ __forceinline__ float beta_factor(const int32_t* __restrict__ dropped, int64_t b) {
    if (!dropped) return 1.f;
    const int64_t eta = *dropped;
    return eta < b ? (float)((double)b / (double)(b - eta)) : 0.f;
}

// ---- storage types ----------------------------------------------------------
template <typename T> struct Vec16;   // 16 bytes of T
template <> struct Vec16<float> {
    static constexpr int N = 4;
    float v[4];
};
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int N = 8;
    uint32_t w[4];
};

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// Load up to 16 bytes of a row starting at element `col`; elements at or beyond
// `ncols` read as zero.  `row` is 16-byte aligned and `col` a multiple of N.
template <typename T>
__device__ __forceinline__ void load_vec(const T* row, int64_t col, int64_t ncols, float (&out)[Vec16<T>::N]);

template <>
__device__ __forceinline__ void load_vec<float>(const float* row, int64_t col, int64_t ncols, float (&out)[4]) {
    if (col + 4 <= ncols) {
        float4 t = __ldg(reinterpret_cast<const float4*>(row + col));
        out[0] = t.x; out[1] = t.y; out[2] = t.z; out[3] = t.w;
    } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) out[e] = (col + e < ncols) ? __ldg(row + col + e) : 0.f;
    }
}

template <>
__device__ __forceinline__ void load_vec<__nv_bfloat16>(const __nv_bfloat16* row, int64_t col, int64_t ncols,
                                                        float (&out)[8]) {
    if (col + 8 <= ncols) {
        uint4 t = __ldg(reinterpret_cast<const uint4*>(row + col));
        out[0] = bf16_lo(t.x); out[1] = bf16_hi(t.x); out[2] = bf16_lo(t.y); out[3] = bf16_hi(t.y);
        out[4] = bf16_lo(t.z); out[5] = bf16_hi(t.z); out[6] = bf16_lo(t.w); out[7] = bf16_hi(t.w);
    } else {
        const unsigned short* r16 = reinterpret_cast<const unsigned short*>(row);
#pragma unroll
        for (int e = 0; e < 8; ++e)
            out[e] = (col + e < ncols) ? __uint_as_float(((uint32_t)__ldg(r16 + col + e)) << 16) : 0.f;
    }
}

// 16 bytes already in a register -> floats
template <typename T>
__device__ __forceinline__ void unpack_vec(const uint4& raw, float (&out)[Vec16<T>::N]);
template <>
__device__ __forceinline__ void unpack_vec<float>(const uint4& raw, float (&out)[4]) {
    out[0] = __uint_as_float(raw.x); out[1] = __uint_as_float(raw.y);
    out[2] = __uint_as_float(raw.z); out[3] = __uint_as_float(raw.w);
}
template <>
__device__ __forceinline__ void unpack_vec<__nv_bfloat16>(const uint4& raw, float (&out)[8]) {
    out[0] = bf16_lo(raw.x); out[1] = bf16_hi(raw.x); out[2] = bf16_lo(raw.y); out[3] = bf16_hi(raw.y);
    out[4] = bf16_lo(raw.z); out[5] = bf16_hi(raw.z); out[6] = bf16_lo(raw.w); out[7] = bf16_hi(raw.w);
}
// floats that are exactly representable in T -> 16 bytes of T
template <typename T>
__device__ __forceinline__ uint4 pack_vec(const float (&x)[Vec16<T>::N]);
template <>
__device__ __forceinline__ uint4 pack_vec<float>(const float (&x)[4]) {
    return make_uint4(__float_as_uint(x[0]), __float_as_uint(x[1]), __float_as_uint(x[2]), __float_as_uint(x[3]));
}
template <>
__device__ __forceinline__ uint4 pack_vec<__nv_bfloat16>(const float (&x)[8]) {
    // the values are bf16 already: their upper halves are the bit patterns
    return make_uint4((__float_as_uint(x[0]) >> 16) | (__float_as_uint(x[1]) & 0xFFFF0000u),
                      (__float_as_uint(x[2]) >> 16) | (__float_as_uint(x[3]) & 0xFFFF0000u),
                      (__float_as_uint(x[4]) >> 16) | (__float_as_uint(x[5]) & 0xFFFF0000u),
                      (__float_as_uint(x[6]) >> 16) | (__float_as_uint(x[7]) & 0xFFFF0000u));
}
// one element through a generic (e.g. shared-memory) pointer
__device__ __forceinline__ float load_scalar_generic(const float* p) { return *p; }
__device__ __forceinline__ float load_scalar_generic(const __nv_bfloat16* p) {
    return __uint_as_float(((uint32_t)*reinterpret_cast<const unsigned short*>(p)) << 16);
}

// ---- keyed permutation of [0,b) used to sample generators ---------------------
// A 6-round balanced Feistel network on w bits (w even, 2^w >= b), cycle-walked
// until the value falls below b.  Round keys come from splitmix64(seed).
struct PermKey {
    uint32_t key[6];
    uint32_t half_bits;
    uint32_t half_mask;
    uint32_t b;
};

__host__ __device__ inline uint64_t splitmix64(uint64_t x) {
    x += 0x9E3779B97F4A7C15ull;
    x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
    x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
    return x ^ (x >> 31);
}

__host__ __device__ inline PermKey make_perm_key(uint64_t seed, uint32_t b) {
    PermKey pk;
    uint32_t w = 2;
    while (w < 32 && (1ull << w) < (uint64_t)b) w += 2;
    pk.half_bits = w / 2;
    pk.half_mask = (1u << (w / 2)) - 1u;
    pk.b = b;
    uint64_t s = seed;
    for (int r = 0; r < 6; ++r) {
        s = splitmix64(s);
        pk.key[r] = (uint32_t)(s >> 32);
    }
    return pk;
}

__host__ __device__ inline uint32_t feistel_round_fn(uint32_t r, uint32_t key) {
    uint32_t h = r * 0x9E3779B1u + key;
    h ^= h >> 16; h *= 0x85EBCA6Bu;
    h ^= h >> 13; h *= 0xC2B2AE35u;
    h ^= h >> 16;
    return h;
}

__host__ __device__ inline uint32_t perm_apply(const PermKey& pk, uint32_t x) {
    // bounded cycle walk: the domain is < 4b, so the expected walk is < 4 steps
    for (int walk = 0; walk < 4096; ++walk) {
        uint32_t L = x >> pk.half_bits, R = x & pk.half_mask;
        for (int r = 0; r < 6; ++r) {
            uint32_t t = (L ^ feistel_round_fn(R, pk.key[r])) & pk.half_mask;
            L = R;
            R = t;
        }
        x = (L << pk.half_bits) | R;
        if (x < pk.b) return x;
    }
    return x % pk.b;   // unreachable in practice; keeps the walk bounded
}

inline int64_t round_up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }

// Text behind the last PAMM_ERR_CUDA of the calling thread (which CUDA call failed and how).
void note_cuda_failure(const char* what, cudaError_t err);
// cudaGetLastError as a status, with the failure noted.
inline pamm_status launch_result(const char* what) {
    const cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) return PAMM_OK;
    note_cuda_failure(what, e);
    return PAMM_ERR_CUDA;
}

pamm_status tensor_map_failed();     // notes what the failed encoding was asked for

// Raises a kernel's dynamic shared-memory limit when a launch needs more than the
// 48 KiB default, remembering per device and kernel what has been granted already
// so that the driver call is not repeated on every launch.
bool ensure_dynamic_smem(const void* kernel, size_t bytes);
// Whether clusters of two CTAs of this kernel can be scheduled on the current device (asked once per
// kernel, device and shared-memory size); where they cannot, the one-CTA kernels serve.
bool cta_pairs_can_launch(const void* kernel, int threads, size_t dynamic_smem);

}  // namespace pamm
