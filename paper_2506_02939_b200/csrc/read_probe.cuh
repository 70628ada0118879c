// Read-only streaming probes: the practical ceiling of the read-dominated passes (the
// compression reads X once, the contraction reads dY once), measured on the data and in the
// row order those passes use.  Nothing of the method is computed here; a 32-bit wrap-around
// sum of what was read keeps the reads alive and lets a test check that every row was visited.
//   PROBE_SUM    every 16-byte word of every row through ordinary loads, summed
//   PROBE_ROWS   whole rows by cp.async.bulk through a shared-memory ring, two CTAs per SM,
//                in natural order or in the order given (the contraction's sorted order):
//                the access pattern of contract_stream_kernel without its arithmetic
#pragma once
#include "pamm_common.cuh"
#include "sm100_ptx.cuh"

namespace pamm {

constexpr int RP_SUM_THREADS = 512;
constexpr int RP_ROW_THREADS = 64;
constexpr int RP_MAX_SLOTS = 16;
constexpr int RP_RING_BYTES = 88 * 1024;      // the ring of the contraction's main pass

// rows x row_bytes (a multiple of 16), ld_bytes apart; the sum of all 32-bit words goes to *sum.
__global__ void __launch_bounds__(RP_SUM_THREADS)
read_probe_sum_kernel(const uint8_t* __restrict__ base, int64_t rows, int64_t row_bytes, int64_t ld_bytes,
                      unsigned int* __restrict__ sum) {
    __shared__ unsigned int s_part[RP_SUM_THREADS / 32];
    const int64_t vecs = row_bytes / 16, total = rows * vecs;
    unsigned int acc = 0;
    int64_t i = (int64_t)blockIdx.x * RP_SUM_THREADS + threadIdx.x;
    const int64_t step = (int64_t)gridDim.x * RP_SUM_THREADS;
    for (; i + 3 * step < total; i += 4 * step) {       // four independent loads in flight per thread
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int64_t j = i + u * step;
            v[u] = __ldg(reinterpret_cast<const uint4*>(base + (j / vecs) * ld_bytes + (j % vecs) * 16));
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) acc += v[u].x + v[u].y + v[u].z + v[u].w;
    }
    for (; i < total; i += step) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(base + (i / vecs) * ld_bytes + (i % vecs) * 16));
        acc += v.x + v.y + v.z + v.w;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned int t = 0;
        for (int w = 0; w < RP_SUM_THREADS / 32; ++w) t += s_part[w];
        atomicAdd(sum, t);          // integers: exact in any order
    }
}

// One CTA per contiguous range of positions; position p reads row order[p] (or p).  Thread 0 keeps
// the ring full, thread 32 takes the slots back as they land and adds the first word of every row.
__global__ void __launch_bounds__(RP_ROW_THREADS, 2)
read_probe_rows_kernel(const uint8_t* __restrict__ base, int64_t rows, uint32_t row_bytes, int64_t ld_bytes,
                       const int32_t* __restrict__ order, int slots, int slot_pitch, unsigned int* __restrict__ sum) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_full[RP_MAX_SLOTS], s_empty[RP_MAX_SLOTS];
    __shared__ int s_abort;
    uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
    const int64_t per = (rows + gridDim.x - 1) / gridDim.x;
    const int64_t r0 = min(rows, (int64_t)blockIdx.x * per), r1 = min(rows, r0 + per);
    if (threadIdx.x == 0) {
        for (int s = 0; s < slots; ++s) { ptx::mbar_init(&s_full[s], 1); ptx::mbar_init(&s_empty[s], 1); }
        s_abort = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async();
    }
    __syncthreads();
    volatile int* abort_flag = &s_abort;
    if (threadIdx.x == 0) {
        const uint64_t policy = ptx::l2_policy_evict_first();
        uint32_t ph = 0;
        int s = 0;
        int64_t r = r0;
        for (; r < r1; ++r) {
            if (!ptx::mbar_wait(&s_empty[s], ph ^ 1u, abort_flag)) break;
            int64_t row = order ? (int64_t)order[r] : r;
            if (row < 0 || row >= rows) { raise_status(DEV_BAD_INDEX); row = 0; }
            ptx::mbar_arrive_expect_tx(&s_full[s], row_bytes);
            ptx::bulk_load_hint(ring + (size_t)s * slot_pitch, base + row * ld_bytes, row_bytes, &s_full[s], policy);
            if (++s == slots) { s = 0; ph ^= 1u; }
        }
        if (r < r1) {      // a wait ran out: let the copies already issued land before the CTA leaves
            raise_status(DEV_TIMEOUT);
            int never = 0;
            volatile int* no_abort = &never;
            const int64_t issued = r - r0;
            for (int64_t d = 1; d <= min(issued, (int64_t)slots); ++d) {
                const int64_t j = issued - d;
                ptx::mbar_wait(&s_full[j % slots], (uint32_t)((j / slots) & 1), no_abort);
            }
        }
    } else if (threadIdx.x == 32) {
        uint32_t ph = 0;
        int s = 0;
        unsigned int acc = 0;
        for (int64_t r = r0; r < r1; ++r) {
            if (!ptx::mbar_wait(&s_full[s], ph, abort_flag)) { raise_status(DEV_TIMEOUT); break; }
            acc += *reinterpret_cast<const volatile unsigned int*>(ring + (size_t)s * slot_pitch);
            ptx::mbar_arrive(&s_empty[s]);
            if (++s == slots) { s = 0; ph ^= 1u; }
        }
        atomicAdd(sum, acc);
    }
}

}  // namespace pamm
