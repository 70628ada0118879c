// Step 3, main pass (Algorithm 1, ApproxMM: alpha-scaling of B and index_add):
// B~[j,:] = sum_{i: f_i = j} alpha_i * dY[i,:] over the rows sorted by f, with the
// rows of dY staged through shared memory by bulk asynchronous copies.
//
// The sorted rows (those with alpha != 0: the others add nothing and are never read) are cut
// into equal contiguous ranges, one CTA per range, two
// CTAs per SM in a single balanced wave (two independent pipelines per SM hide
// each other's waits; measured 17% faster than one CTA with twice the ring).
// Inside a CTA:
//   warp 0      producer: lane l owns ring slot l (a slot holds R = 1, 2 or 4 rows, so that
//               a slot is 8-16 KB whatever the row width and the per-slot handshake is
//               amortised over narrow rows).  A round of the ring is handled by
//               all lanes at once: each looks its row up (perm -> row id, alpha, f; one
//               round ahead), waits for its slot to be free and issues one
//               cp.async.bulk for the row, so the whole ring (88 KB per CTA) is in
//               flight whatever the consumers are doing
//   warps 1..   consumers: thread c owns 16-byte chunks c, c + #consumers, ... of
//               the row and accumulates alpha_i * dY_i in fp32 registers in ascending
//               sorted order; when the generator changes, the finished sum goes
//               straight to B~ if the whole segment lies inside this CTA's range,
//               else to a partial row that contract_reduce_kernel adds up later
// dY is read exactly once; no floating-point atomics, so results are
// bit-reproducible.  Every wait is bounded.
#pragma once
#include "pamm_common.cuh"
#include "sm100_ptx.cuh"
#include "contract.cuh"

namespace pamm {

constexpr int CS_CTAS_PER_SM = 2;                // the ring budget is per CTA
constexpr int CS_MAX_CONSUMERS = 384;            // consumer threads
constexpr int CS_MIN_VPT = 1;
constexpr int CS_MAX_VPT = 4;                    // 16-byte chunks per consumer thread
constexpr int CS_MAX_SLOTS = 32;
constexpr int CS_MAX_RPS = 4;                    // rows per ring slot, at most
constexpr int CS_SLOT_TARGET_BYTES = 16 * 1024;  // rows are grouped while the slot stays within this
constexpr uint32_t CS_PRODUCER_SPINS = 1u << 22;  // idle polls before the producer gives up
constexpr int CS_RING_BYTES = 88 * 1024;

struct ContractStreamPlan {
    int consumers;      // consumer threads, a multiple of 32
    int vpt;            // chunks per consumer thread (1, 2 or 4)
    int rps;            // rows per ring slot (1, 2 or 4; more than 1 only with vpt == 1)
    int slots;
    int row_pitch;      // bytes between the rows of a slot
    uint32_t bulk_bytes;   // bytes of a row copied by the bulk engine (a multiple of 16)
    size_t smem_bytes;
};

// Rows up to CS_MAX_CONSUMERS * CS_MAX_VPT * 16 bytes wide are streamed.
inline bool contract_stream_supported(int64_t m, size_t esz) {
    const int64_t vecs = (m * (int64_t)esz + 15) / 16;
    return vecs <= (int64_t)CS_MAX_CONSUMERS * CS_MAX_VPT;
}

inline ContractStreamPlan contract_stream_plan(int64_t m, size_t esz) {
    ContractStreamPlan p;
    const int64_t row_bytes = m * (int64_t)esz;
    const int64_t vecs = (row_bytes + 15) / 16;
    p.vpt = CS_MIN_VPT;
    while ((vecs + p.vpt - 1) / p.vpt > CS_MAX_CONSUMERS) p.vpt *= 2;
    p.consumers = (int)round_up((vecs + p.vpt - 1) / p.vpt, 32);
    p.bulk_bytes = (uint32_t)(row_bytes & ~(int64_t)15);
    p.row_pitch = (int)round_up(std::max<int64_t>(p.bulk_bytes, 16), 128);
    p.rps = 1;
    if (p.vpt == 1)
        while (p.rps < CS_MAX_RPS && 2 * p.rps * p.row_pitch <= CS_SLOT_TARGET_BYTES) p.rps *= 2;
    p.slots = std::max(2, std::min(CS_MAX_SLOTS, CS_RING_BYTES / (p.rps * p.row_pitch)));
    p.smem_bytes = 128 + (size_t)p.slots * p.rps * p.row_pitch;
    return p;
}

template <typename T, int VPT, int RPS>
__global__ void __launch_bounds__(CS_MAX_CONSUMERS + 32, CS_CTAS_PER_SM)
contract_stream_kernel(const void* __restrict__ f, int f_type, const float* __restrict__ alpha, const T* __restrict__ dY,
                       int64_t ldy, int64_t b, int64_t m, int k, const int32_t* __restrict__ seg_start,
                       const int32_t* __restrict__ perm, int ranges, int slots, int row_pitch,
                       uint32_t bulk_bytes, float* __restrict__ partials, int64_t m_pad,
                       float* __restrict__ Bt, int64_t ldb) {
    constexpr int V = Vec16<T>::N;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t s_full[CS_MAX_SLOTS], s_empty[CS_MAX_SLOTS];
    __shared__ int4 s_meta[CS_MAX_SLOTS][RPS];      // row id, generator, alpha bits of every row in the slot
    __shared__ int s_abort;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int consumers = blockDim.x - 32;
    uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
    const int slot_bytes = RPS * row_pitch;
    const int c = blockIdx.x;

    if (tid == 0) {
        for (int s = 0; s < slots; ++s) {
            ptx::mbar_init(&s_full[s], 1);
            ptx::mbar_init(&s_empty[s], (uint32_t)(consumers / 32));
        }
        s_abort = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async();
    }
    __syncthreads();
    volatile int* abort_flag = &s_abort;
    grid_dependency_wait();       // seg_start and perm come from the kernel before
    grid_launch_dependents();

    const int32_t total = (int32_t)min((int64_t)max(seg_start[k], 0), b);     // the rows with alpha != 0
    const int rows_per_cta = range_rows(total, ranges);
    const int32_t r_begin = (int32_t)min((int64_t)c * rows_per_cta, (int64_t)total);
    const int32_t r_end = (int32_t)min((int64_t)r_begin + rows_per_cta, (int64_t)total);
    const int nrows = r_end - r_begin;

    if (warp == 0) {
        // ---------------- producer ----------------
        // Lane l owns slot l and, in every round of the ring, the RPS consecutive sorted
        // rows that go into it.  Every lane refills its slot as soon as the consumers hand
        // it back, independently of the other lanes (a non-blocking test per poll).
        // Look-ups run ahead: the row ids two rounds ahead, alpha and f one round ahead,
        // so no poll waits on them.
        const int32_t round_rows = slots * RPS;
        int32_t r = lane < slots ? r_begin + lane * RPS : r_end;     // first sorted position of my next slot load
        int32_t i_cur[RPS], i_nxt[RPS], j_cur[RPS];
        float a_cur[RPS];
        // A sorted position holds a row id in [0, b) unless the sort was fed counts that do not
        // belong to this f; such an entry is reported and replaced by row 0 with weight zero.
        bool bad_perm = false;
        auto row_at = [&](int32_t pos) {
            int32_t i = perm[pos];
            if ((uint32_t)i >= (uint32_t)b) { bad_perm = true; i = -1; }
            return i;
        };
        auto weight_of = [&](int32_t i) { return i >= 0 ? alpha[i] : 0.f; };
        auto segment_of_row = [&](int32_t i) {
            const int32_t j = i >= 0 ? load_index(f, f_type, i) : 0;
            return min(max(j, 0), k - 1);
        };
#pragma unroll
        for (int u = 0; u < RPS; ++u) {
            i_cur[u] = -1; i_nxt[u] = -1; j_cur[u] = 0; a_cur[u] = 0.f;
            if (r + u < r_end) {
                i_cur[u] = row_at(r + u);
                a_cur[u] = weight_of(i_cur[u]);
                j_cur[u] = segment_of_row(i_cur[u]);
            }
            if (r + round_rows + u < r_end) i_nxt[u] = row_at(r + round_rows + u);
        }
        const uint64_t stream_policy = ptx::l2_policy_evict_first();   // dY is read once
        uint32_t phase = 0, idle = 0;
        bool issued = false, ok = true;
        uint32_t issued_phase = 0;
        while (__any_sync(0xffffffffu, r < r_end)) {
            bool progressed = false;
            if (r < r_end && ptx::mbar_test_wait(&s_empty[lane], phase ^ 1u)) {
                const int valid = min(RPS, r_end - r);
#pragma unroll
                for (int u = 0; u < RPS; ++u) s_meta[lane][u] = make_int4(i_cur[u], j_cur[u], __float_as_int(a_cur[u]), 0);
                if (bulk_bytes) {
                    ptx::mbar_arrive_expect_tx(&s_full[lane], (uint32_t)valid * bulk_bytes);
#pragma unroll
                    for (int u = 0; u < RPS; ++u)
                        if (u < valid)
                            ptx::bulk_load_hint(ring + (size_t)lane * slot_bytes + (size_t)u * row_pitch,
                                                dY + (int64_t)max(i_cur[u], 0) * ldy, bulk_bytes, &s_full[lane], stream_policy);
                } else {
                    ptx::mbar_arrive(&s_full[lane]);
                }
                issued = true;
                issued_phase = phase;
                phase ^= 1u;
                r += round_rows;
#pragma unroll
                for (int u = 0; u < RPS; ++u) {
                    i_cur[u] = i_nxt[u];
                    if (r + u < r_end) {
                        a_cur[u] = weight_of(i_cur[u]);
                        j_cur[u] = segment_of_row(i_cur[u]);
                    }
                    i_nxt[u] = r + round_rows + u < r_end ? row_at(r + round_rows + u) : -1;
                }
                progressed = true;
            }
            if (__any_sync(0xffffffffu, progressed)) {
                idle = 0;
            } else {
                if (++idle > CS_PRODUCER_SPINS || *abort_flag) { ok = false; break; }
                __nanosleep(32);
            }
        }
        if (bad_perm) raise_status(DEV_BAD_INDEX);
        if (!ok) {
            if (lane == 0) {
                *abort_flag = 1;
                raise_status(DEV_TIMEOUT);
            }
            if (issued) {      // let the copies already issued land before the CTA leaves
                int never = 0;
                volatile int* no_abort = &never;
                ptx::mbar_wait(&s_full[lane], issued_phase, no_abort);
            }
        }
    } else {
        // ---------------- consumers ----------------
        const int ct = tid - 32;
        const int64_t nvec_bulk = bulk_bytes / 16;          // chunks that arrive through the ring
        const int64_t nvec = (m + V - 1) / V;               // all chunks (the last may be ragged)
        float acc[VPT][V];
#pragma unroll
        for (int v = 0; v < VPT; ++v)
#pragma unroll
            for (int e = 0; e < V; ++e) acc[v][e] = 0.f;

        auto flush = [&](int seg) {
            const bool inside = seg_start[seg] >= r_begin && seg_start[seg + 1] <= r_end;
#pragma unroll
            for (int v = 0; v < VPT; ++v) {
                const int64_t vec = ct + (int64_t)v * consumers;
                const int64_t col = vec * V;
                if (vec < nvec) {
                    if (inside) {
                        float* out = Bt + (int64_t)seg * ldb + col;
#pragma unroll
                        for (int e = 0; e < V; e += 4) {
                            if (col + e + 4 <= m) {
                                *reinterpret_cast<float4*>(out + e) = make_float4(acc[v][e], acc[v][e + 1], acc[v][e + 2], acc[v][e + 3]);
                            } else {
                                for (int t = 0; t < 4 && col + e + t < m; ++t) out[e + t] = acc[v][e + t];
                            }
                        }
                    } else {
                        float* out = partials + (int64_t)(c + seg) * m_pad + col;   // m_pad % 4 == 0, col % V == 0
#pragma unroll
                        for (int e = 0; e < V; e += 4)
                            if (col + e < m_pad) *reinterpret_cast<float4*>(out + e) = make_float4(acc[v][e], acc[v][e + 1], acc[v][e + 2], acc[v][e + 3]);
                    }
                }
#pragma unroll
                for (int e = 0; e < V; ++e) acc[v][e] = 0.f;
            }
        };

        int cur = -1;
        int slot = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (int t = 0; t < nrows; t += RPS) {
            ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_full[slot], phase, abort_flag));   // warp-uniform
            if (!ok) break;
            const int valid = min(RPS, nrows - t);
            const uint8_t* src = ring + (size_t)slot * slot_bytes;
            int4 meta[RPS];
            uint4 raw[RPS][VPT];
#pragma unroll
            for (int u = 0; u < RPS; ++u) {           // every load of the slot first, then the arithmetic
                meta[u] = s_meta[slot][u];
#pragma unroll
                for (int v = 0; v < VPT; ++v) {
                    const int64_t vec = ct + (int64_t)v * consumers;
                    raw[u][v] = (u < valid && vec < nvec_bulk)
                                    ? *reinterpret_cast<const uint4*>(src + (size_t)u * row_pitch + vec * 16)
                                    : make_uint4(0u, 0u, 0u, 0u);
                }
            }
#pragma unroll
            for (int u = 0; u < RPS; ++u) {
                if (u < valid) {
                    const int32_t row = meta[u].x;
                    const int32_t j = meta[u].y;
                    const float a = __int_as_float(meta[u].z);
                    if (j != cur) {
                        if (cur >= 0) flush(cur);
                        cur = j;
                    }
#pragma unroll
                    for (int v = 0; v < VPT; ++v) {
                        const int64_t vec = ct + (int64_t)v * consumers;
                        if (vec < nvec_bulk) {
                            fma_raw<T>(acc[v], a, raw[u][v]);
                        } else if (vec < nvec) {     // the ragged last chunk of the row comes straight from global memory
                            float x[V];
                            load_vec<T>(dY + (int64_t)max(row, 0) * ldy, vec * V, m, x);
#pragma unroll
                            for (int e = 0; e < V; ++e) acc[v][e] = fmaf(a, x[e], acc[v][e]);
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&s_empty[slot]);
            if (++slot == slots) { slot = 0; phase ^= 1u; }
        }
        if (ok && cur >= 0) flush(cur);
        if (!ok && lane == 0) raise_status(DEV_TIMEOUT);
    }
}

}  // namespace pamm
