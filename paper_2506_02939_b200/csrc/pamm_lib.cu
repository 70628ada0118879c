// C ABI of the PAMM sm_100a library: argument checks, kernel selection, launches.
// Every step of the path runs in the kernels included below; nothing here
// computes on the host apart from pamm_draw_indices_host.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <map>
#include <tuple>
#include <mutex>
#include <utility>
#include <vector>

#include "pamm_common.cuh"
#include "select.cuh"
#include "compress_simt.cuh"
#include "compress_umma.cuh"
#include "contract.cuh"
#include "contract_stream.cuh"
#include "weight_grad_simt.cuh"
#include "weight_grad_persist.cuh"
#include "weight_grad_chunked.cuh"
#include "weight_grad_planes.cuh"
#include "compress_pair.cuh"
#include "linear_forward.cuh"
#include "linear_forward_pair.cuh"
#include "small_k.cuh"
#include "read_probe.cuh"

using namespace pamm;

namespace pamm {
static thread_local char g_cuda_detail[256] = "";
void note_cuda_failure(const char* what, cudaError_t err) {
    snprintf(g_cuda_detail, sizeof g_cuda_detail, "%s: %s (%s)", what, cudaGetErrorName(err), cudaGetErrorString(err));
}

pamm_status tensor_map_failed() {
    const TmapFailure& f = last_tmap_failure();
    snprintf(g_cuda_detail, sizeof g_cuda_detail,
             "cuTensorMapEncodeTiled failed (CUresult %d; no driver entry point if 0) for a %llu x %llu matrix of %u-byte elements "
             "at %p, leading dimension %llu, boxes of %u rows",
             f.result, (unsigned long long)f.rows, (unsigned long long)f.cols, f.elem_bytes, f.base, (unsigned long long)f.ld,
             f.box_rows);
    return PAMM_ERR_CUDA;
}

bool ensure_dynamic_smem(const void* kernel, size_t bytes) {
    if (bytes <= 48 * 1024) return true;
    static std::mutex mu;
    static std::map<std::pair<int, const void*>, size_t> granted;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    std::lock_guard<std::mutex> lock(mu);
    size_t& have = granted[{dev, kernel}];
    if (have >= bytes) return true;
    const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e != cudaSuccess) {
        note_cuda_failure("cudaFuncSetAttribute(MaxDynamicSharedMemorySize)", e);
        cudaGetLastError();
        return false;
    }
    have = bytes;
    return true;
}

bool cta_pairs_can_launch(const void* kernel, int threads, size_t dynamic_smem) {
    if (!ensure_dynamic_smem(kernel, dynamic_smem)) return false;
    static std::mutex mu;
    static std::map<std::tuple<int, const void*, size_t>, bool> known;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    std::lock_guard<std::mutex> lock(mu);
    const auto key = std::make_tuple(dev, kernel, dynamic_smem);
    const auto it = known.find(key);
    if (it != known.end()) return it->second;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2);
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = dynamic_smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int clusters = 0;
    const cudaError_t e = cudaOccupancyMaxActiveClusters(&clusters, kernel, &cfg);
    if (e != cudaSuccess) cudaGetLastError();
    return known[key] = (e == cudaSuccess && clusters >= 1);
}
}  // namespace pamm

namespace {

inline size_t esize(pamm_dtype dt) { return dt == PAMM_BF16 ? 2 : 4; }
inline bool dtype_ok(pamm_dtype dt) { return dt == PAMM_F32 || dt == PAMM_BF16; }
inline bool layout_ok(pamm_layout l) { return l == PAMM_DW_NM || l == PAMM_DW_MN; }
inline bool index_type_ok(pamm_index_type t) { return t == PAMM_IDX_I32 || t == PAMM_IDX_U16 || t == PAMM_IDX_U8; }
inline size_t index_size(pamm_index_type t) { return t == PAMM_IDX_I32 ? 4 : t == PAMM_IDX_U16 ? 2 : 1; }
inline int64_t index_limit(pamm_index_type t) { return t == PAMM_IDX_I32 ? (1ll << 31) - 1 : t == PAMM_IDX_U16 ? 65536 : 256; }
inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline bool ld_ok(int64_t ld, int64_t cols, size_t es) { return ld >= cols && (ld * (int64_t)es) % 16 == 0; }
inline pamm_status launch_status() { return launch_result("kernel launch"); }
constexpr int64_t MAX_ROWS = (1ll << 31) - 1024;   // row ids, counts and offsets are int32

// Kernel launches issued so far (all streams), and optional event pairs that
// bracket the dominant kernel of a step so a benchmark can time it in place.
unsigned long long g_launches = 0;
cudaEvent_t g_prof[3][2] = {{nullptr, nullptr}, {nullptr, nullptr}, {nullptr, nullptr}};
inline void prof_begin(int kind, cudaStream_t st) { if (g_prof[kind][0]) cudaEventRecord(g_prof[kind][0], st); }
inline void prof_end(int kind, cudaStream_t st) { if (g_prof[kind][1]) cudaEventRecord(g_prof[kind][1], st); }

// Launch with or without the programmatic-serialization attribute.  With it, the
// kernel may begin while the previous kernel of the stream is still running and
// must call grid_dependency_wait() before it depends on that kernel.
template <typename... P, typename... A>
inline void launch(void (*kern)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool overlap_prev, A... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap_prev ? 1 : 0;
    cudaLaunchKernelEx(&cfg, kern, P(args)...);
    g_launches += 1;
}

int sm_count() {
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
            sms = 148;
    }
    return sms;
}

// The row partition shared by the compress pass and the counting sort of the backward pass.
inline int64_t sort_rows_per_block(int64_t b) { return compress_rows_per_cta(b, sm_count()); }
inline ContractWs contract_ws(void* base, int64_t b, int64_t m, int64_t k) {
    return contract_ws_layout(base, b, m, k, sort_rows_per_block(b));
}
// Bytes of the per-block histograms of f for one generator set (the "sort products").
inline size_t sort_products_bytes(int64_t b, int64_t k) {
    const int64_t rpb = sort_rows_per_block(b);
    return (size_t)round_up(((b + rpb - 1) / rpb) * k * 4, 256);
}

struct StepArena {
    char *X, *dY, *C, *dW, *Bt, *ws, *products;
    float *invnorm, *alpha;
    int32_t *idx, *f;
    int64_t ldx, ldy, ldc, ldw, ldb;
    size_t ws_bytes, bytes;
};

StepArena step_arena_layout(void* base, int64_t b, int64_t n, int64_t m, int64_t k, pamm_dtype dt) {
    StepArena a;
    const size_t es = esize(dt);
    const int64_t v = 16 / (int64_t)es;
    a.ldx = round_up(n, v); a.ldy = round_up(m, v); a.ldc = a.ldx;
    a.ldw = round_up(m, 4); a.ldb = a.ldw;
    char* p = (char*)base;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = (size_t)round_up((int64_t)(off + bytes), 256); return p ? p + o : (char*)0; };
    a.X = take((size_t)b * a.ldx * es);
    a.dY = take((size_t)b * a.ldy * es);
    a.C = take((size_t)k * a.ldc * es);
    a.invnorm = (float*)take((size_t)2 * k * 4);
    a.idx = (int32_t*)take((size_t)k * 4);
    a.f = (int32_t*)take((size_t)b * 4);
    a.alpha = (float*)take((size_t)b * 4);
    a.Bt = take((size_t)k * a.ldb * 4);
    a.dW = take((size_t)n * a.ldw * 4);
    a.ws_bytes = contract_ws(nullptr, b, m, k).bytes_with_planes;
    a.ws = take(a.ws_bytes);
    a.products = take(sort_products_bytes(b, k));
    a.bytes = off;
    return a;
}

template <typename T>
pamm_status launch_select(const void* X, int64_t ldx, int64_t b, int64_t n, int64_t k, uint64_t seed,
                          const int32_t* idx_in, int32_t* idx_out, void* C, int64_t ldc, float* c_invnorm,
                          cudaStream_t st, int32_t* zero_words = nullptr, int64_t zero_count = 0) {
    const size_t smem = (size_t)k * 4;
    if (!ensure_dynamic_smem((const void*)select_kernel<T>, smem)) return PAMM_ERR_CUDA;
    const PermKey pk = make_perm_key(seed, (uint32_t)b);
    const int grid = (int)k;
    launch(select_kernel<T>, dim3(grid), dim3(SEL_THREADS), smem, st, true, (const T*)X, ldx, b, n, (int)k, pk, idx_in,
           idx_out, (T*)C, ldc, c_invnorm, zero_words, zero_count);
    return launch_status();
}

// The neighbourhood condition (Eq. 2) applied or not: eps as given by the caller, the
// device counter of dropped rows (zeroed on the stream before the kernel).
struct Neighbourhood {
    bool on;
    float eps;
    int32_t* dropped;
};
constexpr Neighbourhood NO_NEIGHBOURHOOD = {false, 0.f, nullptr};

template <typename T>
pamm_status launch_compress_simt(const void* X, int64_t ldx, int64_t b, int64_t n, const void* C, int64_t ldc,
                                 int64_t k, const float* c_invnorm, void* f, int f_type, float* alpha,
                                 const Neighbourhood& nb, cudaStream_t st) {
    const int64_t want = (b + CS_WARPS - 1) / CS_WARPS;
    const int grid = (int)std::min<int64_t>(want, 148 * 8);
    const float eps2 = nb.eps * nb.eps, slack = neighbourhood_slack(n);
    auto kern = nb.on ? (k <= 4 ? compress_simt_kernel<T, 4, true> : compress_simt_kernel<T, 8, true>)
                      : (k <= 4 ? compress_simt_kernel<T, 4, false> : compress_simt_kernel<T, 8, false>);
    prof_begin(PAMM_PROF_COMPRESS, st);
    launch(kern, dim3(grid), dim3(CS_THREADS), 0, st, true, (const T*)X, ldx, b, n, (const T*)C, ldc, (int)k, c_invnorm, f,
           f_type, alpha, eps2, slack, nb.dropped);
    prof_end(PAMM_PROF_COMPRESS, st);
    return launch_status();
}

// Largest nb * nb * k (histogram words read by all scatter blocks together) for
// which every block rebuilds the scan on its own instead of a separate launch.
constexpr int64_t FUSED_SCAN_LIMIT = 1ll << 24;

// The counting sort of the rows by f.  `products` (the per-block histograms the compress
// pass left behind) saves the histogram launch.
pamm_status launch_sort(const void* f, int f_type, const float* alpha, int64_t b, int64_t k, const int32_t* products,
                        const ContractWs& w, cudaStream_t st) {
    if (k <= SK_MAX_K) products = nullptr;     // the forward pass for so few generators leaves no counts
    const size_t hsmem = (size_t)k * 4;
    const int rpb = (int)w.rows_per_block;
    const int tbl_warps = scatter_table_warps(rpb, k);
    const size_t ssmem = (size_t)(1 + tbl_warps) * k * 4;
    if (!ensure_dynamic_smem((const void*)contract_hist_kernel, hsmem) ||
        !ensure_dynamic_smem((const void*)contract_scatter_kernel, ssmem) ||
        !ensure_dynamic_smem((const void*)contract_scan_scatter_kernel, ssmem))
        return PAMM_ERR_CUDA;
    const bool fused_scan = w.nb * w.nb * k <= FUSED_SCAN_LIMIT;
    const int32_t* hist = w.hist;
    if (products && fused_scan) {
        hist = products;            // read in place
    } else if (products) {          // the scan below rewrites the table: work on a copy
        if (cudaMemcpyAsync(w.hist, products, (size_t)w.nb * k * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
            return PAMM_ERR_CUDA;
    } else {
        launch(contract_hist_kernel, dim3((unsigned)w.nb), dim3(SORT_BLK), hsmem, st, true, f, f_type, alpha, b, (int)k, rpb, w.hist);
    }
    if (fused_scan) {
        launch(contract_scan_scatter_kernel, dim3((unsigned)w.nb), dim3(SORT_BLK), ssmem, st, true, f, f_type, alpha, b, (int)k,
               rpb, tbl_warps, hist, (int)w.nb, w.seg_start, w.perm);
    } else {
        launch(contract_scan_kernel, dim3(1), dim3(SCAN_THREADS), 0, st, true, w.hist, (int)w.nb, (int)k, w.seg_start);
        launch(contract_scatter_kernel, dim3((unsigned)w.nb), dim3(SORT_BLK), ssmem, st, true, f, f_type, alpha, b, (int)k, rpb,
               tbl_warps, (const int32_t*)w.hist, (const int32_t*)w.seg_start, w.perm);
    }
    return launch_status();
}

template <typename T>
pamm_status launch_contract(const void* f, int f_type, const float* alpha, const void* dY, int64_t ldy, int64_t b,
                            int64_t m, int64_t k, float* Bt, int64_t ldb, const int32_t* products, const ContractWs& w,
                            cudaStream_t st, bool with_planes = false) {
    constexpr int V = Vec16<T>::N;
    uint16_t* planes = with_planes ? w.planes : nullptr;     // B~ also as bf16 hi / lo, for the product that follows
    pamm_status s = launch_sort(f, f_type, alpha, b, k, products, w, st);
    if (s != PAMM_OK) return s;
    if (contract_stream_supported(m, sizeof(T))) {
        // one balanced wave, two CTAs per SM: rows of dY stream through a shared-memory ring
        const ContractStreamPlan p = contract_stream_plan(m, sizeof(T));
        int64_t ranges = std::min<int64_t>(CT_MAX_CTAS, (int64_t)sm_count() * CS_CTAS_PER_SM);
        const int64_t rows_per_cta = std::max<int64_t>(32, (b + ranges - 1) / ranges);
        ranges = (b + rows_per_cta - 1) / rows_per_cta;
        auto kern = p.vpt == 4   ? contract_stream_kernel<T, 4, 1>
                    : p.vpt == 2 ? contract_stream_kernel<T, 2, 1>
                    : p.rps == 4 ? contract_stream_kernel<T, 1, 4>
                    : p.rps == 2 ? contract_stream_kernel<T, 1, 2>
                                 : contract_stream_kernel<T, 1, 1>;
        if (!ensure_dynamic_smem((const void*)kern, p.smem_bytes)) return PAMM_ERR_CUDA;
        prof_begin(PAMM_PROF_CONTRACT, st);
        launch(kern, dim3((unsigned)ranges), dim3(p.consumers + 32), p.smem_bytes, st, true, f, f_type, alpha, (const T*)dY,
               ldy, b, m, (int)k, (const int32_t*)w.seg_start, (const int32_t*)w.perm, (int)ranges, p.slots,
               p.row_pitch, p.bulk_bytes, w.partials, w.m_pad, Bt, ldb);
        prof_end(PAMM_PROF_CONTRACT, st);
        launch(contract_reduce_kernel, dim3((unsigned)((w.m_pad / 4 + RED_THREADS - 1) / RED_THREADS), (unsigned)std::min<int64_t>(k, 65535)), dim3(RED_THREADS), 0, st,
               true, (const float*)w.partials, w.m_pad, m, (int)k, b, (const int32_t*)w.seg_start, (int)ranges, Bt, ldb, planes, w.plane_ld);
        return launch_status();
    }
    // very wide rows: column slabs, register staging
    const int64_t vecs = (m + V - 1) / V;
    const int64_t slabs = (vecs + CT_MAX_THREADS - 1) / CT_MAX_THREADS;
    const int threads = (int)round_up((vecs + slabs - 1) / slabs, 32);
    int occ = 1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, contract_main_kernel<T>, threads, 0) != cudaSuccess || occ < 1)
        occ = 1;
    int64_t ranges = std::max<int64_t>(1, std::min<int64_t>(CT_MAX_CTAS, (int64_t)sm_count() * occ / slabs));
    const int64_t rows_per_cta = std::max<int64_t>(32, (b + ranges - 1) / ranges);
    ranges = (b + rows_per_cta - 1) / rows_per_cta;
    dim3 grid((unsigned)ranges, (unsigned)slabs);
    prof_begin(PAMM_PROF_CONTRACT, st);
    launch(contract_main_kernel<T>, grid, dim3(threads), 0, st, true, alpha, (const T*)dY, ldy, b, m, (int)k,
           (const int32_t*)w.seg_start, (const int32_t*)w.perm, (int)ranges, w.partials, w.m_pad, Bt, ldb);
    prof_end(PAMM_PROF_CONTRACT, st);
    launch(contract_reduce_kernel, dim3((unsigned)((w.m_pad / 4 + RED_THREADS - 1) / RED_THREADS), (unsigned)std::min<int64_t>(k, 65535)), dim3(RED_THREADS), 0, st, true,
           (const float*)w.partials, w.m_pad, m, (int)k, b, (const int32_t*)w.seg_start, (int)ranges, Bt, ldb, planes, w.plane_ld);
    return launch_status();
}

// How the weight gradient is stored.
struct DwSpec {
    void* ptr;
    int64_t ld;
    pamm_dtype dt;
    pamm_layout layout;
};

template <typename T>
pamm_status launch_weight_grad_simt(const void* C, int64_t ldc, int64_t k, int64_t n, const float* Bt, int64_t ldb,
                                    int64_t m, const DwSpec& dw, cudaStream_t st, int64_t b_rows,
                                    const int32_t* dropped, bool accumulate) {
    const bool swap = dw.layout == PAMM_DW_MN;
    const int64_t rows = swap ? m : n, cols = swap ? n : m;
    const int64_t items = rows * ((cols + 3) / 4);
    const dim3 grid((unsigned)((items + WG_THREADS - 1) / WG_THREADS)), block(WG_THREADS);
    prof_begin(PAMM_PROF_WEIGHT_GRAD, st);
    if (dw.dt == PAMM_F32) {
        auto kern = swap ? weight_grad_simt_kernel<T, float, true> : weight_grad_simt_kernel<T, float, false>;
        launch(kern, grid, block, 0, st, true, (const T*)C, ldc, (int)k, n, Bt, ldb, m, (float*)dw.ptr, dw.ld, b_rows, dropped,
               accumulate ? 1 : 0);
    } else {
        auto kern = swap ? weight_grad_simt_kernel<T, __nv_bfloat16, true> : weight_grad_simt_kernel<T, __nv_bfloat16, false>;
        launch(kern, grid, block, 0, st, true, (const T*)C, ldc, (int)k, n, Bt, ldb, m, (__nv_bfloat16*)dw.ptr, dw.ld, b_rows,
               dropped, accumulate ? 1 : 0);
    }
    prof_end(PAMM_PROF_WEIGHT_GRAD, st);
    return launch_status();
}

// ---- a handful of generators (k <= 8): three launches for the whole path ----
template <typename T>
pamm_status launch_small_forward(const void* X, int64_t ldx, int64_t b, int64_t n, int64_t k, uint64_t seed,
                                 const int32_t* idx_in, int32_t* idx_out, void* C, int64_t ldc, float* c_invnorm,
                                 void* f, int f_type, float* alpha, cudaStream_t st) {
    constexpr int V = Vec16<T>::N;
    const size_t smem = (size_t)k * round_up(n, V) * sizeof(T);
    if (!ensure_dynamic_smem((const void*)compress_small_kernel<T>, smem)) return PAMM_ERR_CUDA;
    // a row per warp while there are few rows; enough rows per CTA to pay for its copy of the generators otherwise
    const int64_t rows_per_cta = std::max<int64_t>(SK_WARPS, (b + 4 * sm_count() - 1) / (4 * sm_count()));
    const PermKey pk = make_perm_key(seed, (uint32_t)b);
    prof_begin(PAMM_PROF_COMPRESS, st);
    launch(compress_small_kernel<T>, dim3((unsigned)((b + rows_per_cta - 1) / rows_per_cta)), dim3(SK_THREADS), smem, st, true,
           (const T*)X, ldx, b, n, (int)k, pk, idx_in, idx_out, (T*)C, ldc, c_invnorm, f, f_type, alpha, (int)rows_per_cta);
    prof_end(PAMM_PROF_COMPRESS, st);
    return launch_status();
}

template <typename T, typename OutT>
void launch_wgrad_small(const void* C, int64_t ldc, int64_t k, int64_t n, const float* partials, int ranges, int64_t m_pad,
                        int64_t m, float* Bt, int64_t ldb, const DwSpec& dw, bool accumulate, cudaStream_t st) {
    const dim3 grid((unsigned)((m + SK_WG_COLS - 1) / SK_WG_COLS), (unsigned)((n + SK_WG_ROWS - 1) / SK_WG_ROWS));
    if (dw.layout == PAMM_DW_MN)
        launch(wgrad_small_kernel<T, OutT, true>, grid, dim3(SK_THREADS), 0, st, true, (const T*)C, ldc, (int)k, n, partials, ranges,
               m_pad, m, Bt, ldb, (OutT*)dw.ptr, dw.ld, accumulate ? 1 : 0);
    else
        launch(wgrad_small_kernel<T, OutT, false>, grid, dim3(SK_THREADS), 0, st, true, (const T*)C, ldc, (int)k, n, partials, ranges,
               m_pad, m, Bt, ldb, (OutT*)dw.ptr, dw.ld, accumulate ? 1 : 0);
}

template <typename T>
pamm_status launch_small_backward(const void* C, int64_t ldc, int64_t n, const void* f, int f_type, const float* alpha,
                                  const void* dY, int64_t ldy, int64_t b, int64_t m, int64_t k, float* Bt, int64_t ldb,
                                  const DwSpec& dw, const ContractWs& w, cudaStream_t st) {
    constexpr int V = Vec16<T>::N;
    // one partial B~ (k rows) per row range, in the workspace's partial rows
    int64_t ranges = std::max<int64_t>(1, std::min<int64_t>((b + 31) / 32, std::min<int64_t>(CT_MAX_CTAS / k, 2 * sm_count())));
    const int64_t rows_per_range = (b + ranges - 1) / ranges;
    ranges = (b + rows_per_range - 1) / rows_per_range;
    const int64_t vecs = (m + V - 1) / V;
    const int threads = (int)std::min<int64_t>(SK_CT_THREADS, round_up(vecs, 32));
    const int64_t slabs = (vecs + threads - 1) / threads;
    prof_begin(PAMM_PROF_CONTRACT, st);
    launch(contract_small_kernel<T>, dim3((unsigned)ranges, (unsigned)slabs), dim3(threads), 0, st, true, f, f_type, alpha,
           (const T*)dY, ldy, b, m, (int)k, (int)rows_per_range, w.partials, w.m_pad);
    prof_end(PAMM_PROF_CONTRACT, st);
    prof_begin(PAMM_PROF_WEIGHT_GRAD, st);
    if (dw.dt == PAMM_F32)
        launch_wgrad_small<T, float>(C, ldc, k, n, w.partials, (int)ranges, w.m_pad, m, Bt, ldb, dw, false, st);
    else
        launch_wgrad_small<T, __nv_bfloat16>(C, ldc, k, n, w.partials, (int)ranges, w.m_pad, m, Bt, ldb, dw, false, st);
    prof_end(PAMM_PROF_WEIGHT_GRAD, st);
    return launch_status();
}

pamm_status check_select(const void* X, int64_t ldx, int64_t b, int64_t n, pamm_dtype dt, int64_t k,
                         int32_t* idx_out, void* C, int64_t ldc, float* c_invnorm) {
    if (!dtype_ok(dt)) return PAMM_ERR_UNSUPPORTED;
    if (!X || !idx_out || !C || !c_invnorm) return PAMM_ERR_INVALID_ARG;
    if (b < 1 || n < 1 || k < 1 || k > b || b > MAX_ROWS) return PAMM_ERR_INVALID_ARG;
    if (!ld_ok(ldx, n, esize(dt)) || !ld_ok(ldc, n, esize(dt))) return PAMM_ERR_INVALID_ARG;
    if (!aligned(X, 16) || !aligned(C, 16) || !aligned(idx_out, 4) || !aligned(c_invnorm, 4)) return PAMM_ERR_INVALID_ARG;
    if (k > SEL_MAX_K) return PAMM_ERR_UNSUPPORTED;
    return PAMM_OK;
}

// The sort products are optional: no buffer, none written.
pamm_status check_products_out(const void* ws, size_t ws_bytes, int64_t b, int64_t k, int groups) {
    if (!ws) return PAMM_OK;
    if (!aligned(ws, 256) || ws_bytes < (size_t)groups * sort_products_bytes(b, k)) return PAMM_ERR_WORKSPACE;
    return PAMM_OK;
}

pamm_status check_compress(const void* X, int64_t ldx, int64_t b, int64_t n, pamm_dtype dt, const void* C,
                           int64_t ldc, int64_t k, const float* c_invnorm, void* f, pamm_index_type f_type, float* alpha) {
    if (!dtype_ok(dt) || !index_type_ok(f_type)) return PAMM_ERR_UNSUPPORTED;
    if (!X || !C || !c_invnorm || !f || !alpha) return PAMM_ERR_INVALID_ARG;
    if (b < 1 || n < 1 || k < 1 || k > b || b > MAX_ROWS) return PAMM_ERR_INVALID_ARG;
    if (k > index_limit(f_type)) return PAMM_ERR_INVALID_ARG;     // f_i would not fit its storage type
    if (!ld_ok(ldx, n, esize(dt)) || !ld_ok(ldc, n, esize(dt))) return PAMM_ERR_INVALID_ARG;
    if (!aligned(X, 16) || !aligned(C, 16) || !aligned(f, index_size(f_type)) || !aligned(alpha, 4) || !aligned(c_invnorm, 4))
        return PAMM_ERR_INVALID_ARG;
    return PAMM_OK;
}

pamm_status check_contract(const void* f, pamm_index_type f_type, const float* alpha, const void* dY, int64_t ldy,
                           int64_t b, int64_t m, pamm_dtype dt, int64_t k, const float* Bt, int64_t ldb, bool bt_required,
                           const void* products, const void* ws, size_t ws_bytes) {
    if (!dtype_ok(dt) || !index_type_ok(f_type)) return PAMM_ERR_UNSUPPORTED;
    if (!f || !alpha || !dY || (bt_required && !Bt)) return PAMM_ERR_INVALID_ARG;
    if (b < 1 || m < 1 || k < 1 || k > b || b > MAX_ROWS) return PAMM_ERR_INVALID_ARG;
    if (k > index_limit(f_type)) return PAMM_ERR_INVALID_ARG;
    if (!ld_ok(ldy, m, esize(dt)) || (Bt && !ld_ok(ldb, m, 4))) return PAMM_ERR_INVALID_ARG;
    if (!aligned(dY, 16) || (Bt && !aligned(Bt, 16)) || !aligned(f, index_size(f_type)) || !aligned(alpha, 4))
        return PAMM_ERR_INVALID_ARG;
    if (products && !aligned(products, 256)) return PAMM_ERR_INVALID_ARG;
    if (k > CT_MAX_K) return PAMM_ERR_UNSUPPORTED;
    if (!ws || !aligned(ws, 256)) return PAMM_ERR_WORKSPACE;
    if (ws_bytes < contract_ws(nullptr, b, m, k).bytes) return PAMM_ERR_WORKSPACE;
    return PAMM_OK;
}

pamm_status check_weight_grad(const void* C, int64_t ldc, int64_t k, int64_t n, pamm_dtype dt, const float* Bt,
                              int64_t ldb, int64_t m, const DwSpec& dw) {
    if (!dtype_ok(dt) || !dtype_ok(dw.dt) || !layout_ok(dw.layout)) return PAMM_ERR_UNSUPPORTED;
    if (!C || !Bt || !dw.ptr) return PAMM_ERR_INVALID_ARG;
    if (k < 1 || n < 1 || m < 1) return PAMM_ERR_INVALID_ARG;
    const int64_t out_cols = dw.layout == PAMM_DW_MN ? n : m;
    if (!ld_ok(ldc, n, esize(dt)) || !ld_ok(ldb, m, 4) || !ld_ok(dw.ld, out_cols, esize(dw.dt))) return PAMM_ERR_INVALID_ARG;
    if (!aligned(C, 16) || !aligned(Bt, 16) || !aligned(dw.ptr, 16)) return PAMM_ERR_INVALID_ARG;
    return PAMM_OK;
}

// x_is_ready: X was complete before the previous kernel of the stream started (true
// after our own select kernel), so the compress kernel may read it before that
// kernel has finished.  `groups` generator sets are served by one pass over X where the
// tensor-core kernel applies, else by one CUDA-core pass per set.  `products` (optional)
// receives the per-block histograms of f.
pamm_status do_compress(const void* X, int64_t ldx, int64_t b, int64_t n, pamm_dtype dt, const void* C, int64_t ldc,
                        int64_t k, int groups, const float* c_invnorm, void* f, pamm_index_type f_type, float* alpha,
                        int64_t out_stride, int32_t* products, bool x_is_ready, cudaStream_t st,
                        const Neighbourhood& nb = NO_NEIGHBOURHOOD) {
    if (dt == PAMM_BF16 && compress_umma_usable(b, n, k, groups, sm_count(), nb.on)) {
        const CompressOut out = {f, alpha, out_stride, products, (int64_t)(sort_products_bytes(b, k) / 4), (int)f_type};
        // many generators per chunk (tensor-bound): pairs of CTAs on one MMA tile; the same rows, results and counts
        const bool pairs = !nb.on && compress_pair_usable(b, n, k, groups, sm_count());
        prof_begin(PAMM_PROF_COMPRESS, st);
        const pamm_status s = pairs
            ? launch_compress_pair(X, ldx, b, n, C, ldc, k, groups, c_invnorm, out, sm_count(), x_is_ready, st)
            : launch_compress_umma(X, ldx, b, n, C, ldc, k, groups, c_invnorm, out, sm_count(), x_is_ready, st, nb.on, nb.eps,
                                   nb.dropped);
        prof_end(PAMM_PROF_COMPRESS, st);
        g_launches += 1;
        return s;
    }
    const size_t es = esize(dt), fs = index_size(f_type);
    const int64_t rpb = sort_rows_per_block(b), nblk = (b + rpb - 1) / rpb;
    if (products && !ensure_dynamic_smem((const void*)contract_hist_kernel, (size_t)k * 4)) return PAMM_ERR_CUDA;
    for (int g = 0; g < groups; ++g) {
        const char* Cg = (const char*)C + (size_t)g * k * ldc * es;
        void* fg = (char*)f + (size_t)g * out_stride * fs;
        float* ag = alpha + (size_t)g * out_stride;
        const pamm_status s = dt == PAMM_F32
            ? launch_compress_simt<float>(X, ldx, b, n, Cg, ldc, k, c_invnorm + (size_t)g * 2 * k, fg, (int)f_type, ag, nb, st)
            : launch_compress_simt<__nv_bfloat16>(X, ldx, b, n, Cg, ldc, k, c_invnorm + (size_t)g * 2 * k, fg, (int)f_type, ag, nb, st);
        if (s != PAMM_OK) return s;
        if (products)
            launch(contract_hist_kernel, dim3((unsigned)nblk), dim3(SORT_BLK), (size_t)k * 4, st, true, (const void*)fg,
                   (int)f_type, (const float*)ag, b, (int)k, (int)rpb, products + (size_t)g * (sort_products_bytes(b, k) / 4));
    }
    return launch_status();
}

pamm_status do_weight_grad(const void* C, int64_t ldc, int64_t k, int64_t n, pamm_dtype dt, const float* Bt,
                           int64_t ldb, int64_t m, const DwSpec& dw, cudaStream_t st, int64_t b_rows = 0,
                           const int32_t* dropped = nullptr, bool accumulate = false) {
    if (dt == PAMM_F32)
        return launch_weight_grad_simt<float>(C, ldc, k, n, Bt, ldb, m, dw, st, b_rows, dropped, accumulate);
    const bool bf16_out = dw.dt == PAMM_BF16, swap = dw.layout == PAMM_DW_MN;
    // the TMA stores need at least one whole 16-byte unit per output row
    const bool tma_ok = (swap ? n : m) * (int64_t)esize(dw.dt) >= 16;
    if (tma_ok && weight_grad_persist_supported(k, n, m)) {
        prof_begin(PAMM_PROF_WEIGHT_GRAD, st);
        const pamm_status s = launch_weight_grad_persist(C, ldc, k, n, Bt, ldb, m, dw.ptr, dw.ld, bf16_out, swap, sm_count(), st,
                                                          b_rows, dropped, accumulate);
        prof_end(PAMM_PROF_WEIGHT_GRAD, st);
        g_launches += 1;
        return s;
    }
    if (tma_ok && weight_grad_chunked_supported(k, n, m)) {
        prof_begin(PAMM_PROF_WEIGHT_GRAD, st);
        const pamm_status s = launch_weight_grad_chunked(C, ldc, k, n, Bt, ldb, m, dw.ptr, dw.ld, bf16_out, swap, sm_count(), st,
                                                         b_rows, dropped, accumulate);
        prof_end(PAMM_PROF_WEIGHT_GRAD, st);
        g_launches += 1;
        return s;
    }
    return launch_weight_grad_simt<__nv_bfloat16>(C, ldc, k, n, Bt, ldb, m, dw, st, b_rows, dropped, accumulate);
}

}  // namespace

// One CTA waits, with the library's bounded wait and a short limit, on a barrier that
// nothing will ever complete; the wait must give up, raise the status word and let the
// kernel end normally.
__global__ void selftest_bounded_wait_kernel(uint32_t polls) {
    __shared__ uint64_t s_bar;
    __shared__ int s_abort;
    if (threadIdx.x == 0) {
        ptx::mbar_init(&s_bar, 1);
        s_abort = 0;
        ptx::fence_barrier_init();
    }
    __syncthreads();
    volatile int* abort_flag = &s_abort;
    const bool done = ptx::mbar_wait(&s_bar, 0, abort_flag, polls);
    if (!done && (threadIdx.x & 31) == 0) raise_status(DEV_TIMEOUT);
}

extern "C" {

pamm_status pamm_selftest_bounded_wait(void* stream) {
    launch(selftest_bounded_wait_kernel, dim3(1), dim3(64), 0, (cudaStream_t)stream, false, (uint32_t)2048);
    return launch_status();
}

pamm_status pamm_probe_read(pamm_probe_kind kind, const void* base, int64_t rows, int64_t row_bytes, int64_t ld_bytes,
                            const int32_t* order, uint32_t* sum32, void* stream) {
    if (!base || !sum32 || rows < 1 || row_bytes < 16 || row_bytes % 16 || ld_bytes < row_bytes || ld_bytes % 16 ||
        !aligned(base, 16) || !aligned(sum32, 4) || rows > MAX_ROWS)
        return PAMM_ERR_INVALID_ARG;
    if (kind != PAMM_PROBE_SUM && kind != PAMM_PROBE_ROWS) return PAMM_ERR_INVALID_ARG;
    if (kind == PAMM_PROBE_SUM && order) return PAMM_ERR_INVALID_ARG;
    if (kind == PAMM_PROBE_ROWS && (row_bytes > 24576 || (order && !aligned(order, 4)))) return PAMM_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(sum32, 0, 4, st) != cudaSuccess) return PAMM_ERR_CUDA;
    if (kind == PAMM_PROBE_SUM) {
        const int64_t vecs = rows * (row_bytes / 16);
        const int64_t want = (vecs + RP_SUM_THREADS - 1) / RP_SUM_THREADS;
        const unsigned grid = (unsigned)std::max<int64_t>(1, std::min<int64_t>(want, (int64_t)sm_count() * 4));
        launch(read_probe_sum_kernel, dim3(grid), dim3(RP_SUM_THREADS), 0, st, false, (const uint8_t*)base, rows, row_bytes,
               ld_bytes, sum32);
        return launch_status();
    }
    const int pitch = (int)round_up(row_bytes, 128);
    const int slots = std::max(2, std::min(RP_MAX_SLOTS, RP_RING_BYTES / pitch));
    const size_t smem = 128 + (size_t)slots * pitch;
    if (!ensure_dynamic_smem((const void*)read_probe_rows_kernel, smem)) return PAMM_ERR_CUDA;
    const unsigned grid = (unsigned)std::max<int64_t>(1, std::min<int64_t>(rows, (int64_t)sm_count() * 2));
    launch(read_probe_rows_kernel, dim3(grid), dim3(RP_ROW_THREADS), smem, st, false, (const uint8_t*)base, rows,
           (uint32_t)row_bytes, ld_bytes, order, slots, pitch, sum32);
    return launch_status();
}

const char* pamm_status_string(pamm_status s) {
    switch (s) {
        case PAMM_OK: return "ok";
        case PAMM_ERR_INVALID_ARG: return "invalid argument";
        case PAMM_ERR_UNSUPPORTED: return "unsupported dtype or shape";
        case PAMM_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case PAMM_ERR_CUDA: return "CUDA error";
        case PAMM_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case PAMM_ERR_BAD_INDEX: return "index out of range or duplicated on the device";
    }
    return "unknown status";
}

int pamm_version(void) { return 200; }

const char* pamm_last_error_detail(void) { return g_cuda_detail; }

unsigned long long pamm_launch_count(void) { return g_launches; }

pamm_status pamm_set_profile_events(pamm_prof_kind kind, void* start_event, void* stop_event) {
    if ((int)kind < 0 || (int)kind > 2) return PAMM_ERR_INVALID_ARG;
    g_prof[kind][0] = (cudaEvent_t)start_event;
    g_prof[kind][1] = (cudaEvent_t)stop_event;
    return PAMM_OK;
}

size_t pamm_workspace_bytes(pamm_ws_kind kind, int64_t b, int64_t n, int64_t m, int64_t k, pamm_dtype dt) {
    if (!dtype_ok(dt) || b < 1 || k < 1 || k > b || b > MAX_ROWS) return (size_t)-1;
    switch (kind) {
        case PAMM_WS_COMPRESS:
            if (n < 1) return (size_t)-1;
            return sort_products_bytes(b, k);
        case PAMM_WS_CONTRACT:
            if (m < 1) return (size_t)-1;
            return contract_ws(nullptr, b, m, k).bytes_with_planes;     // pamm_contract itself needs less
        case PAMM_WS_STEP_HOST:
            if (n < 1 || m < 1) return (size_t)-1;
            return step_arena_layout(nullptr, b, n, m, k, dt).bytes;
    }
    return (size_t)-1;
}

pamm_status pamm_saved_bytes(int64_t b, int64_t n, int64_t k, pamm_dtype dt, pamm_index_type f_type, int64_t out[4]) {
    if (!dtype_ok(dt) || !index_type_ok(f_type)) return PAMM_ERR_UNSUPPORTED;
    if (!out || b < 1 || n < 1 || k < 1 || k > b || k > index_limit(f_type)) return PAMM_ERR_INVALID_ARG;
    const int64_t e = (int64_t)esize(dt);
    out[0] = b * n * e;                                             // X itself
    out[1] = k * n * e + b * (int64_t)index_size(f_type) + b * 4;   // C, f, alpha
    out[2] = b * n;                                                 // scalars, as the paper counts them
    out[3] = k * n + 2 * b;
    return PAMM_OK;
}

pamm_status pamm_draw_indices_host(int64_t b, int64_t k, uint64_t seed, int32_t* idx_out) {
    if (!idx_out || b < 1 || k < 1 || k > b || b > MAX_ROWS) return PAMM_ERR_INVALID_ARG;
    const PermKey pk = make_perm_key(seed, (uint32_t)b);
    for (int64_t j = 0; j < k; ++j) idx_out[j] = (int32_t)perm_apply(pk, (uint32_t)j);
    std::sort(idx_out, idx_out + k);
    return PAMM_OK;
}

pamm_status pamm_select_generators(const void* X, int64_t ldx, int64_t b, int64_t n, pamm_dtype dt, int64_t k,
                                   uint64_t seed, const int32_t* idx_in, int32_t* idx_out, void* C, int64_t ldc,
                                   float* c_invnorm, void* stream) {
    pamm_status s = check_select(X, ldx, b, n, dt, k, idx_out, C, ldc, c_invnorm);
    if (s != PAMM_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    return dt == PAMM_F32 ? launch_select<float>(X, ldx, b, n, k, seed, idx_in, idx_out, C, ldc, c_invnorm, st)
                          : launch_select<__nv_bfloat16>(X, ldx, b, n, k, seed, idx_in, idx_out, C, ldc, c_invnorm, st);
}

pamm_status pamm_compress(const void* X, int64_t ldx, int64_t b, int64_t n, pamm_dtype dt, const void* C, int64_t ldc,
                          int64_t k, const float* c_invnorm, void* f, pamm_index_type f_type, float* alpha,
                          void* workspace, size_t ws_bytes, void* stream) {
    pamm_status s = check_compress(X, ldx, b, n, dt, C, ldc, k, c_invnorm, f, f_type, alpha);
    if (s != PAMM_OK) return s;
    s = check_products_out(workspace, ws_bytes, b, k, 1);
    if (s != PAMM_OK) return s;
    return do_compress(X, ldx, b, n, dt, C, ldc, k, 1, c_invnorm, f, f_type, alpha, b, (int32_t*)workspace, false,
                       (cudaStream_t)stream);
}

pamm_status pamm_compress_projections(const void* X, int64_t ldx, int64_t b, int64_t n, pamm_dtype dt, const void* C,
                                      int64_t ldc, int64_t k, int64_t sets, const float* c_invnorm, void* f,
                                      pamm_index_type f_type, float* alpha, int64_t out_stride, void* workspace,
                                      size_t ws_bytes, void* stream) {
    pamm_status s = check_compress(X, ldx, b, n, dt, C, ldc, k, c_invnorm, f, f_type, alpha);
    if (s != PAMM_OK) return s;
    if (sets < 1 || sets > 64 || out_stride < b || (out_stride * (int64_t)index_size(f_type)) % 4) return PAMM_ERR_INVALID_ARG;
    s = check_products_out(workspace, ws_bytes, b, k, (int)sets);
    if (s != PAMM_OK) return s;
    return do_compress(X, ldx, b, n, dt, C, ldc, k, (int)sets, c_invnorm, f, f_type, alpha, out_stride, (int32_t*)workspace,
                       false, (cudaStream_t)stream);
}

pamm_status pamm_compress_fused(const void* X, int64_t ldx, int64_t b, int64_t n, pamm_dtype dt, int64_t k,
                                uint64_t seed, const int32_t* idx_in, int32_t* idx_out, void* C, int64_t ldc,
                                float* c_invnorm, void* f, pamm_index_type f_type, float* alpha, void* workspace,
                                size_t ws_bytes, void* stream) {
    pamm_status s = check_select(X, ldx, b, n, dt, k, idx_out, C, ldc, c_invnorm);
    if (s != PAMM_OK) return s;
    s = check_compress(X, ldx, b, n, dt, C, ldc, k, c_invnorm, f, f_type, alpha);
    if (s != PAMM_OK) return s;
    s = check_products_out(workspace, ws_bytes, b, k, 1);
    if (s != PAMM_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    // a handful of generators: selection and compression in one launch, generator rows kept in shared memory
    if (dt == PAMM_F32 && small_k_compress_supported<float>(n, k))
        return launch_small_forward<float>(X, ldx, b, n, k, seed, idx_in, idx_out, C, ldc, c_invnorm, f, (int)f_type, alpha, st);
    if (dt == PAMM_BF16 && small_k_compress_supported<__nv_bfloat16>(n, k))
        return launch_small_forward<__nv_bfloat16>(X, ldx, b, n, k, seed, idx_in, idx_out, C, ldc, c_invnorm, f, (int)f_type,
                                                   alpha, st);
    s = dt == PAMM_F32 ? launch_select<float>(X, ldx, b, n, k, seed, idx_in, idx_out, C, ldc, c_invnorm, st)
                       : launch_select<__nv_bfloat16>(X, ldx, b, n, k, seed, idx_in, idx_out, C, ldc, c_invnorm, st);
    if (s != PAMM_OK) return s;
    return do_compress(X, ldx, b, n, dt, C, ldc, k, 1, c_invnorm, f, f_type, alpha, b, (int32_t*)workspace, true, st);
}

pamm_status pamm_linear_forward(const void* X, int64_t ldx, int64_t b, int64_t n, const void* W, int64_t ldw, int64_t m,
                                pamm_dtype dt, int64_t k, uint64_t seed, const int32_t* idx_in, int32_t* idx_out,
                                void* C, int64_t ldc, float* c_invnorm, void* Z, int64_t ldz, void* f,
                                pamm_index_type f_type, float* alpha, void* workspace, size_t ws_bytes, void* stream) {
    if (!dtype_ok(dt)) return PAMM_ERR_UNSUPPORTED;
    if (!X || !W || !Z || b < 1 || n < 1 || m < 1 || k < 0 || b > MAX_ROWS) return PAMM_ERR_INVALID_ARG;
    if (!ld_ok(ldx, n, esize(dt)) || !ld_ok(ldw, m, esize(dt)) || !ld_ok(ldz, m, esize(dt))) return PAMM_ERR_INVALID_ARG;
    if (!aligned(X, 16) || !aligned(W, 16) || !aligned(Z, 16)) return PAMM_ERR_INVALID_ARG;
    pamm_status s = PAMM_OK;
    if (k > 0) {
        s = check_select(X, ldx, b, n, dt, k, idx_out, C, ldc, c_invnorm);
        if (s != PAMM_OK) return s;
        s = check_compress(X, ldx, b, n, dt, C, ldc, k, c_invnorm, f, f_type, alpha);
        if (s != PAMM_OK) return s;
        s = check_products_out(workspace, ws_bytes, b, k, 1);
        if (s != PAMM_OK) return s;
    }
    // the tensor-core kernel is the only implementation: no CUDA-core or library GEMM stands in for it
    if (dt != PAMM_BF16 || !linear_forward_supported(b, n, m, k) ||
        linear_forward_plan_for(b, m, k, sm_count()).stages < 2)
        return PAMM_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    const int64_t rpb = sort_rows_per_block(b);
    int32_t* hist = k > 0 ? (int32_t*)workspace : nullptr;
    if (k > 0) {
        s = launch_select<__nv_bfloat16>(X, ldx, b, n, k, seed, idx_in, idx_out, C, ldc, c_invnorm, st, hist,
                                         hist ? ((b + rpb - 1) / rpb) * k : 0);
        if (s != PAMM_OK) return s;
    }
    const LinearForwardOut out = {f, alpha, hist, (int)rpb, (int)f_type};
    // pairs of CTAs on one 256-row tile wherever there are at least 256 rows; else one CTA per 128-row tile
    const LinearForwardPlan pp = linear_forward_pair_plan_for(b, m, k, sm_count());
    const bool pairs = b >= LP_PAIR_M && sm_count() >= 2 && pp.stages >= 2 &&
                       cta_pairs_can_launch((const void*)linear_forward_pair_kernel, LF_THREADS, pp.smem_bytes);
    prof_begin(PAMM_PROF_COMPRESS, st);
    s = pairs ? launch_linear_forward_pair(X, ldx, b, n, W, ldw, m, C, ldc, k, c_invnorm, Z, ldz, out, sm_count(), st)
              : launch_linear_forward(X, ldx, b, n, W, ldw, m, C, ldc, k, c_invnorm, Z, ldz, out, sm_count(), st);
    prof_end(PAMM_PROF_COMPRESS, st);
    g_launches += 1;
    return s;
}

pamm_status pamm_linear_backward_input(const void* dZ, int64_t lddz, int64_t b, int64_t m, const void* W, int64_t ldw,
                                       int64_t n, pamm_dtype dt, void* dX, int64_t lddx, void* stream) {
    if (!dtype_ok(dt)) return PAMM_ERR_UNSUPPORTED;
    if (!dZ || !W || !dX || b < 1 || n < 1 || m < 1 || b > MAX_ROWS) return PAMM_ERR_INVALID_ARG;
    if (!ld_ok(lddz, m, esize(dt)) || !ld_ok(ldw, m, esize(dt)) || !ld_ok(lddx, n, esize(dt))) return PAMM_ERR_INVALID_ARG;
    if (!aligned(dZ, 16) || !aligned(W, 16) || !aligned(dX, 16)) return PAMM_ERR_INVALID_ARG;
    // the forward kernel with the roles renamed: rows of dZ, contraction over m, n output columns, W as columns x hidden
    if (dt != PAMM_BF16 || !linear_forward_supported(b, m, n, 0) || linear_forward_plan_for(b, n, 0, sm_count()).stages < 2)
        return PAMM_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    const LinearForwardOut out = {nullptr, nullptr, nullptr, 1, (int)PAMM_IDX_I32};
    const LinearForwardPlan pp = linear_forward_pair_plan_for(b, n, 0, sm_count());
    const bool pairs = b >= LP_PAIR_M && sm_count() >= 2 && pp.stages >= 2 &&
                       cta_pairs_can_launch((const void*)linear_forward_pair_kernel, LF_THREADS, pp.smem_bytes);
    const pamm_status s = pairs
        ? launch_linear_forward_pair(dZ, lddz, b, m, W, ldw, n, nullptr, 0, 0, nullptr, dX, lddx, out, sm_count(), st, true)
        : launch_linear_forward(dZ, lddz, b, m, W, ldw, n, nullptr, 0, 0, nullptr, dX, lddx, out, sm_count(), st, true);
    g_launches += 1;
    return s;
}

pamm_status pamm_contract(const void* f, pamm_index_type f_type, const float* alpha, const void* dY, int64_t ldy,
                          int64_t b, int64_t m, pamm_dtype dt, int64_t k, float* Btilde, int64_t ldb,
                          const void* sort_products, void* workspace, size_t ws_bytes, void* stream) {
    pamm_status s = check_contract(f, f_type, alpha, dY, ldy, b, m, dt, k, Btilde, ldb, true, sort_products, workspace, ws_bytes);
    if (s != PAMM_OK) return s;
    const ContractWs w = contract_ws(workspace, b, m, k);
    cudaStream_t st = (cudaStream_t)stream;
    const int32_t* pr = (const int32_t*)sort_products;
    return dt == PAMM_F32 ? launch_contract<float>(f, (int)f_type, alpha, dY, ldy, b, m, k, Btilde, ldb, pr, w, st)
                          : launch_contract<__nv_bfloat16>(f, (int)f_type, alpha, dY, ldy, b, m, k, Btilde, ldb, pr, w, st);
}

pamm_status pamm_weight_grad(const void* C, int64_t ldc, int64_t k, int64_t n, pamm_dtype dt, const float* Btilde,
                             int64_t ldb, int64_t m, void* dW, int64_t ldw, pamm_dtype dw_dt, pamm_layout layout,
                             void* stream) {
    const DwSpec dw = {dW, ldw, dw_dt, layout};
    pamm_status s = check_weight_grad(C, ldc, k, n, dt, Btilde, ldb, m, dw);
    if (s != PAMM_OK) return s;
    return do_weight_grad(C, ldc, k, n, dt, Btilde, ldb, m, dw, (cudaStream_t)stream);
}

pamm_status pamm_compress_eps(const void* X, int64_t ldx, int64_t b, int64_t n, pamm_dtype dt, const void* C,
                              int64_t ldc, int64_t k, const float* c_invnorm, float eps, void* f,
                              pamm_index_type f_type, float* alpha, int32_t* dropped, void* workspace, size_t ws_bytes,
                              void* stream) {
    pamm_status s = check_compress(X, ldx, b, n, dt, C, ldc, k, c_invnorm, f, f_type, alpha);
    if (s != PAMM_OK) return s;
    if (!dropped || !aligned(dropped, 4) || !(eps >= 0.f)) return PAMM_ERR_INVALID_ARG;     // also rejects NaN
    s = check_products_out(workspace, ws_bytes, b, k, 1);
    if (s != PAMM_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(dropped, 0, sizeof(int32_t), st) != cudaSuccess) return PAMM_ERR_CUDA;
    // ||X_i - alpha C_f|| <= ||X_i|| always, so eps >= 1 keeps every row: the plain kernel does
    const bool on = eps < 1.f;
    return do_compress(X, ldx, b, n, dt, C, ldc, k, 1, c_invnorm, f, f_type, alpha, b, (int32_t*)workspace, false, st,
                       Neighbourhood{on, eps, dropped});
}

pamm_status pamm_weight_grad_beta(const void* C, int64_t ldc, int64_t k, int64_t n, pamm_dtype dt, const float* Btilde,
                                  int64_t ldb, int64_t m, int64_t b, const int32_t* dropped, void* dW, int64_t ldw,
                                  pamm_dtype dw_dt, pamm_layout layout, void* stream) {
    const DwSpec dw = {dW, ldw, dw_dt, layout};
    pamm_status s = check_weight_grad(C, ldc, k, n, dt, Btilde, ldb, m, dw);
    if (s != PAMM_OK) return s;
    if (b < 1 || (dropped && !aligned(dropped, 4))) return PAMM_ERR_INVALID_ARG;
    return do_weight_grad(C, ldc, k, n, dt, Btilde, ldb, m, dw, (cudaStream_t)stream, b, dropped);
}

pamm_status pamm_weight_grad_accumulate(const void* C, int64_t ldc, int64_t k, int64_t n, pamm_dtype dt,
                                        const float* Btilde, int64_t ldb, int64_t m, float* dW, int64_t ldw,
                                        pamm_layout layout, void* stream) {
    const DwSpec dw = {dW, ldw, PAMM_F32, layout};
    pamm_status s = check_weight_grad(C, ldc, k, n, dt, Btilde, ldb, m, dw);
    if (s != PAMM_OK) return s;
    return do_weight_grad(C, ldc, k, n, dt, Btilde, ldb, m, dw, (cudaStream_t)stream, 0, nullptr, true);
}

pamm_status pamm_contract_weight_grad(const void* C, int64_t ldc, int64_t n, const void* f, pamm_index_type f_type,
                                      const float* alpha, const void* dY, int64_t ldy, int64_t b, int64_t m,
                                      pamm_dtype dt, int64_t k, float* Btilde, int64_t ldb, void* dW, int64_t ldw,
                                      pamm_dtype dw_dt, pamm_layout layout, const void* sort_products, void* workspace,
                                      size_t ws_bytes, void* stream) {
    pamm_status s = check_contract(f, f_type, alpha, dY, ldy, b, m, dt, k, Btilde, ldb, false, sort_products, workspace, ws_bytes);
    if (s != PAMM_OK) return s;
    const ContractWs w = contract_ws(workspace, b, m, k);
    float* Bt = Btilde ? Btilde : w.btilde;
    const int64_t ldbt = Btilde ? ldb : w.m_pad;
    const DwSpec dw = {dW, ldw, dw_dt, layout};
    s = check_weight_grad(C, ldc, k, n, dt, Bt, ldbt, m, dw);
    if (s != PAMM_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    if (k <= SK_MAX_K)      // a handful of generators: no sort, two launches (the caller's B~, if any, is still filled)
        return dt == PAMM_F32
            ? launch_small_backward<float>(C, ldc, n, f, (int)f_type, alpha, dY, ldy, b, m, k, Btilde, ldb, dw, w, st)
            : launch_small_backward<__nv_bfloat16>(C, ldc, n, f, (int)f_type, alpha, dY, ldy, b, m, k, Btilde, ldb, dw, w, st);
    const int32_t* pr = (const int32_t*)sort_products;
    // Many generators: the reduction also leaves B~ split into bf16 hi / lo planes and the product takes all its
    // operands by TMA (a workspace of the size pamm_workspace_bytes gives has room for the planes).
    const bool swap = layout == PAMM_DW_MN;
    const bool planes = dt == PAMM_BF16 && ws_bytes >= w.bytes_with_planes && !weight_grad_persist_supported(k, n, m) &&
                        weight_grad_chunked_supported(k, n, m) && (swap ? n : m) * (int64_t)esize(dw_dt) >= 16;
    s = dt == PAMM_F32 ? launch_contract<float>(f, (int)f_type, alpha, dY, ldy, b, m, k, Bt, ldbt, pr, w, st)
                       : launch_contract<__nv_bfloat16>(f, (int)f_type, alpha, dY, ldy, b, m, k, Bt, ldbt, pr, w, st, planes);
    if (s != PAMM_OK) return s;
    if (planes) {
        prof_begin(PAMM_PROF_WEIGHT_GRAD, st);
        s = launch_weight_grad_planes(C, ldc, k, n, w.planes, w.plane_ld, m, dW, ldw, dw_dt == PAMM_BF16, swap, sm_count(), st);
        prof_end(PAMM_PROF_WEIGHT_GRAD, st);
        g_launches += 1;
        return s;
    }
    return do_weight_grad(C, ldc, k, n, dt, Bt, ldbt, m, dw, st);
}

pamm_status pamm_qkv_step_host(const void* X_host, const void* dY_host, int64_t b, int64_t n, int64_t m,
                               pamm_dtype dt, int64_t k, uint64_t seed, float* dW_host, int32_t* f_host,
                               float* alpha_host, void* arena, size_t arena_bytes, void* stream) {
    if (!dtype_ok(dt)) return PAMM_ERR_UNSUPPORTED;
    if (!X_host || !dY_host || !dW_host) return PAMM_ERR_INVALID_ARG;
    if (b < 1 || n < 1 || m < 1 || k < 1 || k > b || b > MAX_ROWS) return PAMM_ERR_INVALID_ARG;
    if (k > SEL_MAX_K) return PAMM_ERR_UNSUPPORTED;
    if (!arena || !aligned(arena, 256)) return PAMM_ERR_WORKSPACE;
    const StepArena a = step_arena_layout(arena, b, n, m, k, dt);
    if (arena_bytes < a.bytes) return PAMM_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t es = esize(dt);
    if (cudaMemcpy2DAsync(a.X, a.ldx * es, X_host, n * es, n * es, b, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpy2DAsync(a.dY, a.ldy * es, dY_host, m * es, m * es, b, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return PAMM_ERR_CUDA;
    pamm_status s = pamm_compress_fused(a.X, a.ldx, b, n, dt, k, seed, nullptr, a.idx, a.C, a.ldc, a.invnorm, a.f,
                                        PAMM_IDX_I32, a.alpha, a.products, sort_products_bytes(b, k), stream);
    if (s != PAMM_OK) return s;
    s = pamm_contract_weight_grad(a.C, a.ldc, n, a.f, PAMM_IDX_I32, a.alpha, a.dY, a.ldy, b, m, dt, k, (float*)a.Bt, a.ldb,
                                  a.dW, a.ldw, PAMM_F32, PAMM_DW_NM, a.products, a.ws, a.ws_bytes, stream);
    if (s != PAMM_OK) return s;
    if (cudaMemcpy2DAsync(dW_host, m * 4, a.dW, a.ldw * 4, m * 4, n, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return PAMM_ERR_CUDA;
    if (f_host && cudaMemcpyAsync(f_host, a.f, (size_t)b * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return PAMM_ERR_CUDA;
    if (alpha_host && cudaMemcpyAsync(alpha_host, a.alpha, (size_t)b * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return PAMM_ERR_CUDA;
    return PAMM_OK;
}

// One small pinned host word and one private stream per device carry the status word
// to the host without touching the caller's streams.
namespace {
struct StatusReader {
    cudaStream_t stream = nullptr;
    int* host_word = nullptr;
    int* dev_word = nullptr;
};
StatusReader g_status_reader[64];
std::mutex g_status_mutex;
}  // namespace

pamm_status pamm_last_device_status(void* stream) {
    (void)stream;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return PAMM_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_status_mutex);
    StatusReader& r = g_status_reader[dev];
    if (!r.stream) {
        void* sym = nullptr;
        if (cudaGetSymbolAddress(&sym, g_status_word) != cudaSuccess || !sym) return PAMM_ERR_CUDA;
        if (cudaHostAlloc((void**)&r.host_word, sizeof(int), cudaHostAllocDefault) != cudaSuccess) return PAMM_ERR_CUDA;
        if (cudaStreamCreateWithFlags(&r.stream, cudaStreamNonBlocking) != cudaSuccess) {
            cudaFreeHost(r.host_word);
            r.host_word = nullptr;
            r.stream = nullptr;
            return PAMM_ERR_CUDA;
        }
        r.dev_word = (int*)sym;
    }
    // a copy on the private stream: it waits for no kernel and blocks no stream of the caller
    if (cudaMemcpyAsync(r.host_word, r.dev_word, sizeof(int), cudaMemcpyDeviceToHost, r.stream) != cudaSuccess ||
        cudaStreamSynchronize(r.stream) != cudaSuccess)
        return PAMM_ERR_CUDA;
    const int word = *r.host_word;
    if (word) {
        if (cudaMemsetAsync(r.dev_word, 0, sizeof(int), r.stream) != cudaSuccess ||
            cudaStreamSynchronize(r.stream) != cudaSuccess)
            return PAMM_ERR_CUDA;
    }
    if (word & DEV_TIMEOUT) return PAMM_ERR_TIMEOUT;
    if (word & DEV_BAD_INDEX) return PAMM_ERR_BAD_INDEX;
    return PAMM_OK;
}

}  // extern "C"

// ---- scratch of pamm_contract_no_alloc -----------------------------------------
// Lives in the library image, one copy per device that loads it.  In host code
// the name below is only a stand-in for the symbol: the device address has to be
// asked for with cudaGetSymbolAddress, once per device, with that device current.
static __device__ __align__(256) unsigned char g_no_alloc_scratch[PAMM_NO_ALLOC_SCRATCH_BYTES];

namespace {
constexpr int NO_ALLOC_MAX_DEVICES = 64;
void* g_no_alloc_ptr[NO_ALLOC_MAX_DEVICES] = {};
std::mutex g_no_alloc_mutex;

// Device address of the fixed scratch on the current device (nullptr on failure).
void* no_alloc_scratch_ptr() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NO_ALLOC_MAX_DEVICES) return nullptr;
    std::lock_guard<std::mutex> lock(g_no_alloc_mutex);
    if (!g_no_alloc_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_no_alloc_scratch) != cudaSuccess || !p) return nullptr;
        g_no_alloc_ptr[dev] = p;
    }
    return g_no_alloc_ptr[dev];
}
}  // namespace

extern "C" pamm_status pamm_contract_no_alloc(const int32_t* f, const float* alpha, const void* dY, int64_t ldy,
                                              int64_t b, int64_t m, pamm_dtype dt, int64_t k, float* Btilde,
                                              int64_t ldb, void* stream) {
    // sizes first: the fixed array is the only scratch there is
    if (!dtype_ok(dt)) return PAMM_ERR_UNSUPPORTED;
    if (b < 1 || m < 1 || k < 1 || k > b || b > MAX_ROWS) return PAMM_ERR_INVALID_ARG;
    if (contract_ws(nullptr, b, m, k).bytes > (size_t)PAMM_NO_ALLOC_SCRATCH_BYTES) return PAMM_ERR_WORKSPACE;
    void* scratch = no_alloc_scratch_ptr();
    if (!scratch) return PAMM_ERR_CUDA;
    pamm_status s = check_contract(f, PAMM_IDX_I32, alpha, dY, ldy, b, m, dt, k, Btilde, ldb, true, nullptr, scratch,
                                   (size_t)PAMM_NO_ALLOC_SCRATCH_BYTES);
    if (s != PAMM_OK) return s;
    const ContractWs w = contract_ws(scratch, b, m, k);
    cudaStream_t st = (cudaStream_t)stream;
    return dt == PAMM_F32
        ? launch_contract<float>(f, PAMM_IDX_I32, alpha, dY, ldy, b, m, k, Btilde, ldb, nullptr, w, st)
        : launch_contract<__nv_bfloat16>(f, PAMM_IDX_I32, alpha, dY, ldy, b, m, k, Btilde, ldb, nullptr, w, st);
}
