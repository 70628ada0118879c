/*
 * pamm.h -- C ABI of the B200 (sm_100a) library for the hot path of
 * Point-Approximate Matrix Multiplication (PAMM) on one fused Q|K|V layer.
 *
 * Notation follows the paper: A = X is the saved layer input (b tokens x n
 * hidden), B = dY = [dQ|dK|dV] is the upstream gradient (b x m), C holds k
 * generator rows of X, f in [0,k)^b assigns every row to a generator, alpha in
 * R^b scales it, B~ (k x m) is the contracted gradient and dW~ = C^T B~ (n x m)
 * approximates X^T dY.  epsilon = infinity (the paper's chosen setting, Section
 * 4.1: no row is dropped, beta = 1) except in pamm_compress_eps /
 * pamm_weight_grad_beta, which add the neighbourhood condition and beta.
 *
 * Conventions for every entry point unless its comment says otherwise:
 *  - Matrices are row-major with a leading dimension given in ELEMENTS.
 *  - All matrix / vector pointers are DEVICE pointers owned by the caller.  The
 *    library never allocates or frees device memory; scratch comes from the
 *    caller as `workspace` (size from pamm_workspace_bytes).
 *  - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Calls
 *    only enqueue work; they never synchronise the host.
 *  - Base pointers of X, dY, C, B~, dW must be 16-byte aligned and leading
 *    dimensions must make every row start 16-byte aligned (ld * element size a
 *    multiple of 16).  f, alpha, index arrays need 4-byte alignment, the
 *    workspace 256-byte alignment.
 *  - Argument errors (NULL, b < 1, k < 1, k > b, ld < columns, misalignment,
 *    workspace too small, sizes over the documented limits) are reported
 *    synchronously with nothing launched.  Unsupported dtype/shape
 *    combinations return PAMM_ERR_UNSUPPORTED; there is no CPU fallback.
 *  - Problems only the device can see (a generator index out of range, a
 *    duplicated index, an assignment f_i outside [0,k), a bounded wait that ran
 *    out) never trap: the kernel skips the access, ORs a bit into a status
 *    word and finishes.  There is ONE word per device, shared by every stream
 *    (two streams cannot tell their errors apart); read it with
 *    pamm_last_device_status after synchronising the work you ask about.
 *  - Outputs are fully overwritten.  Results are deterministic: the same
 *    inputs give bit-identical outputs from run to run.
 */
#ifndef PAMM_H_
#define PAMM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PAMM_OK = 0,
    PAMM_ERR_INVALID_ARG = 1,
    PAMM_ERR_UNSUPPORTED = 2,
    PAMM_ERR_WORKSPACE = 3,
    PAMM_ERR_CUDA = 4,
    PAMM_ERR_TIMEOUT = 5,      /* a bounded device-side wait gave up            */
    PAMM_ERR_BAD_INDEX = 6     /* device saw an out-of-range / duplicate index  */
} pamm_status;

typedef enum { PAMM_F32 = 0, PAMM_BF16 = 1 } pamm_dtype;

/* Layout of the weight gradient.  The paper writes O~ = C^T B~ as n x m (hidden
 * x outputs, Section 3.1); a framework's linear layer usually keeps its weight
 * as out x in, i.e. m x n. */
typedef enum { PAMM_DW_NM = 0, PAMM_DW_MN = 1 } pamm_layout;

/* Storage type of the assignment f (Appendix "Complexity Analysis" counts b
 * scalars for it; with k <= 256 or k <= 65536 generators a byte or two suffice).
 * Values are 0-based generator indices, unsigned for the narrow types. */
typedef enum { PAMM_IDX_I32 = 0, PAMM_IDX_U16 = 1, PAMM_IDX_U8 = 2 } pamm_index_type;

/* Which scratch size is asked for. */
typedef enum {
    PAMM_WS_COMPRESS = 0,            /* sort products pamm_compress_fused leaves for the backward pass */
    PAMM_WS_CONTRACT = 1,            /* also covers pamm_contract_weight_grad */
    PAMM_WS_STEP_HOST = 2            /* device arena of pamm_qkv_step_host    */
} pamm_ws_kind;

/* Human-readable name of a status code (static string, never NULL). */
const char* pamm_status_string(pamm_status s);

/* Which CUDA call was behind the calling thread's last PAMM_ERR_CUDA, and the runtime's
 * name for the failure ("" if there was none).  The string belongs to the library. */
const char* pamm_last_error_detail(void);

/* Bytes of 256-byte-aligned device scratch the named call needs for these
 * sizes (0 is a valid answer).  Returns (size_t)-1 for invalid sizes. */
size_t pamm_workspace_bytes(pamm_ws_kind kind, int64_t b, int64_t n, int64_t m, int64_t k, pamm_dtype dt);

/*
 * Generator sampling on the host (Algorithm 1, "Sample indices I subset [b]
 * uniformly without replacement, |I| = k").  The paper fixes no generator, so
 * this library defines one: I = sort({pi_seed(0), ..., pi_seed(k-1)}) where
 * pi_seed is a keyed pseudo-random permutation of [0,b) (a 6-round Feistel
 * network on the smallest even-width power of two >= b, cycle-walked into
 * range).  A pure function of (b, k, seed); the device path draws the same set.
 * idx_out: HOST array of k int32, ascending.  No GPU is touched.
 */
pamm_status pamm_draw_indices_host(int64_t b, int64_t k, uint64_t seed, int32_t* idx_out);

/*
 * Step 1 -- choose generators (Algorithm 1, Compress: the index sampling, the gather of C,
 * and the norms eta_C of the generator rows).
 *   X        b x n, dtype dt, leading dimension ldx
 *   idx_in   NULL: draw I from `seed` as pamm_draw_indices_host does (ascending);
 *            else k caller-chosen row indices, used in the given order.  They
 *            are checked on the device: an index outside [0,b) is clamped and a
 *            repeated index is kept, both raising PAMM_ERR_BAD_INDEX in the
 *            status word.
 *   idx_out  k int32: the indices used
 *   C        k x n, dtype dt, leading dimension ldc: exact copies of the rows
 *   c_invnorm  2k fp32: [0,k) = 1/||C_j||, [k,2k) = 1/||C_j||^2; both 0 for a
 *            zero row (such a generator scores 0 and yields alpha = 0)
 * Limit: k <= 49152.
 */
pamm_status pamm_select_generators(const void* X, int64_t ldx, int64_t b, int64_t n, pamm_dtype dt,
                                   int64_t k, uint64_t seed, const int32_t* idx_in,
                                   int32_t* idx_out, void* C, int64_t ldc, float* c_invnorm,
                                   void* stream);

/*
 * Step 2 -- compress (Section 3.2 "Compressing A", Eq. 1, Lemma 1; Algorithm 1,
 * Compress: cosine similarities, assignment, scales).  One streaming pass over X:
 *   S = X C^T;  f_i = the lowest j maximising |S_ij| / ||C_j||  (equivalently
 *   |csim(X_i, C_j)|, Lemma 1);  alpha_i = S_{i,f_i} / ||C_{f_i}||^2  (Eq. 1).
 * Products are exact, sums are accumulated in fp32.  A zero row gets f = 0,
 * alpha = 0.
 *   f      b entries of f_type, 0-based (k must fit the type: PAMM_ERR_INVALID_ARG otherwise)
 *   alpha  b fp32
 *   workspace  NULL, or pamm_workspace_bytes(PAMM_WS_COMPRESS, ...) bytes that receive
 *          the "sort products": how many rows of every block of rows chose each
 *          generator, counted on the fly by the pass over the rows whose alpha is not
 *          zero (a row with alpha = 0 adds nothing to B~ and the backward pass leaves it
 *          out of its sorted order, so dY of such a row is never read).  They are an optional by-product
 *          for the backward pass (pamm_contract, pamm_contract_weight_grad), which then
 *          skips its own counting launch; they must be kept next to f until then and
 *          are valid only for this f on a device with the same number of SMs.  With
 *          k <= 8 the backward pass does not sort at all: the argument is then ignored by
 *          both sides and the buffer may be left untouched.
 */
pamm_status pamm_compress(const void* X, int64_t ldx, int64_t b, int64_t n, pamm_dtype dt,
                          const void* C, int64_t ldc, int64_t k, const float* c_invnorm,
                          void* f, pamm_index_type f_type, float* alpha,
                          void* workspace, size_t ws_bytes, void* stream);

/*
 * Steps 1+2 in one call (Algorithm 2: the Compress call on the flattened X):
 * draws I from `seed` (or uses idx_in), then compresses.  Arguments as above.
 */
pamm_status pamm_compress_fused(const void* X, int64_t ldx, int64_t b, int64_t n, pamm_dtype dt,
                                int64_t k, uint64_t seed, const int32_t* idx_in,
                                int32_t* idx_out, void* C, int64_t ldc, float* c_invnorm,
                                void* f, pamm_index_type f_type, float* alpha,
                                void* workspace, size_t ws_bytes, void* stream);

/*
 * The forward pass of the linear layer with the compression fused into it (Algorithm 2:
 * Z = X W; (C, alpha, f) = Compress(flatten(X)); keep C, alpha, f instead of X).  The
 * scores X C^T are k more output columns of the product X [W | C^T]: ONE tensor-core
 * kernel computes Z and, from the row blocks of X it has in flight anyway, f and alpha,
 * so the compression costs no pass over X of its own.  Generators are drawn (or taken
 * from idx_in) as in pamm_compress_fused; f, alpha and the sort products are bit for bit
 * those of pamm_compress_fused.
 *   X  b x n   W  n x m (Z_ic = sum_l X_il W_lc)   Z  b x m, all of dtype dt, row-major
 *   dt  PAMM_BF16 only (fp32 accumulation, Z rounded to nearest even); anything else, or
 *       0 < k < 16 or k > 4096, returns PAMM_ERR_UNSUPPORTED -- there is no other
 *       implementation behind this call
 *   k   0 computes Z alone (a layer whose input needs no gradient, or evaluation): the
 *       compression arguments are then ignored and may be NULL
 * X and W must be complete when the call is enqueued in the sense of every other call
 * (work enqueued earlier on the stream has produced them).
 */
pamm_status pamm_linear_forward(const void* X, int64_t ldx, int64_t b, int64_t n,
                                const void* W, int64_t ldw, int64_t m, pamm_dtype dt,
                                int64_t k, uint64_t seed, const int32_t* idx_in,
                                int32_t* idx_out, void* C, int64_t ldc, float* c_invnorm,
                                void* Z, int64_t ldz,
                                void* f, pamm_index_type f_type, float* alpha,
                                void* workspace, size_t ws_bytes, void* stream);

/*
 * The other product of the layer's backward pass (Algorithm 3: "grad X = grad Z W^T"), through the
 * same tensor-core kernel as pamm_linear_forward: dX (b x n) = dZ (b x m) W^T with W (n x m) the
 * layer's weight exactly as the forward pass takes it (here it is the operand whose contraction
 * index, m, is contiguous).  bf16 only (PAMM_ERR_UNSUPPORTED otherwise); pointers are device
 * pointers, 16-byte aligned, leading dimensions in elements (multiples of 8).  It does not share
 * the read of dZ with the contraction: pamm_contract_weight_grad reads dZ once more.
 */
pamm_status pamm_linear_backward_input(const void* dZ, int64_t lddz, int64_t b, int64_t m, const void* W, int64_t ldw,
                                       int64_t n, pamm_dtype dt, void* dX, int64_t lddx, void* stream);

/*
 * Step 2 for several generator sets at once -- one compression per projection
 * (Section 4: the method "is applied to the Q, K and V projections"; the worked
 * example of the appendix "Complexity Analysis" has m = n per projection) -- in ONE
 * pass over X.  Set s has its k generators in rows [s k, (s+1) k) of C, its norms in
 * c_invnorm[2 k s, 2 k (s+1)) (fill both with one pamm_select_generators call per
 * set, each with its own seed), and receives f and alpha at entry offset
 * s * out_stride.  Every set's result equals what pamm_compress gives for that set
 * alone.  The backward pass then runs per projection on its own columns of dY and dW
 * (pamm_contract / pamm_weight_grad with pointer offsets and the leading dimensions).
 *   sets        1..64
 *   out_stride  >= b, in entries; out_stride * sizeof(f entry) a multiple of 4
 *   workspace   NULL or sets * pamm_workspace_bytes(PAMM_WS_COMPRESS, ...) bytes:
 *               the sort products of set s start at byte s * that size
 */
pamm_status pamm_compress_projections(const void* X, int64_t ldx, int64_t b, int64_t n, pamm_dtype dt,
                                      const void* C, int64_t ldc, int64_t k, int64_t sets,
                                      const float* c_invnorm, void* f, pamm_index_type f_type, float* alpha,
                                      int64_t out_stride, void* workspace, size_t ws_bytes, void* stream);

/*
 * Step 3 -- contract (Section 3.2 "Approximate Matrix Multiplication";
 * Algorithm 1, ApproxMM: the alpha-scaling of B and the index_add into B~):
 *   B~[j,:] = sum over {i : f_i = j} of alpha_i * dY[i,:]      (k x m, fp32)
 * Rows with alpha_i = 0 (dropped by the neighbourhood condition, all-zero rows) are skipped:
 * a non-finite value in their dY rows does not reach B~ (with k > 8 those rows are not even read).
 * B' is never materialised.  dY is read once; rows are grouped by f with a
 * stable counting sort, summed in fp32 in ascending row order inside fixed-size
 * chunks, and chunk sums are added in ascending order -- no floating-point
 * atomics, so the result is reproducible bit for bit.  A row whose f_i is
 * outside [0,k) is skipped and raises PAMM_ERR_BAD_INDEX in the status word.
 *   dY  b x m, dtype dt, leading dimension ldy     Btilde  k x m fp32, ldb
 *   sort_products  NULL, or what a compress call left in its workspace for this
 *       very f (same b, k, device).  Counts that belong to another f give a wrong
 *       B~ and PAMM_ERR_BAD_INDEX in the status word, never an access out of bounds.
 */
pamm_status pamm_contract(const void* f, pamm_index_type f_type, const float* alpha,
                          const void* dY, int64_t ldy, int64_t b, int64_t m, pamm_dtype dt, int64_t k,
                          float* Btilde, int64_t ldb, const void* sort_products,
                          void* workspace, size_t ws_bytes, void* stream);

/*
 * Step 4 -- weight gradient (Algorithm 1, ApproxMM: the final product; Algorithm 3,
 * the weight gradient through ApproxMM):
 *   dW[r,c] = sum_j C[j,r] * B~[j,c]
 *   C  k x n, dtype dt, ldc      Btilde  k x m fp32, ldb
 *   dW      layout PAMM_DW_NM: n x m (the paper's O~);  PAMM_DW_MN: its transpose,
 *           m x n (out x in);  leading dimension ldw in elements of dw_dt
 *   dw_dt   PAMM_F32, or PAMM_BF16 (the fp32 accumulator is rounded to nearest even
 *           once, on the way out)
 */
pamm_status pamm_weight_grad(const void* C, int64_t ldc, int64_t k, int64_t n, pamm_dtype dt,
                             const float* Btilde, int64_t ldb, int64_t m,
                             void* dW, int64_t ldw, pamm_dtype dw_dt, pamm_layout layout, void* stream);

/*
 * Step 2 with the neighbourhood condition (Section 3.2, Eq. 2; Algorithm 1,
 * Compress: the distance e and the masked assignment of alpha).  As pamm_compress;
 * in addition a row whose representative is farther than eps ||X_i|| is dropped,
 * i.e. gets alpha_i = 0 (f_i is still reported).  The test follows Eq. 2 (relative
 * to ||X_i||; Algorithm 1 prints it without the norm).  It is evaluated in fp32 as
 *     ||X_i||^2 - S_{i,f}^2 / ||C_f||^2  <=  (eps^2 + 2 n 2^-24) ||X_i||^2
 * with ||X_i||^2 summed during the same pass over X: the second term on the right
 * is the rounding allowance of the two n-term sums, so a row lying exactly on its
 * generator's line is kept for every eps (eps = 0 is uniform column-row sampling,
 * Section 4.1), and rows within that allowance of the threshold may fall on either
 * side of it.  eps >= 1 (or infinite) keeps every row, like pamm_compress.
 *   eps      >= 0
 *   dropped  device int32: overwritten with eta, the number of dropped rows
 */
pamm_status pamm_compress_eps(const void* X, int64_t ldx, int64_t b, int64_t n, pamm_dtype dt,
                              const void* C, int64_t ldc, int64_t k, const float* c_invnorm, float eps,
                              void* f, pamm_index_type f_type, float* alpha, int32_t* dropped,
                              void* workspace, size_t ws_bytes, void* stream);

/*
 * Step 4 with the normalisation factor (Section 3.2, "Normalization factor beta",
 * Eq. 4-5): dW = beta C^T B~ with beta = b / (b - eta), eta read from `dropped` on
 * the device when the kernel runs (no host synchronisation).  dropped = NULL means
 * beta = 1; eta = b (every row dropped) gives dW = 0.
 *   b        number of rows that were compressed (b of pamm_compress_eps)
 */
pamm_status pamm_weight_grad_beta(const void* C, int64_t ldc, int64_t k, int64_t n, pamm_dtype dt,
                                  const float* Btilde, int64_t ldb, int64_t m,
                                  int64_t b, const int32_t* dropped,
                                  void* dW, int64_t ldw, pamm_dtype dw_dt, pamm_layout layout, void* stream);

/*
 * Step 4, accumulating: dW += C^T B~ (Algorithm 3's weight gradient added to what dW
 * already holds, as gradient accumulation over micro-batches needs).  Every element
 * of dW receives exactly one addition per call, so the result is reproducible.
 * dW is fp32 (the type gradients are accumulated in), in either layout.
 */
pamm_status pamm_weight_grad_accumulate(const void* C, int64_t ldc, int64_t k, int64_t n, pamm_dtype dt,
                                        const float* Btilde, int64_t ldb, int64_t m,
                                        float* dW, int64_t ldw, pamm_layout layout, void* stream);

/*
 * Steps 3+4 in one call (Algorithm 3, backward of the linear layer, the
 * weight-gradient half): contract dY into B~ and multiply by C^T.  Btilde may
 * be NULL, in which case B~ lives in the workspace only.  dW, dw_dt, layout as in
 * pamm_weight_grad; sort_products as in pamm_contract.
 */
pamm_status pamm_contract_weight_grad(const void* C, int64_t ldc, int64_t n,
                                      const void* f, pamm_index_type f_type, const float* alpha,
                                      const void* dY, int64_t ldy, int64_t b, int64_t m, pamm_dtype dt,
                                      int64_t k, float* Btilde, int64_t ldb,
                                      void* dW, int64_t ldw, pamm_dtype dw_dt, pamm_layout layout,
                                      const void* sort_products,
                                      void* workspace, size_t ws_bytes, void* stream);

/*
 * The whole path from HOST buffers (Algorithm 2's Compress followed by
 * Algorithm 3's ApproxMM for one layer): copies X and dY host->device into the
 * caller's device arena, runs steps 1-4 there, and copies dW (fp32, n x m; and, if the
 * pointers are non-NULL, f as int32 and alpha) back to the host.  X_host / dY_host /
 * dW_host should be pinned for the copies to be asynchronous.  `arena` is
 * pamm_workspace_bytes(PAMM_WS_STEP_HOST, ...) bytes of device memory.
 * The call enqueues everything on `stream` and returns; synchronise the stream
 * before reading the host outputs.
 */
pamm_status pamm_qkv_step_host(const void* X_host, const void* dY_host,
                               int64_t b, int64_t n, int64_t m, pamm_dtype dt,
                               int64_t k, uint64_t seed,
                               float* dW_host, int32_t* f_host, float* alpha_host,
                               void* arena, size_t arena_bytes, void* stream);

/*
 * What is kept for the backward pass (appendix "Complexity Analysis": k n + 2 b scalars
 * instead of b n).  No GPU is touched.
 *   out[0]  bytes of X (b n elements of dt)
 *   out[1]  bytes of (C in dt, f in f_type, alpha fp32)
 *   out[2]  b n, out[3]  k n + 2 b: the paper's scalar counts
 */
pamm_status pamm_saved_bytes(int64_t b, int64_t n, int64_t k, pamm_dtype dt, pamm_index_type f_type, int64_t out[4]);

/*
 * Contract without any caller-provided or library-allocated scratch (the paper
 * has no counterpart: this entry exists for the benefit of some callers, not
 * for the method).  It computes exactly what pamm_contract computes, with the
 * same kernels, but its scratch is a fixed array of PAMM_NO_ALLOC_SCRATCH_BYTES
 * that is part of the library image, so nothing is allocated or freed by this
 * call: no cudaMalloc / cudaFree, no allocating library routine.
 *
 * Who needs it: code that is not allowed to allocate device memory at the
 * point where it needs B~ -- a plugin running inside a host application that
 * owns the whole memory budget, a step running between the stages of a
 * latency-critical loop where cudaMalloc's implicit device synchronisation is
 * unacceptable, or a callback that runs while the framework's allocator is
 * locked.  Such a caller still owns f, alpha, dY and Btilde and passes them in.
 *
 * Limits and sharing:
 *  - the problem must be small enough for the fixed array:
 *    pamm_workspace_bytes(PAMM_WS_CONTRACT, b, n, m, k, dt) must not exceed
 *    PAMM_NO_ALLOC_SCRATCH_BYTES, otherwise PAMM_ERR_WORKSPACE is returned and
 *    nothing is launched;
 *  - every device that loads the library holds the array until the process
 *    exits, whether or not this entry is ever called;
 *  - the first call on a device looks up the array's device address (once per
 *    device, with that device current) before it launches anything; make that
 *    first call outside any stream capture;
 *  - all calls on one device share the one array and find in it whatever the
 *    previous call left.  The kernels write every word of it before they read
 *    it, so nothing has to be cleared between calls, but two calls that overlap
 *    on the GPU (different streams, no ordering between them) race on it and
 *    give wrong results.  Calls on one stream are ordered and safe.
 * Arguments, layout and error behaviour are those of pamm_contract.
 */
#define PAMM_NO_ALLOC_SCRATCH_BYTES (8u << 20)
pamm_status pamm_contract_no_alloc(const int32_t* f, const float* alpha, const void* dY, int64_t ldy,
                                   int64_t b, int64_t m, pamm_dtype dt, int64_t k,
                                   float* Btilde, int64_t ldb, void* stream);

/*
 * Reads and clears the current device's status word WITHOUT waiting for any of the
 * caller's streams: it reports what kernels that have already finished left there, so
 * synchronise the work you ask about first.  The word is per device, not per stream;
 * `stream` is accepted for symmetry with the other calls and not used.  The first
 * call on a device creates a small private stream and a pinned host word (no device
 * memory).  Returns PAMM_OK, PAMM_ERR_TIMEOUT, PAMM_ERR_BAD_INDEX, or PAMM_ERR_CUDA
 * if the read itself failed.
 */
pamm_status pamm_last_device_status(void* stream);

/*
 * Measurement hooks (no counterpart in the paper).  pamm_launch_count returns
 * the number of kernels this library has launched in this process.
 * pamm_set_profile_events makes later calls record the two given cudaEvent_t
 * (passed as void*, NULL to stop) on the call's stream immediately before and
 * after the named step's main kernel, so a benchmark can time that kernel in
 * place.  The events stay owned by the caller.  Not thread-safe.
 */
typedef enum { PAMM_PROF_COMPRESS = 0, PAMM_PROF_CONTRACT = 1, PAMM_PROF_WEIGHT_GRAD = 2 } pamm_prof_kind;
unsigned long long pamm_launch_count(void);
pamm_status pamm_set_profile_events(pamm_prof_kind kind, void* start_event, void* stop_event);

/*
 * Self-test of the failure path (no counterpart in the paper): launches one small
 * kernel that waits, with the library's bounded wait and a limit of 2048 polls, on a
 * barrier nothing completes.  The wait gives up, the kernel ends normally, and
 * pamm_last_device_status(stream) then reports PAMM_ERR_TIMEOUT once; the context
 * stays usable.  Nothing faults, traps or spins without a limit.
 */
pamm_status pamm_selftest_bounded_wait(void* stream);

/*
 * Read-only streaming probes (no counterpart in the paper): what a pass that only reads a
 * matrix once can reach on this device, as the practical ceiling of the compression (reads X)
 * and of the contraction (reads dY).  `base` (device): `rows` rows of `row_bytes` bytes (a
 * multiple of 16), `ld_bytes` apart (a multiple of 16, >= row_bytes), 16-byte aligned.
 *   PAMM_PROBE_SUM   ordinary loads of every 16-byte word; *sum32 receives the wrap-around
 *                    sum of all 32-bit words
 *   PAMM_PROBE_ROWS  whole rows by bulk copies through a shared-memory ring, two CTAs per SM,
 *                    the access pattern of the contraction's main pass; position p reads row
 *                    order[p] (device, `rows` entries of int32 in [0, rows); NULL = natural
 *                    order); *sum32 receives the sum of the first 32-bit word of every row read.
 *                    row_bytes <= 24576.
 * sum32 (device, 4 bytes) is zeroed on the stream first.  Enqueues on `stream`; time it with
 * events around the call.  An entry of `order` out of range sets PAMM_ERR_BAD_INDEX in the
 * device status (row 0 is read instead).
 */
typedef enum { PAMM_PROBE_SUM = 0, PAMM_PROBE_ROWS = 1 } pamm_probe_kind;
pamm_status pamm_probe_read(pamm_probe_kind kind, const void* base, int64_t rows, int64_t row_bytes, int64_t ld_bytes,
                            const int32_t* order, uint32_t* sum32, void* stream);

/* Library version as major*10000 + minor*100 + patch. */
int pamm_version(void);

#ifdef __cplusplus
}
#endif
#endif /* PAMM_H_ */
