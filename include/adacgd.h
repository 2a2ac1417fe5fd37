/*
 * adacgd.h -- C ABI of the B200 (sm_100a) implementation of one AdaCGD iteration
 * (Makarenko, Gasanov, Islamov, Sadiev, Richtarik: "Adaptive Compression for
 * Communication-Efficient Distributed Training", arXiv 2211.00188).
 *
 * The n workers of the paper's problem statement (Eq. 1) are simulated as n rows
 * of row-major [n x d] binary32 arrays on ONE GPU.  One iteration is, in the
 * order of Algorithm 1 (with the three-point arguments of Algorithm 2):
 *
 *   a0  x <- x - gamma * g                                   (Alg. 1, x-update)
 *   a1  X_i = grad f_i(x) for every worker i                 (Alg. 1, worker step; Section 6 objective)
 *   a2  v_i = X_i - g_i,  D_i = ||X_i - Y_i||^2              (Eq. 7 shift; right side of Eq. 10)
 *   a3  error ||v_i - C_j(v_i)||^2 of every candidate C_j    (left side of Eq. 10)
 *   a4  level_i = first j whose trigger holds, g_i update    (Eq. 11)
 *   a5  g~ = (1/n) sum_i g_i, master compression g           (Alg. 1 aggregation; Alg. 2 master step)
 *
 * Conventions
 *   - "dev" pointers are CUDA device pointers, "host" pointers are ordinary host
 *     memory.  The library never frees or reallocates a caller's buffer.
 *   - All device work is enqueued on the stream given to adacgd_init.  A call
 *     that returns results to the host synchronises that stream; the others
 *     return as soon as the work is enqueued.
 *   - A context is bound to the CUDA device that is current when adacgd_init is
 *     called (its workspace and stream must belong to it).  Every later call on the
 *     context must be made with that device current and returns
 *     ADACGD_ERR_INVALID_ARG otherwise.
 *   - Every entry point returns an adacgd_status and never aborts; a message for
 *     the last failure is available from adacgd_last_error.
 *   - Arithmetic: every elementwise operation is one IEEE binary32 operation
 *     (round to nearest even, no fused multiply-add, subnormals kept).  Squared
 *     norms that feed the trigger are exact sums rounded once to binary64.
 *     Top-K keeps the first K entries in the order (|v| descending, index
 *     ascending), |v| compared on its bit pattern (so -0 == +0).
 */
#ifndef ADACGD_H
#define ADACGD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct adacgd_ctx adacgd_ctx; /* opaque; created by adacgd_init, released by adacgd_destroy */

typedef enum {
  ADACGD_OK = 0,
  ADACGD_ERR_INVALID_ARG = 1, /* null pointer, size out of range, misaligned pointer */
  ADACGD_ERR_BAD_ORDER = 2,   /* candidate list not ordered strongest compression first */
  ADACGD_ERR_NONFINITE = 3,   /* an input held Inf/NaN; the estimators of that call are left unchanged */
  ADACGD_ERR_WORKSPACE = 4,   /* workspace smaller than adacgd_workspace_bytes reports */
  ADACGD_ERR_CUDA = 5,        /* a CUDA runtime call failed (no device, launch failure, ...) */
  ADACGD_ERR_UNSUPPORTED = 6  /* valid request that this build does not implement */
} adacgd_status;

#define ADACGD_MAX_CANDS 8

/* Candidate kinds of the user's compressor set (Section 4.3: "a set of m EF21
 * compressors sorted from the highest compression level to the lowest"). */
#define ADACGD_TOPK 0  /* param = K >= 1; K >= d is the identity (Section 2.1) */
#define ADACGD_QUANT 1 /* param = bits in [2,16]; deterministic uniform quantiser, 2^(bits-1)-1 positive levels */

typedef struct {
  int32_t kind;
  int32_t reserved; /* must be 0 */
  int64_t param;
} adacgd_cand;

/* Trigger of one level.  The adaptive compressor of Definition 3 (Eq. 9) applies the first compressor whose
 * condition P_j(h, y, x) holds and the last one when none does; AdaCGD (Eq. 11) is the case where every P_j is the
 * lazy-aggregation test of Eq. 10.  The library evaluates the conditions below, all of them comparisons of
 * squared norms it computes anyway (exact sums rounded once to binary64, as for Eq. 10); with
 * E_j = ||x - C^j_{h,y}(x)||^2 for candidate j and E_0 = ||x - h||^2 for the skip level: */
#define ADACGD_PRED_LAZY 0     /* E_j <= param * ||x - y||^2   Eq. 10 with the level's own zeta */
#define ADACGD_PRED_ABSOLUTE 1 /* E_j <= param                  an absolute error budget */
#define ADACGD_PRED_RELATIVE 2 /* E_j <= param * ||x - h||^2    a fraction of what skipping would leave */
#define ADACGD_PRED_NEVER 3    /* false: the level is never chosen by its trigger (level 0: no skipping) */
#define ADACGD_PRED_ALWAYS 4   /* true: the level is chosen whenever it is reached */
typedef struct {
  int32_t kind;  /* ADACGD_PRED_* */
  float param;   /* finite, >= 0; ignored by NEVER and ALWAYS */
} adacgd_pred;

/* A compressor set: m candidates in the order they are tried, and the trigger
 * zeta >= 0 of Eq. 10.  m = 0 is the identity compressor (no trigger).  Host memory;
 * copied by the call that receives it.  Top-K parameters must be strictly
 * increasing along the list and quantiser widths strictly increasing.
 *   preds: NULL for AdaCGD (Eq. 11: Eq. 10 with zeta at every level), or m triggers:
 *   preds[0] for the skip level, preds[j] for candidate j, 1 <= j <= m - 1; the last
 *   candidate is the "otherwise" of Eq. 9 and has none.  zeta is ignored then. */
typedef struct {
  const adacgd_cand* cands;
  int32_t m;
  float zeta;
  const adacgd_pred* preds;
} adacgd_cset;

/* Objectives f_i (Eq. 1). m_rows samples per worker, features a_l, targets t_l. */
#define ADACGD_LOSS_LOGISTIC_NCVX 0 /* (1/m) sum log(1+exp(-t a.x)) + lambda sum x_j^2/(1+x_j^2)  (Section 6) */
#define ADACGD_LOSS_LOGISTIC_L2 1   /* (1/m) sum log(1+exp(-t a.x)) + (lambda/2) ||x||^2 */
#define ADACGD_LOSS_LEAST_SQUARES 2 /* ||A x - t||^2 / (2m) */
#define ADACGD_LOSS_NONE 3          /* no data: the context only serves adacgd_compress */

#define ADACGD_LAYOUT_DENSE 0 /* A: [n][m_rows][d] row-major binary32 */
#define ADACGD_LAYOUT_CSR 1   /* CSR over all n*m_rows sample rows: row l of worker i is row i*m_rows + l; column
                                 indices in [0, d); adacgd_init builds the transposed (CSC) copy it needs for
                                 A_i^T r in the workspace, on the host, once */

typedef struct {
  int32_t loss;
  float lambda;
  int32_t n;          /* workers, 1 <= n <= 65535 */
  int32_t layout;
  int64_t d;          /* 1 <= d < 2^31 */
  int64_t m_rows;     /* samples per worker */
  const float* A;           /* dev, dense layout */
  const float* target;      /* dev, [n][m_rows]: labels in {-1,+1} or least-squares targets */
  const int64_t* csr_rowptr;/* dev, [n*m_rows + 1], offsets into csr_col / csr_val */
  const int32_t* csr_col;   /* dev, [csr_nnz] */
  const float* csr_val;     /* dev, [csr_nnz] */
  int64_t csr_nnz;          /* stored entries over all workers (CSR layout only) */
} adacgd_problem; /* device arrays are BORROWED for the lifetime of the context */

#define ADACGD_FLAG_HOST_STAGING 1 /* reserve device staging so that adacgd_compress_host can be used */
#define ADACGD_FLAG_INCREMENTAL_FORWARD 2 /* dense layout only: reserve a column-major copy of A (as large as A) and
                                             keep z_i = A_i x between iterations; see adacgd_set_refresh_period */

/* Bytes of device workspace adacgd_init needs for this problem and these sets.
 * adacgd_compress later accepts any shape with rows <= n and d <= problem->d.
 * Returns ADACGD_ERR_INVALID_ARG / ADACGD_ERR_BAD_ORDER for bad descriptors. */
adacgd_status adacgd_workspace_bytes(const adacgd_problem* problem, const adacgd_cset* worker,
                                     const adacgd_cset* master, int32_t flags, size_t* bytes_out);

/* Inputs of Algorithm 1: x^0, the estimators g_i^0 (g0_mode 0: zero; 1: grad f_i(x^0);
 * 2: C^1(grad f_i(x^0)) with the first candidate, the CLAG start of Section 2.3),
 * g~^0 = mean, g^0 = g~^0; step size gamma > 0.
 *   master = NULL or m = 0: identity master (the setting of the paper's experiments).
 *   x0_dev: dev [d], copied.  workspace_dev: dev, 256-byte aligned, caller-owned, must
 *   outlive the context.  cuda_stream: a cudaStream_t (NULL = default stream).
 * On success *ctx_out owns host-side bookkeeping only. */
adacgd_status adacgd_init(adacgd_ctx** ctx_out, const adacgd_problem* problem,
                          const adacgd_cset* worker, const adacgd_cset* master,
                          const float* x0_dev, float gamma, int32_t g0_mode, int32_t flags,
                          void* workspace_dev, size_t workspace_bytes, void* cuda_stream);

/* Per-iteration record written by adacgd_step. */
typedef struct {
  double loss;           /* f(x^{t+1}) = (1/n) sum_i f_i, by-product of a1 */
  uint64_t bits_up;      /* sum over workers of the bits of the chosen level (this iteration) */
  uint64_t bits_down;    /* bits of the master's chosen level (32 d for the identity) */
  int32_t master_level;  /* 0 = skip, j = j-th master candidate; 0 for the identity */
  int32_t exact_rechecks;/* trigger comparisons that had to be re-evaluated in exact integer arithmetic */
} adacgd_step_report;

/* n_steps iterations a0..a5 of Algorithm 1 / Algorithm 2.
 *   report_host: NULL or host array of n_steps records.
 *   levels_host: NULL or host int32 [n_steps][n], the level each worker chose (Eq. 11:
 *                0 = skip, j = j-th candidate).
 * Synchronises the stream iff a host pointer is given. */
adacgd_status adacgd_step(adacgd_ctx* ctx, int32_t n_steps, adacgd_step_report* report_host,
                          int32_t* levels_host);

/* Incremental forward pass (contexts created with ADACGD_FLAG_INCREMENTAL_FORWARD).  Algorithm 1 moves the
 * iterate by x^{t+1} = x^t - gamma g^t, so z_i = A_i x moves by -gamma A_i g^t, and g^t differs from g^{t-1}
 * only in the entries some worker's message touched (identity master: g is the mean of the estimators) or the
 * master's message touched (Algorithm 2).  adacgd_step then keeps z_i and u_i = A_i g and advances them by the
 * changed entries alone, u_i += sum_c A_i[:, c] (g^t[c] - g^{t-1}[c]) and z_i <- fl(z_i - fl(gamma u_i)), instead
 * of reading A for z_i = A_i x; the backward product A_i^T r is unchanged.  An iteration in which more than half
 * of the entries of g changed recomputes z_i = A_i x instead (gathering that many columns would cost as much),
 * and the change is carried over to the next iteration's difference.  Rounding makes the kept z_i drift from
 * A_i x, so every `period` iterations (and after any adacgd_set_state) both products are recomputed in full.
 * period >= 1; 1 recomputes every iteration; the default is 16, which keeps the gradients within the 1e-5
 * relative agreement the library is tested to.  Returns ADACGD_ERR_INVALID_ARG for a context without the flag. */
adacgd_status adacgd_set_refresh_period(adacgd_ctx* ctx, int32_t period);

/* Stages a2-a4 (and the mean of a5) on caller arrays: for every row i
 *     G_i <- AdaCGD_{h=G_i, y=Y_i}(X_i)      (Eq. 11 with EF21 candidates, Eq. 7)
 * and, if mean_out_dev != NULL, mean_out = (1/rows) sum_i G_i (binary32, summed in row
 * order, one division).  The master step of Algorithm 2 is the same call with rows = 1,
 * X = g~^{t+1}, G = g^t, Y = g~^t.
 *   X_dev, Y_dev: dev [rows][d], read only.  G_dev: dev [rows][d], updated in place.
 *   cset: host; m = 0 copies X into G.  rows*d must fit the shape given at init.
 *   Outputs, all dev, each may be NULL:
 *     level_dev int32[rows]; bits_dev uint64[rows]; err_dev double[rows][m+1] (||v||^2 then
 *     one value per candidate); D_dev double[rows]; these two are diagnostics accurate to a
 *     relative 4e-6 (the level choice itself is exact);
 *     kept_idx_dev int32[rows][kept_stride]: indices written by a Top-K level, in no
 *     particular order, kept_cnt_dev int64[rows] their number (0 for other levels).
 * Returns ADACGD_ERR_NONFINITE only from the _host variant and from adacgd_step (the
 * device-side flag is read where the stream is synchronised anyway); see
 * adacgd_get_state(ADACGD_STATE_FLAGS). */
adacgd_status adacgd_compress(adacgd_ctx* ctx, const float* X_dev, float* G_dev, const float* Y_dev,
                              int32_t rows, int64_t d, const adacgd_cset* cset, float* mean_out_dev,
                              int32_t* level_dev, uint64_t* bits_dev, double* err_dev, double* D_dev,
                              int32_t* kept_idx_dev, int64_t kept_stride, int64_t* kept_cnt_dev);

/* The same operation on HOST arrays: copies X, G, Y to the context's staging area
 * (requires ADACGD_FLAG_HOST_STAGING), runs adacgd_compress, copies G (and the mean,
 * levels, bits if requested) back, and synchronises.  The rows are taken in up to four
 * groups so that a group's results go back (on a second stream the context creates at
 * the first call) while the next group is still coming in; the results are those of one
 * adacgd_compress call on all rows.  Pinned host memory makes the copies asynchronous
 * but is not required. */
adacgd_status adacgd_compress_host(adacgd_ctx* ctx, const float* X_host, float* G_host,
                                   const float* Y_host, int32_t rows, int64_t d,
                                   const adacgd_cset* cset, float* mean_out_host,
                                   int32_t* level_host, uint64_t* bits_host);

/* adacgd_compress for callers that cannot allocate device memory (the paper has no
 * counterpart; this is a packaging variant of the same kernels).  Meant for code that is
 * only ever handed buffers: a plug-in inside a host application whose own allocator has
 * claimed the whole device, so that cudaMalloc would fail; a control loop that cannot
 * afford the device-wide synchronisation an allocation implies; a component running
 * under a policy that forbids it to grow the process's device footprint.  There is no
 * context and no workspace: the histograms, accumulators and per-row records live in a
 * 2 MiB array that is compiled into the library, so every GPU that loads the library
 * holds those 2 MiB until the process exits.  The call itself allocates nothing on the
 * host or the device and frees nothing.
 *   Limits: rows <= ADACGD_NOALLOC_MAX_ROWS, d <= ADACGD_NOALLOC_MAX_D; larger shapes
 *   return ADACGD_ERR_INVALID_ARG (message via adacgd_last_error(NULL)).
 *   X_dev, G_dev, Y_dev, cset, mean_out_dev, level_dev, bits_dev: as in adacgd_compress
 *   (the last three may be NULL); results are identical to adacgd_compress.  With no
 *   context there is no status word to read back: a row that holds Inf or NaN is
 *   reported only through level_dev (level 0) and its untouched row of G, and the call
 *   still returns ADACGD_OK.
 *   Cost: the built-in scratch has no room for the key lists of the sampled single-pass
 *   pipeline, so rows longer than 32 768 entries take the three-pass radix select (about
 *   44 bytes of traffic per entry and row, against about 21 for adacgd_compress with a
 *   workspace).
 *   cuda_stream: the cudaStream_t the work is enqueued on (NULL = default stream); the
 *   call does not synchronise.
 *   The first call on each device looks up the array's device address, with the current
 *   device being the one that owns the buffers; make that first call before any stream
 *   capture is started.
 *   All calls on a device share the one array and it keeps the previous call's
 *   contents (the call clears what has to start from zero).  Two calls whose kernels can
 *   overlap on the GPU -- different streams without an ordering between them, or two
 *   host threads -- race on it and give wrong results: serialise them. */
#define ADACGD_NOALLOC_MAX_ROWS 4
#define ADACGD_NOALLOC_MAX_D 4194304
adacgd_status adacgd_compress_noalloc(const float* X_dev, float* G_dev, const float* Y_dev,
                                      int32_t rows, int64_t d, const adacgd_cset* cset,
                                      float* mean_out_dev, int32_t* level_dev, uint64_t* bits_dev,
                                      void* cuda_stream);

/* Stage a1 alone: grads_out_dev [n][d] = grad f_i(x_dev); loss_out_host (may be NULL,
 * synchronises) = (1/n) sum_i f_i(x). */
adacgd_status adacgd_gradient(adacgd_ctx* ctx, const float* x_dev, float* grads_out_dev,
                              double* loss_out_host);

/* State of Algorithm 1 (its inputs line) plus what the three-point arguments of
 * Algorithm 2 need.  get/set copy `bytes` bytes (must equal the item's size). */
#define ADACGD_STATE_X 0        /* x^t            float [d] */
#define ADACGD_STATE_G 1        /* g~_i^t         float [n][d] */
#define ADACGD_STATE_GRAD 2     /* grad f_i(x^t)  float [n][d]  (the y of the next worker step) */
#define ADACGD_STATE_GT 3       /* g~^t           float [d] */
#define ADACGD_STATE_GM 4       /* g^t            float [d] */
#define ADACGD_STATE_STEP 5     /* t              int64 */
#define ADACGD_STATE_BITS_UP 6  /* cumulative     uint64 */
#define ADACGD_STATE_BITS_DOWN 7/* cumulative     uint64 */
#define ADACGD_STATE_LEVELS 8   /* last step      int32 [n] */
#define ADACGD_STATE_FLAGS 9    /* uint32: bit 0 = a non-finite input was seen since init; bit 1 is reserved for a
                                   device-side wait that gave up (no kernel of this version waits) (get only) */
#define ADACGD_STATE_RECHECKS 10/* uint32: trigger comparisons redone in exact arithmetic since init (get only) */
#define ADACGD_STATE_FALLBACKS 11/* uint32: rows whose sampled threshold bracket failed and that took the full
                                   three-pass radix select instead, since init (get only) */
#define ADACGD_STATE_LIST_LEVELS 12/* uint32: rows whose threshold shared the first digit of its bracket with more keys
                                   than the collection buffer holds (many equal or nearly equal magnitudes) and
                                   that went through the three-level passes over the key lists, since init (get only) */
#define ADACGD_STATE_DEVICE 13  /* int32: ordinal of the CUDA device the context is bound to (the device that was
                                   current at adacgd_init); host destination only (get only) */
#define ADACGD_STATE_INC_COLUMNS 14 /* uint64: entries of g the incremental forward passes found changed since init,
                                      summed over iterations; every worker gathers that many columns of its A (get only) */
#define ADACGD_STATE_REFRESHES 15  /* uint64: iterations since init whose forward products were recomputed in full;
                                      host destination only (get only) */
adacgd_status adacgd_get_state(adacgd_ctx* ctx, int32_t which, void* dst, size_t bytes,
                               int32_t dst_is_device);
adacgd_status adacgd_set_state(adacgd_ctx* ctx, int32_t which, const void* src, size_t bytes,
                               int32_t src_is_device);

/* Message of the last failure on this context (ctx = NULL: of the last failed
 * adacgd_init / adacgd_workspace_bytes on this thread).  Never NULL. */
const char* adacgd_last_error(const adacgd_ctx* ctx);

/* Releases host bookkeeping.  Device memory belongs to the caller. */
void adacgd_destroy(adacgd_ctx* ctx);

/* Bits of the message one worker sends when it applies candidate `cand` to a vector of d entries.  The paper
 * measures communication cost (Appendix C stops every method at a bit budget) but prints no formula; this is
 * the library's reading and its only definition: Top-K with K < d sends K values of 32 bits, each with an
 * index of ceil(log2 d) bits; Top-K with K >= d sends the d values; a b-bit quantiser sends its 32-bit scale
 * and b bits per entry; skipping sends nothing.  The bit counts that adacgd_compress and adacgd_step report
 * are this function of the chosen level.  Host only, needs no device.  Returns 0 for an invalid candidate
 * (NULL, unknown kind, K < 1, width outside [2,16]) or d outside [1, 2^31). */
uint64_t adacgd_message_bits(const adacgd_cand* cand, int64_t d);

/* Number of kernels this library has launched on behalf of ctx since init. */
int64_t adacgd_launch_count(const adacgd_ctx* ctx);

/* Per-kernel timing with CUDA events recorded on the context's stream around every
 * launch (measurement aid; the paper has no counterpart).  adacgd_profile_enable
 * reserves max_records event pairs (<= 0 switches timing off); records beyond that are
 * dropped.  adacgd_profile_read synchronises the stream, writes for every kernel id in
 * [0, adacgd_profile_kernel_count()) the summed device time in milliseconds and the
 * number of timed launches, and clears the records. */
int32_t adacgd_profile_kernel_count(void);
const char* adacgd_profile_kernel_name(int32_t id);
adacgd_status adacgd_profile_enable(adacgd_ctx* ctx, int32_t max_records);
adacgd_status adacgd_profile_read(adacgd_ctx* ctx, double* ms_out, int64_t* records_out);

#ifdef __cplusplus
}
#endif
#endif /* ADACGD_H */
