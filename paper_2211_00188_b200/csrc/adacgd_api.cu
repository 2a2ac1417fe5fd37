// C ABI of libadacgd: context, workspace carving and the iteration driver
// (Algorithm 1 with the three-point arguments of Algorithm 2).
#include <new>
#include <string>
#include <vector>

#include "adacgd_device.cuh"

using namespace adacgd;

namespace {

constexpr int LOG_CAP = 256;  // iterations logged on the device between two host reads

struct StepLog {  // one record per iteration, device resident
  double loss;
  unsigned long long bits_up, bits_down;
  int master_level, rechecks;
};

struct Counters {  // device resident, cumulative
  long long step;
  unsigned long long bits_up, bits_down;
  unsigned int rechecks_seen;
  unsigned int log_pos;  // next free record of the step log; the host rewinds it before each batch
  unsigned int pending;  // 1: the iteration that ran last has no record yet (written by the next x update or by k_log_step)
};

thread_local std::string g_err = "";

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct WsLayout {
  size_t scratch, grad, x, G, gradA, gradB, gtA, gtB, gm, levels, bits, mlevel, mbits, counters, log,
      loglevels, stage, total;
};

WsLayout ws_layout(const adacgd_problem& p, bool master_compresses, int flags) {
  WsLayout L;
  size_t o = 0;
  const size_t nd = (size_t)p.n * (size_t)p.d * 4, dd = (size_t)p.d * 4;
  L.scratch = o; o = align_up(o + scratch_bytes(p.n, p.d, true), 256);
  L.grad = o; o = align_up(o + grad_scratch_bytes(p, flags), 256);
  L.levels = o; o = align_up(o + (size_t)p.n * 4, 256);
  L.bits = o; o = align_up(o + (size_t)p.n * 8, 256);
  L.mlevel = o; o = align_up(o + 4, 256);
  L.mbits = o; o = align_up(o + 8, 256);
  L.counters = o; o = align_up(o + sizeof(Counters), 256);
  L.log = o; o = align_up(o + sizeof(StepLog) * LOG_CAP, 256);
  L.loglevels = o; o = align_up(o + (size_t)LOG_CAP * p.n * 4, 256);
  L.x = L.G = L.gradA = L.gradB = L.gtA = L.gtB = L.gm = o;
  if (p.loss != ADACGD_LOSS_NONE) {
    L.x = o; o = align_up(o + dd, 256);
    L.G = o; o = align_up(o + nd, 256);
    L.gradA = o; o = align_up(o + nd, 256);
    L.gradB = o; o = align_up(o + nd, 256);
    L.gtA = o; o = align_up(o + dd, 256);
    L.gtB = o; o = align_up(o + dd, 256);
    L.gm = o;
    if (master_compresses) o = align_up(o + dd, 256);
  }
  L.stage = o;
  if (flags & ADACGD_FLAG_HOST_STAGING) o = align_up(o + 3 * nd + dd, 256);
  L.total = o;
  return L;
}

adacgd_status check_problem(const adacgd_problem* p, const char** msg) {
  if (!p) { *msg = "problem is NULL"; return ADACGD_ERR_INVALID_ARG; }
  if (p->n < 1 || p->n > 65535) { *msg = "n must be in [1, 65535]"; return ADACGD_ERR_INVALID_ARG; }
  if (p->d < 1 || p->d >= (1ll << 31)) { *msg = "d must be in [1, 2^31)"; return ADACGD_ERR_INVALID_ARG; }
  if (p->loss < 0 || p->loss > ADACGD_LOSS_NONE) { *msg = "unknown loss"; return ADACGD_ERR_INVALID_ARG; }
  if (p->loss != ADACGD_LOSS_NONE) {
    if (p->m_rows < 1) { *msg = "m_rows must be >= 1"; return ADACGD_ERR_INVALID_ARG; }
    if (p->layout == ADACGD_LAYOUT_DENSE) {
      if (!p->A || !p->target) { *msg = "dense layout needs A and target"; return ADACGD_ERR_INVALID_ARG; }
    } else if (p->layout == ADACGD_LAYOUT_CSR) {
      if (!p->csr_rowptr || !p->csr_col || !p->csr_val || !p->target || p->csr_nnz < 0) {
        *msg = "CSR layout needs csr_rowptr, csr_col, csr_val, target and csr_nnz >= 0";
        return ADACGD_ERR_INVALID_ARG;
      }
    } else {
      *msg = "unknown layout";
      return ADACGD_ERR_INVALID_ARG;
    }
    if (!(p->lambda >= 0.f)) { *msg = "lambda must be >= 0"; return ADACGD_ERR_INVALID_ARG; }
  }
  return ADACGD_OK;
}

// The record of the iteration that just ran: bits sent, levels, loss, exact rechecks.  Run by one CTA.
__device__ void log_body(int n, const int* __restrict__ levels, const unsigned long long* __restrict__ bits,
                         const int* __restrict__ mlevel, const unsigned long long* __restrict__ mbits,
                         const double* __restrict__ loss, const unsigned int* __restrict__ flags,
                         Counters* cnt, StepLog* log, int* loglevels) {
  __shared__ unsigned long long sh[32];
  const int slot = (int)cnt->log_pos;
  unsigned long long a = 0;
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    a += bits[i];
    loglevels[(long long)slot * n + i] = levels[i];
  }
  for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = a;
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long up = 0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) up += sh[w];
    StepLog r;
    r.loss = loss ? *loss : 0.0;
    r.bits_up = up;
    r.bits_down = *mbits;
    r.master_level = *mlevel;
    r.rechecks = (int)(flags[1] - cnt->rechecks_seen);
    cnt->rechecks_seen = flags[1];
    cnt->log_pos = (unsigned int)slot + 1u;
    cnt->step += 1;
    cnt->bits_up += up;
    cnt->bits_down += r.bits_down;
    log[slot] = r;
  }
}

// Closes a batch of iterations: writes the record of the last one, if it has none yet.
__global__ void k_log_step(int n, const int* __restrict__ levels, const unsigned long long* __restrict__ bits,
                           const int* __restrict__ mlevel, const unsigned long long* __restrict__ mbits,
                           const double* __restrict__ loss, const unsigned int* __restrict__ flags,
                           Counters* cnt, StepLog* log, int* loglevels) {
  if (!cnt->pending) return;
  log_body(n, levels, bits, mlevel, mbits, loss, flags, cnt, log, loglevels);
  __syncthreads();
  if (threadIdx.x == 0) cnt->pending = 0u;
}

// Opens an iteration: x^{t+1} = x^t - gamma g^t (Algorithm 1).  Its first CTA also writes the record of the iteration
// before, whose results (levels, bits, loss) stay in place until later kernels of this iteration overwrite them:
// one launch per iteration less than a record kernel at the end of every iteration.
__global__ void __launch_bounds__(256) k_axpy_log(float* __restrict__ x, const float* __restrict__ g, float gamma, long long d,
                                                  int n, const int* __restrict__ levels,
                                                  const unsigned long long* __restrict__ bits, const int* __restrict__ mlevel,
                                                  const unsigned long long* __restrict__ mbits, const double* __restrict__ loss,
                                                  const unsigned int* __restrict__ flags, Counters* cnt, StepLog* log,
                                                  int* loglevels) {
  pdl_begin();     // the forward kernel may become resident (it waits for this grid before it reads x); this grid
                   // itself may have become resident while the last kernel of the iteration before was running
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < d) x[i] = __fsub_rn(x[i], __fmul_rn(gamma, g[i]));   // two binary32 roundings: the product, then the difference
  if (blockIdx.x != 0) return;
  if (cnt->pending) log_body(n, levels, bits, mlevel, mbits, loss, flags, cnt, log, loglevels);
  __syncthreads();
  if (threadIdx.x == 0) cnt->pending = 1u;
}

__global__ void k_set_master_identity(int* mlevel, unsigned long long* mbits, long long d) {
  *mlevel = 0;
  *mbits = 32ull * (unsigned long long)d;
}

}  // namespace

namespace adacgd {
void set_thread_error(const char* msg) { g_err = msg ? msg : ""; }
}  // namespace adacgd

struct adacgd_ctx {
  adacgd_problem p;
  CsetDev wcs, mcs;
  bool master_compresses;
  float gamma;
  int flags;
  cudaStream_t stream;
  int device;                  // ordinal of the device that was current at adacgd_init; every later call must find it current
  Scratch scr;
  GradScratch gs;
  float *x, *G, *grad_cur, *grad_nxt, *gt_cur, *gt_nxt, *gm, *gm_buf;
  int* levels;
  unsigned long long* bits;
  int* mlevel;
  unsigned long long* mbits;
  Counters* counters;
  StepLog* log;
  int* loglevels;
  float* stage;
  cudaStream_t copy_stream;    // second stream of adacgd_compress_host (created at its first call): results go back
  cudaEvent_t copy_ev[5];      // to the host while the next group of rows is still coming in
  long long launches;
  cudaGraphExec_t pair_exec;   // two captured iterations (the buffers ping-pong with period 2)
  long long pair_launches;
  bool graph_tried;
  bool odd;                    // parity of the iterations run since the graph's reference state
  // incremental forward pass: z_i = A_i x and u_i = A_i g live in the workspace
  int refresh_period;          // iterations between full recomputations
  int since_refresh;           // iterations run since the last one
  bool inc_dirty;              // the kept products do not belong to the current x and g (fresh context, set_state)
  unsigned long long refreshes;
  Prof* prof;
  Prof prof_store;
  std::vector<cudaEvent_t> ev_beg, ev_end;
  std::vector<int> ev_id;
  std::string err;
};

namespace {

adacgd_status fail(adacgd_ctx* c, adacgd_status s, const std::string& m) {
  if (c) c->err = m;
  else g_err = m;
  return s;
}

adacgd_status cuda_fail(adacgd_ctx* c, const char* what) {
  cudaError_t e = cudaGetLastError();
  return fail(c, ADACGD_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

adacgd_status cuda_fail(adacgd_ctx* c, const char* what, cudaError_t e) {
  cudaGetLastError();  // the sticky copy of the same error
  return fail(c, ADACGD_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

// Runs a CUDA runtime call and leaves the entry point with a message that names it when it fails.
#define CK(c, call, what)                                          \
  do {                                                             \
    const cudaError_t ck_e_ = (call);                              \
    if (ck_e_ != cudaSuccess) return cuda_fail((c), (what), ck_e_); \
  } while (0)

// A context is bound to the device that was current when it was created: its workspace, its stream and
// the per-device kernel attributes belong to that device.
adacgd_status check_device(adacgd_ctx* c, const char* entry) {
  int dev = -1;
  const cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(c, (std::string(entry) + " (cudaGetDevice)").c_str(), e);
  if (dev != c->device)
    return fail(c, ADACGD_ERR_INVALID_ARG, std::string(entry) + ": the current CUDA device is " + std::to_string(dev) +
                                               " but the context was created on device " + std::to_string(c->device));
  return ADACGD_OK;
}

// Worker side + mean, then master side, on the context's own state.
adacgd_status run_server_and_master(adacgd_ctx* c) {
  CompressOut mo;
  memset(&mo, 0, sizeof(mo));
  if (c->master_compresses) {
    mo.level = c->mlevel;
    mo.bits = (uint64_t*)c->mbits;
    int r = launch_compress(c->scr, c->mcs, c->gt_nxt, c->gm_buf, c->gt_cur, 1, c->p.d, mo, c->stream);
    if (r < 0) return cuda_fail(c, "master compression");
    c->launches += r;
    c->gm = c->gm_buf;
  } else {
    c->gm = c->gt_nxt;
  }
  float* t = c->gt_cur;
  c->gt_cur = c->gt_nxt;
  c->gt_nxt = t;
  return ADACGD_OK;
}

}  // namespace

extern "C" {

adacgd_status adacgd_workspace_bytes(const adacgd_problem* problem, const adacgd_cset* worker,
                                     const adacgd_cset* master, int32_t flags, size_t* bytes_out) {
  const char* msg = "";
  adacgd_status s = check_problem(problem, &msg);
  if (s != ADACGD_OK) return fail(nullptr, s, msg);
  if (!bytes_out) return fail(nullptr, ADACGD_ERR_INVALID_ARG, "bytes_out is NULL");
  CsetDev tmp;
  if ((s = make_cset(worker, problem->d, &tmp, &msg)) != ADACGD_OK) return fail(nullptr, s, msg);
  if ((s = make_cset(master, problem->d, &tmp, &msg)) != ADACGD_OK) return fail(nullptr, s, msg);
  const bool mc = master && master->m > 0;
  *bytes_out = ws_layout(*problem, mc, flags).total;
  return ADACGD_OK;
}

// Everything of adacgd_init that can fail after the context object exists; messages go to the thread's
// slot because the caller gets no context back on failure.
static adacgd_status init_body(adacgd_ctx* c, const adacgd_problem* problem, const adacgd_cset* worker,
                               const adacgd_cset* master, const float* x0_dev, float gamma, int32_t g0_mode,
                               int32_t flags, void* workspace_dev, size_t workspace_bytes, void* cuda_stream) {
  const char* msg = "";
  adacgd_status s;
  c->p = *problem;
  if ((s = make_cset(worker, problem->d, &c->wcs, &msg)) != ADACGD_OK ||
      (s = make_cset(master, problem->d, &c->mcs, &msg)) != ADACGD_OK)
    return fail(nullptr, s, msg);
  c->master_compresses = master && master->m > 0;
  c->gamma = gamma;
  c->flags = flags;
  c->stream = (cudaStream_t)cuda_stream;
  c->launches = 0;
  c->pair_exec = nullptr;
  c->pair_launches = 0;
  c->graph_tried = false;
  c->odd = false;
  c->refresh_period = 16;
  c->since_refresh = 0;
  c->inc_dirty = true;
  c->refreshes = 0;
  c->prof = nullptr;
  c->copy_stream = nullptr;
  for (cudaEvent_t& e : c->copy_ev) e = nullptr;
  c->x = c->G = c->grad_cur = c->grad_nxt = c->gt_cur = c->gt_nxt = c->gm = c->gm_buf = nullptr;
  const bool has_loss = problem->loss != ADACGD_LOSS_NONE;
  if (has_loss && (!x0_dev || !(gamma > 0.f) || g0_mode < 0 || g0_mode > 2))
    return fail(nullptr, ADACGD_ERR_INVALID_ARG, "x0_dev must be non-NULL, gamma > 0, g0_mode in {0,1,2}");
  if (has_loss && g0_mode == 2 && c->wcs.m == 0)
    return fail(nullptr, ADACGD_ERR_INVALID_ARG, "g0_mode 2 needs a worker candidate");
  const WsLayout L = ws_layout(*problem, c->master_compresses, flags);
  if (!workspace_dev || ((uintptr_t)workspace_dev & 255))
    return fail(nullptr, ADACGD_ERR_INVALID_ARG, "workspace_dev must be non-NULL and 256-byte aligned");
  if (workspace_bytes < L.total)
    return fail(nullptr, ADACGD_ERR_WORKSPACE, "workspace smaller than adacgd_workspace_bytes reports");
  CK(nullptr, cudaGetDevice(&c->device), "adacgd_init (cudaGetDevice)");
  if (!current_device()) return cuda_fail(nullptr, "adacgd_init (device attributes)");
  char* b = (char*)workspace_dev;
  carve_scratch(&c->scr, b + L.scratch, problem->n, problem->d, true);
  c->levels = (int*)(b + L.levels);
  c->bits = (unsigned long long*)(b + L.bits);
  c->mlevel = (int*)(b + L.mlevel);
  c->mbits = (unsigned long long*)(b + L.mbits);
  c->counters = (Counters*)(b + L.counters);
  c->log = (StepLog*)(b + L.log);
  c->loglevels = (int*)(b + L.loglevels);
  c->stage = (flags & ADACGD_FLAG_HOST_STAGING) ? (float*)(b + L.stage) : nullptr;

  CK(nullptr, cudaMemsetAsync(c->scr.flags, 0, 64, c->stream), "adacgd_init (clearing the status words)");
  CK(nullptr, cudaMemsetAsync(c->counters, 0, sizeof(Counters), c->stream), "adacgd_init (clearing the counters)");
  if (has_loss) {
    carve_grad_scratch(&c->gs, b + L.grad, *problem, flags);
    CK(nullptr, cudaMemsetAsync(c->gs.loss_ticket, 0, c->gs.ticket_bytes, c->stream), "adacgd_init (clearing the gradient tickets)");
    if (c->gs.inc && build_transposed_features(*problem, c->gs, c->stream) < 0)
      return cuda_fail(nullptr, "adacgd_init (column-major copy of the features)");
    if (problem->layout == ADACGD_LAYOUT_CSR) {
      const char* why = build_csc(*problem, &c->gs, c->stream);
      if (why) return fail(nullptr, ADACGD_ERR_INVALID_ARG, why);
    }
    c->x = (float*)(b + L.x);
    c->G = (float*)(b + L.G);
    c->grad_cur = (float*)(b + L.gradA);
    c->grad_nxt = (float*)(b + L.gradB);
    c->gt_cur = (float*)(b + L.gtA);
    c->gt_nxt = (float*)(b + L.gtB);
    c->gm_buf = c->master_compresses ? (float*)(b + L.gm) : nullptr;
    const size_t nd = (size_t)problem->n * problem->d * 4, dd = (size_t)problem->d * 4;
    CK(nullptr, cudaMemcpyAsync(c->x, x0_dev, dd, cudaMemcpyDeviceToDevice, c->stream), "adacgd_init (copy of x0)");
    int r = launch_gradient(c->p, c->gs, c->x, c->grad_cur, c->stream);
    if (r < 0) return cuda_fail(nullptr, "adacgd_init (gradient)");
    c->launches += r;
    if (g0_mode == 0) {
      CK(nullptr, cudaMemsetAsync(c->G, 0, nd, c->stream), "adacgd_init (zero estimators)");
    } else if (g0_mode == 1) {
      CK(nullptr, cudaMemcpyAsync(c->G, c->grad_cur, nd, cudaMemcpyDeviceToDevice, c->stream), "adacgd_init (estimators = gradients)");
    } else {
      CK(nullptr, cudaMemsetAsync(c->G, 0, nd, c->stream), "adacgd_init (zero estimators)");
      adacgd_cand first = worker->cands[0];
      adacgd_cset one = {&first, 1, 0.f, nullptr};
      CsetDev cs1;
      make_cset(&one, problem->d, &cs1, &msg);
      CompressOut o;
      memset(&o, 0, sizeof(o));
      r = launch_compress(c->scr, cs1, c->grad_cur, c->G, c->grad_cur, problem->n, problem->d, o, c->stream);
      if (r < 0) return cuda_fail(nullptr, "adacgd_init (g0)");
      c->launches += r;
    }
    r = launch_mean_rows(c->G, problem->n, problem->d, c->gt_cur, c->stream);
    if (r < 0) return cuda_fail(nullptr, "adacgd_init (mean)");
    c->launches += r;
    if (c->master_compresses) {
      CK(nullptr, cudaMemcpyAsync(c->gm_buf, c->gt_cur, dd, cudaMemcpyDeviceToDevice, c->stream), "adacgd_init (copy of the mean)");
      c->gm = c->gm_buf;
    } else {
      c->gm = c->gt_cur;
      k_set_master_identity<<<1, 1, 0, c->stream>>>(c->mlevel, c->mbits, problem->d);
      c->launches += 1;
    }
  }
  CK(nullptr, cudaStreamSynchronize(c->stream), "adacgd_init (synchronising the stream)");
  CK(nullptr, cudaGetLastError(), "adacgd_init");
  return ADACGD_OK;
}

adacgd_status adacgd_init(adacgd_ctx** ctx_out, const adacgd_problem* problem, const adacgd_cset* worker,
                          const adacgd_cset* master, const float* x0_dev, float gamma, int32_t g0_mode,
                          int32_t flags, void* workspace_dev, size_t workspace_bytes, void* cuda_stream) {
  const char* msg = "";
  if (!ctx_out) return fail(nullptr, ADACGD_ERR_INVALID_ARG, "ctx_out is NULL");
  *ctx_out = nullptr;
  adacgd_status s = check_problem(problem, &msg);
  if (s != ADACGD_OK) return fail(nullptr, s, msg);
  adacgd_ctx* c = new (std::nothrow) adacgd_ctx();
  if (!c) return fail(nullptr, ADACGD_ERR_INVALID_ARG, "out of host memory");
  s = init_body(c, problem, worker, master, x0_dev, gamma, g0_mode, flags, workspace_dev, workspace_bytes, cuda_stream);
  if (s != ADACGD_OK) {
    delete c;
    return s;
  }
  *ctx_out = c;
  return ADACGD_OK;
}

adacgd_status adacgd_compress(adacgd_ctx* ctx, const float* X_dev, float* G_dev, const float* Y_dev, int32_t rows,
                              int64_t d, const adacgd_cset* cset, float* mean_out_dev, int32_t* level_dev,
                              uint64_t* bits_dev, double* err_dev, double* D_dev, int32_t* kept_idx_dev,
                              int64_t kept_stride, int64_t* kept_cnt_dev) {
  if (!ctx) return fail(nullptr, ADACGD_ERR_INVALID_ARG, "ctx is NULL");
  if (!X_dev || !G_dev || !Y_dev) return fail(ctx, ADACGD_ERR_INVALID_ARG, "X, G, Y must be non-NULL");
  if (rows < 1 || rows > ctx->p.n || d < 1 || d > ctx->p.d)
    return fail(ctx, ADACGD_ERR_INVALID_ARG, "rows/d exceed the shape given at init");
  if ((kept_idx_dev != nullptr) != (kept_cnt_dev != nullptr) || (kept_idx_dev && kept_stride < 1))
    return fail(ctx, ADACGD_ERR_INVALID_ARG, "kept_idx_dev and kept_cnt_dev go together, kept_stride >= 1");
  const char* msg = "";
  CsetDev cs;
  adacgd_status s = make_cset(cset, d, &cs, &msg);
  if (s != ADACGD_OK) return fail(ctx, s, msg);
  if ((s = check_device(ctx, "adacgd_compress")) != ADACGD_OK) return s;
  CompressOut o;
  o.mean_out = mean_out_dev; o.level = level_dev; o.bits = bits_dev; o.err = err_dev; o.D = D_dev;
  o.kept_idx = kept_idx_dev; o.kept_stride = kept_stride; o.kept_cnt = (long long*)kept_cnt_dev;
  int r = launch_compress(ctx->scr, cs, X_dev, G_dev, Y_dev, rows, d, o, ctx->stream);
  if (r < 0) return cuda_fail(ctx, "adacgd_compress");
  ctx->launches += r;
  return ADACGD_OK;
}

adacgd_status adacgd_compress_host(adacgd_ctx* ctx, const float* X_host, float* G_host, const float* Y_host,
                                   int32_t rows, int64_t d, const adacgd_cset* cset, float* mean_out_host,
                                   int32_t* level_host, uint64_t* bits_host) {
  if (!ctx) return fail(nullptr, ADACGD_ERR_INVALID_ARG, "ctx is NULL");
  if (!ctx->stage) return fail(ctx, ADACGD_ERR_INVALID_ARG, "context was created without ADACGD_FLAG_HOST_STAGING");
  if (!X_host || !G_host || !Y_host) return fail(ctx, ADACGD_ERR_INVALID_ARG, "X, G, Y must be non-NULL");
  if (rows < 1 || rows > ctx->p.n || d < 1 || d > ctx->p.d)
    return fail(ctx, ADACGD_ERR_INVALID_ARG, "rows/d exceed the shape given at init");
  const size_t cap = (size_t)ctx->p.n * (size_t)ctx->p.d;
  float* Xs = ctx->stage;
  float* Gs = Xs + cap;
  float* Ys = Gs + cap;
  float* Ms = Ys + cap;
  unsigned int flags_before = 0, flags_after = 0;
  {
    const adacgd_status sd = check_device(ctx, "adacgd_compress_host");
    if (sd != ADACGD_OK) return sd;
  }
  CK(ctx, cudaMemcpyAsync(&flags_before, ctx->scr.flags, 4, cudaMemcpyDeviceToHost, ctx->stream), "adacgd_compress_host (status words to the host)");
  // The rows are taken in up to four groups: while a group's estimators travel back to the host on a second
  // stream, the next group's operands are still coming in (the link carries both directions at once).  The
  // mean needs every row and follows in a kernel of its own, summed in row order like the fused one.
  if (!ctx->copy_stream) {
    if (cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking) != cudaSuccess) return cuda_fail(ctx, "stream for host copies");
    for (cudaEvent_t& e : ctx->copy_ev)
      if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return cuda_fail(ctx, "event for host copies");
  }
  const int ngroups = rows < 4 ? rows : 4;
  for (int g = 0; g < ngroups; ++g) {
    const int r0 = (int)((long long)rows * g / ngroups), r1 = (int)((long long)rows * (g + 1) / ngroups);
    const size_t off = (size_t)r0 * (size_t)d, bytes = (size_t)(r1 - r0) * (size_t)d * 4;
    CK(ctx, cudaMemcpyAsync(Xs + off, X_host + off, bytes, cudaMemcpyHostToDevice, ctx->stream), "adacgd_compress_host (copy of X to the device)");
    CK(ctx, cudaMemcpyAsync(Gs + off, G_host + off, bytes, cudaMemcpyHostToDevice, ctx->stream), "adacgd_compress_host (copy of G to the device)");
    CK(ctx, cudaMemcpyAsync(Ys + off, Y_host + off, bytes, cudaMemcpyHostToDevice, ctx->stream), "adacgd_compress_host (copy of Y to the device)");
    adacgd_status s = adacgd_compress(ctx, Xs + off, Gs + off, Ys + off, r1 - r0, d, cset, nullptr,
                                      level_host ? ctx->levels + r0 : nullptr,
                                      bits_host ? (uint64_t*)ctx->bits + r0 : nullptr, nullptr, nullptr, nullptr, 0, nullptr);
    if (s != ADACGD_OK) { cudaStreamSynchronize(ctx->copy_stream); return s; }   // earlier groups may still be on their way back
    CK(ctx, cudaEventRecord(ctx->copy_ev[g], ctx->stream), "adacgd_compress_host (event after a group of rows)");
    CK(ctx, cudaStreamWaitEvent(ctx->copy_stream, ctx->copy_ev[g], 0), "adacgd_compress_host (copy stream waiting for a group)");
    CK(ctx, cudaMemcpyAsync(G_host + off, Gs + off, bytes, cudaMemcpyDeviceToHost, ctx->copy_stream), "adacgd_compress_host (copy of G to the host)");
  }
  if (mean_out_host) {
    if (launch_mean_rows(Gs, rows, d, Ms, ctx->stream) < 0) return cuda_fail(ctx, "mean over rows");
    ctx->launches += 1;
    CK(ctx, cudaMemcpyAsync(mean_out_host, Ms, (size_t)d * 4, cudaMemcpyDeviceToHost, ctx->stream), "adacgd_compress_host (copy of the mean to the host)");
  }
  if (level_host) CK(ctx, cudaMemcpyAsync(level_host, ctx->levels, (size_t)rows * 4, cudaMemcpyDeviceToHost, ctx->stream), "adacgd_compress_host (copy of the levels to the host)");
  if (bits_host) CK(ctx, cudaMemcpyAsync(bits_host, ctx->bits, (size_t)rows * 8, cudaMemcpyDeviceToHost, ctx->stream), "adacgd_compress_host (copy of the bit counts to the host)");
  CK(ctx, cudaEventRecord(ctx->copy_ev[4], ctx->copy_stream), "adacgd_compress_host (event after the last copy)");
  CK(ctx, cudaStreamWaitEvent(ctx->stream, ctx->copy_ev[4], 0), "adacgd_compress_host (waiting for the copy stream)");
  CK(ctx, cudaMemcpyAsync(&flags_after, ctx->scr.flags, 4, cudaMemcpyDeviceToHost, ctx->stream), "adacgd_compress_host (status words to the host)");
  CK(ctx, cudaStreamSynchronize(ctx->stream), "adacgd_compress_host (synchronising the stream)");
  if (flags_after & 2u) return fail(ctx, ADACGD_ERR_CUDA, "a device-side wait for an asynchronous copy timed out");
  if ((flags_after & 1u) && !(flags_before & 1u))
    return fail(ctx, ADACGD_ERR_NONFINITE, "an input row held Inf or NaN; its estimator was left unchanged");
  return ADACGD_OK;
}

adacgd_status adacgd_gradient(adacgd_ctx* ctx, const float* x_dev, float* grads_out_dev, double* loss_out_host) {
  if (!ctx) return fail(nullptr, ADACGD_ERR_INVALID_ARG, "ctx is NULL");
  if (ctx->p.loss == ADACGD_LOSS_NONE) return fail(ctx, ADACGD_ERR_INVALID_ARG, "context has no objective");
  if (!x_dev || !grads_out_dev) return fail(ctx, ADACGD_ERR_INVALID_ARG, "x_dev and grads_out_dev must be non-NULL");
  {
    const adacgd_status sd = check_device(ctx, "adacgd_gradient");
    if (sd != ADACGD_OK) return sd;
  }
  int r = launch_gradient(ctx->p, ctx->gs, x_dev, grads_out_dev, ctx->stream);
  if (r < 0) return cuda_fail(ctx, "adacgd_gradient");
  ctx->launches += r;
  if (loss_out_host) {
    CK(ctx, cudaMemcpyAsync(loss_out_host, ctx->gs.loss, 8, cudaMemcpyDeviceToHost, ctx->stream), "adacgd_gradient (copy of the loss to the host)");
    CK(ctx, cudaStreamSynchronize(ctx->stream), "adacgd_gradient (synchronising the stream)");
  }
  return ADACGD_OK;
}

// Enqueues one iteration a0..a5 on the context's stream.  `capturing`: the iteration is being recorded into the
// graph of incremental iterations, so it takes the incremental forward pass and leaves the refresh counters alone.
static adacgd_status enqueue_iteration(adacgd_ctx* c, bool capturing = false) {
  const int n = c->p.n;
  const long long d = c->p.d;
  // a0: x^{t+1} = x^t - gamma g^t
  prof_begin(c->prof, KID_AXPY, c->stream);
  launch_k(k_axpy_log, dim3((unsigned)((d + 255) / 256)), dim3(256), 0, c->stream, c->prof == nullptr, c->x, (const float*)c->gm, c->gamma,
           (long long)d, n, (const int*)c->levels, (const unsigned long long*)c->bits, (const int*)c->mlevel,
           (const unsigned long long*)c->mbits, (const double*)c->gs.loss, (const unsigned int*)c->scr.flags, c->counters, c->log,
           c->loglevels);
  prof_end(c->prof, c->stream);
  if (cudaGetLastError() != cudaSuccess) return cuda_fail(c, "x update");
  c->launches += 1;
  int r = 0;
  // a1: X_i = grad f_i(x^{t+1})
  if (c->gs.inc) {
    const bool refresh = !capturing && (c->inc_dirty || c->since_refresh + 1 >= c->refresh_period);
    r = launch_gradient_incremental(c->p, c->gs, c->x, c->gm, c->gamma, refresh, c->grad_nxt, c->stream);
    if (!capturing) {
      if (refresh) { c->since_refresh = 0; c->inc_dirty = false; c->refreshes += 1; }
      else c->since_refresh += 1;
    }
  } else {
    r = launch_gradient(c->p, c->gs, c->x, c->grad_nxt, c->stream);
  }
  if (r < 0) return cuda_fail(c, "gradient");
  c->launches += r;
  // a2-a4 and the mean of a5: h = g~_i^t, y = grad f_i(x^t), x = grad f_i(x^{t+1})
  CompressOut o;
  memset(&o, 0, sizeof(o));
  o.mean_out = c->gt_nxt;
  o.level = c->levels;
  o.bits = (uint64_t*)c->bits;
  r = launch_compress(c->scr, c->wcs, c->grad_nxt, c->G, c->grad_cur, n, d, o, c->stream);
  if (r < 0) return cuda_fail(c, "worker compression");
  c->launches += r;
  // a5: master step h = g^t, y = g~^t, x = g~^{t+1}
  adacgd_status s = run_server_and_master(c);
  if (s != ADACGD_OK) return s;
  float* t2 = c->grad_cur;
  c->grad_cur = c->grad_nxt;
  c->grad_nxt = t2;
  return ADACGD_OK;   // the iteration's record is written by the next x update, or by close_batch()
}

// The record of the last iteration enqueued, before the host reads the step log or other calls touch its inputs.
static void close_batch(adacgd_ctx* c) {
  prof_begin(c->prof, KID_LOG, c->stream);
  k_log_step<<<1, 256, 0, c->stream>>>(c->p.n, c->levels, c->bits, c->mlevel, c->mbits, c->gs.loss, c->scr.flags,
                                       c->counters, c->log, c->loglevels);
  prof_end(c->prof, c->stream);
  c->launches += 1;
}

// Captures two iterations into one graph: after two steps every ping-pong pointer is back where it
// was, so the graph can be replayed from any even step on.  A workload whose iteration is a few
// dozen short kernels is otherwise bound by launch latency.
static void try_capture_pair(adacgd_ctx* c) {
  c->graph_tried = true;
  // one plain iteration pair first: lazy per-kernel attributes are set outside the capture
  const long long before = c->launches;
  cudaGraph_t graph = nullptr;
  if (cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
    cudaGetLastError();
    return;
  }
  adacgd_status s1 = enqueue_iteration(c, true);
  adacgd_status s2 = (s1 == ADACGD_OK) ? enqueue_iteration(c, true) : s1;
  const cudaError_t e = cudaStreamEndCapture(c->stream, &graph);
  c->pair_launches = c->launches - before;
  c->launches = before;
  if (s1 != ADACGD_OK || s2 != ADACGD_OK || e != cudaSuccess || !graph) {
    cudaGetLastError();
    if (graph) cudaGraphDestroy(graph);
    return;
  }
  if (cudaGraphInstantiate(&c->pair_exec, graph, 0) != cudaSuccess) {
    cudaGetLastError();
    c->pair_exec = nullptr;
  }
  cudaGraphDestroy(graph);
}

adacgd_status adacgd_step(adacgd_ctx* c, int32_t n_steps, adacgd_step_report* report_host, int32_t* levels_host) {
  if (!c) return fail(nullptr, ADACGD_ERR_INVALID_ARG, "ctx is NULL");
  if (c->p.loss == ADACGD_LOSS_NONE) return fail(c, ADACGD_ERR_INVALID_ARG, "context has no objective");
  if (n_steps < 0) return fail(c, ADACGD_ERR_INVALID_ARG, "n_steps must be >= 0");
  {
    const adacgd_status sd = check_device(c, "adacgd_step");
    if (sd != ADACGD_OK) return sd;
  }
  const int n = c->p.n;
  std::vector<StepLog> hostlog;
  for (int done = 0; done < n_steps;) {
    const int batch = (n_steps - done < LOG_CAP) ? (n_steps - done) : LOG_CAP;
    CK(c, cudaMemsetAsync(&c->counters->log_pos, 0, 4, c->stream), "adacgd_step (rewinding the step log)");
    int t = 0;
    // graphs hold the buffer pointers of the step parity they were captured at (always even here,
    // because pairs are replayed whole and single iterations toggle `odd`)
    const bool use_graph = !c->prof && batch >= 4;
    if (use_graph && c->odd) {
      adacgd_status s = enqueue_iteration(c);
      if (s != ADACGD_OK) return s;
      c->odd = !c->odd;
      ++t;
    }
    if (use_graph && !c->graph_tried) {
      // the first pair runs uncaptured so that one-time kernel attributes are set before the capture
      for (int k = 0; k < 2 && t < batch; ++k, ++t) {
        adacgd_status s = enqueue_iteration(c);
        if (s != ADACGD_OK) return s;
        c->odd = !c->odd;
      }
      if (!c->odd) try_capture_pair(c);
    }
    while (t < batch) {
      // a recorded pair holds two incremental iterations: it is replayed while no refresh falls inside it
      const bool pair_ok = use_graph && c->pair_exec && !c->odd && t + 2 <= batch &&
                           (!c->gs.inc || (!c->inc_dirty && c->since_refresh + 2 < c->refresh_period));
      if (pair_ok) {
        if (cudaGraphLaunch(c->pair_exec, c->stream) != cudaSuccess) return cuda_fail(c, "graph launch");
        c->launches += c->pair_launches;
        if (c->gs.inc) c->since_refresh += 2;
        t += 2;
      } else {
        adacgd_status s = enqueue_iteration(c);
        if (s != ADACGD_OK) return s;
        c->odd = !c->odd;
        ++t;
      }
    }
    if (batch > 0) close_batch(c);
    if (report_host || levels_host) {
      hostlog.resize(batch);
      CK(c, cudaMemcpyAsync(hostlog.data(), c->log, sizeof(StepLog) * batch, cudaMemcpyDeviceToHost, c->stream), "adacgd_step (copy of the step log to the host)");
      if (levels_host)
        CK(c, cudaMemcpyAsync(levels_host + (size_t)done * n, c->loglevels, (size_t)batch * n * 4, cudaMemcpyDeviceToHost, c->stream),
           "adacgd_step (copy of the levels to the host)");
      CK(c, cudaStreamSynchronize(c->stream), "adacgd_step (synchronising the stream)");
      if (report_host)
        for (int q = 0; q < batch; ++q) {
          adacgd_step_report& rr = report_host[done + q];
          rr.loss = hostlog[q].loss;
          rr.bits_up = hostlog[q].bits_up;
          rr.bits_down = hostlog[q].bits_down;
          rr.master_level = hostlog[q].master_level;
          rr.exact_rechecks = hostlog[q].rechecks;
        }
    }
    done += batch;
  }
  if (report_host || levels_host) {
    unsigned int fl = 0;
    CK(c, cudaMemcpyAsync(&fl, c->scr.flags, 4, cudaMemcpyDeviceToHost, c->stream), "adacgd_step (status words to the host)");
    CK(c, cudaStreamSynchronize(c->stream), "adacgd_step (synchronising the stream)");
    if (fl & 2u) return fail(c, ADACGD_ERR_CUDA, "a device-side wait for an asynchronous copy timed out");
    if (fl & 1u) return fail(c, ADACGD_ERR_NONFINITE, "a gradient or estimator held Inf or NaN");
  }
  if (cudaGetLastError() != cudaSuccess) return cuda_fail(c, "adacgd_step");
  return ADACGD_OK;
}

static adacgd_status state_ptr(adacgd_ctx* c, int32_t which, void** p, size_t* bytes) {
  const size_t nd = (size_t)c->p.n * c->p.d * 4, dd = (size_t)c->p.d * 4;
  const bool has = c->p.loss != ADACGD_LOSS_NONE;
  switch (which) {
    case ADACGD_STATE_X: *p = c->x; *bytes = dd; break;
    case ADACGD_STATE_G: *p = c->G; *bytes = nd; break;
    case ADACGD_STATE_GRAD: *p = c->grad_cur; *bytes = nd; break;
    case ADACGD_STATE_GT: *p = c->gt_cur; *bytes = dd; break;
    case ADACGD_STATE_GM: *p = c->gm; *bytes = dd; break;
    case ADACGD_STATE_STEP: *p = &c->counters->step; *bytes = 8; return ADACGD_OK;
    case ADACGD_STATE_BITS_UP: *p = &c->counters->bits_up; *bytes = 8; return ADACGD_OK;
    case ADACGD_STATE_BITS_DOWN: *p = &c->counters->bits_down; *bytes = 8; return ADACGD_OK;
    case ADACGD_STATE_LEVELS: *p = c->levels; *bytes = (size_t)c->p.n * 4; return ADACGD_OK;
    case ADACGD_STATE_FLAGS: *p = c->scr.flags; *bytes = 4; return ADACGD_OK;
    case ADACGD_STATE_RECHECKS: *p = c->scr.flags + 1; *bytes = 4; return ADACGD_OK;
    case ADACGD_STATE_FALLBACKS: *p = c->scr.flags + 2; *bytes = 4; return ADACGD_OK;
    case ADACGD_STATE_LIST_LEVELS: *p = c->scr.flags + 3; *bytes = 4; return ADACGD_OK;
    case ADACGD_STATE_DEVICE: *p = nullptr; *bytes = 4; return ADACGD_OK;   // host-side value, handled by the caller
    case ADACGD_STATE_REFRESHES: *p = nullptr; *bytes = 8; return ADACGD_OK;   // host-side value
    case ADACGD_STATE_INC_COLUMNS:
      if (!c->gs.inc) return fail(c, ADACGD_ERR_INVALID_ARG, "context was created without ADACGD_FLAG_INCREMENTAL_FORWARD");
      *p = c->gs.inc_cols; *bytes = 8; return ADACGD_OK;
    default: return fail(c, ADACGD_ERR_INVALID_ARG, "unknown state item");
  }
  if (!has) return fail(c, ADACGD_ERR_INVALID_ARG, "context has no objective, hence no iterate state");
  return ADACGD_OK;
}

adacgd_status adacgd_get_state(adacgd_ctx* c, int32_t which, void* dst, size_t bytes, int32_t dst_is_device) {
  if (!c) return fail(nullptr, ADACGD_ERR_INVALID_ARG, "ctx is NULL");
  if (!dst) return fail(c, ADACGD_ERR_INVALID_ARG, "dst is NULL");
  void* p;
  size_t want;
  adacgd_status s = state_ptr(c, which, &p, &want);
  if (s != ADACGD_OK) return s;
  if (bytes != want) return fail(c, ADACGD_ERR_INVALID_ARG, "bytes does not match the item's size");
  if (which == ADACGD_STATE_DEVICE) {   // needs no device work, so it also answers when another device is current
    if (dst_is_device) return fail(c, ADACGD_ERR_INVALID_ARG, "ADACGD_STATE_DEVICE is returned to host memory");
    *(int32_t*)dst = c->device;
    return ADACGD_OK;
  }
  if (which == ADACGD_STATE_REFRESHES) {
    if (dst_is_device) return fail(c, ADACGD_ERR_INVALID_ARG, "ADACGD_STATE_REFRESHES is returned to host memory");
    *(uint64_t*)dst = c->refreshes;
    return ADACGD_OK;
  }
  if ((s = check_device(c, "adacgd_get_state")) != ADACGD_OK) return s;
  CK(c, cudaMemcpyAsync(dst, p, bytes, dst_is_device ? cudaMemcpyDeviceToDevice : cudaMemcpyDeviceToHost, c->stream), "adacgd_get_state (copy)");
  CK(c, cudaStreamSynchronize(c->stream), "adacgd_get_state (synchronising the stream)");
  return ADACGD_OK;
}

adacgd_status adacgd_set_state(adacgd_ctx* c, int32_t which, const void* src, size_t bytes, int32_t src_is_device) {
  if (!c) return fail(nullptr, ADACGD_ERR_INVALID_ARG, "ctx is NULL");
  if (!src) return fail(c, ADACGD_ERR_INVALID_ARG, "src is NULL");
  if (which == ADACGD_STATE_FLAGS || which == ADACGD_STATE_LEVELS || which == ADACGD_STATE_RECHECKS ||
      which == ADACGD_STATE_FALLBACKS || which == ADACGD_STATE_LIST_LEVELS || which == ADACGD_STATE_DEVICE ||
      which == ADACGD_STATE_INC_COLUMNS || which == ADACGD_STATE_REFRESHES)
    return fail(c, ADACGD_ERR_INVALID_ARG, "this item is read-only");
  void* p;
  size_t want;
  adacgd_status s = state_ptr(c, which, &p, &want);
  if (s != ADACGD_OK) return s;
  if (bytes != want) return fail(c, ADACGD_ERR_INVALID_ARG, "bytes does not match the item's size");
  if ((s = check_device(c, "adacgd_set_state")) != ADACGD_OK) return s;
  c->inc_dirty = true;   // the kept forward products no longer belong to the state
  CK(c, cudaMemcpyAsync(p, src, bytes, src_is_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice, c->stream), "adacgd_set_state (copy)");
  CK(c, cudaStreamSynchronize(c->stream), "adacgd_set_state (synchronising the stream)");
  return ADACGD_OK;
}

adacgd_status adacgd_set_refresh_period(adacgd_ctx* c, int32_t period) {
  if (!c) return fail(nullptr, ADACGD_ERR_INVALID_ARG, "ctx is NULL");
  if (!c->gs.inc) return fail(c, ADACGD_ERR_INVALID_ARG, "context was created without ADACGD_FLAG_INCREMENTAL_FORWARD (dense layout)");
  if (period < 1) return fail(c, ADACGD_ERR_INVALID_ARG, "period must be >= 1");
  c->refresh_period = period;
  return ADACGD_OK;
}

const char* adacgd_last_error(const adacgd_ctx* ctx) { return ctx ? ctx->err.c_str() : g_err.c_str(); }

void adacgd_destroy(adacgd_ctx* ctx) {
  if (!ctx) return;
  for (cudaEvent_t e : ctx->ev_beg) cudaEventDestroy(e);
  for (cudaEvent_t e : ctx->ev_end) cudaEventDestroy(e);
  if (ctx->pair_exec) cudaGraphExecDestroy(ctx->pair_exec);
  for (cudaEvent_t e : ctx->copy_ev) if (e) cudaEventDestroy(e);
  if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
  delete ctx;
}

static const char* const kKernelNames[KID_COUNT] = {
    "memset", "k_hist<1>", "k_hist<2>", "k_hist<3>", "k_scan", "k_energy", "k_quant_err", "k_pick",
    "k_exact_sums+k_pick_exact", "k_tiecount+k_tiescan", "k_update", "k_dense_fwd", "k_dense_bwd",
    "k_grad_reduce", "k_loss_reduce", "k_axpy_log", "k_log_step", "k_sample", "k_bracket", "k_pass1", "k_lhist", "k_lcollect", "k_small_rows",
    "k_csr_fwd", "k_csc_bwd", "k_csr_residual", "k_delta_scan", "k_dense_inc", "k_inc_finish", "k_side"};

int32_t adacgd_profile_kernel_count(void) { return KID_COUNT; }

const char* adacgd_profile_kernel_name(int32_t id) { return (id >= 0 && id < KID_COUNT) ? kKernelNames[id] : ""; }

adacgd_status adacgd_profile_enable(adacgd_ctx* c, int32_t max_records) {
  if (!c) return fail(nullptr, ADACGD_ERR_INVALID_ARG, "ctx is NULL");
  if (max_records <= 0) {
    c->prof = nullptr;
    c->scr.prof = nullptr;
    c->gs.prof = nullptr;
    return ADACGD_OK;
  }
  while ((int)c->ev_beg.size() < max_records) {
    cudaEvent_t a, b;
    if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess)
      return cuda_fail(c, "adacgd_profile_enable");
    c->ev_beg.push_back(a);
    c->ev_end.push_back(b);
  }
  c->ev_id.assign(c->ev_beg.size(), 0);
  c->prof_store.cap = max_records;
  c->prof_store.used = 0;
  c->prof_store.beg = c->ev_beg.data();
  c->prof_store.end = c->ev_end.data();
  c->prof_store.id = c->ev_id.data();
  c->prof = &c->prof_store;
  c->scr.prof = c->prof;
  c->gs.prof = c->prof;
  return ADACGD_OK;
}

adacgd_status adacgd_profile_read(adacgd_ctx* c, double* ms_out, int64_t* records_out) {
  if (!c) return fail(nullptr, ADACGD_ERR_INVALID_ARG, "ctx is NULL");
  if (!ms_out || !records_out) return fail(c, ADACGD_ERR_INVALID_ARG, "output arrays must be non-NULL");
  for (int i = 0; i < KID_COUNT; ++i) { ms_out[i] = 0.0; records_out[i] = 0; }
  if (!c->prof) return ADACGD_OK;
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return cuda_fail(c, "adacgd_profile_read");
  for (int i = 0; i < c->prof->used; ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, c->prof->beg[i], c->prof->end[i]) != cudaSuccess)
      return cuda_fail(c, "adacgd_profile_read");
    ms_out[c->prof->id[i]] += (double)ms;
    records_out[c->prof->id[i]] += 1;
  }
  c->prof->used = 0;
  return ADACGD_OK;
}

int64_t adacgd_launch_count(const adacgd_ctx* ctx) { return ctx ? ctx->launches : 0; }

uint64_t adacgd_message_bits(const adacgd_cand* cand, int64_t d) {
  if (!cand || d < 1 || d >= (1ll << 31)) return 0;
  if (cand->kind == ADACGD_TOPK ? cand->param < 1 : (cand->kind != ADACGD_QUANT || cand->param < 2 || cand->param > 16)) return 0;
  CsetDev cs;
  memset(&cs, 0, sizeof(cs));
  cs.m = 1;
  cs.kind[0] = cand->kind;
  cs.param[0] = cand->param;
  return level_bits(cs, 1, d);
}

}  // extern "C"
