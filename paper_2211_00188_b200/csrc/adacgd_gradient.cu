// Stage a1: every worker's local gradient X_i = grad f_i(x) of the finite-sum
// objective (Eq. 1) for the three objectives of the workloads:
//   logistic loss + non-convex regulariser (Section 6), logistic + l2, least squares.
// A memory-bound GEMV pair per worker: z = A_i x (forward), X_i = A_i^T r(z) (backward).
#include <vector>

#include "adacgd_internal.cuh"

namespace adacgd {

constexpr int LOSS_BLOCK_ROWS = 8;  // sample rows per CTA in warp-per-row mode

__device__ __forceinline__ float warp_sum_f32(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Residual r = dl/dz / m and the sample's loss, from z = a.x and the target t.
__device__ __forceinline__ void residual(int loss, float z, float t, float inv_m, float* r, double* l) {
  if (loss == ADACGD_LOSS_LEAST_SQUARES) {
    const float e = z - t;
    *r = e * inv_m;
    *l = 0.5 * (double)e * (double)e;
  } else {
    // log(1+exp(-t z)); derivative -t * sigma(-t z), sigma(u) = 1/(1+exp(-u))
    const float u = -t * z;
    const float sig = 1.f / (1.f + expf(-u));
    *r = -t * sig * inv_m;
    const double du = (double)u;
    *l = fmax(du, 0.0) + log1p(exp(-fabs(du)));
  }
}

// One warp (CTA_ROW = false) or one CTA (CTA_ROW = true) per sample row.
template <bool CTA_ROW, bool ALIGNED>
__global__ void __launch_bounds__(TPB) k_dense_fwd(const float* __restrict__ A, const float* __restrict__ target,
                                                   const float* __restrict__ x, long long d, long long m_rows,
                                                   int loss, float* __restrict__ r, double* __restrict__ losspart) {
  const int worker = blockIdx.y;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const long long row = CTA_ROW ? (long long)blockIdx.x : (long long)blockIdx.x * LOSS_BLOCK_ROWS + wid;
  const bool live = row < m_rows;
  float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
  if (live) {
    const float* a = A + ((long long)worker * m_rows + row) * d;
    const int tid = CTA_ROW ? threadIdx.x : lane;
    const int nth = CTA_ROW ? TPB : 32;
    if (ALIGNED) {
      const float4* a4 = reinterpret_cast<const float4*>(a);
      const float4* x4 = reinterpret_cast<const float4*>(x);
      const long long n4 = d >> 2;
      long long c = tid;
      for (; c + nth < n4; c += 2 * nth) {
        const float4 p = a4[c], q = a4[c + nth];
        const float4 xp = x4[c], xq = x4[c + nth];
        acc0 = fmaf(p.x, xp.x, acc0); acc1 = fmaf(p.y, xp.y, acc1);
        acc2 = fmaf(p.z, xp.z, acc2); acc3 = fmaf(p.w, xp.w, acc3);
        acc0 = fmaf(q.x, xq.x, acc0); acc1 = fmaf(q.y, xq.y, acc1);
        acc2 = fmaf(q.z, xq.z, acc2); acc3 = fmaf(q.w, xq.w, acc3);
      }
      for (; c < n4; c += nth) {
        const float4 p = a4[c];
        const float4 xp = x4[c];
        acc0 = fmaf(p.x, xp.x, acc0); acc1 = fmaf(p.y, xp.y, acc1);
        acc2 = fmaf(p.z, xp.z, acc2); acc3 = fmaf(p.w, xp.w, acc3);
      }
    } else {
      for (long long c = tid; c < d; c += nth) acc0 = fmaf(a[c], x[c], acc0);
    }
  }
  float z = warp_sum_f32((acc0 + acc1) + (acc2 + acc3));
  __shared__ float zs[TPB / 32];
  __shared__ double ls[TPB / 32];
  if (CTA_ROW) {
    if (lane == 0) zs[wid] = z;
    __syncthreads();
    z = 0.f;
    for (int w = 0; w < TPB / 32; ++w) z += zs[w];
  }
  double l = 0.0;
  if (live && lane == 0 && (!CTA_ROW || wid == 0)) {
    float rr;
    residual(loss, z, target[(long long)worker * m_rows + row], 1.f / (float)m_rows, &rr, &l);
    r[(long long)worker * m_rows + row] = rr;
  }
  if (CTA_ROW) {
    if (threadIdx.x == 0) losspart[(long long)worker * gridDim.x + blockIdx.x] = l;
  } else {
    if (lane == 0) ls[wid] = l;
    __syncthreads();
    if (threadIdx.x == 0) {
      double s = 0.0;
      for (int w = 0; w < TPB / 32; ++w) s += ls[w];
      losspart[(long long)worker * gridDim.x + blockIdx.x] = s;
    }
  }
}

__device__ __forceinline__ float reg_grad(int loss, float lambda, float x) {
  if (loss == ADACGD_LOSS_LOGISTIC_NCVX) {
    const float t = 1.f + x * x;
    return lambda * 2.f * x / (t * t);
  }
  if (loss == ADACGD_LOSS_LOGISTIC_L2) return lambda * x;
  return 0.f;
}

// Thread owns 4 consecutive columns; blockIdx.y = worker * split + s walks the rows of slice s.
template <bool ALIGNED>
__global__ void __launch_bounds__(TPB) k_dense_bwd(const float* __restrict__ A, const float* __restrict__ r,
                                                   const float* __restrict__ x, long long d, long long m_rows,
                                                   int split, int loss, float lambda, float* __restrict__ grads,
                                                   float* __restrict__ part, int n) {
  const int worker = blockIdx.y / split, s = blockIdx.y % split;
  const long long per = (m_rows + split - 1) / split;
  const long long l0 = s * per, l1 = (l0 + per < m_rows) ? l0 + per : m_rows;
  const long long c0 = (long long)blockIdx.x * (TPB * 4) + threadIdx.x * 4;
  __shared__ float rs[1024];
  float acc[4][4];
#pragma unroll
  for (int u = 0; u < 4; ++u)
#pragma unroll
    for (int k = 0; k < 4; ++k) acc[u][k] = 0.f;
  const float* Aw = A + (long long)worker * m_rows * d;
  for (long long base = l0; base < l1; base += 1024) {
    const int cnt = (int)((l1 - base < 1024) ? (l1 - base) : 1024);
    __syncthreads();
    for (int i = threadIdx.x; i < cnt; i += TPB) rs[i] = r[(long long)worker * m_rows + base + i];
    __syncthreads();
    if (c0 < d) {
      int i = 0;
      if (ALIGNED) {
        for (; i + 4 <= cnt; i += 4) {
          float4 a[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) a[u] = *reinterpret_cast<const float4*>(Aw + (base + i + u) * d + c0);
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const float ru = rs[i + u];
            acc[u][0] = fmaf(a[u].x, ru, acc[u][0]); acc[u][1] = fmaf(a[u].y, ru, acc[u][1]);
            acc[u][2] = fmaf(a[u].z, ru, acc[u][2]); acc[u][3] = fmaf(a[u].w, ru, acc[u][3]);
          }
        }
      }
      for (; i < cnt; ++i) {
        const float ru = rs[i];
        const float* a = Aw + (base + i) * d + c0;
#pragma unroll
        for (int k = 0; k < 4; ++k)
          if (c0 + k < d) acc[0][k] = fmaf(a[k], ru, acc[0][k]);
      }
    }
  }
  if (c0 >= d) return;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    if (c0 + k >= d) break;
    const float v = (acc[0][k] + acc[1][k]) + (acc[2][k] + acc[3][k]);
    if (split == 1) grads[(long long)worker * d + c0 + k] = v + reg_grad(loss, lambda, x[c0 + k]);
    else part[((long long)s * n + worker) * d + c0 + k] = v;
  }
}

__global__ void k_grad_reduce(const float* __restrict__ part, const float* __restrict__ x, long long d, int n,
                              int split, int loss, float lambda, float* __restrict__ grads) {
  const long long c = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int worker = blockIdx.y;
  if (c >= d) return;
  float v = 0.f;
  for (int s = 0; s < split; ++s) v += part[((long long)s * n + worker) * d + c];
  grads[(long long)worker * d + c] = v + reg_grad(loss, lambda, x[c]);
}

// CSR forward: one warp per sample row.
__global__ void __launch_bounds__(TPB) k_csr_fwd(const long long* __restrict__ rowptr, const int* __restrict__ col,
                                                 const float* __restrict__ val, const float* __restrict__ target,
                                                 const float* __restrict__ x, long long m_rows, int loss,
                                                 float* __restrict__ r, double* __restrict__ losspart) {
  const int worker = blockIdx.y;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const long long row = (long long)blockIdx.x * LOSS_BLOCK_ROWS + wid;
  const bool live = row < m_rows;
  float acc = 0.f;
  if (live) {
    const long long g = (long long)worker * m_rows + row;
    const long long e0 = rowptr[g], e1 = rowptr[g + 1];
    // eight entries per lane in flight: their values and column indices first, then the eight gathers;
    // a lane still adds its products in ascending entry order
    for (long long e = e0 + lane; e < e1; e += 32 * 8) {
      int c[8];
      float v[8], xv[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const long long ee = e + 32 * k;
        const bool ok = ee < e1;
        c[k] = ok ? __ldcs(&col[ee]) : 0;
        v[k] = ok ? __ldcs(&val[ee]) : 0.f;
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) xv[k] = __ldg(&x[c[k]]);
#pragma unroll
      for (int k = 0; k < 8; ++k)
        if (e + 32 * k < e1) acc = fmaf(v[k], xv[k], acc);
    }
  }
  const float z = warp_sum_f32(acc);
  __shared__ double ls[TPB / 32];
  double l = 0.0;
  if (live && lane == 0) {
    float rr;
    residual(loss, z, target[(long long)worker * m_rows + row], 1.f / (float)m_rows, &rr, &l);
    r[(long long)worker * m_rows + row] = rr;
  }
  if (lane == 0) ls[wid] = l;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int w = 0; w < TPB / 32; ++w) s += ls[w];
    losspart[(long long)worker * gridDim.x + blockIdx.x] = s;
  }
}

// CSR backward on the transposed copy: one thread per column, entries in ascending sample row.
__global__ void __launch_bounds__(TPB) k_csc_bwd(const long long* __restrict__ cptr, const int* __restrict__ crow,
                                                 const float* __restrict__ cval, const float* __restrict__ r,
                                                 const float* __restrict__ x, long long d, long long m_rows, int loss,
                                                 float lambda, float* __restrict__ grads) {
  const int worker = blockIdx.y;
  const long long c = (long long)blockIdx.x * TPB + threadIdx.x;
  if (c >= d) return;
  const long long e0 = cptr[(long long)worker * d + c], e1 = cptr[(long long)worker * d + c + 1];
  const float* rw = r + (long long)worker * m_rows;
  float acc = 0.f;
  for (long long e = e0; e < e1; ++e) acc = fmaf(cval[e], rw[crow[e]], acc);
  grads[(long long)worker * d + c] = acc + reg_grad(loss, lambda, x[c]);
}

// f(x) = (1/n) sum_i [ (1/m) sum_l loss_l + reg(x) ]  in binary64, fixed summation order.
__global__ void __launch_bounds__(1024) k_loss_reduce(const double* __restrict__ losspart, int n, int blocks,
                                                      long long m_rows, const float* __restrict__ x, long long d,
                                                      int loss, float lambda, double* __restrict__ out) {
  __shared__ double red[32];
  double a = 0.0;
  for (long long i = threadIdx.x; i < (long long)n * blocks; i += blockDim.x) a += losspart[i];
  a /= ((double)m_rows * (double)n);
  double rg = 0.0;
  if (loss == ADACGD_LOSS_LOGISTIC_NCVX || loss == ADACGD_LOSS_LOGISTIC_L2) {
    for (long long c = threadIdx.x; c < d; c += blockDim.x) {
      const double xv = (double)x[c];
      rg += (loss == ADACGD_LOSS_LOGISTIC_NCVX) ? xv * xv / (1.0 + xv * xv) : 0.5 * xv * xv;
    }
    rg *= (double)lambda;
  }
  a += rg;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = a;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) s += red[w];
    *out = s;
  }
}

// --------------------------------------------------------------------------
static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// The split decides the size of the partial-sum buffer, so it is part of the workspace layout and must not
// depend on the device a context later runs on: it is taken for a nominal 148 SMs.
static int choose_split(const adacgd_problem& p) {
  if (p.layout == ADACGD_LAYOUT_CSR) return 1;
  constexpr int NOMINAL_SMS = 148;
  const long long ctas = (long long)p.n * ((p.d + TPB * 4 - 1) / (TPB * 4));
  long long split = (NOMINAL_SMS * 4 + ctas - 1) / ctas;
  if (split < 1) split = 1;
  if (split > 16) split = 16;
  if (split > p.m_rows) split = p.m_rows;
  return (int)split;
}

static bool cta_row_mode(const adacgd_problem& p) { return p.layout == ADACGD_LAYOUT_DENSE && p.d >= 32768; }

static int loss_blocks_of(const adacgd_problem& p) {
  return cta_row_mode(p) ? (int)p.m_rows : (int)((p.m_rows + LOSS_BLOCK_ROWS - 1) / LOSS_BLOCK_ROWS);
}

size_t grad_scratch_bytes(const adacgd_problem& p) {
  if (p.loss == ADACGD_LOSS_NONE) return 0;
  size_t o = 0;
  o = align_up(o + (size_t)p.n * p.m_rows * 4, 256);
  const int split = choose_split(p);
  if (split > 1) o = align_up(o + (size_t)split * p.n * p.d * 4, 256);
  o = align_up(o + (size_t)p.n * loss_blocks_of(p) * 8, 256);
  o = align_up(o + 8, 256);
  if (p.layout == ADACGD_LAYOUT_CSR) {
    o = align_up(o + ((size_t)p.n * p.d + 1) * 8, 256);
    o = align_up(o + (size_t)p.csr_nnz * 4, 256);
    o = align_up(o + (size_t)p.csr_nnz * 4, 256);
  }
  return o;
}

void carve_grad_scratch(GradScratch* g, void* base, const adacgd_problem& p) {
  char* b = (char*)base;
  size_t o = 0;
  g->split = choose_split(p);
  g->loss_blocks = loss_blocks_of(p);
  g->r = (float*)(b + o); o = align_up(o + (size_t)p.n * p.m_rows * 4, 256);
  g->part = nullptr;
  if (g->split > 1) { g->part = (float*)(b + o); o = align_up(o + (size_t)g->split * p.n * p.d * 4, 256); }
  g->losspart = (double*)(b + o); o = align_up(o + (size_t)p.n * g->loss_blocks * 8, 256);
  g->loss = (double*)(b + o); o = align_up(o + 8, 256);
  g->csc_ptr = nullptr; g->csc_row = nullptr; g->csc_val = nullptr;
  if (p.layout == ADACGD_LAYOUT_CSR) {
    g->csc_ptr = (long long*)(b + o); o = align_up(o + ((size_t)p.n * p.d + 1) * 8, 256);
    g->csc_row = (int*)(b + o); o = align_up(o + (size_t)p.csr_nnz * 4, 256);
    g->csc_val = (float*)(b + o);
  }
  g->prof = nullptr;
}

int launch_gradient(const adacgd_problem& p, const GradScratch& g, const float* x, float* grads,
                    cudaStream_t stream) {
  if (p.layout == ADACGD_LAYOUT_CSR) {
    int launches = 0;
    prof_begin(g.prof, KID_CSR_FWD, stream);
    k_csr_fwd<<<dim3((unsigned)g.loss_blocks, p.n), TPB, 0, stream>>>((const long long*)p.csr_rowptr, p.csr_col, p.csr_val,
                                                                      p.target, x, p.m_rows, p.loss, g.r, g.losspart);
    prof_end(g.prof, stream);
    ++launches;
    prof_begin(g.prof, KID_CSC_BWD, stream);
    k_csc_bwd<<<dim3((unsigned)((p.d + TPB - 1) / TPB), p.n), TPB, 0, stream>>>(g.csc_ptr, g.csc_row, g.csc_val, g.r, x,
                                                                                p.d, p.m_rows, p.loss, p.lambda, grads);
    prof_end(g.prof, stream);
    ++launches;
    prof_begin(g.prof, KID_LOSS, stream);
    k_loss_reduce<<<1, 1024, 0, stream>>>(g.losspart, p.n, g.loss_blocks, p.m_rows, x, p.d, p.loss, p.lambda, g.loss);
    prof_end(g.prof, stream);
    ++launches;
    return cudaGetLastError() == cudaSuccess ? launches : -1;
  }
  const bool al = (p.d % 4 == 0) && (((uintptr_t)p.A | (uintptr_t)x | (uintptr_t)grads) & 15) == 0;
  int launches = 0;
  prof_begin(g.prof, KID_GRAD_FWD, stream);
  if (cta_row_mode(p)) {
    const dim3 grid((unsigned)p.m_rows, p.n);
    if (al) k_dense_fwd<true, true><<<grid, TPB, 0, stream>>>(p.A, p.target, x, p.d, p.m_rows, p.loss, g.r, g.losspart);
    else k_dense_fwd<true, false><<<grid, TPB, 0, stream>>>(p.A, p.target, x, p.d, p.m_rows, p.loss, g.r, g.losspart);
  } else {
    const dim3 grid((unsigned)g.loss_blocks, p.n);
    if (al) k_dense_fwd<false, true><<<grid, TPB, 0, stream>>>(p.A, p.target, x, p.d, p.m_rows, p.loss, g.r, g.losspart);
    else k_dense_fwd<false, false><<<grid, TPB, 0, stream>>>(p.A, p.target, x, p.d, p.m_rows, p.loss, g.r, g.losspart);
  }
  prof_end(g.prof, stream);
  ++launches;
  const dim3 bgrid((unsigned)((p.d + TPB * 4 - 1) / (TPB * 4)), p.n * g.split);
  prof_begin(g.prof, KID_GRAD_BWD, stream);
  if (al) k_dense_bwd<true><<<bgrid, TPB, 0, stream>>>(p.A, g.r, x, p.d, p.m_rows, g.split, p.loss, p.lambda, grads, g.part, p.n);
  else k_dense_bwd<false><<<bgrid, TPB, 0, stream>>>(p.A, g.r, x, p.d, p.m_rows, g.split, p.loss, p.lambda, grads, g.part, p.n);
  prof_end(g.prof, stream);
  ++launches;
  if (g.split > 1) {
    prof_begin(g.prof, KID_GRAD_REDUCE, stream);
    k_grad_reduce<<<dim3((unsigned)((p.d + 255) / 256), p.n), 256, 0, stream>>>(g.part, x, p.d, p.n, g.split, p.loss, p.lambda, grads);
    prof_end(g.prof, stream);
    ++launches;
  }
  prof_begin(g.prof, KID_LOSS, stream);
  k_loss_reduce<<<1, 1024, 0, stream>>>(g.losspart, p.n, g.loss_blocks, p.m_rows, x, p.d, p.loss, p.lambda, g.loss);
  prof_end(g.prof, stream);
  ++launches;
  return cudaGetLastError() == cudaSuccess ? launches : -1;
}

}  // namespace adacgd

namespace adacgd {

// Builds the transposed copy of a CSR problem (host side, once per context): stable counting sort by
// (worker, column), so that the entries of a column keep ascending sample-row order and the
// backward sums have a fixed order.  Returns a message on failure, nullptr on success.
const char* build_csc(const adacgd_problem& p, const GradScratch& g, cudaStream_t stream) {
  const long long rows = (long long)p.n * p.m_rows, nnz = p.csr_nnz, cols = (long long)p.n * p.d;
  std::vector<long long> rowptr((size_t)rows + 1), cptr((size_t)cols + 1, 0);
  std::vector<int> col((size_t)nnz), crow((size_t)nnz);
  std::vector<float> val((size_t)nnz), cval((size_t)nnz);
  if (cudaMemcpyAsync(rowptr.data(), p.csr_rowptr, (rows + 1) * 8, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
      cudaMemcpyAsync(col.data(), p.csr_col, nnz * 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
      cudaMemcpyAsync(val.data(), p.csr_val, nnz * 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
      cudaStreamSynchronize(stream) != cudaSuccess)
    return "copying the CSR arrays to the host failed";
  if (rowptr[0] != 0 || rowptr[(size_t)rows] != nnz) return "csr_rowptr must start at 0 and end at csr_nnz";
  for (long long r = 0; r < rows; ++r) {
    if (rowptr[(size_t)r + 1] < rowptr[(size_t)r]) return "csr_rowptr must be non-decreasing";
    const long long w = r / p.m_rows;
    for (long long e = rowptr[(size_t)r]; e < rowptr[(size_t)r + 1]; ++e) {
      if (col[(size_t)e] < 0 || col[(size_t)e] >= p.d) return "csr_col out of range";
      ++cptr[(size_t)(w * p.d + col[(size_t)e]) + 1];
    }
  }
  for (long long c = 0; c < cols; ++c) cptr[(size_t)c + 1] += cptr[(size_t)c];
  std::vector<long long> fill(cptr.begin(), cptr.end() - 1);
  for (long long r = 0; r < rows; ++r) {
    const long long w = r / p.m_rows;
    for (long long e = rowptr[(size_t)r]; e < rowptr[(size_t)r + 1]; ++e) {
      const long long at = fill[(size_t)(w * p.d + col[(size_t)e])]++;
      crow[(size_t)at] = (int)(r - w * p.m_rows);
      cval[(size_t)at] = val[(size_t)e];
    }
  }
  if (cudaMemcpyAsync(g.csc_ptr, cptr.data(), (cols + 1) * 8, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
      cudaMemcpyAsync(g.csc_row, crow.data(), nnz * 4, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
      cudaMemcpyAsync(g.csc_val, cval.data(), nnz * 4, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
      cudaStreamSynchronize(stream) != cudaSuccess)
    return "copying the transposed arrays to the device failed";
  return nullptr;
}

}  // namespace adacgd
