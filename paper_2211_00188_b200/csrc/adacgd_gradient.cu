// Stage a1: every worker's local gradient X_i = grad f_i(x) of the finite-sum
// objective (Eq. 1) for the three objectives of the workloads:
//   logistic loss + non-convex regulariser (Section 6), logistic + l2, least squares.
// A memory-bound GEMV pair per worker: z = A_i x (forward), X_i = A_i^T r(z) (backward).
#include <vector>

#include "adacgd_device.cuh"

namespace adacgd {

constexpr int LOSS_BLOCK_ROWS = 8;  // sample rows per CTA in warp-per-row mode

__device__ __forceinline__ u32 warp_sum_u32_g(u32 v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

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

// f(x) = (1/n) sum_i [ (1/m) sum_l loss_l + reg(x) ] in binary64, finished by whichever CTA of the forward kernel
// comes last.  Every CTA leaves the loss of its sample rows and the regulariser of its share of x; the last one
// (a ticket that it resets for the next launch) adds both lists up, thread t taking entries t, t + blockDim, ...
// and then lanes and warps, so the sum depends on the launch shape only.
struct LossTail {
  double* losspart;   // [CTAs of the launch]
  double* regpart;    // [CTAs of the launch]
  u32* ticket;
  const float* x;
  long long d, m_rows;
  int loss, n;
  float lambda;
  double* out;
  int fused;          // 0: the CTAs only leave their losses; k_loss_reduce adds them up (grids of thousands of short CTAs,
                      // where a completion count at the end of every CTA costs more than one more launch)
};
__device__ __forceinline__ double block_sum_f64(double v, double* red32) {   // result valid in thread 0
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if (lane == 0) red32[wid] = v;
  __syncthreads();
  double t = 0.0;
  if (threadIdx.x == 0)
    for (int w = 0; w < nw; ++w) t += red32[w];
  return t;
}
// Called by every thread of every CTA (a 2-D grid); `cta_loss` is read from thread 0.  The regulariser is left to
// the first ceil(d / REG_SLICE) CTAs (the others have nothing to add), and the completion count has two levels, one
// word per grid row and one for the rows, so that thousands of short CTAs do not queue up on a single address.
constexpr int REG_SLICE = 4096;
__device__ void loss_tail(const LossTail& t, double cta_loss) {
  __shared__ double lt_red[32];
  __shared__ u32 lt_last;
  const long long ncta = (long long)gridDim.x * gridDim.y;
  const long long cta = (long long)blockIdx.y * gridDim.x + blockIdx.x;
  if (!t.fused) {
    if (threadIdx.x == 0) t.losspart[cta] = cta_loss;
    return;
  }
  const bool has_reg = t.loss == ADACGD_LOSS_LOGISTIC_NCVX || t.loss == ADACGD_LOSS_LOGISTIC_L2;
  long long per = REG_SLICE;
  while ((t.d + per - 1) / per > ncta) per *= 2;
  const long long nreg = has_reg ? (t.d + per - 1) / per : 0;
  if (cta < nreg) {
    double rg = 0.0;
    const long long c0 = cta * per, c1 = (c0 + per < t.d) ? c0 + per : t.d;
    for (long long c = c0 + threadIdx.x; c < c1; c += blockDim.x) {
      const double xv = (double)t.x[c];
      rg += (t.loss == ADACGD_LOSS_LOGISTIC_NCVX) ? xv * xv / (1.0 + xv * xv) : 0.5 * xv * xv;
    }
    rg = block_sum_f64(rg, lt_red);
    if (threadIdx.x == 0) t.regpart[cta] = rg;
  }
  if (threadIdx.x == 0) {
    t.losspart[cta] = cta_loss;
    __threadfence();
    u32 last = 0u;
    if (atomicAdd(&t.ticket[1 + blockIdx.y], 1u) == gridDim.x - 1u) {        // last CTA of this grid row
      t.ticket[1 + blockIdx.y] = 0u;
      __threadfence();
      last = (atomicAdd(&t.ticket[0], 1u) == gridDim.y - 1u) ? 1u : 0u;       // last grid row
    }
    lt_last = last;
  }
  __syncthreads();
  if (!lt_last) return;
  __threadfence();
  double a = 0.0, b = 0.0;
  for (long long i = threadIdx.x; i < ncta; i += blockDim.x) a += __ldcg(&t.losspart[i]);
  for (long long i = threadIdx.x; i < nreg; i += blockDim.x) b += __ldcg(&t.regpart[i]);
  a = block_sum_f64(a, lt_red);
  b = block_sum_f64(b, lt_red);
  if (threadIdx.x == 0) {
    *t.out = a / ((double)t.m_rows * (double)t.n) + (double)t.lambda * b;
    t.ticket[0] = 0u;
  }
}

// One warp (CTA_ROW = false) or one CTA (CTA_ROW = true) per sample row.
// FUSED: the last CTA adds up the loss (loss_tail); otherwise every CTA only leaves its share for k_loss_reduce.
template <bool CTA_ROW, bool ALIGNED, bool FUSED>
__global__ void __launch_bounds__(TPB) k_dense_fwd(const float* __restrict__ A, const float* __restrict__ target,
                                                   const float* __restrict__ x, long long d, long long m_rows,
                                                   int loss, float* __restrict__ r, LossTail lt,
                                                   float* __restrict__ zout, const u32* __restrict__ gate) {
  // r == nullptr: only the products z = A x are wanted (zout); gate != nullptr: the launch only runs when the
  // word is zero (the incremental pass found too many changed columns and leaves the products to this kernel)
  pdl_wait();      // may be resident while the x update runs; the backward kernel is not let in early
  if (gate && *gate != 0u) return;
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
    if (zout) zout[(long long)worker * m_rows + row] = z;
    if (r) {
      float rr;
      residual(loss, z, target[(long long)worker * m_rows + row], 1.f / (float)m_rows, &rr, &l);
      r[(long long)worker * m_rows + row] = rr;
    }
  }
  if (r == nullptr) return;
  if (!CTA_ROW) {
    if (lane == 0) ls[wid] = l;
    __syncthreads();
    if (threadIdx.x == 0) {
      l = 0.0;
      for (int w = 0; w < TPB / 32; ++w) l += ls[w];
    }
  }
  if (FUSED) loss_tail(lt, l);
  else if (threadIdx.x == 0) lt.losspart[(long long)worker * gridDim.x + blockIdx.x] = l;
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
                                                   float* __restrict__ part, int n, u32* __restrict__ tickets) {
  pdl_wait();
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
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    if (c0 + k >= d) break;
    const float v = (acc[0][k] + acc[1][k]) + (acc[2][k] + acc[3][k]);
    if (split == 1) grads[(long long)worker * d + c0 + k] = v + reg_grad(loss, lambda, x[c0 + k]);
    else part[((long long)s * n + worker) * d + c0 + k] = v;
  }
  if (split == 1) return;
  // the slice of a column tile that finishes last adds the slices up, in slice order
  __shared__ u32 is_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    u32* t = &tickets[(long long)worker * gridDim.x + blockIdx.x];
    is_last = (atomicAdd(t, 1u) == (u32)(split - 1)) ? 1u : 0u;
    if (is_last) *t = 0u;   // ready for the next launch
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    if (c0 + k >= d) break;
    float v = 0.f;
    for (int q = 0; q < split; ++q) v += __ldcg(&part[((long long)q * n + worker) * d + c0 + k]);
    grads[(long long)worker * d + c0 + k] = v + reg_grad(loss, lambda, x[c0 + k]);
  }
}

// CSR forward: one warp per sample row.
__global__ void __launch_bounds__(TPB) k_csr_fwd(const long long* __restrict__ rowptr, const int* __restrict__ col,
                                                 const float* __restrict__ val, const float* __restrict__ target,
                                                 const float* __restrict__ x, long long m_rows, int loss,
                                                 float* __restrict__ r, LossTail lt) {
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
    l = 0.0;
    for (int w = 0; w < TPB / 32; ++w) l += ls[w];
  }
  loss_tail(lt, l);
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


// ---- CSR, column-blocked forward ------------------------------------------------------------------
// A gathered word of x costs a whole L1 wavefront when it comes from global memory but only a bank
// access when it comes from shared memory, and the forward pass gathers one word per stored entry.  So the
// columns are cut into nb blocks of `blk` columns that fit in shared memory; a CTA keeps one block of x
// there and walks the sample rows of ALL workers (they share x), one warp per row, over the entries of
// that block only.  Column indices ascend inside a row, so those entries are the contiguous span
// [split[b][row], split[b+1][row]) found once at init.  zpart[b][row] receives the block's share of
// a_row . x; k_csr_residual adds the shares in block order.
constexpr int CSR_BLK_MAX = 49152;   // columns of x per block: 192 KB of shared memory
constexpr int CSR_FWD_TPB = 1024;
constexpr int CSR_NB_MAX = 8;        // wider problems take the plain warp-per-row kernel
constexpr int CSR_FWD_UNR = 3;       // groups of four entries a lane requests at once

__global__ void __launch_bounds__(CSR_FWD_TPB) k_csr_fwd_blocked(const long long* __restrict__ qptr, const u16* __restrict__ col16,
                                                                 const float* __restrict__ val, const float* __restrict__ x,
                                                                 long long rows, long long d, int blk,
                                                                 float* __restrict__ zpart) {
  pdl_begin();
  // val / col16: the entries regrouped at init, block-major, every (block, row) span padded with zero entries to a
  // multiple of four so that a lane reads four values (16 bytes) and four 16-bit block-relative columns (8 bytes) per
  // request: 6 bytes per stored entry.  qptr[b * rows + row]: first group of four of the span.
  extern __shared__ __align__(16) float xs[];
  const int b = blockIdx.y;
  const long long cbase = (long long)b * blk;
  const int ncol = (int)((d - cbase < blk) ? (d - cbase) : blk);
  for (int i = threadIdx.x; i < ncol; i += CSR_FWD_TPB) xs[i] = x[cbase + i];
  __syncthreads();
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const long long* q = qptr + (long long)b * rows;
  const float4* vq = (const float4*)val;
  const uint2* cq = (const uint2*)col16;
  const long long stride = (long long)gridDim.x * (CSR_FWD_TPB / 32);
  long long row = (long long)blockIdx.x * (CSR_FWD_TPB / 32) + wid;
  // Two rows ahead the span is known, one row ahead its first CSR_FWD_UNR groups per lane are already requested
  // while the current row is summed: a warp always has a row's worth of entries in flight.
  struct Batch { uint2 c[CSR_FWD_UNR]; float4 v[CSR_FWD_UNR]; };
  auto request = [&](long long e0, long long e1, int o, Batch& t) {
    const float4* vp = vq + e0 + lane;                    // offsets are 32-bit and relative to the lane's first group
    const uint2* cp = cq + e0 + lane;
    const int cnt = (int)(e1 - e0) - lane;                // this lane owns groups 32 k with 32 k < cnt
#pragma unroll
    for (int k = 0; k < CSR_FWD_UNR; ++k) {
      const bool ok = o + 32 * k < cnt;
      t.c[k] = ok ? __ldcs(cp + o + 32 * k) : make_uint2(0u, 0u);
      t.v[k] = ok ? __ldcs(vp + o + 32 * k) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };
  auto add = [&](const Batch& t, float acc) {             // a lane adds its products in ascending entry order;
#pragma unroll
    for (int k = 0; k < CSR_FWD_UNR; ++k) {               // absent and padding entries add 0 * xs[0]
      acc = fmaf(t.v[k].x, xs[t.c[k].x & 0xffffu], acc);
      acc = fmaf(t.v[k].y, xs[t.c[k].x >> 16], acc);
      acc = fmaf(t.v[k].z, xs[t.c[k].y & 0xffffu], acc);
      acc = fmaf(t.v[k].w, xs[t.c[k].y >> 16], acc);
    }
    return acc;
  };
  long long e0 = 0, e1 = 0, n0 = 0, n1 = 0;
  Batch cur, nxt;
  if (row < rows) { e0 = q[row]; e1 = q[row + 1]; request(e0, e1, 0, cur); }
  if (row + stride < rows) { n0 = q[row + stride]; n1 = q[row + stride + 1]; }
  for (; row < rows; row += stride) {
    const long long nnrow = row + 2 * stride;
    long long m0 = 0, m1 = 0;
    if (nnrow < rows) { m0 = q[nnrow]; m1 = q[nnrow + 1]; }
    if (row + stride < rows) request(n0, n1, 0, nxt);
    float acc = add(cur, 0.f);
    for (int o = 32 * CSR_FWD_UNR; o < (int)(e1 - e0); o += 32 * CSR_FWD_UNR) {   // the rest of a long span
      request(e0, e1, o, cur);
      acc = add(cur, acc);
    }
    acc = warp_sum_f32(acc);
    if (lane == 0) zpart[(long long)b * rows + row] = acc;
    e0 = n0; e1 = n1; n0 = m0; n1 = m1;
    cur = nxt;
  }
}

// z = sum over the column blocks (in block order), residual and loss of every sample row.
__global__ void __launch_bounds__(TPB) k_csr_residual(const float* __restrict__ zpart, int nb, long long rows,
                                                      const float* __restrict__ target, long long m_rows, int loss,
                                                      float* __restrict__ r, LossTail lt) {
  pdl_wait();      // the large backward kernel that follows is let in once this one runs, not before
  pdl_trigger();
  const int worker = blockIdx.y;
  const long long l = (long long)blockIdx.x * TPB + threadIdx.x;
  double ls = 0.0;
  if (l < m_rows) {
    const long long g = (long long)worker * m_rows + l;
    float z = zpart[g];
    for (int b = 1; b < nb; ++b) z += zpart[(long long)b * rows + g];
    float rr;
    residual(loss, z, target[g], 1.f / (float)m_rows, &rr, &ls);
    r[g] = rr;
  }
  __shared__ double red[TPB / 32];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ls += __shfl_xor_sync(0xffffffffu, ls, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ls;
  __syncthreads();
  double t = 0.0;
  if (threadIdx.x == 0)
    for (int w = 0; w < TPB / 32; ++w) t += red[w];
  loss_tail(lt, t);
}

// ---- CSR backward on the transposed copy, one contiguous span per warp --------------------------------
// A warp owns CSC_WCOLS consecutive columns of one worker at a time (two per lane).  Their entries are one contiguous
// span of the transposed arrays: it is read with coalesced loads, every entry is multiplied by its
// sample's residual (the worker's residuals sit in shared memory) and the products are parked in the
// warp's part of shared memory; then each lane adds the products of its columns in ascending sample
// order, so the sums have a fixed order.  A span that does not fit (the columns hold more than CSC_WPCAP
// entries) is walked column by column instead.  The warps of a CTA work on their own: the only CTA-wide
// barrier follows the load of the residuals.
constexpr int CSC_WCOLS = 64;      // columns a warp takes at a time (two per lane)
constexpr int CSC_WPCAP = 768;     // products parked per warp
constexpr int CSC_UNR = 6;         // entries a lane requests at once
constexpr int CSC_RCAP = 8192;     // residuals of a worker kept in shared memory
#ifndef CSC_TPB_N
#define CSC_TPB_N 64
#endif
constexpr int CSC_TPB = CSC_TPB_N;   // threads per CTA of the span kernel: small CTAs (c3: 512 threads 242 us, 256 117, 128 115, 64 113, 32 133)
__global__ void __launch_bounds__(CSC_TPB) k_csc_bwd_span(const long long* __restrict__ wbase, const u32* __restrict__ ptr32,
                                                      const u16* __restrict__ crow, const float* __restrict__ cval,
                                                      const float* __restrict__ r, const float* __restrict__ x,
                                                      long long d, long long m_rows, int loss, float lambda,
                                                      float* __restrict__ grads) {
  // crow: 16-bit sample indices (a worker has at most CSC_RCAP samples here)
  pdl_wait();      // no early launch of the kernel after this one: its CTAs would take room from this grid
  extern __shared__ __align__(16) float bsm[];   // [m_rows] residuals, then [CSC_TPB / 32][CSC_WPCAP] products
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  float* rs = bsm;
  float* prod = bsm + m_rows + (size_t)wid * CSC_WPCAP;
  const int worker = blockIdx.y;
  const u32* ptr = ptr32 + (long long)worker * (d + 1);
  const long long base = wbase[worker];
  const float* rw = r + (long long)worker * m_rows;
  for (int i = threadIdx.x; i < (int)m_rows; i += CSC_TPB) rs[i] = rw[i];
  __syncthreads();
  const long long ngroups = (d + CSC_WCOLS - 1) / CSC_WCOLS;
  const long long gstride = (long long)gridDim.x * (CSC_TPB / 32);
  // Column pointers and x of a group: this lane's columns c0 + lane and c0 + lane + 32, and the ends of the
  // warp's span.  The next group's are requested before the current group's entries.
  struct Grp { u32 pa[2], pb[2], e0, e1; float xv[2]; };
  auto fetch = [&](long long grp, Grp& q) {
    const long long c0 = grp * CSC_WCOLS;
    const long long c1 = (c0 + CSC_WCOLS < d) ? c0 + CSC_WCOLS : d;
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const long long c = c0 + lane + 32 * k;
      const bool ok = c < c1;
      q.pa[k] = ok ? ptr[c] : 0u;
      q.pb[k] = ok ? ptr[c + 1] : 0u;
      q.xv[k] = ok ? x[c] : 0.f;
    }
    q.e0 = ptr[c0];
    q.e1 = ptr[c1];
  };
  long long grp = (long long)blockIdx.x * (CSC_TPB / 32) + wid;
  Grp cur, nxt;
  if (grp < ngroups) fetch(grp, cur);
  for (; grp < ngroups; grp += gstride) {
    if (grp + gstride < ngroups) fetch(grp + gstride, nxt);
    const long long c0 = grp * CSC_WCOLS;
    const long long c1 = (c0 + CSC_WCOLS < d) ? c0 + CSC_WCOLS : d;
    const u32 e0 = cur.e0, span = cur.e1 - cur.e0;
    const u16* er = crow + base + e0;
    const float* ev = cval + base + e0;
    float acc[2] = {0.f, 0.f};
    if (span <= (u32)CSC_WPCAP) {
      const u16* erl = er + lane;
      const float* evl = ev + lane;
      float* pl = prod + lane;
      const int cnt = (int)span - lane;                  // this lane owns entries 32 k with 32 k < cnt
      for (int o = 0; o < cnt; o += 32 * CSC_UNR) {
        u16 rr[CSC_UNR];
        float vv[CSC_UNR];
#pragma unroll
        for (int k = 0; k < CSC_UNR; ++k) {
          const bool ok = o + 32 * k < cnt;
          rr[k] = ok ? __ldcs(erl + o + 32 * k) : (u16)0;
          vv[k] = ok ? __ldcs(evl + o + 32 * k) : 0.f;
        }
#pragma unroll
        for (int k = 0; k < CSC_UNR; ++k)
          if (o + 32 * k < cnt) pl[o + 32 * k] = vv[k] * rs[rr[k]];
      }
      __syncwarp();
#pragma unroll
      for (int k = 0; k < 2; ++k)
        for (u32 j = cur.pa[k] - e0; j < cur.pb[k] - e0; ++j) acc[k] += prod[j];   // empty for columns past the end
      __syncwarp();
    } else {
#pragma unroll
      for (int k = 0; k < 2; ++k)
        for (u32 j = cur.pa[k] - e0; j < cur.pb[k] - e0; ++j) acc[k] += ev[j] * rs[er[j]];
    }
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const long long c = c0 + lane + 32 * k;
      if (c < c1) grads[(long long)worker * d + c] = acc[k] + reg_grad(loss, lambda, cur.xv[k]);
    }
    cur = nxt;
  }
}

// The same sum by a kernel of its own, for forward launches whose CTAs do not count themselves.
__global__ void __launch_bounds__(1024) k_loss_reduce(const double* __restrict__ losspart, long long nparts, int n,
                                                      long long m_rows, const float* __restrict__ x, long long d,
                                                      int loss, float lambda, double* __restrict__ out) {
  pdl_wait();
  pdl_trigger();   // one CTA: the backward kernel may become resident beside it
  __shared__ double red[32];
  double a = 0.0;
  for (long long i = threadIdx.x; i < nparts; i += blockDim.x) a += losspart[i];
  a /= ((double)m_rows * (double)n);
  double rg = 0.0;
  if (loss == ADACGD_LOSS_LOGISTIC_NCVX || loss == ADACGD_LOSS_LOGISTIC_L2) {
    for (long long c = threadIdx.x; c < d; c += blockDim.x) {
      const double xv = (double)x[c];
      rg += (loss == ADACGD_LOSS_LOGISTIC_NCVX) ? xv * xv / (1.0 + xv * xv) : 0.5 * xv * xv;
    }
    rg *= (double)lambda;
  }
  a = block_sum_f64(a + rg, red);
  if (threadIdx.x == 0) *out = a;
}

// ---- incremental forward: z_i = A_i x kept up to date from the entries of g that changed -----------------
// x moves by -gamma g every iteration (Algorithm 1), so z_i = A_i x moves by -gamma u_i with u_i = A_i g, and g
// itself changes only where a worker (identity master) or the master sent something.  u_i is therefore
// kept between iterations and corrected by the changed entries alone: u_i += sum_c A_i[:, c] (g[c] - g_prev[c]),
// columns read from a column-major copy of the features.  Sums run in ascending column order inside a chunk
// of INC_CHUNK columns and the chunks are added in chunk order, so the result does not depend on scheduling.

// AT[w][c][l] = A[w][l][c]
__global__ void k_transpose_features(const float* __restrict__ A, float* __restrict__ AT, long long m_rows, long long d) {
  __shared__ float tile[32][33];
  const int w = blockIdx.z;
  const long long c0 = (long long)blockIdx.x * 32, l0 = (long long)blockIdx.y * 32;
  const float* a = A + (long long)w * m_rows * d;
  float* at = AT + (long long)w * m_rows * d;
  for (int j = threadIdx.y; j < 32; j += 8) {
    const long long l = l0 + j, c = c0 + threadIdx.x;
    tile[j][threadIdx.x] = (l < m_rows && c < d) ? a[l * d + c] : 0.f;
  }
  __syncthreads();
  for (int j = threadIdx.y; j < 32; j += 8) {
    const long long c = c0 + j, l = l0 + threadIdx.x;
    if (c < d && l < m_rows) at[c * m_rows + l] = tile[threadIdx.x][j];
  }
}

// One CTA per chunk of INC_CHUNK columns: the entries where g differs from g_prev, compacted in ascending
// column order with their differences.  The last CTA to finish adds the counts up and decides the route of the
// iteration: dl_flag[0] = 1, the changed columns are few enough to be gathered (k_dense_inc), or 0, z = A x is
// recomputed in full (u and g_prev then stay as they are and the next scan sees the accumulated change).
__global__ void __launch_bounds__(TPB) k_delta_scan(const float* __restrict__ g, const float* __restrict__ g_prev, long long d,
                                                    u32* __restrict__ count, int* __restrict__ idx, float* __restrict__ val,
                                                    u32* __restrict__ dl_flag, u64* __restrict__ inc_cols, u32 max_cols) {
  static_assert(INC_CHUNK == 2 * TPB, "two columns per thread");
  __shared__ u32 wsum[TPB / 32];
  __shared__ u32 last;
  const int chunk = blockIdx.x;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const long long c0 = (long long)chunk * INC_CHUNK + 2 * threadIdx.x;
  float dv[2] = {0.f, 0.f};
#pragma unroll
  for (int k = 0; k < 2; ++k)
    if (c0 + k < d) dv[k] = __fsub_rn(g[c0 + k], g_prev[c0 + k]);
  const u32 mine = (dv[0] != 0.f ? 1u : 0u) + (dv[1] != 0.f ? 1u : 0u);
  u32 inc = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const u32 t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  if (lane == 31) wsum[wid] = inc;
  __syncthreads();
  u32 before = 0, total = 0;
  for (int w = 0; w < TPB / 32; ++w) {
    if (w < wid) before += wsum[w];
    total += wsum[w];
  }
  u32 pos = before + inc - mine;
#pragma unroll
  for (int k = 0; k < 2; ++k) {
    if (dv[k] != 0.f) {
      idx[(long long)chunk * INC_CHUNK + pos] = (int)(c0 + k);
      val[(long long)chunk * INC_CHUNK + pos] = dv[k];
      ++pos;
    }
  }
  if (threadIdx.x == 0) {
    count[chunk] = total;
    __threadfence();
    last = (atomicAdd(&dl_flag[1], 1u) == gridDim.x - 1u) ? 1u : 0u;   // dl_flag[1]: completion ticket, cleared by the last CTA
  }
  __syncthreads();
  if (!last) return;
  __threadfence();
  u32 sum = 0;
  for (int c = threadIdx.x; c < (int)gridDim.x; c += TPB) sum += __ldcg(&count[c]);
  sum = warp_sum_u32_g(sum);
  if (lane == 0) wsum[wid] = sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    u32 all = 0;
    for (int w = 0; w < TPB / 32; ++w) all += wsum[w];
    const u32 go = (all <= max_cols) ? 1u : 0u;
    dl_flag[0] = go;
    dl_flag[1] = 0u;
    if (go && all) atomicAdd(inc_cols, (u64)all);
  }
}

// Contribution of one chunk's changed columns to u of one worker: ipart[w][chunk][l] = sum_c AT[w][c][l] dv[c],
// columns in ascending order, a thread per sample row (coalesced along l), four columns in flight.  The CTA of
// worker 0 and the first row tile also moves g_prev to g at those columns.
__global__ void __launch_bounds__(TPB) k_dense_inc(const float* __restrict__ AT, const u32* __restrict__ count,
                                                   const int* __restrict__ idx, const float* __restrict__ val, long long d,
                                                   long long m_rows, float* __restrict__ ipart, const u32* __restrict__ dl_flag,
                                                   const float* __restrict__ g, float* __restrict__ g_prev) {
  if (dl_flag[0] == 0u) return;
  const int chunk = blockIdx.x, w = blockIdx.z;
  const u32 cnt = count[chunk];
  if (cnt == 0) return;
  __shared__ int s_idx[INC_CHUNK];
  __shared__ float s_val[INC_CHUNK];
  for (u32 i = threadIdx.x; i < cnt; i += TPB) {
    s_idx[i] = idx[(long long)chunk * INC_CHUNK + i];
    s_val[i] = val[(long long)chunk * INC_CHUNK + i];
  }
  __syncthreads();
  if (w == 0 && blockIdx.y == 0)
    for (u32 i = threadIdx.x; i < cnt; i += TPB) g_prev[s_idx[i]] = g[s_idx[i]];
  const float* at = AT + (long long)w * d * m_rows;
  float* out = ipart + ((long long)w * gridDim.x + chunk) * m_rows;
  const long long l = (long long)blockIdx.y * TPB + threadIdx.x;
  if (l >= m_rows) return;
  float acc = 0.f;
  u32 e = 0;
  for (; e + 8 <= cnt; e += 8) {
    float a[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) a[k] = __ldcs(at + (long long)s_idx[e + k] * m_rows + l);
#pragma unroll
    for (int k = 0; k < 8; ++k) acc = fmaf(a[k], s_val[e + k], acc);
  }
  for (; e < cnt; ++e) acc = fmaf(__ldcs(at + (long long)s_idx[e] * m_rows + l), s_val[e], acc);
  out[l] = acc;
}

// Gathered route (dl_flag[0] = 1): u += the chunks' contributions, z <- z - gamma u (two roundings, like the
// update of x).  Full route: z has just been recomputed.  Then the residual and the loss of every sample row
// from z.  A CTA serves FIN_ROWS sample rows with FIN_SLICES threads per row: each adds a contiguous range of
// chunks in chunk order (the ranges are latency chains of dependent loads, so there are many of them), and the
// ranges are added to u in range order.
constexpr int FIN_ROWS = 64;
constexpr int FIN_SLICES = 16;
__global__ void __launch_bounds__(FIN_ROWS * FIN_SLICES) k_inc_finish(const float* __restrict__ ipart, const u32* __restrict__ count,
                                                                      int nchunk, long long m_rows, float gamma,
                                                                      const float* __restrict__ target, int loss, float* __restrict__ u,
                                                                      float* __restrict__ z, float* __restrict__ r,
                                                                      LossTail lt, const u32* __restrict__ dl_flag) {
  __shared__ float part[FIN_SLICES][FIN_ROWS];
  __shared__ double red[FIN_ROWS / 32];
  const int w = blockIdx.y;
  const int row = threadIdx.x % FIN_ROWS, slice = threadIdx.x / FIN_ROWS;
  const long long l = (long long)blockIdx.x * FIN_ROWS + row;
  const bool gathered = dl_flag != nullptr && dl_flag[0] != 0u;   // nullptr: z has just been recomputed (refresh)
  if (gathered) {
    float s = 0.f;
    if (l < m_rows) {
      const int c0 = (int)((long long)nchunk * slice / FIN_SLICES), c1 = (int)((long long)nchunk * (slice + 1) / FIN_SLICES);
      for (int c = c0; c < c1; ++c)
        if (__ldg(&count[c])) s += ipart[((long long)w * nchunk + c) * m_rows + l];
    }
    part[slice][row] = s;
  }
  __syncthreads();
  double ls = 0.0;
  if (slice == 0 && l < m_rows) {
    const long long gi = (long long)w * m_rows + l;
    float zn = z[gi];
    if (gathered) {
      float s = u[gi];
#pragma unroll
      for (int q = 0; q < FIN_SLICES; ++q) s += part[q][row];
      u[gi] = s;
      zn = __fsub_rn(zn, __fmul_rn(gamma, s));
      z[gi] = zn;
    }
    float rr;
    residual(loss, zn, target[gi], 1.f / (float)m_rows, &rr, &ls);
    r[gi] = rr;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ls += __shfl_xor_sync(0xffffffffu, ls, o);
  if (slice == 0 && (threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ls;
  __syncthreads();
  double t = 0.0;
  if (threadIdx.x == 0)
    for (int k = 0; k < FIN_ROWS / 32; ++k) t += red[k];
  loss_tail(lt, t);
}

// --------------------------------------------------------------------------
static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

void launch_dense_fwd(const adacgd_problem& p, const GradScratch& g, const float* v, float* r, float* zout, cudaStream_t stream,
                      const u32* gate = nullptr, bool pdl = false);
// Above this many short CTAs (a few sample rows each) in a forward launch the loss is added up by k_loss_reduce
// instead of the last CTA; a CTA that walks a whole long row does not notice the count at its end.
constexpr long long FUSED_LOSS_MAX_CTAS = 1024;
static long long dense_fwd_short_ctas(const adacgd_problem& p, const GradScratch& g);
static LossTail make_tail(const adacgd_problem& p, const GradScratch& g, const float* x, long long ctas = 0) {
  LossTail t;
  t.fused = ctas <= FUSED_LOSS_MAX_CTAS ? 1 : 0;
  t.losspart = g.losspart; t.regpart = g.regpart; t.ticket = g.loss_ticket; t.x = x; t.d = p.d; t.m_rows = p.m_rows;
  t.loss = p.loss; t.n = p.n; t.lambda = p.lambda; t.out = g.loss;
  return t;
}
int launch_dense_bwd_and_loss(const adacgd_problem& p, const GradScratch& g, const float* x, float* grads, int loss_blocks, bool al,
                              cudaStream_t stream, bool pdl = false);

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

// Column blocks of the CSR forward pass (0: the plain kernel) and the route of the backward pass, from
// the shape alone so that sizing and carving agree.
static int csr_blocks_of(const adacgd_problem& p) {
  const long long nb = (p.d + CSR_BLK_MAX - 1) / CSR_BLK_MAX;
  return nb <= CSR_NB_MAX ? (int)nb : 0;
}
static int csr_block_cols(const adacgd_problem& p, int nb) {
  if (nb == 0) return 0;
  const long long blk = (p.d + nb - 1) / nb;
  return (int)((blk + 3) / 4 * 4);
}
// Entries of the regrouped forward copy: every (block, row) span padded to a multiple of four.
static size_t csr_fwd_cap(const adacgd_problem& p, int nb) {
  return (size_t)p.csr_nnz + 3 * (size_t)nb * (size_t)p.n * (size_t)p.m_rows + 4;
}
// Whether the backward pass walks spans (1) or takes one thread per column (0).
static int csc_cols_per_cta(const adacgd_problem& p) {
  if (p.m_rows > CSC_RCAP) return 0;
  const double avg = (double)p.csr_nnz / ((double)p.n * (double)p.d);   // stored entries per column of a worker
  return avg * CSC_WCOLS <= 0.75 * CSC_WPCAP ? 1 : 0;                    // a warp's span fits its buffer on average
}

static bool incremental_wanted(const adacgd_problem& p, int flags) {
  return (flags & ADACGD_FLAG_INCREMENTAL_FORWARD) && p.loss != ADACGD_LOSS_NONE && p.layout == ADACGD_LAYOUT_DENSE;
}

size_t grad_scratch_bytes(const adacgd_problem& p, int flags) {
  if (p.loss == ADACGD_LOSS_NONE) return 0;
  size_t o = 0;
  if (incremental_wanted(p, flags)) {
    const size_t nm = (size_t)p.n * p.m_rows, chunks = ((size_t)p.d + INC_CHUNK - 1) / INC_CHUNK;
    o = align_up(o + nm * (size_t)p.d * 4, 256);         // AT
    o = align_up(o + nm * 4, 256);                        // z
    o = align_up(o + nm * 4, 256);                        // u
    o = align_up(o + (size_t)p.d * 4, 256);               // g_prev
    o = align_up(o + chunks * 4, 256);                    // dl_count
    o = align_up(o + chunks * INC_CHUNK * 4, 256);        // dl_idx
    o = align_up(o + chunks * INC_CHUNK * 4, 256);        // dl_val
    o = align_up(o + nm * chunks * 4, 256);               // ipart
    o = align_up(o + 8, 256);                             // inc_cols
    o = align_up(o + 8, 256);                             // dl_flag
  }
  o = align_up(o + (size_t)p.n * p.m_rows * 4, 256);
  const int split = choose_split(p);
  if (split > 1) o = align_up(o + (size_t)split * p.n * p.d * 4, 256);
  o = align_up(o + (size_t)p.n * loss_blocks_of(p) * 8, 256);
  o = align_up(o + (size_t)p.n * loss_blocks_of(p) * 8, 256);   // regpart
  o = align_up(o + 8, 256);
  o = align_up(o + 4 * (1 + (size_t)p.n) + (size_t)p.n * ((p.d + TPB * 4 - 1) / (TPB * 4)) * 4, 256);   // loss tickets, backward tickets
  if (p.layout == ADACGD_LAYOUT_CSR) {
    o = align_up(o + ((size_t)p.n * p.d + 1) * 8, 256);
    o = align_up(o + (size_t)p.csr_nnz * 4, 256);
    o = align_up(o + (size_t)p.csr_nnz * 4, 256);
    const int nb = csr_blocks_of(p);
    const size_t rows = (size_t)p.n * p.m_rows;
    if (nb) {
      o = align_up(o + ((size_t)nb * rows + 1) * 8, 256);
      o = align_up(o + (size_t)nb * rows * 4, 256);
      o = align_up(o + csr_fwd_cap(p, nb) * 4, 256);   // regrouped values
      o = align_up(o + csr_fwd_cap(p, nb) * 2, 256);   // regrouped 16-bit columns
    }
    o = align_up(o + ((size_t)p.n + 1) * 8, 256);
    o = align_up(o + (size_t)p.n * ((size_t)p.d + 1) * 4, 256);
    o = align_up(o + (size_t)p.csr_nnz * 2, 256);   // 16-bit sample indices of the transposed copy
  }
  return o;
}

void carve_grad_scratch(GradScratch* g, void* base, const adacgd_problem& p, int flags) {
  char* b = (char*)base;
  size_t o = 0;
  g->inc = incremental_wanted(p, flags) ? 1 : 0;
  g->AT = g->z = g->u = g->g_prev = g->dl_val = g->ipart = nullptr;
  g->dl_count = nullptr; g->dl_idx = nullptr; g->inc_cols = nullptr; g->dl_flag = nullptr; g->inc_chunks = 0;
  if (g->inc) {
    const size_t nm = (size_t)p.n * p.m_rows, chunks = ((size_t)p.d + INC_CHUNK - 1) / INC_CHUNK;
    g->inc_chunks = (int)chunks;
    g->AT = (float*)(b + o); o = align_up(o + nm * (size_t)p.d * 4, 256);
    g->z = (float*)(b + o); o = align_up(o + nm * 4, 256);
    g->u = (float*)(b + o); o = align_up(o + nm * 4, 256);
    g->g_prev = (float*)(b + o); o = align_up(o + (size_t)p.d * 4, 256);
    g->dl_count = (u32*)(b + o); o = align_up(o + chunks * 4, 256);
    g->dl_idx = (int*)(b + o); o = align_up(o + chunks * INC_CHUNK * 4, 256);
    g->dl_val = (float*)(b + o); o = align_up(o + chunks * INC_CHUNK * 4, 256);
    g->ipart = (float*)(b + o); o = align_up(o + nm * chunks * 4, 256);
    g->inc_cols = (u64*)(b + o); o = align_up(o + 8, 256);
    g->dl_flag = (u32*)(b + o); o = align_up(o + 8, 256);
  }
  g->split = choose_split(p);
  g->loss_blocks = loss_blocks_of(p);
  g->r = (float*)(b + o); o = align_up(o + (size_t)p.n * p.m_rows * 4, 256);
  g->part = nullptr;
  if (g->split > 1) { g->part = (float*)(b + o); o = align_up(o + (size_t)g->split * p.n * p.d * 4, 256); }
  g->losspart = (double*)(b + o); o = align_up(o + (size_t)p.n * g->loss_blocks * 8, 256);
  g->regpart = (double*)(b + o); o = align_up(o + (size_t)p.n * g->loss_blocks * 8, 256);
  g->loss = (double*)(b + o); o = align_up(o + 8, 256);
  g->loss_ticket = (u32*)(b + o);
  g->bwd_tickets = g->loss_ticket + 1 + p.n;
  g->ticket_bytes = 4 * (1 + (size_t)p.n) + (size_t)p.n * ((p.d + TPB * 4 - 1) / (TPB * 4)) * 4;
  o = align_up(o + g->ticket_bytes, 256);
  g->csc_ptr = nullptr; g->csc_row = nullptr; g->csc_val = nullptr;
  g->nb = 0; g->blk = 0; g->csr_split = nullptr; g->zpart = nullptr; g->ccols = 0; g->wbase = nullptr; g->ptr32 = nullptr;
  g->csc_row16 = nullptr; g->csr_col16 = nullptr; g->fwd_val = nullptr;
  if (p.layout == ADACGD_LAYOUT_CSR) {
    g->csc_ptr = (long long*)(b + o); o = align_up(o + ((size_t)p.n * p.d + 1) * 8, 256);
    g->csc_row = (int*)(b + o); o = align_up(o + (size_t)p.csr_nnz * 4, 256);
    g->csc_val = (float*)(b + o); o = align_up(o + (size_t)p.csr_nnz * 4, 256);
    g->nb = csr_blocks_of(p);
    g->blk = csr_block_cols(p, g->nb);
    const size_t rows = (size_t)p.n * p.m_rows;
    if (g->nb) {
      g->csr_split = (long long*)(b + o); o = align_up(o + ((size_t)g->nb * rows + 1) * 8, 256);
      g->zpart = (float*)(b + o); o = align_up(o + (size_t)g->nb * rows * 4, 256);
      g->fwd_val = (float*)(b + o); o = align_up(o + csr_fwd_cap(p, g->nb) * 4, 256);
      g->csr_col16 = (u16*)(b + o); o = align_up(o + csr_fwd_cap(p, g->nb) * 2, 256);
    }
    g->ccols = csc_cols_per_cta(p);
    g->wbase = (long long*)(b + o); o = align_up(o + ((size_t)p.n + 1) * 8, 256);
    g->ptr32 = (u32*)(b + o); o = align_up(o + (size_t)p.n * ((size_t)p.d + 1) * 4, 256);
    g->csc_row16 = (u16*)(b + o);
  }
  g->prof = nullptr;
}

int launch_gradient(const adacgd_problem& p, const GradScratch& g, const float* x, float* grads,
                    cudaStream_t stream) {
  if (p.layout == ADACGD_LAYOUT_CSR) {
    int launches = 0;
    const DevProps* dp = current_device();
    if (!dp) return -1;
    int loss_blocks = g.loss_blocks;
    // chained as programmatic dependents (the x update before them lets the forward kernel in early); not under the
    // per-kernel event timers, whose records would sit between the kernels
    const bool pdl = g.prof == nullptr;
    if (g.nb) {
      const long long rows = (long long)p.n * p.m_rows;
      long long gx = dp->sms / g.nb;            // one 1024-thread CTA per SM over all column blocks
      if (gx < 1) gx = 1;
      if (gx > (rows + 31) / 32) gx = (rows + 31) / 32;
      prof_begin(g.prof, KID_CSR_FWD, stream);
      launch_k(k_csr_fwd_blocked, dim3((unsigned)gx, g.nb), dim3(CSR_FWD_TPB), (size_t)g.blk * 4, stream, pdl,
               (const long long*)g.csr_split, (const u16*)g.csr_col16, (const float*)g.fwd_val, x, rows, (long long)p.d, g.blk, g.zpart);
      prof_end(g.prof, stream);
      ++launches;
      loss_blocks = (int)((p.m_rows + TPB - 1) / TPB);
      prof_begin(g.prof, KID_CSR_RES, stream);
      launch_k(k_csr_residual, dim3((unsigned)loss_blocks, p.n), dim3(TPB), 0, stream, pdl, (const float*)g.zpart, g.nb, rows,
               (const float*)p.target, (long long)p.m_rows, (int)p.loss, g.r, make_tail(p, g, x));
      prof_end(g.prof, stream);
      ++launches;
    } else {
      prof_begin(g.prof, KID_CSR_FWD, stream);
      k_csr_fwd<<<dim3((unsigned)g.loss_blocks, p.n), TPB, 0, stream>>>((const long long*)p.csr_rowptr, p.csr_col, p.csr_val,
                                                                        p.target, x, p.m_rows, p.loss, g.r, make_tail(p, g, x));
      prof_end(g.prof, stream);
      ++launches;
    }
    prof_begin(g.prof, KID_CSC_BWD, stream);
    if (g.ccols) {
      // about eight CTAs per SM over all workers, each walking groups of columns of its worker
      const long long ngroups = (p.d + CSC_WCOLS - 1) / CSC_WCOLS;
      long long gx = (8ll * (TPB / CSC_TPB) * dp->sms + p.n - 1) / p.n;
      if (gx > (ngroups + CSC_TPB / 32 - 1) / (CSC_TPB / 32)) gx = (ngroups + CSC_TPB / 32 - 1) / (CSC_TPB / 32);
      if (gx < 1) gx = 1;
      launch_k(k_csc_bwd_span, dim3((unsigned)gx, p.n), dim3(CSC_TPB), ((size_t)p.m_rows + (size_t)(CSC_TPB / 32) * CSC_WPCAP) * 4, stream,
               pdl && g.nb != 0, (const long long*)g.wbase, (const u32*)g.ptr32, (const u16*)g.csc_row16, (const float*)g.csc_val,
               (const float*)g.r, x, (long long)p.d, (long long)p.m_rows, (int)p.loss, (float)p.lambda, grads);
    }
    else
      k_csc_bwd<<<dim3((unsigned)((p.d + TPB - 1) / TPB), p.n), TPB, 0, stream>>>(g.csc_ptr, g.csc_row, g.csc_val, g.r, x,
                                                                                  p.d, p.m_rows, p.loss, p.lambda, grads);
    prof_end(g.prof, stream);
    ++launches;
    return cudaGetLastError() == cudaSuccess ? launches : -1;
  }
  const bool al = (p.d % 4 == 0) && (((uintptr_t)p.A | (uintptr_t)x | (uintptr_t)grads) & 15) == 0;
  int launches = 0;
  const bool pdl = g.prof == nullptr;   // the kernels of the pass as programmatic dependents of one another
  launch_dense_fwd(p, g, x, g.r, nullptr, stream, nullptr, pdl);
  ++launches;
  if (dense_fwd_short_ctas(p, g) > FUSED_LOSS_MAX_CTAS) {
    prof_begin(g.prof, KID_LOSS, stream);
    launch_k(k_loss_reduce, dim3(1), dim3(1024), 0, stream, pdl, (const double*)g.losspart, (long long)p.n * g.loss_blocks, (int)p.n,
             (long long)p.m_rows, x, (long long)p.d, (int)p.loss, (float)p.lambda, g.loss);
    prof_end(g.prof, stream);
    ++launches;
  }
  return launches + launch_dense_bwd_and_loss(p, g, x, grads, g.loss_blocks, al, stream, pdl);
}

static long long dense_fwd_short_ctas(const adacgd_problem& p, const GradScratch& g) {
  return cta_row_mode(p) ? 0 : (long long)p.n * g.loss_blocks;
}

// The forward kernel in the shape the problem calls for: z = A v for a d-vector v, residuals if r != nullptr.
void launch_dense_fwd(const adacgd_problem& p, const GradScratch& g, const float* v, float* r, float* zout,
                      cudaStream_t stream, const u32* gate, bool pdl) {
  const bool al = (p.d % 4 == 0) && (((uintptr_t)p.A | (uintptr_t)v) & 15) == 0;
  prof_begin(g.prof, KID_GRAD_FWD, stream);
  const long long fwd_ctas = dense_fwd_short_ctas(p, g);
  const LossTail lt = make_tail(p, g, v, fwd_ctas);
  const bool cta_row = cta_row_mode(p);
  const dim3 grid((unsigned)(cta_row ? p.m_rows : g.loss_blocks), p.n);
#define FWD(CR, AL, FU)                                                                                                   \
  launch_k(k_dense_fwd<CR, AL, FU>, grid, dim3(TPB), 0, stream, pdl && g.prof == nullptr, (const float*)p.A, (const float*)p.target, v, \
           (long long)p.d, (long long)p.m_rows, (int)p.loss, r, lt, zout, gate)
  if (cta_row) { if (al) FWD(true, true, true); else FWD(true, false, true); }      // long CTAs always count themselves
  else if (lt.fused) { if (al) FWD(false, true, true); else FWD(false, false, true); }
  else { if (al) FWD(false, true, false); else FWD(false, false, false); }
#undef FWD
  prof_end(g.prof, stream);
}

// X_i = A_i^T r + reg'(x) and the loss from `loss_blocks` partial sums per worker; returns the launches.
int launch_dense_bwd_and_loss(const adacgd_problem& p, const GradScratch& g, const float* x, float* grads, int loss_blocks,
                              bool al, cudaStream_t stream, bool pdl) {
  int launches = 0;
  const dim3 bgrid((unsigned)((p.d + TPB * 4 - 1) / (TPB * 4)), p.n * g.split);
  prof_begin(g.prof, KID_GRAD_BWD, stream);
#define BWD(AL)                                                                                                              \
  launch_k(k_dense_bwd<AL>, bgrid, dim3(TPB), 0, stream, pdl, (const float*)p.A, (const float*)g.r, x, (long long)p.d, (long long)p.m_rows, \
           (int)g.split, (int)p.loss, (float)p.lambda, grads, g.part, (int)p.n, g.bwd_tickets)
  if (al) BWD(true); else BWD(false);
#undef BWD
  prof_end(g.prof, stream);
  ++launches;
  return cudaGetLastError() == cudaSuccess ? launches : -1;
}

int launch_gradient_incremental(const adacgd_problem& p, const GradScratch& g, const float* x, const float* gvec,
                                float gamma, bool refresh, float* grads, cudaStream_t stream) {
  const bool al = (p.d % 4 == 0) && (((uintptr_t)p.A | (uintptr_t)x | (uintptr_t)grads) & 15) == 0;
  int launches = 0;
  const int fin_blocks = (int)((p.m_rows + FIN_ROWS - 1) / FIN_ROWS);
  const int inc_tiles = (int)((p.m_rows + TPB - 1) / TPB);
  if (refresh) {
    // z = A x, u = A g, and g is remembered as the vector u belongs to
    launch_dense_fwd(p, g, x, nullptr, g.z, stream);
    launch_dense_fwd(p, g, gvec, nullptr, g.u, stream);
    launches += 2;
    if (cudaMemcpyAsync(g.g_prev, gvec, (size_t)p.d * 4, cudaMemcpyDeviceToDevice, stream) != cudaSuccess) return -1;
  } else {
    // more changed entries than this and the gathered columns cost as much as reading A in order
    const u32 max_cols = (u32)(p.d / 2);
    prof_begin(g.prof, KID_DELTA, stream);
    k_delta_scan<<<g.inc_chunks, TPB, 0, stream>>>(gvec, g.g_prev, p.d, g.dl_count, g.dl_idx, g.dl_val, g.dl_flag, g.inc_cols, max_cols);
    prof_end(g.prof, stream);
    prof_begin(g.prof, KID_INC, stream);
    k_dense_inc<<<dim3((unsigned)g.inc_chunks, (unsigned)inc_tiles, p.n), TPB, 0, stream>>>(g.AT, g.dl_count, g.dl_idx, g.dl_val, p.d, p.m_rows,
                                                                                             g.ipart, g.dl_flag, gvec, g.g_prev);
    prof_end(g.prof, stream);
    launch_dense_fwd(p, g, x, nullptr, g.z, stream, g.dl_flag);   // runs only if the scan chose the full route
    launches += 3;
  }
  prof_begin(g.prof, KID_INC_FINISH, stream);
  k_inc_finish<<<dim3((unsigned)fin_blocks, p.n), FIN_ROWS * FIN_SLICES, 0, stream>>>(g.ipart, g.dl_count, g.inc_chunks, p.m_rows, gamma, p.target, p.loss,
                                                                    g.u, g.z, g.r, make_tail(p, g, x), refresh ? nullptr : g.dl_flag);
  prof_end(g.prof, stream);
  ++launches;
  return launches + launch_dense_bwd_and_loss(p, g, x, grads, fin_blocks, al, stream);
}

// Column-major copy of the dense features, once per context.
int build_transposed_features(const adacgd_problem& p, const GradScratch& g, cudaStream_t stream) {
  const dim3 grid((unsigned)((p.d + 31) / 32), (unsigned)((p.m_rows + 31) / 32), p.n);
  k_transpose_features<<<grid, dim3(32, 8), 0, stream>>>(p.A, g.AT, p.m_rows, p.d);
  if (cudaMemsetAsync(g.inc_cols, 0, 8, stream) != cudaSuccess || cudaMemsetAsync(g.dl_flag, 0, 8, stream) != cudaSuccess) return -1;
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace adacgd

namespace adacgd {

// Builds the transposed copy of a CSR problem (host side, once per context): stable counting sort by
// (worker, column), so that the entries of a column keep ascending sample-row order and the
// backward sums have a fixed order.  Returns a message on failure, nullptr on success.
const char* build_csc(const adacgd_problem& p, GradScratch* gp, cudaStream_t stream) {
  GradScratch& g = *gp;
  const long long rows = (long long)p.n * p.m_rows, nnz = p.csr_nnz, cols = (long long)p.n * p.d;
  std::vector<long long> rowptr((size_t)rows + 1), cptr((size_t)cols + 1, 0);
  std::vector<int> col((size_t)nnz), crow((size_t)nnz);
  std::vector<float> val((size_t)nnz), cval((size_t)nnz);
  std::vector<u16> crow16, col16;
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
  // column pointers relative to each worker's first entry (32 bits: half the pointer traffic of the backward pass)
  std::vector<long long> wbase((size_t)p.n + 1);
  std::vector<u32> ptr32((size_t)p.n * ((size_t)p.d + 1));
  for (long long w = 0; w <= p.n; ++w) wbase[(size_t)w] = cptr[(size_t)(w * p.d)];
  for (long long w = 0; w < p.n; ++w) {
    if (wbase[(size_t)w + 1] - wbase[(size_t)w] >= (1ll << 32)) g.ccols = 0;   // would not fit: one thread per column instead
    for (long long c = 0; c <= p.d; ++c)
      ptr32[(size_t)(w * (p.d + 1) + c)] = (u32)(cptr[(size_t)(w * p.d + c)] - wbase[(size_t)w]);
  }
  // first entry of every column block inside every sample row (needs ascending columns inside a row)
  std::vector<long long> split;
  if (g.nb) {
    split.resize((size_t)(g.nb + 1) * (size_t)rows);
    for (long long r = 0; r < rows && g.nb; ++r) {
      long long e = rowptr[(size_t)r];
      const long long e1 = rowptr[(size_t)r + 1];
      for (long long q = e + 1; q < e1; ++q)
        if (col[(size_t)q] < col[(size_t)q - 1]) { g.nb = 0; break; }   // unsorted row: the plain forward kernel
      if (!g.nb) break;
      for (int b = 0; b <= g.nb; ++b) {
        const long long first_col = (long long)b * g.blk;
        while (e < e1 && col[(size_t)e] < first_col) ++e;
        split[(size_t)b * (size_t)rows + (size_t)r] = (b == g.nb) ? e1 : e;
      }
    }
  }
  // narrow copies of the indices for the two span kernels: what they read per stored entry drops from 8 to 6 bytes
  if (g.ccols) {
    crow16.resize((size_t)nnz);
    for (long long e = 0; e < nnz; ++e) crow16[(size_t)e] = (u16)crow[(size_t)e];          // m_rows <= CSC_RCAP
  }
  std::vector<float> fval;
  std::vector<long long> qptr;
  if (g.nb) {
    // the forward copy: block-major, spans padded with (0, column 0) to a multiple of four entries
    const size_t cap = csr_fwd_cap(p, g.nb);
    fval.assign(cap, 0.f);
    col16.assign(cap, (u16)0);
    qptr.resize((size_t)g.nb * (size_t)rows + 1);
    long long at = 0;   // in entries, always a multiple of four
    for (int b = 0; b < g.nb; ++b) {
      for (long long r = 0; r < rows; ++r) {
        qptr[(size_t)b * (size_t)rows + (size_t)r] = at / 4;
        const long long e0 = split[(size_t)b * (size_t)rows + (size_t)r], e1 = split[(size_t)(b + 1) * (size_t)rows + (size_t)r];
        for (long long e = e0; e < e1; ++e) {
          fval[(size_t)(at + e - e0)] = val[(size_t)e];
          col16[(size_t)(at + e - e0)] = (u16)(col[(size_t)e] - (long long)b * g.blk);     // blk <= CSR_BLK_MAX
        }
        at += (e1 - e0 + 3) / 4 * 4;
      }
    }
    qptr[(size_t)g.nb * (size_t)rows] = at / 4;
  }
  if (cudaMemcpyAsync(g.csc_ptr, cptr.data(), (cols + 1) * 8, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
      cudaMemcpyAsync(g.csc_row, crow.data(), nnz * 4, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
      cudaMemcpyAsync(g.csc_val, cval.data(), nnz * 4, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
      cudaMemcpyAsync(g.wbase, wbase.data(), wbase.size() * 8, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
      cudaMemcpyAsync(g.ptr32, ptr32.data(), ptr32.size() * 4, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
      (g.nb && cudaMemcpyAsync(g.csr_split, qptr.data(), qptr.size() * 8, cudaMemcpyHostToDevice, stream) != cudaSuccess) ||
      (g.nb && cudaMemcpyAsync(g.csr_col16, col16.data(), col16.size() * 2, cudaMemcpyHostToDevice, stream) != cudaSuccess) ||
      (g.nb && cudaMemcpyAsync(g.fwd_val, fval.data(), fval.size() * 4, cudaMemcpyHostToDevice, stream) != cudaSuccess) ||
      (g.ccols && cudaMemcpyAsync(g.csc_row16, crow16.data(), (size_t)nnz * 2, cudaMemcpyHostToDevice, stream) != cudaSuccess) ||
      cudaStreamSynchronize(stream) != cudaSuccess)
    return "copying the transposed arrays to the device failed";
  if (g.nb) cudaFuncSetAttribute(k_csr_fwd_blocked, cudaFuncAttributeMaxDynamicSharedMemorySize, CSR_BLK_MAX * 4);
  if (g.ccols) cudaFuncSetAttribute(k_csc_bwd_span, cudaFuncAttributeMaxDynamicSharedMemorySize, (CSC_RCAP + (CSC_TPB / 32) * CSC_WPCAP) * 4);
  return nullptr;
}

}  // namespace adacgd
