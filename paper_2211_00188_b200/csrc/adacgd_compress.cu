// Stages a2-a4 of one AdaCGD iteration and the server mean of a5:
//   v = X - G (EF21 shift, Eq. 7), D = ||X - Y||^2 and the error of every candidate
//   (both sides of the trigger, Eq. 10), the adaptive level choice and the
//   estimator update (Eq. 11), and g~ = (1/n) sum_i g_i (Algorithm 1).
//
// Three routes to the same results, chosen by size in launch_compress():
//   - large problems: thresholds are bracketed from a sample (k_sample), one streaming pass over
//     X, G, Y (k_pass1) gathers the sums and lists the few keys inside a bracket, the exact
//     selection runs on those lists (k_lcollect), one cooperative launch holds what only some rows need
//     (k_side), k_update applies the chosen level;
//   - the three-pass radix select on the bit pattern of |v| (11 + 11 + 9 bits: k_hist, k_energy),
//     shared by all Top-K candidates of a row: mid-size problems, and the per-row fallback of
//     the first route;
//   - short rows: everything in one CTA per row (k_small_rows).
// Energies are sums of non-negative exact terms; a comparison whose margin is below the
// worst-case summation error is redone in exact integer arithmetic.
#include <mutex>

#include <cooperative_groups.h>
#include "adacgd_device.cuh"

namespace adacgd {

// --------------------------------------------------------------------------
// radix-select passes
// --------------------------------------------------------------------------
// Run by the last CTA of a row's histogram pass: locates every candidate's K-th key in the table.
template <int PASS>
__device__ void scan_row(const CsetDev& cs, int row, const u32* __restrict__ hist, SelRow* __restrict__ sel,
                         bool count_fallback, u32* __restrict__ flags) {
  __shared__ u32 res[2];
  if (PASS == 1 && count_fallback && threadIdx.x == 0) atomicAdd(&flags[2], 1u);  // rows sent through the full select
  constexpr int NB = (PASS == 3) ? BINS3 : BINS1;
  SelRow* s = sel + row;
  for (int j = 0; j < cs.nsel; ++j) {
    const u32 K = (u32)cs.param[cs.sel[j]];
    const u32* h = hist + (long long)row * ((PASS == 1) ? NB : MAXC * NB) + ((PASS == 1) ? 0 : j * NB);
    const u32 before = (PASS == 1) ? 0u : (PASS == 2 ? s->above1[j] : s->above2[j]);
    block_find_kth_desc(h, NB, K - before, res);
    if (threadIdx.x == 0) {
      if (PASS == 1) {
        s->b1[j] = res[0];
        s->above1[j] = res[1];
      } else if (PASS == 2) {
        s->p2[j] = (s->b1[j] << 11) | res[0];
        s->above2[j] = before + res[1];
      } else {
        s->T[j] = (s->p2[j] << 9) | res[0];
        s->above[j] = before + res[1];
        s->ntie[j] = __ldcg(&h[res[0]]);
        s->q[j] = K - (before + res[1]);
        s->extraE[j] = 0.0;
        s->tiemode[j] = (s->q[j] < s->ntie[j]) ? 2u : 0u;
        s->cut[j] = 0xffffffffu;
      }
    }
    __syncthreads();
  }
}

// PASS 1: histogram of key[30:20] (one table per row) and the row maximum.
// PASS 2: for every selecting candidate, histogram of key[19:9] over the keys in its pass-1 bin.
// PASS 3: histogram of key[8:0] over the keys that share its 22-bit prefix.
// Body of one CTA (bx of gx CTAs of row by) of the histogram passes: shared by the kernel of that name and by k_side.
template <int PASS, bool ALIGNED>
__device__ __forceinline__ void d_hist(int bx, int by, int gx, u32* sh, const float* __restrict__ X, const float* __restrict__ G,
                                              long long d, const CsetDev& cs, SelRow* sel,
                                              u32* hist, u32* maxkey,
                                              const u32* rowflag, u32* tickets,
                                              u32* flags) {
  const int row = by;
  const int nsel = cs.nsel;
  if (rowflag && !__ldcg(&rowflag[row])) return;  // single-pass mode: only rows whose bracket failed
  constexpr int NB = (PASS == 3) ? BINS3 : BINS1;
  const int ntab = (PASS == 1) ? 1 : nsel;
  for (int i = threadIdx.x; i < ntab * NB; i += TPB) sh[i] = 0;
  u32 pref[MAXC];
#pragma unroll
  for (int j = 0; j < MAXC; ++j) {
    pref[j] = 0xffffffffu;
    if (PASS == 2 && j < nsel) pref[j] = __ldcg(&sel[row].b1[j]);
    if (PASS == 3 && j < nsel) pref[j] = __ldcg(&sel[row].p2[j]);
  }
  __syncthreads();
  const float* xr = X + (long long)row * d;
  const float* gr = G + (long long)row * d;
  u32 mx = 0;
  const long long ntile = (d + TPB * 4 - 1) / (TPB * 4);
  for (long long t = bx; t < ntile; t += gx) {
    const long long c0 = t * (TPB * 4) + threadIdx.x * 4;
    if (c0 >= d) continue;
    float x[4], g[4];
    load4<ALIGNED>(xr, c0, d, x);
    load4<ALIGNED>(gr, c0, d, g);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (!ALIGNED && c0 + k >= d) break;
      const u32 key = key_of(__fsub_rn(x[k], g[k]));
      if (PASS == 1) {
        mx = max(mx, key);
        atomicAdd(&sh[key >> 20], 1u);
      } else if (PASS == 2) {
#pragma unroll
        for (int j = 0; j < MAXC; ++j)
          if (j < nsel && (key >> 20) == pref[j]) atomicAdd(&sh[j * NB + ((key >> 9) & 0x7ffu)], 1u);
      } else {
#pragma unroll
        for (int j = 0; j < MAXC; ++j)
          if (j < nsel && (key >> 9) == pref[j]) atomicAdd(&sh[j * NB + (key & 0x1ffu)], 1u);
      }
    }
  }
  __syncthreads();
  u32* gh = hist + (long long)row * ((PASS == 1) ? NB : MAXC * NB);
  for (int i = threadIdx.x; i < ntab * NB; i += TPB)
    if (sh[i]) atomicAdd(&gh[i], sh[i]);
  if (PASS == 1) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if ((threadIdx.x & 31) == 0 && mx) atomicMax(&maxkey[row], mx);
  }
  if (nsel && last_cta_of_row(&tickets[row * NTICKET + 3 + PASS], gx))
    scan_row<PASS>(cs, row, hist, sel, rowflag != nullptr, flags);
}

template <int PASS, bool ALIGNED>
__global__ void __launch_bounds__(TPB) k_hist(const float* __restrict__ X, const float* __restrict__ G,
                                              long long d, CsetDev cs, SelRow* __restrict__ sel,
                                              u32* __restrict__ hist, u32* __restrict__ maxkey,
                                              const u32* __restrict__ rowflag, u32* __restrict__ tickets,
                                              u32* __restrict__ flags) {
  pdl_begin();
  extern __shared__ u32 sh[];
  d_hist<PASS, ALIGNED>(blockIdx.x, blockIdx.y, gridDim.x, sh, X, G, d, cs, sel, hist, maxkey, rowflag, tickets, flags);
}

// --------------------------------------------------------------------------
// energies (binary64, non-negative exact terms)
// --------------------------------------------------------------------------
// slot 0: D = sum (x-y)^2; slot 1: sum v^2; slot 2+c (Top-K candidate c with a
// threshold): sum of v^2 over keys strictly below its threshold.
template <bool ALIGNED>
__device__ __forceinline__ void d_energy(int bx, int by, int gx, const float* __restrict__ X, const float* __restrict__ G,
                                                const float* __restrict__ Y, long long d, const CsetDev& cs,
                                                const SelRow* sel, double* partial,
                                                const u32* rowflag, u32* diffflag) {
  const int row = by;
  if (rowflag && !__ldcg(&rowflag[row])) return;
  u32 T[MAXC];
#pragma unroll
  for (int j = 0; j < MAXC; ++j) T[j] = (j < cs.nsel) ? __ldcg(&sel[row].T[j]) : 0u;
  double aD = 0, aE = 0, aB[MAXC];
  u32 mxw = 0, dfl = 0;
#pragma unroll
  for (int j = 0; j < MAXC; ++j) aB[j] = 0;
  const float* xr = X + (long long)row * d;
  const float* gr = G + (long long)row * d;
  const float* yr = Y + (long long)row * d;
  const long long ntile = (d + TPB * 4 - 1) / (TPB * 4);
  for (long long t = bx; t < ntile; t += gx) {
    const long long c0 = t * (TPB * 4) + threadIdx.x * 4;
    if (c0 >= d) continue;
    float x[4], g[4], y[4];
    load4<ALIGNED>(xr, c0, d, x);
    load4<ALIGNED>(gr, c0, d, g);
    load4<ALIGNED>(yr, c0, d, y);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (!ALIGNED && c0 + k >= d) break;
      const float v = __fsub_rn(x[k], g[k]);
      const float w = __fsub_rn(x[k], y[k]);
      const double dv = (double)v, dw = (double)w;
      mxw = max(mxw, key_of(w));
      dfl |= __float_as_uint(v) ^ __float_as_uint(w);
      const double sq = __dmul_rn(dv, dv);
      aD = __dadd_rn(aD, __dmul_rn(dw, dw));
      aE = __dadd_rn(aE, sq);
      const u32 key = key_of(v);
#pragma unroll
      for (int j = 0; j < MAXC; ++j)
        if (j < cs.nsel && key < T[j]) aB[j] = __dadd_rn(aB[j], sq);
    }
  }
  if (mxw >= 0x7f800000u) atomicOr(&diffflag[row], 0x80000000u);
  if (dfl & 0x7fffffffu) atomicOr(&diffflag[row], dfl & 0x7fffffffu);  // some |X-G| differs from |X-Y|
  __shared__ double red[NSLOT][TPB / 32];
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  double v0 = warp_sum_f64(aD), v1 = warp_sum_f64(aE);
  if (lane == 0) { red[0][wid] = v0; red[1][wid] = v1; }
#pragma unroll
  for (int j = 0; j < MAXC; ++j) {
    if (j < cs.nsel) {
      double vb = warp_sum_f64(aB[j]);
      if (lane == 0) red[2 + cs.sel[j]][wid] = vb;
    }
  }
  __syncthreads();
  if (threadIdx.x < NSLOT) {
    const int s = threadIdx.x;
    bool used = (s < 2);
    for (int j = 0; j < cs.nsel; ++j) used |= (s == 2 + cs.sel[j]);
    if (used) {
      double acc = 0;
      for (int w = 0; w < TPB / 32; ++w) acc += red[s][w];
      partial[((long long)row * MAX_BLK_PER_ROW + bx) * NSLOT + s] = acc;
    }
  }
}

template <bool ALIGNED>
__global__ void __launch_bounds__(TPB) k_energy(const float* __restrict__ X, const float* __restrict__ G,
                                                const float* __restrict__ Y, long long d, CsetDev cs,
                                                const SelRow* __restrict__ sel, double* __restrict__ partial,
                                                const u32* __restrict__ rowflag, u32* __restrict__ diffflag) {
  pdl_begin();
  d_energy<ALIGNED>(blockIdx.x, blockIdx.y, gridDim.x, X, G, Y, d, cs, sel, partial, rowflag, diffflag);
}


// slot 2+c for quantiser candidate c: sum (v - Q_c(v))^2 with the row scale s = max|v|.
template <bool ALIGNED>
__global__ void __launch_bounds__(TPB) k_quant_err(const float* __restrict__ X, const float* __restrict__ G,
                                                   long long d, CsetDev cs, const u32* __restrict__ maxkey,
                                                   double* __restrict__ partial) {
  pdl_begin();
  const int row = blockIdx.y;
  const float s = __uint_as_float(maxkey[row]);
  float L[MAXC], inv[MAXC], step[MAXC];
  double acc[MAXC];
#pragma unroll
  for (int j = 0; j < MAXC; ++j) {
    acc[j] = 0;
    L[j] = inv[j] = step[j] = 0.f;
    if (j < cs.nquant) {
      L[j] = (float)((1 << ((int)cs.param[cs.qsel[j]] - 1)) - 1);
      if (s > 0.f) { inv[j] = __fdiv_rn(L[j], s); step[j] = __fdiv_rn(s, L[j]); }
    }
  }
  const float* xr = X + (long long)row * d;
  const float* gr = G + (long long)row * d;
  const long long ntile = (d + TPB * 4 - 1) / (TPB * 4);
  for (long long t = blockIdx.x; t < ntile; t += gridDim.x) {
    const long long c0 = t * (TPB * 4) + threadIdx.x * 4;
    if (c0 >= d) continue;
    float x[4], g[4];
    load4<ALIGNED>(xr, c0, d, x);
    load4<ALIGNED>(gr, c0, d, g);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (!ALIGNED && c0 + k >= d) break;
      const float v = __fsub_rn(x[k], g[k]);
#pragma unroll
      for (int j = 0; j < MAXC; ++j) {
        if (j < cs.nquant) {
          const double r = (double)__fsub_rn(v, quant_value(v, L[j], inv[j], step[j]));
          acc[j] = __dadd_rn(acc[j], __dmul_rn(r, r));
        }
      }
    }
  }
  __shared__ double red[MAXC][TPB / 32];
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
  for (int j = 0; j < MAXC; ++j) {
    if (j < cs.nquant) {
      double vb = warp_sum_f64(acc[j]);
      if (lane == 0) red[j][wid] = vb;
    }
  }
  __syncthreads();
  if (threadIdx.x < cs.nquant) {
    double a = 0;
    for (int w = 0; w < TPB / 32; ++w) a += red[threadIdx.x][w];
    partial[((long long)row * MAX_BLK_PER_ROW + blockIdx.x) * NSLOT + 2 + cs.qsel[threadIdx.x]] = a;
  }
}

// `picked` (may be null): per-row ticket words; a row whose word 9 is set was already decided.
// (rows decided here are not marked: nothing reads the mark after the level choice)
__device__ __forceinline__ void picked_mark(const u32*, int) {}
__device__ __forceinline__ void d_pick(int row, const CsetDev& cs, long long d, int nblk_main, int nblk_full, const u32* rowflag,
                                       const double* partial, const SelRow* sel, const u32* maxkey, RowDec* dec, u32* flags,
                                       const CompressOut& out, const u32* diffflag, const u32* picked, double tol) {
  if (picked && __ldcg(&picked[row * NTICKET + 9])) return;
  const int nblk = (rowflag && __ldcg(&rowflag[row])) ? nblk_full : nblk_main;  // which pass produced this row's partial sums
  pick_row(cs, d, row, nblk, nblk_main, partial, sel, maxkey, dec, flags, out, diffflag, tol);  // k_quant_err: main grid
  if (picked && threadIdx.x == 0) picked_mark(picked, row);
}

__global__ void __launch_bounds__(TPB) k_pick(CsetDev cs_param, long long d, int nblk_main, int nblk_full,
                                             const u32* __restrict__ rowflag, const double* __restrict__ partial,
                                             const SelRow* __restrict__ sel, const u32* __restrict__ maxkey,
                                             RowDec* __restrict__ dec, u32* __restrict__ flags, CompressOut out,
                                             const u32* __restrict__ diffflag, const u32* __restrict__ picked,
                                             double tol) {
  pdl_begin();
  __shared__ CsetDev cs;   // indexed with run-time values below: a shared copy instead of a local one per thread
  if (threadIdx.x == 0) cs_copy_static(cs, cs_param);
  __syncthreads();
  d_pick(blockIdx.x, cs, d, nblk_main, nblk_full, rowflag, partial, sel, maxkey, dec, flags, out, diffflag, picked, tol);
}

template <bool ALIGNED>
__device__ __forceinline__ void d_exact_sums(int bx, int by, int gx, const float* __restrict__ X, const float* __restrict__ G,
                                                    const float* __restrict__ Y, long long d, const CsetDev& cs,
                                                    const SelRow* sel, const u32* maxkey,
                                                    RowDec* dec, u64* limbs,
                                                    u32* diffflag, long long d_full, const CompressOut& out,
                                                    u32* tickets, u32* flags) {
  const int row = by;
  if (!__ldcg(&dec[row].need_exact)) return;
  __shared__ u64 sh[NSLOT * NLIMB];
  for (int i = threadIdx.x; i < NSLOT * NLIMB; i += TPB) sh[i] = 0;
  __syncthreads();
  const float s = __uint_as_float(__ldcg(&maxkey[row]));
  const float* xr = X + (long long)row * d;
  const float* gr = G + (long long)row * d;
  const float* yr = Y + (long long)row * d;
  const long long ntile = (d + TPB * 4 - 1) / (TPB * 4);
  for (long long t = bx; t < ntile; t += gx) {
    const long long c0 = t * (TPB * 4) + threadIdx.x * 4;
    if (c0 >= d) continue;
    float x[4], g[4], y[4];
    load4<ALIGNED>(xr, c0, d, x);
    load4<ALIGNED>(gr, c0, d, g);
    load4<ALIGNED>(yr, c0, d, y);
    for (int k = 0; k < 4; ++k) {
      if (!ALIGNED && c0 + k >= d) break;
      const float v = __fsub_rn(x[k], g[k]);
      int kk; u32 p[3];
      if (key_of(__fsub_rn(x[k], y[k])) >= 0x7f800000u || key_of(v) >= 0x7f800000u) {
        atomicOr(&diffflag[row], 0x80000000u);   // Inf/NaN in X - Y or X - G: the row is reported, not summed
        continue;
      }
      sq_pieces(__fsub_rn(x[k], y[k]), &kk, p);
      limb_add(sh + 0 * NLIMB, kk, p);
      sq_pieces(v, &kk, p);
      limb_add(sh + 1 * NLIMB, kk, p);
      const u32 key = key_of(v);
      for (int j = 0; j < cs.nsel; ++j)
        if (key < __ldcg(&sel[row].T[j])) limb_add(sh + (2 + cs.sel[j]) * NLIMB, kk, p);
      for (int j = 0; j < cs.nquant; ++j) {
        const int c = cs.qsel[j];
        const float L = (float)((1 << ((int)cs.param[c] - 1)) - 1);
        float inv = 0.f, step = 0.f;
        if (s > 0.f) { inv = __fdiv_rn(L, s); step = __fdiv_rn(s, L); }
        int k2; u32 p2[3];
        sq_pieces(__fsub_rn(v, quant_value(v, L, inv, step)), &k2, p2);
        limb_add(sh + (2 + c) * NLIMB, k2, p2);
      }
    }
  }
  __syncthreads();
  u64* gl = limbs + (long long)row * NSLOT * NLIMB;
  for (int i = threadIdx.x; i < NSLOT * NLIMB; i += TPB) {
    // split so that the global limb stays below 2^63 for any row length < 2^31
    const u64 vlo = sh[i] & 0xffffffffull, vhi = sh[i] >> 32;
    if (vlo) atomicAdd(&gl[i], vlo);
    if (vhi && (i % NLIMB) + 1 < NLIMB) atomicAdd(&gl[i + 1], vhi);
  }
  if (last_cta_of_row(&tickets[row * NTICKET + 7], gx) && threadIdx.x == 0)
    pick_exact_row(cs, row, d_full, limbs + (long long)row * NSLOT * NLIMB, sel, maxkey, dec, out, diffflag, flags);
}

template <bool ALIGNED>
__global__ void __launch_bounds__(TPB) k_exact_sums(const float* __restrict__ X, const float* __restrict__ G,
                                                    const float* __restrict__ Y, long long d, CsetDev cs,
                                                    const SelRow* __restrict__ sel, const u32* __restrict__ maxkey,
                                                    RowDec* __restrict__ dec, u64* __restrict__ limbs,
                                                    u32* __restrict__ diffflag, long long d_full, CompressOut out,
                                                    u32* __restrict__ tickets, u32* __restrict__ flags) {
  pdl_begin();
  d_exact_sums<ALIGNED>(blockIdx.x, blockIdx.y, gridDim.x, X, G, Y, d, cs, sel, maxkey, dec, limbs, diffflag, d_full, out, tickets, flags);
}

// --------------------------------------------------------------------------
// tie order, estimator update, server mean
// --------------------------------------------------------------------------
template <bool ALIGNED>
__device__ __forceinline__ void d_tiecount(int bx, int by, int gx, const float* __restrict__ X, const float* __restrict__ G,
                                                  long long d, const RowDec* dec,
                                                  u32* tiecnt, long long nchunk,
                                                  u32* tickets) {
  const int row = by;
  if (!__ldcg(&dec[row].need_tie)) return;
  const u32 T = __ldcg(&dec[row].T);
  for (long long chunk = bx; chunk < nchunk; chunk += gx) {
    const long long c0 = chunk * UPD_COLS + threadIdx.x * 4;
    u32 cnt = 0;
    if (c0 < d) {
      float x[4], g[4];
      load4<ALIGNED>(X + (long long)row * d, c0, d, x);
      load4<ALIGNED>(G + (long long)row * d, c0, d, g);
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if ((ALIGNED || c0 + k < d) && key_of(__fsub_rn(x[k], g[k])) == T) ++cnt;
    }
    u32 total;
    block_excl_scan(cnt, &total);
    if (threadIdx.x == 0) tiecnt[(long long)row * nchunk + chunk] = total;
  }
  if (!last_cta_of_row(&tickets[row * NTICKET + 8], gx)) return;
  // exclusive prefix over the row's chunks
  u32* t = tiecnt + (long long)row * nchunk;
  u32 carry = 0;
  for (long long base = 0; base < nchunk; base += TPB) {
    const long long i = base + threadIdx.x;
    const u32 v = (i < nchunk) ? __ldcg(&t[i]) : 0u;
    u32 total;
    const u32 ex = block_excl_scan(v, &total);
    if (i < nchunk) t[i] = carry + ex;
    carry += total;
  }
}

template <bool ALIGNED>
__global__ void __launch_bounds__(TPB) k_tiecount(const float* __restrict__ X, const float* __restrict__ G,
                                                  long long d, const RowDec* __restrict__ dec,
                                                  u32* __restrict__ tiecnt, long long nchunk,
                                                  u32* __restrict__ tickets) {
  pdl_begin();
  d_tiecount<ALIGNED>(blockIdx.x, blockIdx.y, gridDim.x, X, G, d, dec, tiecnt, nchunk, tickets);
}

// Thread owns 4 consecutive columns and walks the rows in order, so that the mean is
// summed in worker order.  Row i: G_i <- G_i + C_level(X_i - G_i) (EF21, Eq. 7).  The next
// row's operands are loaded before the current row is written back.
constexpr int UPD_ROW_TILE = 32;
#ifndef UPD_RB
#define UPD_RB 2    // rows whose operands a thread of the update kernel keeps in flight
#endif
// g <- g + C(x - g) on four columns for a Top-K level given by threshold key T and index cut:
// kept <=> |v| >= T for indices up to the cut, |v| > T (>= the next key value) beyond it; finite
// non-negative binary32 values order like their bit patterns.  Returns whether anything was kept.
__device__ __forceinline__ bool apply_topk4(float (&g)[4], const float (&x)[4], u32 T, u32 cut, u32 c0u) {
  const float Tf = __uint_as_float(T), Tn = __uint_as_float(T + 1u);
  float th[4];
  if (cut >= c0u + 3u) { th[0] = th[1] = th[2] = th[3] = Tf; }
  else if (cut < c0u) { th[0] = th[1] = th[2] = th[3] = Tn; }
  else {
#pragma unroll
    for (int k = 0; k < 4; ++k) th[k] = (c0u + (u32)k <= cut) ? Tf : Tn;
  }
  bool any = false;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const float v = __fsub_rn(x[k], g[k]);
    const bool kept = fabsf(v) >= th[k];
    g[k] = kept ? __fadd_rn(g[k], v) : g[k];
    any = any || kept;
  }
  return any;
}
// Rows r0 .. r0 + nr - 1 of one chunk for a thread's four columns, every row skipped (mode 0), a Top-K
// level with an index cut (1), the identity (2) or a quantiser (3): RB rows in flight as plain 128-bit
// loads, applied in row order so that `acc` sums the mean in worker order.
template <int RB>
__device__ __forceinline__ void update_rows_simple(const float* __restrict__ X, float* __restrict__ G, long long d,
                                                   long long c0, int r0, int nr, const RowDec* rd, bool want_mean,
                                                   float (&acc)[4]) {
  const u32 c0u = (u32)c0;
  for (int q0 = 0; q0 < nr; q0 += RB) {
    float4 gq[RB], xq[RB];
#pragma unroll
    for (int u = 0; u < RB; ++u) {
      gq[u] = make_float4(0.f, 0.f, 0.f, 0.f); xq[u] = gq[u];
      const int ii = q0 + u;
      if (ii < nr) {
        const int m = rd[ii].mode;
        if (m != 0 || want_mean) gq[u] = *reinterpret_cast<const float4*>(G + (long long)(r0 + ii) * d + c0);
        if (m != 0) xq[u] = __ldcs(reinterpret_cast<const float4*>(X + (long long)(r0 + ii) * d + c0));
      }
    }
#pragma unroll
    for (int u = 0; u < RB; ++u) {
      const int ii = q0 + u;
      if (ii >= nr) break;
      float g[4] = {gq[u].x, gq[u].y, gq[u].z, gq[u].w};
      const int m = rd[ii].mode;
      if (m != 0) {
        const float x[4] = {xq[u].x, xq[u].y, xq[u].z, xq[u].w};
        bool any = true;
        if (m == 1) any = apply_topk4(g, x, rd[ii].T, rd[ii].cut, c0u);
        else if (m == 2) {
#pragma unroll
          for (int k = 0; k < 4; ++k) g[k] = __fadd_rn(g[k], __fsub_rn(x[k], g[k]));
        } else {
          const float L = rd[ii].qL, inv = rd[ii].qinv, step = rd[ii].qstep;
#pragma unroll
          for (int k = 0; k < 4; ++k) g[k] = __fadd_rn(g[k], quant_value(__fsub_rn(x[k], g[k]), L, inv, step));
        }
        if (any) *reinterpret_cast<float4*>(G + (long long)(r0 + ii) * d + c0) = make_float4(g[0], g[1], g[2], g[3]);
      }
      if (want_mean) {
#pragma unroll
        for (int k = 0; k < 4; ++k) acc[k] = __fadd_rn(acc[k], g[k]);
      }
    }
  }
}
// The same update for many short rows, one column per thread: a thread of k_update owns four columns of every
// row, which leaves a 100 x 100 000 problem with 98 CTAs; here it is 391.  Only calls whose rows all take the
// simple path (skip, Top-K by threshold and index cut, identity, quantiser) are served: the kernel checks that
// first, and if it does the work it sets `done`, on which the general kernel that follows returns at once.
constexpr int UPDN_RB = 8;   // rows whose operands a thread keeps in flight
__global__ void __launch_bounds__(TPB) k_update_narrow(const float* __restrict__ X, float* __restrict__ G, int rows, long long d,
                                                       const RowDec* __restrict__ dec, CompressOut out, u32* __restrict__ done) {
  pdl_begin();
  __shared__ RowDec shd[UPD_ROW_TILE];
  bool simple = true;
  for (int i = threadIdx.x; i < rows; i += TPB) {
    const int m = dec[i].mode;
    simple = simple && m != 4 && !(m == 1 && dec[i].need_tie);
  }
  if (!__syncthreads_and(simple ? 1 : 0)) return;
  if (blockIdx.x == 0 && threadIdx.x == 0) *done = 1u;
  const bool want_mean = out.mean_out != nullptr;
  const long long c = (long long)blockIdx.x * TPB + threadIdx.x;
  const bool live = c < d;
  const u32 cu = (u32)c;
  float acc = -0.f;   // -0 + g == g bit for bit
  for (int r0 = 0; r0 < rows; r0 += UPD_ROW_TILE) {
    const int nr = (rows - r0 < UPD_ROW_TILE) ? rows - r0 : UPD_ROW_TILE;
    __syncthreads();
    if (threadIdx.x < nr) shd[threadIdx.x] = dec[r0 + threadIdx.x];
    __syncthreads();
    if (!live) continue;
    for (int q0 = 0; q0 < nr; q0 += UPDN_RB) {
      float gq[UPDN_RB], xq[UPDN_RB];
#pragma unroll
      for (int u = 0; u < UPDN_RB; ++u) {
        gq[u] = 0.f; xq[u] = 0.f;
        const int ii = q0 + u;
        if (ii < nr) {
          const int m = shd[ii].mode;
          if (m != 0 || want_mean) gq[u] = G[(long long)(r0 + ii) * d + c];
          if (m != 0) xq[u] = __ldcs(X + (long long)(r0 + ii) * d + c);
        }
      }
#pragma unroll
      for (int u = 0; u < UPDN_RB; ++u) {
        const int ii = q0 + u;
        if (ii >= nr) break;
        float g = gq[u];
        const int m = shd[ii].mode;
        if (m != 0) {
          const float v = __fsub_rn(xq[u], g);
          bool kept = true;
          float add = v;
          if (m == 1) {
            const u32 T = shd[ii].T;
            kept = fabsf(v) >= __uint_as_float(cu <= shd[ii].cut ? T : T + 1u);
          } else if (m == 3) {
            add = quant_value(v, shd[ii].qL, shd[ii].qinv, shd[ii].qstep);
          }
          if (kept) {
            g = __fadd_rn(g, add);
            G[(long long)(r0 + ii) * d + c] = g;
          }
        }
        if (want_mean) acc = __fadd_rn(acc, g);
      }
    }
  }
  if (want_mean && live) out.mean_out[c] = __fdiv_rn(acc, (float)rows);
}

#ifndef UPD_MINB
#define UPD_MINB 4   // resident CTAs per SM the register budget of the update kernel is set for
#endif
template <bool ALIGNED>
__global__ void __launch_bounds__(TPB, UPD_MINB) k_update(const float* __restrict__ X, float* __restrict__ G, int rows,
                                                long long d, const RowDec* __restrict__ dec,
                                                const u32* __restrict__ tiepref, long long nchunk, int copy_mode,
                                                CompressOut out, const u32* __restrict__ skip_flag) {
  pdl_begin();
  if (skip_flag && __ldcg(skip_flag)) return;   // the one-column-per-thread kernel has done the work
  __shared__ RowDec shd[UPD_ROW_TILE];
  const int lane = threadIdx.x & 31;
  const bool want_mean = out.mean_out != nullptr;

  // Streaming mode: all rows fit one tile of decisions, every row either skips or applies a Top-K
  // level decided by threshold and index cut, and no kept-index list is wanted.  A thread keeps the
  // operands of UPD_RB rows of its four columns in flight as plain 128-bit loads; rows are still
  // applied in worker order, so the mean is summed in that order.
  if (ALIGNED && rows <= UPD_ROW_TILE && !copy_mode && out.kept_idx == nullptr) {
    if (threadIdx.x < rows) shd[threadIdx.x] = dec[threadIdx.x];
    __syncthreads();
    bool simple = true;
    if (threadIdx.x < rows) simple = shd[threadIdx.x].mode != 4 && !(shd[threadIdx.x].mode == 1 && shd[threadIdx.x].need_tie);
    if (__syncthreads_and(simple ? 1 : 0)) {
      if (rows == 1 && !want_mean && shd[0].mode == 1) {
        // a single row (the master step): nothing to keep in flight across rows, so four chunks at a time
        const u32 T = shd[0].T, cut = shd[0].cut;
        for (long long chunk = blockIdx.x; chunk < nchunk; chunk += 4ll * gridDim.x) {
          float4 gq[4], xq[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const long long c0 = (chunk + (long long)u * gridDim.x) * UPD_COLS + threadIdx.x * 4;
            gq[u] = make_float4(0.f, 0.f, 0.f, 0.f); xq[u] = gq[u];
            if (c0 < d) {
              gq[u] = *reinterpret_cast<const float4*>(G + c0);
              xq[u] = __ldcs(reinterpret_cast<const float4*>(X + c0));
            }
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const long long c0 = (chunk + (long long)u * gridDim.x) * UPD_COLS + threadIdx.x * 4;
            if (c0 >= d) break;
            float g[4] = {gq[u].x, gq[u].y, gq[u].z, gq[u].w};
            const float x[4] = {xq[u].x, xq[u].y, xq[u].z, xq[u].w};
            if (apply_topk4(g, x, T, cut, (u32)c0)) *reinterpret_cast<float4*>(G + c0) = make_float4(g[0], g[1], g[2], g[3]);
          }
        }
        return;
      }
      for (long long chunk = blockIdx.x; chunk < nchunk; chunk += gridDim.x) {
        const long long c0 = chunk * UPD_COLS + threadIdx.x * 4;
        if (c0 >= d) continue;
        float acc[4] = {-0.f, -0.f, -0.f, -0.f};  // -0 + g == g bit for bit, so the first row needs no special case
        update_rows_simple<UPD_RB>(X, G, d, c0, 0, rows, shd, want_mean, acc);
        if (want_mean) {
          const float n = (float)rows;
          *reinterpret_cast<float4*>(out.mean_out + c0) =
              make_float4(__fdiv_rn(acc[0], n), __fdiv_rn(acc[1], n), __fdiv_rn(acc[2], n), __fdiv_rn(acc[3], n));
        }
      }
      return;
    }
  }

  for (long long chunk = blockIdx.x; chunk < nchunk; chunk += gridDim.x) {
    const long long c0 = chunk * UPD_COLS + threadIdx.x * 4;
    const bool live = c0 < d;
    float acc[4] = {-0.f, -0.f, -0.f, -0.f};  // -0 + g == g bit for bit, so the first row needs no special case
    for (int r0 = 0; r0 < rows; r0 += UPD_ROW_TILE) {
      const int nr = (rows - r0 < UPD_ROW_TILE) ? rows - r0 : UPD_ROW_TILE;
      __syncthreads();
      if (threadIdx.x < nr) {
        RowDec t;
        if (copy_mode) { t.level = 0; t.mode = 4; t.T = 0; t.q = 0; t.need_tie = 0; t.need_exact = 0; t.qL = t.qinv = t.qstep = 0.f; t.cut = 0xffffffffu; }
        else t = dec[r0 + threadIdx.x];
        shd[threadIdx.x] = t;
      }
      __syncthreads();
      // Common case for the whole tile of rows: every row either skips or applies a Top-K level whose
      // threshold-equal keys are decided by the index cut, and no kept-index list is wanted.
      bool simple = true;
      // rows that need no per-key tie ranking; without 16-byte alignment the batched loop below only takes
      // skipped rows and Top-K rows, identity and quantiser rows go through the general loop
      if (threadIdx.x < nr) {
        const int m = shd[threadIdx.x].mode;
        simple = ALIGNED ? (m != 4 && !(m == 1 && shd[threadIdx.x].need_tie)) : (m == 0 || (m == 1 && !shd[threadIdx.x].need_tie));
      }
      simple = __syncthreads_and(simple ? 1 : 0) != 0 && out.kept_idx == nullptr;
      if (simple && ALIGNED) {
        if (live) {   // few chunks (short rows): more rows in flight per thread, the SMs are not full
          if (gridDim.x < 2 * sm_count()) update_rows_simple<4>(X, G, d, c0, r0, nr, shd, want_mean, acc);
          else update_rows_simple<UPD_RB>(X, G, d, c0, r0, nr, shd, want_mean, acc);
        }
        continue;
      }
      if (simple) {
        float sg[4] = {0.f, 0.f, 0.f, 0.f}, sx[4] = {0.f, 0.f, 0.f, 0.f};
        if (live) {
          if (shd[0].mode != 0 || want_mean) load4<ALIGNED>(G + (long long)r0 * d, c0, d, sg);
          if (shd[0].mode != 0) load4<ALIGNED>(X + (long long)r0 * d, c0, d, sx);
        }
        for (int ii = 0; ii < nr; ++ii) {
          const int i = r0 + ii;
          float g[4], x[4];
  #pragma unroll
          for (int k = 0; k < 4; ++k) { g[k] = sg[k]; x[k] = sx[k]; }
          if (ii + 1 < nr && live) {
            const int m1 = shd[ii + 1].mode;
            if (m1 != 0 || want_mean) load4<ALIGNED>(G + (long long)(i + 1) * d, c0, d, sg);
            if (m1 != 0) load4<ALIGNED>(X + (long long)(i + 1) * d, c0, d, sx);
          }
          if (shd[ii].mode != 0) {
            const u32 T = shd[ii].T, cut = shd[ii].cut;
            bool any = false;
  #pragma unroll
            for (int k = 0; k < 4; ++k) {
              const float v = __fsub_rn(x[k], g[k]);
              const u32 key = key_of(v);
              const bool kept = (key > T) || (key == T && (u32)c0 + (u32)k <= cut);
              g[k] = kept ? __fadd_rn(g[k], v) : g[k];
              any = any || kept;
            }
            // dead lanes hold zeros: they are kept only when T == 0, and never stored
            if (any && live) store4<ALIGNED>(G + (long long)i * d, c0, d, g);
          }
          if (want_mean) {
  #pragma unroll
            for (int k = 0; k < 4; ++k) acc[k] = __fadd_rn(acc[k], g[k]);
          }
        }
        continue;
      }
      float gn[4] = {0.f, 0.f, 0.f, 0.f}, xn[4] = {0.f, 0.f, 0.f, 0.f};
      if (live) {
        const int m0 = shd[0].mode;
        if (m0 != 4 && (m0 != 0 || want_mean)) load4<ALIGNED>(G + (long long)r0 * d, c0, d, gn);
        if (m0 != 0) load4<ALIGNED>(X + (long long)r0 * d, c0, d, xn);
      }
      for (int ii = 0; ii < nr; ++ii) {
        const int i = r0 + ii;
        const int mode = shd[ii].mode;
        float* grow = G + (long long)i * d;
        float g[4], x[4];
  #pragma unroll
        for (int k = 0; k < 4; ++k) { g[k] = gn[k]; x[k] = xn[k]; }
        if (ii + 1 < nr && live) {
          const int m1 = shd[ii + 1].mode;
          if (m1 != 4 && (m1 != 0 || want_mean)) load4<ALIGNED>(G + (long long)(i + 1) * d, c0, d, gn);
          if (m1 != 0) load4<ALIGNED>(X + (long long)(i + 1) * d, c0, d, xn);
        }
        if (mode == 1 && !shd[ii].need_tie && !out.kept_idx) {
          // common case: keep every key > T and the threshold-equal keys up to index `cut`
          const u32 T = shd[ii].T, cut = shd[ii].cut;
          bool any = false;
  #pragma unroll
          for (int k = 0; k < 4; ++k) {
            const float v = __fsub_rn(x[k], g[k]);
            const u32 key = key_of(v);
            const bool kept = (key > T || (key == T && (u32)(c0 + k) <= cut)) && (ALIGNED || c0 + k < d);
            g[k] = kept ? __fadd_rn(g[k], v) : g[k];
            any = any || kept;
          }
          if (any && live) store4<ALIGNED>(grow, c0, d, g);
        } else if (mode != 0) {
          bool kept[4] = {false, false, false, false};
          bool any = false;
          if (mode == 4) {
  #pragma unroll
            for (int k = 0; k < 4; ++k) g[k] = x[k];
            any = live;
          } else if (mode == 1) {
            const u32 T = shd[ii].T, q = shd[ii].q;
            const int need_tie = shd[ii].need_tie;
            u32 key[4];
            float v[4];
            u32 nt = 0;
  #pragma unroll
            for (int k = 0; k < 4; ++k) {
              const bool ok = live && (ALIGNED || c0 + k < d);
              v[k] = __fsub_rn(x[k], g[k]);
              key[k] = ok ? key_of(v[k]) : 0xffffffffu;
              if (ok && key[k] == T) ++nt;
            }
            u32 before = 0;
            if (need_tie) before = tiepref[(long long)i * nchunk + chunk] + block_excl_scan(nt, nullptr);
  #pragma unroll
            for (int k = 0; k < 4; ++k) {
              const bool ok = live && (ALIGNED || c0 + k < d);
              if (!ok) continue;
              if (key[k] > T) kept[k] = true;
              else if (key[k] == T) {
                kept[k] = need_tie ? (before < q) : ((u32)(c0 + k) <= shd[ii].cut);
                ++before;
              }
              if (kept[k]) { g[k] = __fadd_rn(g[k], v[k]); any = true; }
            }
          } else if (mode == 2) {
  #pragma unroll
            for (int k = 0; k < 4; ++k) {
              g[k] = __fadd_rn(g[k], __fsub_rn(x[k], g[k]));
              kept[k] = live && (ALIGNED || c0 + k < d);
            }
            any = live;
          } else {  // quantiser
            const float L = shd[ii].qL, inv = shd[ii].qinv, step = shd[ii].qstep;
  #pragma unroll
            for (int k = 0; k < 4; ++k) {
              const float v = __fsub_rn(x[k], g[k]);
              g[k] = __fadd_rn(g[k], quant_value(v, L, inv, step));
            }
            any = live;
          }
          if (any) store4<ALIGNED>(grow, c0, d, g);
          if (out.kept_idx && (mode == 1 || mode == 2)) {
            int mine = 0;
  #pragma unroll
            for (int k = 0; k < 4; ++k) mine += kept[k] ? 1 : 0;
            int inc = mine;
  #pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
              int t = __shfl_up_sync(0xffffffffu, inc, o);
              if (lane >= o) inc += t;
            }
            const int wtotal = __shfl_sync(0xffffffffu, inc, 31);
            long long base = 0;
            if (lane == 31 && wtotal) base = (long long)atomicAdd((u64*)&out.kept_cnt[i], (u64)wtotal);
            base = __shfl_sync(0xffffffffu, base, 31);
            long long pos = base + inc - mine;
  #pragma unroll
            for (int k = 0; k < 4; ++k)
              if (kept[k]) {
                if (pos < out.kept_stride) out.kept_idx[(long long)i * out.kept_stride + pos] = (int32_t)(c0 + k);
                ++pos;
              }
          }
        }
        if (want_mean) {
  #pragma unroll
          for (int k = 0; k < 4; ++k) acc[k] = __fadd_rn(acc[k], g[k]);
        }
      }
    }
    if (want_mean && live) {
      const float n = (float)rows;
      float r[4];
  #pragma unroll
      for (int k = 0; k < 4; ++k) r[k] = __fdiv_rn(acc[k], n);
      store4<ALIGNED>(out.mean_out, c0, d, r);
    }
  }
}

__global__ void k_copy_report(int rows, long long d, int m, CompressOut out) {
  pdl_begin();
  // identity compressor: level 0, bits 32 d, no error values
  const int row = blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= rows) return;
  if (out.level) out.level[row] = 0;
  if (out.bits) out.bits[row] = 32ull * (uint64_t)d;
  if (out.D) out.D[row] = 0.0;
  if (out.err) out.err[row] = 0.0;
}

// --------------------------------------------------------------------------
// single-pass path: brackets from a sample, one streaming pass, selection on short lists
// --------------------------------------------------------------------------
// Finds the bin holding the r-th largest sampled key (1-based); one warp calls, every lane gets the
// answer.  csum/cexcl: counts and exclusive prefixes of the 256 chunks of 256 bins, descending order.
__device__ u32 sample_rank_bin(const u32* __restrict__ h, const u32* csum, const u32* cexcl, u32 r) {
  const int lane = threadIdx.x & 31;
  int c = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int cc = lane + 32 * i;
    const u32 hit = __ballot_sync(0xffffffffu, cexcl[cc] < r && r <= cexcl[cc] + csum[cc]);
    if (hit) c = 32 * i + (__ffs(hit) - 1);
  }
  const int pos0 = 256 * c + 8 * lane;                         // descending position of this lane's first bin
  const uint4* p = reinterpret_cast<const uint4*>(h + (SBINS - 8 - pos0));
  const uint4 a = __ldcg(p), b = __ldcg(p + 1);                // ascending addresses: positions pos0+7 .. pos0
  const u32 v[8] = {b.w, b.z, b.y, b.x, a.w, a.z, a.y, a.x};   // v[k] = bin at descending position pos0 + k
  u32 lsum = 0;
#pragma unroll
  for (int k = 0; k < 8; ++k) lsum += v[k];
  u32 inc = lsum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const u32 t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  u32 run = cexcl[c] + inc - lsum;
  u32 found = 0xffffffffu;
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    if (r > run && r <= run + v[k]) found = (u32)(SBINS - 1 - (pos0 + k));
    run += v[k];
  }
  const u32 who = __ballot_sync(0xffffffffu, found != 0xffffffffu);
  return __shfl_sync(0xffffffffu, found, who ? (__ffs(who) - 1) : 0);
}

// Per row and Top-K candidate: a bracket [lo, hi) of key values, aligned to sample bins, that
// holds the K-th largest key with overwhelming probability (checked exactly afterwards).
// Called by a whole CTA of any size that is a multiple of 32 threads.
__device__ void bracket_row(const CsetDev& cs, int row, long long d, int full_sample,
                            const u32* __restrict__ shist, SelRow* __restrict__ sel, u32* __restrict__ tickets) {
  __shared__ u32 csum[256], cexcl[256];
  __shared__ u32 s_total;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  const u32* h = shist + (long long)row * SBINS;
  // chunk sums, four chunks (eight 16-byte loads) in flight per warp
  for (int c0 = wid * 4; c0 < 256; c0 += nwarp * 4) {
    uint4 a[4], b[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint4* p = reinterpret_cast<const uint4*>(h + (SBINS - 256 * (c0 + u + 1))) + 2 * lane;
      a[u] = __ldcg(p);
      b[u] = __ldcg(p + 1);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const u32 t = warp_sum_u32(a[u].x + a[u].y + a[u].z + a[u].w + b[u].x + b[u].y + b[u].z + b[u].w);
      if (lane == 0) csum[c0 + u] = t;
    }
  }
  __syncthreads();
  if (wid == 0) {  // exclusive prefix over the 256 chunk sums: eight per lane
    u32 loc[8], sum = 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) { loc[k] = csum[lane * 8 + k]; sum += loc[k]; }
    u32 inc = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const u32 t = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += t;
    }
    u32 run = inc - sum;
#pragma unroll
    for (int k = 0; k < 8; ++k) { cexcl[lane * 8 + k] = run; run += loc[k]; }
    if (lane == 31) s_total = inc;
  }
  __syncthreads();
  const u32 S = s_total;
  // one warp per (candidate, edge)
  for (int w = wid; w < 2 * cs.nsel; w += nwarp) {
    const int j = w >> 1;
    const bool upper = (w & 1) == 0;
    const double K = (double)cs.param[cs.sel[j]];
    const double r = K * (double)S / (double)d;
    const double dev = full_sample ? 0.0 : 6.0 * sqrt(r * (1.0 - K / (double)d)) + 8.0;
    const double r_hi = floor(r - dev), r_lo = ceil(r + dev) + 1.0;
    if (upper) {
      u32 hi = 0x80000000u;
      if (r_hi >= 1.0) hi = (sample_rank_bin(h, csum, cexcl, (u32)r_hi) + 1u) << 15;
      if (lane == 0) sel[row].hi[j] = hi;
    } else {
      u32 lo = 0u;
      if (r_lo <= (double)S) lo = sample_rank_bin(h, csum, cexcl, (u32)r_lo) << 15;
      if (lane == 0) sel[row].lo[j] = lo;
    }
  }
  __syncthreads();
  if (threadIdx.x < cs.nsel) {
    const int j = threadIdx.x;
    const u32 span = sel[row].hi[j] - sel[row].lo[j];            // >= 2^15
    const u32 nbits = 32u - (u32)__clz((int)(span - 1u));
    const u32 sh1 = nbits > 11u ? nbits - 11u : 0u;
    const u32 sh2 = sh1 > 11u ? sh1 - 11u : 0u;
    sel[row].sh1[j] = sh1; sel[row].sh2[j] = sh2;
    if (sh2) tickets[row * NTICKET + 10] = 1u;
  }
}

// The sample of a row: its d elements are cut into granules of SAMP_G consecutive elements (64
// bytes), the granules into windows of `win`, and one granule of every window is taken, at an
// offset that changes from window to window (a hash of the window index), so that neither a period
// nor a block structure of the data lines up with the sample.  The histogram has one bin per value
// of key[30:15].  Per-CTA counts are 16 bit (two bins per shared word): a CTA takes fewer than
// 65536 elements.  Four threads share a granule; SAMP_NL granules are in flight per thread.
constexpr int SAMP_TPB = 1024;
constexpr int SAMP_G = 16;
constexpr int SAMP_NL = 4;
__device__ __forceinline__ long long sample_granule(long long w, long long win, long long ngran) {
  const long long first = w * win;
  const long long span = (ngran - first < win) ? (ngran - first) : win;
  u32 h = (u32)w * 2654435761u;
  h ^= h >> 15; h *= 2246822519u; h ^= h >> 13;
  return first + (long long)(h % (u32)span);
}
template <bool ALIGNED>
__global__ void __launch_bounds__(SAMP_TPB) k_sample(const float* __restrict__ X, const float* __restrict__ G,
                                                     long long d, long long nwin, long long win,
                                                     u32* __restrict__ shist, CsetDev cs, SelRow* __restrict__ sel,
                                                     u32* __restrict__ tickets, u32* __restrict__ maxkey,
                                                     CsetDev* __restrict__ cs_global) {
  // maxkey != nullptr: every element is sampled (win == 1) and the row maximum is wanted already here, so that the
  // streaming pass can evaluate the quantisers
  pdl_begin();
  if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) *cs_global = cs;   // for the last CTAs of the collection pass
  extern __shared__ __align__(16) u32 sh[];  // SBINS / 2 words
  const int row = blockIdx.y;
  for (int i = threadIdx.x; i < SBINS / 8; i += SAMP_TPB) reinterpret_cast<uint4*>(sh)[i] = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
  const float* xr = X + (long long)row * d;
  const float* gr = G + (long long)row * d;
  const long long ngran = (d + SAMP_G - 1) / SAMP_G;
  const long long nquad = (long long)gridDim.x * (SAMP_TPB / 4);
  const int ql = threadIdx.x & 3;
  u32 mxs = 0;
  for (long long w0 = (long long)blockIdx.x * (SAMP_TPB / 4) + (threadIdx.x >> 2); w0 < nwin; w0 += nquad * SAMP_NL) {
    float x[SAMP_NL][4], g[SAMP_NL][4];
    long long c0[SAMP_NL];
#pragma unroll
    for (int u = 0; u < SAMP_NL; ++u) {
      const long long w = w0 + (long long)u * nquad;
      c0[u] = d;
      if (w < nwin) {
        c0[u] = sample_granule(w, win, ngran) * SAMP_G + ql * 4;
        if (c0[u] < d) {
          load4<ALIGNED>(xr, c0[u], d, x[u]);
          load4<ALIGNED>(gr, c0[u], d, g[u]);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < SAMP_NL; ++u) {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (c0[u] + k >= d) break;
        const u32 key = key_of(__fsub_rn(x[u][k], g[u][k]));
        mxs = max(mxs, key);
        const u32 bin = key >> 15;
        atomicAdd(&sh[bin >> 1], (bin & 1u) ? 0x10000u : 1u);
      }
    }
  }
  if (maxkey) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mxs = max(mxs, __shfl_xor_sync(0xffffffffu, mxs, o));
    if ((threadIdx.x & 31) == 0 && mxs) atomicMax(&maxkey[row], mxs);
  }
  __syncthreads();
  u32* gh = shist + (long long)row * SBINS;
  for (int i = threadIdx.x; i < SBINS / 2; i += SAMP_TPB) {
    const u32 w = sh[i];
    if (w & 0xffffu) atomicAdd(&gh[2 * i], w & 0xffffu);
    if (w >> 16) atomicAdd(&gh[2 * i + 1], w >> 16);
  }
  if (last_cta_of_row(&tickets[row * NTICKET + 0], gridDim.x))
    bracket_row(cs, row, d, win == 1 ? 1 : 0, shist, sel, tickets);
}

// The same brackets for rows short enough to be read in full by one CTA (d < 2^18) when there are many
// rows: the histogram, on key[30:16], stays in shared memory with 32-bit counts, the bracket of a candidate is
// the bin that holds its K-th largest key (exact, since every element is counted), and nothing goes through
// global memory but the brackets themselves.  Also yields the row maximum.
constexpr int RS_BINS = 32768;
constexpr int RS_SHIFT = 16;
template <bool ALIGNED>
__global__ void __launch_bounds__(SAMP_TPB) k_sample_row(const float* __restrict__ X, const float* __restrict__ G, long long d,
                                                         CsetDev cs, SelRow* __restrict__ sel, u32* __restrict__ tickets,
                                                         u32* __restrict__ maxkey, CsetDev* __restrict__ cs_global,
                                                         u32* __restrict__ rowflag, u32* __restrict__ diffflag,
                                                         u32* __restrict__ flcnt, u32* __restrict__ cntpart,
                                                         u32* __restrict__ fhist) {
  pdl_begin();
  if (blockIdx.x == 0 && threadIdx.x == 0) *cs_global = cs;   // for the last CTAs of the collection pass
  extern __shared__ __align__(16) u32 sh[];   // RS_BINS counts
  __shared__ u32 wsum[SAMP_TPB / 32];
  const int row = blockIdx.x;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  // This kernel is the first of its call and has one CTA per row: it clears the row's per-call words itself (flags,
  // completion counts, first-digit tables; the row maximum is written below), so the call needs no memset.
  for (int i = threadIdx.x; i < MAXC * LB1; i += SAMP_TPB) fhist[(long long)row * MAXC * LB1 + i] = 0u;
  if (threadIdx.x < NTICKET) tickets[row * NTICKET + threadIdx.x] = 0u;
  if (threadIdx.x >= 32 && threadIdx.x < 32 + MAXC) { flcnt[row * MAXC + threadIdx.x - 32] = 0u; cntpart[row * MAXC + threadIdx.x - 32] = 0u; }
  if (threadIdx.x == 64) { rowflag[row] = 0u; diffflag[row] = 0u; }
  for (int i = threadIdx.x; i < RS_BINS / 4; i += SAMP_TPB) reinterpret_cast<uint4*>(sh)[i] = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
  const float* xr = X + (long long)row * d;
  const float* gr = G + (long long)row * d;
  u32 mx = 0;
  for (long long base = (long long)threadIdx.x * 4; base < d; base += (long long)SAMP_TPB * 4 * SAMP_NL) {
    float x[SAMP_NL][4], g[SAMP_NL][4];
#pragma unroll
    for (int u = 0; u < SAMP_NL; ++u) {
      const long long c0 = base + (long long)u * SAMP_TPB * 4;
      if (c0 < d) {
        load4<ALIGNED>(xr, c0, d, x[u]);
        load4<ALIGNED>(gr, c0, d, g[u]);
      }
    }
#pragma unroll
    for (int u = 0; u < SAMP_NL; ++u) {
      const long long c0 = base + (long long)u * SAMP_TPB * 4;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (c0 + k >= d) break;
        const u32 key = key_of(__fsub_rn(x[u][k], g[u][k]));
        mx = max(mx, key);
        atomicAdd(&sh[key >> RS_SHIFT], 1u);
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if (lane == 0) wsum[wid] = mx;
  __syncthreads();
  if (threadIdx.x == 0) {
    u32 m = 0;
    for (int w = 0; w < SAMP_TPB / 32; ++w) m = max(m, wsum[w]);
    maxkey[row] = m;
  }
  __syncthreads();
  // thread t owns the RS_BINS / SAMP_TPB = 32 bins at descending positions 32 t .. 32 t + 31
  constexpr int PER = RS_BINS / SAMP_TPB;
  u32 mine = 0;
#pragma unroll 8
  for (int k = 0; k < PER; ++k) mine += sh[RS_BINS - 1 - (threadIdx.x * PER + k)];
  u32 inc = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const u32 t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  if (lane == 31) wsum[wid] = inc;
  __syncthreads();
  u32 before = 0;
  for (int w = 0; w < wid; ++w) before += wsum[w];
  const u32 excl = before + inc - mine;                 // keys in bins above this thread's
  for (int j = 0; j < cs.nsel; ++j) {
    const u32 K = (u32)cs.param[cs.sel[j]];             // K < d: the K-th largest key exists
    if (K > excl && K <= excl + mine) {
      u32 run = excl;
      for (int k = 0; k < PER; ++k) {
        const u32 bin = (u32)(RS_BINS - 1 - (threadIdx.x * PER + k));
        const u32 c = sh[bin];
        if (K <= run + c) {
          SelRow* sr = sel + row;
          sr->lo[j] = bin << RS_SHIFT;
          sr->hi[j] = (bin + 1u) << RS_SHIFT;
          sr->sh1[j] = RS_SHIFT - 11;                    // digits of key - lo inside a bracket of 2^16 key values
          sr->sh2[j] = 0u;
          break;
        }
        run += c;
      }
    }
  }
}

// Entries of the candidate set by a run-time index, written as compile-time indexed selects: indexing the kernel
// parameter with a run-time value (or handing its address to a function) makes every thread copy the whole
// structure to local memory first.
__device__ __forceinline__ long long cs_param_at(const CsetDev& cs, int c) {
  long long v = 0;
#pragma unroll
  for (int k = 0; k < MAXC; ++k) v = (k == c) ? cs.param[k] : v;
  return v;
}
__device__ __forceinline__ int cs_sel_at(const CsetDev& cs, int j) {
  int v = 0;
#pragma unroll
  for (int k = 0; k < MAXC; ++k) v = (k == j) ? cs.sel[k] : v;
  return v;
}
__device__ __forceinline__ int cs_qsel_at(const CsetDev& cs, int j) {
  int v = 0;
#pragma unroll
  for (int k = 0; k < MAXC; ++k) v = (k == j) ? cs.qsel[k] : v;
  return v;
}

// Shift that leaves the first LB1-valued digit of key - lo for a bracket [lo, hi).
static_assert(LB1 == TPB, "first_digit_scan reads one bin per thread");
__device__ __forceinline__ u32 first_digit_shift(u32 lo, u32 hi) {
  const u32 span = hi - lo;
  const u32 nbits = span > 1u ? 32u - (u32)__clz((int)(span - 1u)) : 0u;
  return nbits > 8u ? nbits - 8u : 0u;
}

// Run by the last CTA of a row's streaming pass, one warp per bracket.  Checks the bracket exactly
// (the K-th largest key must be one of the listed keys; otherwise the row is flagged for the full
// select) and locates the first-digit bin of its threshold.  A bin with more than FINAL_CAP keys
// sends the row through the three-level list passes.
__device__ __noinline__ void first_digit_scan(int nsel, const long long* s_K, int row, const u32* __restrict__ fhist,
                                              const u32* __restrict__ cnttot, SelRow* __restrict__ sel,
                                              u32* __restrict__ rowflag, u32* __restrict__ tickets,
                                              u32* __restrict__ flags) {
  static_assert(MAXC <= TPB / 32 && LB1 == 256, "one warp per bracket, eight bins per lane");
  __shared__ u32 bad, toofull;
  const int lane = threadIdx.x & 31, j = threadIdx.x >> 5;
  SelRow* s = sel + row;
  if (threadIdx.x == 0) { bad = 0; toofull = 0; }
  __syncthreads();
  if (j < nsel) {
    const u32 above = __ldcg(&cnttot[row * MAXC + j]);            // keys >= hi
    const u32* h = fhist + ((long long)row * MAXC + j) * LB1;
    // bins in descending order: this lane holds positions 8*lane .. 8*lane + 7
    const uint4 q0 = __ldcg(reinterpret_cast<const uint4*>(h + (LB1 - 8 - 8 * lane)));
    const uint4 q1 = __ldcg(reinterpret_cast<const uint4*>(h + (LB1 - 4 - 8 * lane)));
    const u32 v[8] = {q1.w, q1.z, q1.y, q1.x, q0.w, q0.z, q0.y, q0.x};
    u32 lsum = 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) lsum += v[k];
    u32 inc = lsum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const u32 t = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += t;
    }
    const u32 total = __shfl_sync(0xffffffffu, inc, 31);
    const long long K = s_K[j];
    if (K <= (long long)above || K > (long long)above + (long long)total) {
      if (lane == 0) bad = 1;
    } else {
      const u32 krem = (u32)K - above;
      u32 run = inc - lsum;
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        if (krem > run && krem <= run + v[k]) {                  // true in exactly one lane, for one k
          s->above_hi[j] = above; s->fb1[j] = (u32)(LB1 - 1 - (8 * lane + k)); s->fabove1[j] = above + run; s->fc1[j] = v[k];
          if (v[k] > (u32)FINAL_CAP) toofull = 1;
        }
        run += v[k];
      }
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    if (bad || __ldcg(&rowflag[row])) rowflag[row] = 1;   // bracket missed, or a segment overflowed
    else if (toofull) { tickets[row * NTICKET + 13] = 1u; atomicAdd(&flags[3], 1u); }
  }
}

// The streaming pass: D, ||v||^2, per bracket the count of keys >= hi and the energy of keys
// < lo, the row maximum, and the keys inside a bracket appended to this CTA's list segment.
// Sums run in binary32 chains of at most 4*FLUSH_TILES fused multiply-adds (relative error
// <= (4*FLUSH_TILES + 1) 2^-24 for non-negative terms), folded into binary64.
// Every warp runs on its own: P1_UNR tiles of plain 128-bit loads are in flight per thread, and
// the keys that reach the lowest bracket edge (about K_max/d of them) go through a per-warp queue
// compacted with warp votes, drained 32 entries at a time; there is no CTA-wide barrier in the loop.
constexpr int P1_UNR = 2;                                         // tiles in flight per CTA iteration (3: 5 % slower, 1: 4 % slower)
constexpr int P1_QCAP = 160;                                      // 31 left over + 128 new entries per warp
constexpr int P1_FLUSH_IT = FLUSH_TILES / P1_UNR;                 // iterations between folds into binary64
#ifndef P1_MINB3
#define P1_MINB3 4
#endif
// resident CTAs per SM the register budget is set for: more brackets need more state per thread
constexpr int p1_min_ctas(int nsel) { return nsel <= 3 ? P1_MINB3 : (nsel <= 5 ? 3 : 2); }
constexpr int P1_NQ = 3;   // quantisers the streaming pass evaluates itself when the row maximum is known beforehand
template <int NSEL, bool ALIGNED, int QM>
__global__ void __launch_bounds__(TPB, p1_min_ctas(NSEL)) k_pass1(const float* __restrict__ X, const float* __restrict__ G,
                                                  const float* __restrict__ Y, long long d, CsetDev cs,
                                                  SelRow* __restrict__ sel, double* __restrict__ partial,
                                                  u32* __restrict__ cntpart, u64* __restrict__ list,
                                                  u32* __restrict__ lcount, long long list_row, u32 segcap,
                                                  u32* __restrict__ maxkey, u32* __restrict__ rowflag,
                                                  u32* __restrict__ diffflag, u32* __restrict__ flags,
                                                  u32* __restrict__ fhist, u32* __restrict__ tickets) {
  pdl_begin();
  constexpr int NS = NSEL > 0 ? NSEL : 1;
  const int row = blockIdx.y;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  __shared__ u32 sh_cnt;
  __shared__ __align__(8) u64 qbuf[TPB / 32][P1_QCAP];
  __shared__ u32 lh[NS * LB1];                                   // first digit of key - lo, per bracket
  if (threadIdx.x == 0) sh_cnt = 0;
  for (int i = threadIdx.x; i < NS * LB1; i += TPB) lh[i] = 0;
  // bracket edges and digit shifts are only read when a queue is drained: kept in shared memory
  __shared__ u32 s_lo[NS], s_hi[NS], s_shq[NS];
  __shared__ long long s_K[NS];
  u32 cnt[NS];
  float fB[NS];
  double dB[NS];
  float lomin = __uint_as_float(0x7f800000u), fBall = 0.f;
  double dBall = 0.0;
#pragma unroll
  for (int j = 0; j < NS; ++j) {
    const u32 lo = (j < NSEL) ? sel[row].lo[j] : 0u;
    const u32 hi = (j < NSEL) ? sel[row].hi[j] : 0u;
    if (threadIdx.x == 0) { s_lo[j] = lo; s_hi[j] = hi; s_shq[j] = first_digit_shift(lo, hi); s_K[j] = cs_param_at(cs, cs_sel_at(cs, j)); }
    cnt[j] = 0; fB[j] = 0.f; dB[j] = 0.0;
    if (j < NSEL) lomin = fminf(lomin, __uint_as_float(lo));       // lo < 2^31 - 2^15: finite or +inf
  }
  float fD = 0.f, fE = 0.f;
  double dD = 0.0, dE = 0.0;
  u32 mx = 0, df = 0;
  // QM == 2: scale, reciprocal and step of the row's quantisers (the maximum comes from the sampling kernel)
  constexpr int NQR = (QM == 2) ? P1_NQ : 1;
  float qL[NQR], qinv[NQR], qstep[NQR], fQ[NQR];
  double dQ[NQR];
#pragma unroll
  for (int q = 0; q < NQR; ++q) {
    qL[q] = qinv[q] = qstep[q] = fQ[q] = 0.f; dQ[q] = 0.0;
    if (QM == 2 && q < cs.nquant) {
      const float smax = __uint_as_float(__ldcg(&maxkey[row]));
      qL[q] = (float)((1 << ((int)cs_param_at(cs, cs_qsel_at(cs, q)) - 1)) - 1);
      if (smax > 0.f) { qinv[q] = __fdiv_rn(qL[q], smax); qstep[q] = __fdiv_rn(smax, qL[q]); }
    }
  }
  __syncthreads();
  const float* xr = X + (long long)row * d;
  const float* gr = G + (long long)row * d;
  const float* yr = Y + (long long)row * d;
  u64* seg = list + (long long)row * list_row + (long long)blockIdx.x * segcap;
  const long long ntile = (d + TPB * 4 - 1) / (TPB * 4);
  const u32 ltmask = (1u << lane) - 1u;
  // A queued entry meets every bracket: count it if it lies above, add its square if it lies
  // below (fB[j] holds only what fBall does not: keys in [lomin, lo_j)), list it if inside one.
  auto drain = [&](u32 slot, bool act) {
    const u64 e = act ? qbuf[wid][slot] : 0ull;
    const u32 ka = (u32)(e >> 32);
    const float a = __uint_as_float(ka);
    bool inb = false;
#pragma unroll
    for (int j = 0; j < NS; ++j) {
      const u32 lo = s_lo[j];
      const bool ge = ka >= s_hi[j];
      const bool below = ka < lo;
      cnt[j] += (act && ge) ? 1u : 0u;
      fB[j] = (act && below) ? fmaf(a, a, fB[j]) : fB[j];
      const bool in = act && !ge && !below && j < NSEL;
      if (in) atomicAdd(&lh[j * LB1 + ((ka - lo) >> s_shq[j])], 1u);
      inb = inb || in;
    }
    const u32 m = __ballot_sync(0xffffffffu, inb);
    if (m) {
      u32 base = 0;
      if (lane == 0) base = atomicAdd(&sh_cnt, (u32)__popc(m));
      base = __shfl_sync(0xffffffffu, base, 0);
      const u32 pos = base + (u32)__popc(m & ltmask);
      if (inb && pos < segcap) seg[pos] = e;
    }
  };
  u32 qc = 0;  // entries waiting in this warp's queue: the same value in every lane
  int it = 0;
  for (long long t0 = blockIdx.x; t0 < ntile; t0 += (long long)gridDim.x * P1_UNR, ++it) {
    float x[P1_UNR][4], g[P1_UNR][4], y[P1_UNR][4];
#pragma unroll
    for (int u = 0; u < P1_UNR; ++u) {
      const long long c0 = (t0 + (long long)u * gridDim.x) * (TPB * 4) + threadIdx.x * 4;
#pragma unroll
      for (int k = 0; k < 4; ++k) { x[u][k] = 0.f; g[u][k] = 0.f; y[u][k] = 0.f; }
      if (c0 < d) {
        if (ALIGNED) {  // streamed once: evict-first loads
          const float4 a = __ldcs(reinterpret_cast<const float4*>(xr + c0));
          const float4 b = __ldcs(reinterpret_cast<const float4*>(gr + c0));
          const float4 c = __ldcs(reinterpret_cast<const float4*>(yr + c0));
          x[u][0] = a.x; x[u][1] = a.y; x[u][2] = a.z; x[u][3] = a.w;
          g[u][0] = b.x; g[u][1] = b.y; g[u][2] = b.z; g[u][3] = b.w;
          y[u][0] = c.x; y[u][1] = c.y; y[u][2] = c.z; y[u][3] = c.w;
        } else {
          load4<false>(xr, c0, d, x[u]);
          load4<false>(gr, c0, d, g[u]);
          load4<false>(yr, c0, d, y[u]);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < P1_UNR; ++u) {
      const long long c0 = (t0 + (long long)u * gridDim.x) * (TPB * 4) + threadIdx.x * 4;
      float av[4];
      u32 rm = 0;  // which of the four entries reach the lowest bracket edge
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float v = __fsub_rn(x[u][k], g[u][k]);
        const float w = __fsub_rn(x[u][k], y[u][k]);
        fE = fmaf(v, v, fE);
        fD = fmaf(w, w, fD);
        av[k] = fabsf(v);
        if (QM == 1) mx = max(mx, __float_as_uint(av[k]));
        if (QM == 2) {
#pragma unroll
          for (int q = 0; q < P1_NQ; ++q) {
            const float rq = __fsub_rn(v, quant_value(v, qL[q], qinv[q], qstep[q]));
            fQ[q] = fmaf(rq, rq, fQ[q]);   // a quantiser that is not in the list has L = 0: its slot is never read
          }
        }
        df |= __float_as_uint(v) ^ __float_as_uint(w);
        if (NSEL > 0) {
          // finite non-negative binary32 values order like their bit patterns: compare as floats
          const bool small = av[k] < lomin;
          fBall = small ? fmaf(v, v, fBall) : fBall;
          if (!small && (ALIGNED || c0 + k < d)) rm |= 1u << k;
        }
      }
      if (ALIGNED && c0 >= d) rm = 0u;                             // zero padding past the row end is never queued
      if (NSEL > 0 && __any_sync(0xffffffffu, rm != 0u)) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const bool p = (rm >> k) & 1u;
          const u32 m = __ballot_sync(0xffffffffu, p);
          if (p) qbuf[wid][qc + (u32)__popc(m & ltmask)] = ((u64)__float_as_uint(av[k]) << 32) | (u64)(u32)(c0 + k);
          qc += (u32)__popc(m);
        }
        if (qc >= 32) {
          __syncwarp();
          do { qc -= 32; drain(qc + lane, true); } while (qc >= 32);
          __syncwarp();
        }
      }
    }
    if (it % P1_FLUSH_IT == P1_FLUSH_IT - 1) {
      dD += (double)fD; fD = 0.f;
      dE += (double)fE; fE = 0.f;
      dBall += (double)fBall; fBall = 0.f;
#pragma unroll
      for (int j = 0; j < NS; ++j) { dB[j] += (double)fB[j]; fB[j] = 0.f; }
      if (QM == 2) {
#pragma unroll
        for (int q = 0; q < NQR; ++q) { dQ[q] += (double)fQ[q]; fQ[q] = 0.f; }
      }
    }
  }
  if (NSEL > 0) {  // what is left in the queue: fewer than 32 entries
    __syncwarp();
    if (qc) drain((u32)lane < qc ? (u32)lane : 0u, (u32)lane < qc);
  }
  dD += (double)fD;
  dE += (double)fE;
  dBall += (double)fBall;
#pragma unroll
  for (int j = 0; j < NS; ++j) dB[j] += (double)fB[j] + dBall;

  __shared__ double red[2 + NS][TPB / 32];
  __shared__ u32 redc[NS][TPB / 32];
  __shared__ double redq[NQR][TPB / 32];
  if (QM == 2) {
#pragma unroll
    for (int q = 0; q < NQR; ++q) {
      const double vq = warp_sum_f64(dQ[q] + (double)fQ[q]);
      if (lane == 0) redq[q][wid] = vq;
    }
  }
  double v0 = warp_sum_f64(dD), v1 = warp_sum_f64(dE);
  if (lane == 0) { red[0][wid] = v0; red[1][wid] = v1; }
#pragma unroll
  for (int j = 0; j < NS; ++j) {
    const double vb = warp_sum_f64(dB[j]);
    const u32 vc = warp_sum_u32(cnt[j]);
    if (lane == 0) { red[2 + j][wid] = vb; redc[j][wid] = vc; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    df |= __shfl_xor_sync(0xffffffffu, df, o);
  }
  if (lane == 0) {
    if (mx) atomicMax(&maxkey[row], mx);
    df &= 0x7fffffffu;  // sign differences do not matter: only |X-G| against |X-Y|
    if (df) atomicOr(&diffflag[row], df);
  }
  __syncthreads();
  const long long pbase = ((long long)row * MAX_BLK_PER_ROW + blockIdx.x);
  if (threadIdx.x < 2 + NSEL) {
    const int s = threadIdx.x;
    double acc = 0;
    for (int w = 0; w < TPB / 32; ++w) acc += red[s][w];
    const int slot = (s < 2) ? s : 2 + cs_sel_at(cs, s - 2);
    partial[pbase * NSLOT + slot] = acc;
  }
  if (QM == 2 && threadIdx.x >= 64 && threadIdx.x < 64 + cs.nquant) {
    const int q = threadIdx.x - 64;
    double acc = 0;
    for (int w = 0; w < TPB / 32; ++w) acc += redq[q][w];
    partial[pbase * NSLOT + 2 + cs_qsel_at(cs, q)] = acc;
  }
  if (threadIdx.x >= 32 && threadIdx.x < 32 + NSEL) {
    const int j = threadIdx.x - 32;
    u32 acc = 0;
    for (int w = 0; w < TPB / 32; ++w) acc += redc[j][w];
    if (acc) atomicAdd(&cntpart[row * MAXC + j], acc);
  }
  if (threadIdx.x == 0 && NSEL > 0) {
    const u32 n = sh_cnt;
    lcount[pbase] = n < segcap ? n : segcap;
    if (n > segcap) atomicOr(&rowflag[row], 1u);
  }
  if (NSEL > 0) {
    u32* gh = fhist + (long long)row * MAXC * LB1;
    for (int i = threadIdx.x; i < NSEL * LB1; i += TPB) {
      const u32 c = lh[i];
      if (c) atomicAdd(&gh[i], c);
    }
    if (last_cta_of_row(&tickets[row * NTICKET + 11], gridDim.x))
      first_digit_scan(NSEL, s_K, row, fhist, cntpart, sel, rowflag, tickets, flags);
  }
}

// ---- exact selection among the listed keys -------------------------------------------------
// Inside its bracket a key is identified by rel = key - lo < hi - lo, split into up to three
// digits: d1 = rel >> sh1 (11 bits), d2 = the next sh1 - sh2 <= 11 bits, d3 = the last sh2 <= 9 bits.
// The first digit is histogrammed by the streaming pass itself, the second by one pass over the
// lists, the third (only for brackets wider than 2^22 key values) by another.
__device__ __forceinline__ u32 digit2(u32 rel, u32 sh1, u32 sh2) { return (rel >> sh2) & ((1u << (sh1 - sh2)) - 1u); }

// Completes bracket j of a row once its threshold key is known (run by a whole CTA).
__device__ void finalize_band(SelRow* s, int row, int j, u32 T, u32 above, u32 ntie, u32 K, double energy,
                              const u64* __restrict__ fl, const u32* __restrict__ flcnt) {
  __shared__ u32 ties[1024];
  __shared__ u32 nties_sh;
  const u32 q = K - above;
  if (threadIdx.x == 0) {
    s->T[j] = T; s->above[j] = above; s->ntie[j] = ntie; s->q[j] = q; s->extraE[j] = energy;
  }
  // Which threshold-equal keys are kept: the q with the lowest indices.  They are all among the
  // entries collected at the last digit level; the q-th smallest of their indices is the cut.
  const u32 nfl = __ldcg(&flcnt[row * MAXC + j]);
  if (q == ntie) {
    if (threadIdx.x == 0) { s->tiemode[j] = 0u; s->cut[j] = 0xffffffffu; }
  } else if (nfl > FINAL_CAP || ntie > 1024u) {
    if (threadIdx.x == 0) { s->tiemode[j] = 2u; s->cut[j] = 0xffffffffu; }
  } else {
    if (threadIdx.x == 0) nties_sh = 0;
    __syncthreads();
    const u64* f = fl + ((long long)row * MAXC + j) * FINAL_CAP;
    for (u32 i = threadIdx.x; i < nfl; i += TPB) {
      const u64 ent = __ldcg(&f[i]);
      if ((u32)(ent >> 32) == T) ties[atomicAdd(&nties_sh, 1u)] = (u32)ent;
    }
    __syncthreads();
    for (u32 i = threadIdx.x; i < ntie; i += TPB) {
      const u32 mine = ties[i];
      u32 rank = 0;
      for (u32 k = 0; k < ntie; ++k) rank += (ties[k] < mine) ? 1u : 0u;
      if (rank == q - 1u) { s->tiemode[j] = 1u; s->cut[j] = mine; }
    }
  }
  __syncthreads();
}

// Sum over the bins below `bin` of count * value^2, every bin being a single key value
// base + b; all TPB threads call, the result is valid in thread 0.
__device__ double bins_energy_below(const u32* __restrict__ h, u32 bin, u32 base) {
  __shared__ double redd[TPB / 32];
  double a = 0.0;
  for (u32 b = threadIdx.x; b < bin; b += TPB) {
    const double kv = (double)__uint_as_float(base + b);
    a += (double)__ldcg(&h[b]) * (kv * kv);
  }
  a = warp_sum_f64(a);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) redd[threadIdx.x >> 5] = a;
  __syncthreads();
  double e = 0.0;
  if (threadIdx.x == 0)
    for (int w = 0; w < TPB / 32; ++w) e += redd[w];
  return e;
}

// Run by the last CTA of a row after digit level LEVEL has been histogrammed.
template <int LEVEL>
__device__ __noinline__ void lscan_row(const CsetDev& cs, int row, int nblk, int nlb, const u32* __restrict__ hist,
                          const u32* __restrict__ cntpart, const double* __restrict__ lepart2,
                          const double* __restrict__ lepart3, SelRow* __restrict__ sel,
                          u32* __restrict__ rowflag, const u64* __restrict__ fl, const u32* __restrict__ flcnt) {
  __shared__ u32 res[2];
  __shared__ u32 bad;
  constexpr int NB = (LEVEL == 3) ? BINS3 : BINS1;
  SelRow* s = sel + row;
  if (LEVEL == 1) {
    // exact check of every bracket: the K-th largest key must be one of the listed keys
    if (threadIdx.x == 0) bad = 0;
    __syncthreads();
    for (int j = 0; j < cs.nsel; ++j) {
      u32 a = 0, tot = 0;
      if (threadIdx.x == 0) a = __ldcg(&cntpart[row * MAXC + j]);
      const u32* h = hist + ((long long)row * MAXC + j) * NB;
      for (int b = threadIdx.x; b < NB; b += TPB) tot += __ldcg(&h[b]);
      u32 above, total;
      block_excl_scan(a, &above);
      block_excl_scan(tot, &total);
      if (threadIdx.x == 0) {
        const long long K = cs.param[cs.sel[j]];
        s->above_hi[j] = above;
        if (K <= (long long)above || K > (long long)above + (long long)total) bad = 1;
      }
    }
    __syncthreads();
    if (bad || __ldcg(&rowflag[row])) {   // bracket missed, or a list segment overflowed
      if (threadIdx.x == 0) rowflag[row] = 1;
      return;
    }
  }
  for (int j = 0; j < cs.nsel; ++j) {
    const u32 sh1 = s->sh1[j], sh2 = s->sh2[j];
    if (LEVEL == 3 && sh2 == 0) continue;  // finished at level 2
    const u32 K = (u32)cs.param[cs.sel[j]];
    const u32* h = hist + ((long long)row * MAXC + j) * NB;
    const u32 before = (LEVEL == 1) ? s->above_hi[j] : (LEVEL == 2 ? s->above1[j] : s->above2[j]);
    block_find_kth_desc(h, NB, K - before, res);
    const u32 bin = res[0], above = before + res[1];
    if (LEVEL == 1) {
      if (threadIdx.x == 0) { s->b1[j] = bin; s->above1[j] = above; }
    } else if (LEVEL == 2 && sh2 != 0) {
      if (threadIdx.x == 0) { s->p2[j] = bin; s->above2[j] = above; }
    } else {
      // last level of this bracket: each bin is one key value
      const u32 base = s->lo[j] + ((LEVEL == 2) ? (s->b1[j] << sh1) : ((s->b1[j] << sh1) | (s->p2[j] << sh2)));
      double e = bins_energy_below(h, bin, base);
      // energies the list passes found below the chosen digits, one partial per CTA (fixed order)
      double part = 0.0;
      for (int b = threadIdx.x; b < nlb; b += TPB) {
        part += __ldcg(&lepart2[((long long)row * LIST_BLK + b) * MAXC + j]);
        if (LEVEL == 3) part += __ldcg(&lepart3[((long long)row * LIST_BLK + b) * MAXC + j]);
      }
      __shared__ double e_sh, part_sh[TPB / 32];
      part = warp_sum_f64(part);
      if ((threadIdx.x & 31) == 0) part_sh[threadIdx.x >> 5] = part;
      __syncthreads();
      if (threadIdx.x == 0) {
        for (int w = 0; w < TPB / 32; ++w) e += part_sh[w];
        e_sh = e;
        res[0] = __ldcg(&h[bin]);
      }
      __syncthreads();
      finalize_band(s, row, j, base + bin, above, res[0], K, e_sh, fl, flcnt);
    }
    __syncthreads();
  }
}

// Pass over the listed keys for digit level LEVEL (1, 2 or 3).
template <int LEVEL>
__device__ __forceinline__ void d_lhist(int bx, int by, int gx, u32* sh, const CsetDev& cs, int nseg, SelRow* sel,
                                               const u64* list, const u32* lcount,
                                               long long list_row, u32 segcap, u32* hist,
                                               double* lepart2, double* lepart3,
                                               u32* rowflag, u64* fl,
                                               u32* flcnt, const u32* cntpart,
                                               u32* tickets) {
  const int row = by;
  const int nsel = cs.nsel;
  if (__ldcg(&rowflag[row]) || !__ldcg(&tickets[row * NTICKET + 13])) return;  // only rows whose first-digit bin is too full
  if (LEVEL == 3 && !__ldcg(&tickets[row * NTICKET + 10])) return;  // no bracket of this row needs a third digit
  constexpr int NB = (LEVEL == 3) ? BINS3 : BINS1;
  for (int i = threadIdx.x; i < nsel * NB; i += TPB) sh[i] = 0;
  u32 lo[MAXC], hi[MAXC], sh1[MAXC], sh2[MAXC], b1[MAXC], b2[MAXC];
  double en[MAXC];
#pragma unroll
  for (int j = 0; j < MAXC; ++j) {
    lo[j] = (j < nsel) ? sel[row].lo[j] : 1u;
    hi[j] = (j < nsel) ? sel[row].hi[j] : 0u;
    sh1[j] = (j < nsel) ? sel[row].sh1[j] : 0u;
    sh2[j] = (j < nsel) ? sel[row].sh2[j] : 0u;
    b1[j] = (j < nsel && LEVEL >= 2) ? __ldcg(&sel[row].b1[j]) : 0u;
    b2[j] = (j < nsel && LEVEL == 3) ? __ldcg(&sel[row].p2[j]) : 0u;
    en[j] = 0.0;
  }
  __syncthreads();
  for (int sg = bx; sg < nseg; sg += gx) {
    const u32 n = lcount[(long long)row * MAX_BLK_PER_ROW + sg];
    const u64* seg = list + (long long)row * list_row + (long long)sg * segcap;
    for (u32 i = threadIdx.x; i < n; i += TPB) {
      const u64 ent = seg[i];
      const u32 key = (u32)(ent >> 32);
#pragma unroll
      for (int j = 0; j < MAXC; ++j) {
        if (j < nsel && key >= lo[j] && key < hi[j]) {
          const u32 rel = key - lo[j];
          const u32 d1 = rel >> sh1[j];
          if (LEVEL == 1) {
            atomicAdd(&sh[j * NB + d1], 1u);
          } else if (LEVEL == 2) {
            if (d1 < b1[j]) { const double kv = (double)__uint_as_float(key); en[j] += kv * kv; }
            else if (d1 == b1[j]) {
              atomicAdd(&sh[j * NB + digit2(rel, sh1[j], sh2[j])], 1u);
              if (sh2[j] == 0) {
                const u32 pos = atomicAdd(&flcnt[row * MAXC + j], 1u);
                if (pos < FINAL_CAP) fl[((long long)row * MAXC + j) * FINAL_CAP + pos] = ent;
              }
            }
          } else if (sh2[j] != 0 && d1 == b1[j]) {
            const u32 d2 = digit2(rel, sh1[j], sh2[j]);
            if (d2 < b2[j]) { const double kv = (double)__uint_as_float(key); en[j] += kv * kv; }
            else if (d2 == b2[j]) {
              atomicAdd(&sh[j * NB + (rel & ((1u << sh2[j]) - 1u))], 1u);
              const u32 pos = atomicAdd(&flcnt[row * MAXC + j], 1u);
              if (pos < FINAL_CAP) fl[((long long)row * MAXC + j) * FINAL_CAP + pos] = ent;
            }
          }
        }
      }
    }
  }
  __syncthreads();
  u32* gh = hist + (long long)row * MAXC * NB;
  for (int i = threadIdx.x; i < nsel * NB; i += TPB)
    if (sh[i]) atomicAdd(&gh[i], sh[i]);
  if (LEVEL >= 2) {
    __shared__ double red[MAXC][TPB / 32];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
    for (int j = 0; j < MAXC; ++j) {
      const double vb = warp_sum_f64(en[j]);
      if (lane == 0) red[j][wid] = vb;
    }
    __syncthreads();
    if (threadIdx.x < MAXC) {
      double a = 0;
      for (int w = 0; w < TPB / 32; ++w) a += red[threadIdx.x][w];
      double* lp = (LEVEL == 2) ? lepart2 : lepart3;
      lp[((long long)row * LIST_BLK + bx) * MAXC + threadIdx.x] = a;
    }
  }
  if (last_cta_of_row(&tickets[row * NTICKET + LEVEL], gx))
    lscan_row<LEVEL>(cs, row, nseg, gx, hist, cntpart, lepart2, lepart3, sel, rowflag, fl, flcnt);
}


// ---- the usual case: the threshold's first-digit bin holds at most FINAL_CAP keys ----------------
// Completes the brackets of a row from the keys collected out of each threshold's bin.  One warp
// per bracket, all brackets at once: a radix select over the remaining low bits of key - lo (8 bits
// per round, 256 bins scanned by the warp) gives the threshold, the counts above and equal, and how
// many threshold-equal keys are kept; those are the ones with the lowest indices, found by ranking
// the equal keys' indices.  `wbuf` is dynamic shared memory, FINISH_WORDS words per bracket.
constexpr int TIE_CAP = 1024;                        // threshold-equal keys ranked here; more go to the chunk-prefix pass
constexpr int FINISH_WORDS = FINAL_CAP + TIE_CAP;
__device__ __noinline__ void collected_finish_row(const CsetDev& cs, int row, int nlb, SelRow* __restrict__ sel,
                                                  const u64* __restrict__ fl, const double* __restrict__ lepart,
                                                  u32* __restrict__ wbuf) {
  static_assert(MAXC <= TPB / 32, "one warp per bracket");
  __shared__ u32 whist[TPB / 32][256];
  const int lane = threadIdx.x & 31, j = threadIdx.x >> 5;
  if (j >= cs.nsel) return;
  SelRow* s = sel + row;
  u32* ek = wbuf + (size_t)j * FINISH_WORDS;
  u32* ties = ek + FINAL_CAP;
  u32* hist = whist[j];
  const u32 c1 = __ldcg(&s->fc1[j]);
  const u32 K = (u32)cs.param[cs.sel[j]];
  const u32 need = K - __ldcg(&s->fabove1[j]);        // 1 <= need <= c1 <= FINAL_CAP
  const u32 lo = __ldcg(&s->lo[j]);
  const u32 shq = first_digit_shift(lo, __ldcg(&s->hi[j]));
  const u32 base = lo + (__ldcg(&s->fb1[j]) << shq);  // every collected key lies in [base, base + 2^shq)
  const u64* f = fl + ((long long)row * MAXC + j) * FINAL_CAP;
  for (u32 i = lane; i < c1; i += 32) ek[i] = (u32)(__ldcg(&f[i]) >> 32);
  __syncwarp();
  u32 prefix = 0, pmask = 0, krem = need, neq = c1;
  for (u32 bits = shq; bits > 0;) {
    const u32 nb = bits < 8u ? bits : 8u, shift = bits - nb;
    for (int b = lane; b < 256; b += 32) hist[b] = 0;
    __syncwarp();
    for (u32 i = lane; i < c1; i += 32) {
      const u32 rel = ek[i] - base;
      if ((rel & pmask) == prefix) atomicAdd(&hist[(rel >> shift) & ((1u << nb) - 1u)], 1u);
    }
    __syncwarp();
    // bins in descending order: this lane holds positions 8*lane .. 8*lane + 7
    u32 v[8], lsum = 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) { v[k] = hist[255 - (8 * lane + k)]; lsum += v[k]; }
    u32 inc = lsum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const u32 t = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += t;
    }
    u32 run = inc - lsum, fbin = 0, fabove = 0, fcnt = 0;
    bool found = false;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      if (!found && krem > run && krem <= run + v[k]) { found = true; fbin = 255u - (u32)(8 * lane + k); fabove = run; fcnt = v[k]; }
      run += v[k];
    }
    const u32 who = __ballot_sync(0xffffffffu, found);
    const int src = who ? (__ffs(who) - 1) : 0;       // exactly one lane finds it: 1 <= krem <= matching keys
    fbin = __shfl_sync(0xffffffffu, fbin, src);
    fabove = __shfl_sync(0xffffffffu, fabove, src);
    fcnt = __shfl_sync(0xffffffffu, fcnt, src);
    prefix |= fbin << shift;
    pmask |= ((1u << nb) - 1u) << shift;
    krem -= fabove;
    neq = fcnt;
    bits = shift;
    __syncwarp();
  }
  const u32 T = base + prefix, q = krem;              // q of the neq keys equal to T are kept
  // energy of the listed keys in [lo, T): collected keys below T, then the per-CTA sums over lower bins
  double e = 0.0;
  for (u32 i = lane; i < c1; i += 32)
    if (ek[i] < T) { const double kv = (double)__uint_as_float(ek[i]); e += kv * kv; }
  for (int b = lane; b < nlb; b += 32) e += __ldcg(&lepart[((long long)row * LIST_BLK + b) * MAXC + j]);
  e = warp_sum_f64(e);
  u32 mode = 0u, cut = 0xffffffffu;
  if (q < neq) {
    mode = 2u;
    if (neq <= (u32)TIE_CAP) {
      mode = 1u;
      // indices of the threshold-equal keys, compacted in any order; the q-th smallest is the cut
      u32 nt = 0;
      for (u32 i0 = 0; i0 < c1; i0 += 32) {
        const u32 i = i0 + lane;
        const bool eq = i < c1 && ek[i] == T;
        const u32 m = __ballot_sync(0xffffffffu, eq);
        if (eq) ties[nt + (u32)__popc(m & ((1u << lane) - 1u))] = (u32)__ldcg(&f[i]);
        nt += (u32)__popc(m);
      }
      __syncwarp();
      for (u32 i = lane; i < neq; i += 32) {
        const u32 mine = ties[i];
        u32 rank = 0;
        for (u32 k = 0; k < neq; ++k) rank += (ties[k] < mine) ? 1u : 0u;
        if (rank == q - 1u) cut = mine;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) cut = min(cut, __shfl_xor_sync(0xffffffffu, cut, o));
    }
  }
  if (lane == 0) {
    s->T[j] = T; s->above[j] = K - q; s->ntie[j] = neq; s->q[j] = q; s->extraE[j] = e;
    s->tiemode[j] = mode; s->cut[j] = cut;
  }
}

// One pass over the listed keys: energies below the threshold's first-digit bin, and the keys of
// that bin collected for collected_finish_row; the last CTA of a row finishes it and, when no other
// kernel has to contribute sums first (pick_here), chooses the row's level at once.
__global__ void __launch_bounds__(TPB) k_lcollect(CsetDev cs, int nseg, SelRow* __restrict__ sel,
                                                  const u64* __restrict__ list, const u32* __restrict__ lcount,
                                                  long long list_row, u32 segcap, double* __restrict__ lepart,
                                                  const u32* __restrict__ rowflag, u64* __restrict__ fl,
                                                  u32* __restrict__ flcnt, u32* __restrict__ tickets,
                                                  int pick_here, long long d, int nblk_main,
                                                  const double* __restrict__ partial, const u32* __restrict__ maxkey,
                                                  RowDec* __restrict__ dec, u32* __restrict__ flags, CompressOut out,
                                                  const u32* __restrict__ diffflag, double tol,
                                                  const CsetDev* __restrict__ cs_global) {
  // cs_global: the same candidate set in global memory (written by the sampling kernel).  The row's last CTA hands
  // the set to functions that index it with run-time values; doing that with the kernel parameter would make every
  // thread of every CTA copy it to local memory first.
  pdl_begin();
  extern __shared__ __align__(16) u32 wbuf[];          // cs.nsel * FINISH_WORDS words, used by the row's last CTA
  const int row = blockIdx.y;
  const int nsel = cs.nsel;
  // everything the pass needs is requested before the first value is looked at
  const u32 skip_a = __ldcg(&rowflag[row]), skip_b = __ldcg(&tickets[row * NTICKET + 13]);
  int sg = blockIdx.x;
  u32 n_next = (sg < nseg) ? __ldcg(&lcount[(long long)row * MAX_BLK_PER_ROW + sg]) : 0u;
  u32 lo[MAXC], hi[MAXC], shq[MAXC], b1[MAXC];
  double en[MAXC];
#pragma unroll
  for (int j = 0; j < MAXC; ++j) {
    lo[j] = (j < nsel) ? __ldcg(&sel[row].lo[j]) : 1u;
    hi[j] = (j < nsel) ? __ldcg(&sel[row].hi[j]) : 0u;
    b1[j] = (j < nsel) ? __ldcg(&sel[row].fb1[j]) : 0u;
    en[j] = 0.0;
  }
  if (skip_a || skip_b) return;
#pragma unroll
  for (int j = 0; j < MAXC; ++j) shq[j] = first_digit_shift(lo[j], hi[j]);
  // the segment lengths are fetched one segment ahead, the entries four per thread at a time
  for (; sg < nseg; sg += gridDim.x) {
    const u32 n = n_next;
    const int sgn = sg + (int)gridDim.x;
    n_next = (sgn < nseg) ? __ldcg(&lcount[(long long)row * MAX_BLK_PER_ROW + sgn]) : 0u;
    const u64* seg = list + (long long)row * list_row + (long long)sg * segcap;
    for (u32 i0 = threadIdx.x; i0 < n; i0 += 4 * TPB) {
      u64 ents[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) ents[u] = (i0 + u * TPB < n) ? __ldcg(&seg[i0 + u * TPB]) : 0ull;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (i0 + u * TPB >= n) break;
        const u64 ent = ents[u];
        const u32 key = (u32)(ent >> 32);
#pragma unroll
        for (int j = 0; j < MAXC; ++j) {
          if (j < nsel && key >= lo[j] && key < hi[j]) {
            const u32 d1 = (key - lo[j]) >> shq[j];
            if (d1 < b1[j]) { const double kv = (double)__uint_as_float(key); en[j] += kv * kv; }
            else if (d1 == b1[j]) {
              const u32 pos = atomicAdd(&flcnt[row * MAXC + j], 1u);
              if (pos < FINAL_CAP) fl[((long long)row * MAXC + j) * FINAL_CAP + pos] = ent;
            }
          }
        }
      }
    }
  }
  __shared__ double red[MAXC][TPB / 32];
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
  for (int j = 0; j < MAXC; ++j) {
    const double vb = warp_sum_f64(en[j]);
    if (lane == 0) red[j][wid] = vb;
  }
  __syncthreads();
  if (threadIdx.x < MAXC) {
    double a = 0;
    for (int w = 0; w < TPB / 32; ++w) a += red[threadIdx.x][w];
    lepart[((long long)row * LIST_BLK + blockIdx.x) * MAXC + threadIdx.x] = a;
  }
  if (!last_cta_of_row(&tickets[row * NTICKET + 12], gridDim.x)) return;
  collected_finish_row(*cs_global, row, (int)gridDim.x, sel, fl, lepart, wbuf);
  __syncthreads();   // the brackets' results, written by one warp each, are read by the level choice
  if (pick_here) {
    pick_row(*cs_global, d, row, nblk_main, nblk_main, partial, sel, maxkey, dec, flags, out, diffflag, tol);
    if (threadIdx.x == 0) tickets[row * NTICKET + 9] = 1u;
  }
}


// --------------------------------------------------------------------------
// the rarely needed steps of the single-pass route, one launch
// --------------------------------------------------------------------------
// After the streaming pass and the collection pass most calls have nothing left to decide.  What may remain:
//   L  rows whose threshold bin holds more keys than the collection buffer: three digit levels over the key lists;
//   F  rows whose bracket missed (or whose list overflowed): the full three-pass select and the energies;
//   P  rows without a level yet (the two above, or every row when quantiser errors come from a separate pass);
//   E  rows whose fast sums could not certify a trigger decision: exact integer sums;
//   T  rows with more threshold-equal keys than the ranking buffers hold: per-chunk tie counts.
// One cooperative grid looks at the per-row flags and returns at once when none is set; otherwise it walks the
// phases in order, its CTAs standing in for the grids of the separate kernels (bx of gx per row), with a grid-wide
// barrier wherever a phase reads what the one before wrote.  Every CTA derives the same phase mask from the same
// memory: a barrier follows each look at the flags before anything that may change them runs.
struct SideArgs {
  const float *X, *G, *Y;
  long long d;
  int rows, nseg, lh_gx, f_gx, t_gx, nblk_main;
  const CsetDev* cs_global;
  SelRow* sel;
  const u64* list;
  const u32* lcount;
  long long list_row;
  u32 segcap;
  u32 *lhist1, *hist1, *hist2, *hist3;
  double *lepart, *lepart3, *partial;
  u32 *rowflag, *flcnt, *tickets, *maxkey, *flags, *diffflag, *tiecnt;
  const u32* cntpart;
  u64 *fl, *limbs;
  RowDec* dec;
  long long nchunk;
  CompressOut out;
  double tol;
};

constexpr u32 SIDE_L = 1u, SIDE_F = 2u, SIDE_P = 4u, SIDE_E = 8u, SIDE_T = 16u;

__device__ __forceinline__ u32 side_mask(const SideArgs& a) {
  u32 m = 0;
  for (int r = threadIdx.x; r < a.rows; r += TPB) {
    if (__ldcg(&a.rowflag[r])) m |= SIDE_F;
    else if (__ldcg(&a.tickets[r * NTICKET + 13])) m |= SIDE_L;
    if (!__ldcg(&a.tickets[r * NTICKET + 9])) m |= SIDE_P;
    if (__ldcg(&a.dec[r].need_exact)) m |= SIDE_E;
    if (__ldcg(&a.dec[r].need_tie)) m |= SIDE_T;
  }
  // bitwise OR over the CTA
  __shared__ u32 all;
  if (threadIdx.x == 0) all = 0;
  __syncthreads();
  m = __reduce_or_sync(0xffffffffu, m);
  if ((threadIdx.x & 31) == 0 && m) atomicOr(&all, m);
  __syncthreads();
  m = all;
  __syncthreads();   // `all` may be cleared by the next call only after everyone has read it
  return m;
}

template <bool ALIGNED>
__global__ void __launch_bounds__(TPB) k_side(SideArgs a) {
  namespace cg = cooperative_groups;
  u32 m = side_mask(a);
  if (!m) return;                                   // the usual call
  cg::grid_group grid = cg::this_grid();
  extern __shared__ u32 sh[];
  __shared__ CsetDev cs;
  if (threadIdx.x == 0) cs = *a.cs_global;
  __syncthreads();
  const int G = (int)gridDim.x, b0 = (int)blockIdx.x;
  // The tables of the phases below are not cleared per call: the grid clears them here, for the rows that use them
  // (the exact sums' limbs, which are small, for every row).  The barrier that follows separates this from their use.
  {
    const long long gtid = (long long)b0 * TPB + threadIdx.x, gsz = (long long)G * TPB;
    for (int r = 0; r < a.rows; ++r) {
      if (!__ldcg(&a.rowflag[r]) && !__ldcg(&a.tickets[r * NTICKET + 13])) continue;
      for (long long i = gtid; i < BINS1; i += gsz) a.hist1[(long long)r * BINS1 + i] = 0u;
      for (long long i = gtid; i < MAXC * BINS2; i += gsz) a.hist2[(long long)r * MAXC * BINS2 + i] = 0u;
      for (long long i = gtid; i < MAXC * BINS3; i += gsz) a.hist3[(long long)r * MAXC * BINS3 + i] = 0u;
      for (long long i = gtid; i < MAXC * BINS1; i += gsz) a.lhist1[(long long)r * MAXC * BINS1 + i] = 0u;
    }
    for (long long i = gtid; i < (long long)a.rows * NSLOT * NLIMB; i += gsz) a.limbs[i] = 0ull;
  }
  grid.sync();
#define SIDE_PHASE(gx, call)                                   \
  for (int v = b0; v < (gx) * a.rows; v += G) {                \
    const int bx = v % (gx), by = v / (gx);                    \
    call;                                                      \
    __syncthreads();                                           \
  }
  if (m & SIDE_L) {
    SIDE_PHASE(a.lh_gx, d_lhist<1>(bx, by, a.lh_gx, sh, cs, a.nseg, a.sel, a.list, a.lcount, a.list_row, a.segcap, a.lhist1,
                                   a.lepart, a.lepart3, a.rowflag, a.fl, a.flcnt, a.cntpart, a.tickets))
    grid.sync();
    SIDE_PHASE(a.lh_gx, d_lhist<2>(bx, by, a.lh_gx, sh, cs, a.nseg, a.sel, a.list, a.lcount, a.list_row, a.segcap, a.hist2,
                                   a.lepart, a.lepart3, a.rowflag, a.fl, a.flcnt, a.cntpart, a.tickets))
    grid.sync();
    SIDE_PHASE(a.lh_gx, d_lhist<3>(bx, by, a.lh_gx, sh, cs, a.nseg, a.sel, a.list, a.lcount, a.list_row, a.segcap, a.hist3,
                                   a.lepart, a.lepart3, a.rowflag, a.fl, a.flcnt, a.cntpart, a.tickets))
    grid.sync();
    m = side_mask(a);                               // the first level may have found a bracket that missed
    grid.sync();
  }
  if (m & SIDE_F) {
    SIDE_PHASE(a.f_gx, (d_hist<1, ALIGNED>(bx, by, a.f_gx, sh, a.X, a.G, a.d, cs, a.sel, a.hist1, a.maxkey, a.rowflag, a.tickets, a.flags)))
    grid.sync();
    SIDE_PHASE(a.f_gx, (d_hist<2, ALIGNED>(bx, by, a.f_gx, sh, a.X, a.G, a.d, cs, a.sel, a.hist2, a.maxkey, a.rowflag, a.tickets, a.flags)))
    grid.sync();
    SIDE_PHASE(a.f_gx, (d_hist<3, ALIGNED>(bx, by, a.f_gx, sh, a.X, a.G, a.d, cs, a.sel, a.hist3, a.maxkey, a.rowflag, a.tickets, a.flags)))
    grid.sync();
    SIDE_PHASE(a.f_gx, d_energy<ALIGNED>(bx, by, a.f_gx, a.X, a.G, a.Y, a.d, cs, a.sel, a.partial, a.rowflag, a.diffflag))
    grid.sync();
  }
  if (m & SIDE_P) {
    for (int row = b0; row < a.rows; row += G) {
      d_pick(row, cs, a.d, a.nblk_main, a.f_gx, a.rowflag, a.partial, a.sel, a.maxkey, a.dec, a.flags, a.out, a.diffflag, a.tickets,
             a.tol);
      __syncthreads();
    }
    grid.sync();
    m = side_mask(a);
    grid.sync();
  }
  if (m & SIDE_E) {
    SIDE_PHASE(a.f_gx, d_exact_sums<ALIGNED>(bx, by, a.f_gx, a.X, a.G, a.Y, a.d, cs, a.sel, a.maxkey, a.dec, a.limbs, a.diffflag, a.d,
                                             a.out, a.tickets, a.flags))
    grid.sync();
    m = side_mask(a);                               // the exact decision may pick another level
    grid.sync();
  }
  if (m & SIDE_T) {
    SIDE_PHASE(a.t_gx, d_tiecount<ALIGNED>(bx, by, a.t_gx, a.X, a.G, a.d, a.dec, a.tiecnt, a.nchunk, a.tickets))
  }
#undef SIDE_PHASE
}

// --------------------------------------------------------------------------
// host side
// --------------------------------------------------------------------------
static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

static long long nchunk_of(long long d) { return (d + UPD_COLS - 1) / UPD_COLS; }

struct Layout {
  size_t hist1, hist2, hist3, maxkey, limbs, flags, csdev, zero_end, zero_rare, sel, dec, partial, energy, tiecnt, total;
  size_t tickets, rowflag, diffflag, shist, lhist1, fhist, list, lcount, cntpart, lepart, lepart3, fl, flcnt;
  long long list_row;
};

static long long list_row_of(long long d) {
  long long a = d / 8, b = d < 65536 ? d : 65536;
  long long r = a > b ? a : b;
  return (r + 31) / 32 * 32;
}

static Layout layout_of(int rows, long long d, bool single_pass) {
  Layout L;
  size_t o = 0;
  // first the tables that only the side paths of the single-pass route use (k_side clears them itself, for the rows
  // that need them), then what every call needs cleared
  L.hist1 = o; o = align_up(o + (size_t)rows * BINS1 * 4, 256);
  L.hist2 = o; o = align_up(o + (size_t)rows * MAXC * BINS2 * 4, 256);
  L.hist3 = o; o = align_up(o + (size_t)rows * MAXC * BINS3 * 4, 256);
  L.limbs = o; o = align_up(o + (size_t)rows * NSLOT * NLIMB * 8, 256);
  L.lhist1 = o;
  if (single_pass) o = align_up(o + (size_t)rows * MAXC * BINS1 * 4, 256);
  L.zero_rare = o;
  L.maxkey = o; o = align_up(o + (size_t)rows * 4, 256);
  L.rowflag = o; o = align_up(o + (size_t)rows * 4, 256);
  L.diffflag = o; o = align_up(o + (size_t)rows * 4, 256);
  L.tickets = o; o = align_up(o + (size_t)rows * NTICKET * 4, 256);
  L.shist = L.fhist = L.flcnt = L.cntpart = o;
  if (single_pass) {
    L.flcnt = o; o = align_up(o + (size_t)rows * MAXC * 4, 256);
    L.cntpart = o; o = align_up(o + (size_t)rows * MAXC * 4, 256);
    L.fhist = o; o = align_up(o + (size_t)rows * MAXC * LB1 * 4, 256);
    L.shist = o; o = align_up(o + (size_t)rows * SBINS * 4, 256);
  }
  L.zero_end = o;
  L.flags = o; o = align_up(o + 64, 256);   // status words 0-3, word 8: completion count of the short-row kernel
  L.csdev = o; o = align_up(o + sizeof(CsetDev), 256);
  L.sel = o; o = align_up(o + (size_t)rows * sizeof(SelRow), 256);
  L.dec = o; o = align_up(o + (size_t)rows * sizeof(RowDec), 256);
  L.partial = o; o = align_up(o + (size_t)rows * MAX_BLK_PER_ROW * NSLOT * 8, 256);
  L.energy = o; o = align_up(o + (size_t)rows * NSLOT * 8, 256);
  L.tiecnt = o; o = align_up(o + (size_t)rows * (size_t)nchunk_of(d) * 4, 256);
  L.list_row = 0;
  L.list = L.lcount = L.lepart = L.lepart3 = L.fl = o;
  if (single_pass) {
    L.list_row = list_row_of(d);
    L.fl = o; o = align_up(o + (size_t)rows * MAXC * FINAL_CAP * 8, 256);
    L.list = o; o = align_up(o + (size_t)rows * (size_t)L.list_row * 8, 256);
    L.lcount = o; o = align_up(o + (size_t)rows * MAX_BLK_PER_ROW * 4, 256);
    L.lepart = o; o = align_up(o + (size_t)rows * LIST_BLK * MAXC * 8, 256);
    L.lepart3 = o; o = align_up(o + (size_t)rows * LIST_BLK * MAXC * 8, 256);
  }
  L.total = o;
  return L;
}

size_t scratch_bytes(int rows, long long d, bool single_pass) { return layout_of(rows, d, single_pass).total; }

void carve_scratch(Scratch* s, void* base, int rows, long long d, bool single_pass) {
  const Layout L = layout_of(rows, d, single_pass);
  char* b = (char*)base;
  s->hist1 = (u32*)(b + L.hist1);
  s->hist2 = (u32*)(b + L.hist2);
  s->hist3 = (u32*)(b + L.hist3);
  s->maxkey = (u32*)(b + L.maxkey);
  s->limbs = (u64*)(b + L.limbs);
  s->flags = (u32*)(b + L.flags);
  s->csdev = (CsetDev*)(b + L.csdev);
  s->zero_begin = b;
  s->zero_bytes = L.zero_end;
  s->zero_rare = L.zero_rare;
  s->sel = (SelRow*)(b + L.sel);
  s->dec = (RowDec*)(b + L.dec);
  s->partial = (double*)(b + L.partial);
  s->energy = (double*)(b + L.energy);
  s->tiecnt = (u32*)(b + L.tiecnt);
  s->rowflag = (u32*)(b + L.rowflag);
  s->diffflag = (u32*)(b + L.diffflag);
  s->tickets = (u32*)(b + L.tickets);
  s->shist = s->lhist1 = s->fhist = s->lcount = s->cntpart = nullptr;
  s->list = nullptr;
  s->lepart = nullptr;
  s->lepart3 = nullptr;
  s->fl = nullptr;
  s->flcnt = nullptr;
  s->list_row = L.list_row;
  if (single_pass) {
    s->shist = (u32*)(b + L.shist);
    s->lhist1 = (u32*)(b + L.lhist1);
    s->fhist = (u32*)(b + L.fhist);
    s->list = (u64*)(b + L.list);
    s->lcount = (u32*)(b + L.lcount);
    s->cntpart = (u32*)(b + L.cntpart);
    s->lepart = (double*)(b + L.lepart);
    s->lepart3 = (double*)(b + L.lepart3);
    s->fl = (u64*)(b + L.fl);
    s->flcnt = (u32*)(b + L.flcnt);
  }
  s->rows_cap = rows;
  s->d_cap = d;
  s->nchunk_cap = nchunk_of(d);
  s->prof = nullptr;
}

adacgd_status make_cset(const adacgd_cset* in, long long d, CsetDev* out, const char** msg) {
  CsetDev cs;
  memset(&cs, 0, sizeof(cs));
  if (!in || in->m == 0) { *out = cs; return ADACGD_OK; }
  if (in->m < 0 || in->m > MAXC || !in->cands) { *msg = "candidate count must be in [0, ADACGD_MAX_CANDS] with a non-null list"; return ADACGD_ERR_INVALID_ARG; }
  if (!(in->zeta >= 0.f) || !(in->zeta <= 3.0e38f)) { *msg = "zeta must be finite and >= 0"; return ADACGD_ERR_INVALID_ARG; }
  cs.m = in->m;
  cs.zeta = in->zeta;
  for (int j = 0; j < in->m; ++j) {
    cs.pkind[j] = ADACGD_PRED_LAZY;   // Eq. 10 at every level unless the caller names other triggers
    cs.pparam[j] = in->zeta;
    if (in->preds) {
      const adacgd_pred& q = in->preds[j];
      if (q.kind < ADACGD_PRED_LAZY || q.kind > ADACGD_PRED_ALWAYS) { *msg = "unknown trigger kind"; return ADACGD_ERR_INVALID_ARG; }
      const bool has_param = q.kind == ADACGD_PRED_LAZY || q.kind == ADACGD_PRED_ABSOLUTE || q.kind == ADACGD_PRED_RELATIVE;
      if (has_param && (!(q.param >= 0.f) || !(q.param <= 3.0e38f))) { *msg = "trigger parameter must be finite and >= 0"; return ADACGD_ERR_INVALID_ARG; }
      cs.pkind[j] = q.kind;
      cs.pparam[j] = has_param ? q.param : 0.f;
    }
  }
  long long lastK = 0, lastB = 0;
  for (int c = 0; c < in->m; ++c) {
    const adacgd_cand& a = in->cands[c];
    if (a.reserved != 0) { *msg = "candidate.reserved must be 0"; return ADACGD_ERR_INVALID_ARG; }
    cs.kind[c] = a.kind;
    cs.param[c] = a.param;
    if (a.kind == ADACGD_TOPK) {
      if (a.param < 1) { *msg = "Top-K needs K >= 1"; return ADACGD_ERR_INVALID_ARG; }
      if (a.param <= lastK) { *msg = "Top-K candidates must have strictly increasing K (strongest compression first)"; return ADACGD_ERR_BAD_ORDER; }
      if (lastK >= d) { *msg = "only the last Top-K candidate may have K >= d"; return ADACGD_ERR_BAD_ORDER; }
      lastK = a.param;
      if (a.param < d) cs.sel[cs.nsel++] = c;
    } else if (a.kind == ADACGD_QUANT) {
      if (a.param < 2 || a.param > 16) { *msg = "quantiser width must be in [2,16] bits"; return ADACGD_ERR_INVALID_ARG; }
      if (a.param <= lastB) { *msg = "quantiser candidates must have strictly increasing width"; return ADACGD_ERR_BAD_ORDER; }
      lastB = a.param;
      cs.qsel[cs.nquant++] = c;
    } else {
      *msg = "unknown candidate kind";
      return ADACGD_ERR_INVALID_ARG;
    }
  }
  *out = cs;
  return ADACGD_OK;
}

// Tables of up to MAXC candidates exceed the default 48 KB of dynamic shared memory.
constexpr int SIDE_SHM = MAXC * BINS2 * 4;   // the largest table any phase of k_side keeps in shared memory
static_assert(BINS2 >= BINS1 && BINS2 >= BINS3, "k_side sizes its shared memory by BINS2");

// Co-resident CTAs per SM of the cooperative kernel (the smaller of its two instantiations); 0 on failure.
int side_ctas_per_sm() {
  int a = 0, b = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, k_side<true>, TPB, SIDE_SHM) != cudaSuccess) return 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, k_side<false>, TPB, SIDE_SHM) != cudaSuccess) return 0;
  return a < b ? a : b;
}

void set_compress_kernel_attributes() {
  cudaFuncSetAttribute(k_hist<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, MAXC * BINS2 * 4);
  cudaFuncSetAttribute(k_hist<2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, MAXC * BINS2 * 4);
  cudaFuncSetAttribute(k_side<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SIDE_SHM);
  cudaFuncSetAttribute(k_side<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SIDE_SHM);
  cudaFuncSetAttribute(k_lcollect, cudaFuncAttributeMaxDynamicSharedMemorySize, MAXC * FINISH_WORDS * 4);
  cudaFuncSetAttribute(k_sample<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SBINS * 2);
  cudaFuncSetAttribute(k_sample<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SBINS * 2);
  cudaFuncSetAttribute(k_sample_row<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, RS_BINS * 4);
  cudaFuncSetAttribute(k_sample_row<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, RS_BINS * 4);
}

// One record per device ordinal, filled at the first use of that device by this process.
const DevProps* current_device() {
  constexpr int MAX_DEVICES = 64;
  static DevProps table[MAX_DEVICES];
  static bool known[MAX_DEVICES] = {false};
  static std::mutex mu;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  if (!known[dev]) {
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return nullptr;
    set_compress_kernel_attributes();
    set_small_kernel_attributes();
    if (cudaGetLastError() != cudaSuccess) return nullptr;
    table[dev].ordinal = dev;
    table[dev].sms = sms;
    table[dev].side_ctas = side_ctas_per_sm();
    if (table[dev].side_ctas < 1) return nullptr;
    known[dev] = true;
  }
  return &table[dev];
}

int launch_compress(const Scratch& s, const CsetDev& cs, const float* X, float* G, const float* Y, int rows,
                    long long d, const CompressOut& out, cudaStream_t stream) {
  int launches = 0;
  const DevProps* dp = current_device();
  if (!dp) return -1;
  const int SMS = dp->sms;
  const bool al = (d % 4 == 0) && aligned16(X) && aligned16(G) && aligned16(Y) &&
                  (!out.mean_out || aligned16(out.mean_out));
  const long long nchunk = nchunk_of(d);
  const dim3 ugrid((unsigned)(nchunk < SMS * 4 ? nchunk : SMS * 4));  // persistent: CTAs walk the column chunks
  Prof* pf = s.prof;
#define TIMED(id, ...)             \
  do {                             \
    prof_begin(pf, id, stream);    \
    __VA_ARGS__;                   \
    prof_end(pf, stream);          \
    ++launches;                    \
  } while (0)
#define TIMED_AL(id, kern, grid, shm, ...)                                               \
  TIMED(id, if (al) launch_k(kern<true>, grid, dim3(TPB), shm, stream, pdl, __VA_ARGS__);   \
            else launch_k(kern<false>, grid, dim3(TPB), shm, stream, pdl, __VA_ARGS__))
  const bool pdl = pf == nullptr;   // event records between kernels would break the pairing anyway

  if (cs.m == 0) {
    prof_begin(pf, KID_MEMSET, stream);
    if (out.kept_cnt) cudaMemsetAsync(out.kept_cnt, 0, (size_t)rows * 8, stream);
    prof_end(pf, stream);
    TIMED(KID_PICK, launch_k(k_copy_report, dim3((rows + 127) / 128), dim3(128), 0, stream, false, rows, d, 0, out));
    TIMED_AL(KID_UPDATE, k_update, ugrid, 0, X, G, rows, d, s.dec, s.tiecnt, nchunk, 1, out, (const u32*)nullptr);
    return cudaGetLastError() == cudaSuccess ? launches : -1;
  }
  // clear the per-call accumulators
  // Small problems live in L2 and are bound by launch latency: the plain three-pass select needs fewer
  // kernels there than sampling + streaming pass + list passes.
  const bool single = (s.list != nullptr) && cs.nsel > 0 && (long long)rows * d >= (1ll << 19);
  if (!single && d <= SMALL_DMAX) {
    // short rows: everything in one launch, one CTA per row, then the mean; the kernel keeps its tables in shared
    // memory and writes every record it reads, so nothing of the scratch has to be cleared
    if (out.kept_cnt) {
      prof_begin(pf, KID_MEMSET, stream);
      cudaMemsetAsync(out.kept_cnt, 0, (size_t)rows * 8, stream);
      prof_end(pf, stream);
    }
    const int n = launch_small_rows(s, cs, X, G, Y, rows, d, out, stream, pdl);
    return n < 0 ? -1 : launches + n;
  }
  prof_begin(pf, KID_MEMSET, stream);
  if (out.kept_cnt) cudaMemsetAsync(out.kept_cnt, 0, (size_t)rows * 8, stream);
  // every element sampled and many rows: one CTA per row samples into shared memory (no global sample histogram)
  const long long ngran_all = (d + SAMP_G - 1) / SAMP_G;
  const bool row_sampler = single && ngran_all / 8192 < 2 && rows >= 32;
  {
    // row flags, tickets, first-digit tables; the three-pass route also needs its histograms and limbs cleared, which
    // in the single-pass route only k_side uses, and clears for the rows that need them (160 KB per row)
    const size_t skip = single ? s.zero_rare : 0;
    if (!row_sampler)   // the per-row sampler clears its row's words itself
      cudaMemsetAsync((char*)s.zero_begin + skip, 0, s.zero_bytes - skip, stream);
  }
  prof_end(pf, stream);

  const long long ntile = (d + TPB * 4 - 1) / (TPB * 4);
  long long want = (SMS * 4 + rows - 1) / rows;   // one wave of the streaming pass: four resident CTAs per SM
  // a CTA takes at least eight tiles (spread over the row by the grid stride) where the row has them, so
  // that its share of the key list is sized for an average over the row rather than for one tile
  if (single && want > (ntile + 7) / 8) want = (ntile + 7) / 8;
  if (want > ntile) want = ntile;
  if (want > MAX_BLK_PER_ROW) want = MAX_BLK_PER_ROW;
  if (want < 1) want = 1;
  const int nblk = (int)want;
  const dim3 sgrid(nblk, rows);
  // in single-pass mode the full select only serves rows whose bracket failed, inside k_side, whose CTAs stand in
  // for this many CTAs per flagged row: as many as the kernel has, so that a single such row still gets the whole
  // machine (with 37 per row one 12.5e6-element row took 1.4 ms; rows that are not flagged cost one flag read each)
  long long want_full = single ? SMS * 2 : nblk;
  if (single && want_full > (ntile + 7) / 8) want_full = (ntile + 7) / 8;   // at least eight tiles per histogram flush
  if (want_full > ntile) want_full = ntile;
  if (want_full < 1) want_full = 1;
  if (want_full > MAX_BLK_PER_ROW) want_full = MAX_BLK_PER_ROW;
  const int nblk_full = (int)want_full;
  const dim3 fgrid(nblk_full, rows);
  const u32* only = single ? s.rowflag : nullptr;  // in single-pass mode the full select serves flagged rows only
  bool qinline = false;                            // the streaming pass evaluates the quantisers itself
  double tol = 4.0 * ((double)d + 16.0) * 1.1102230246251565e-16;  // binary64 sums of <= d exact terms

#define TIMED_HIST(id, PASS, shm, hist)                                                                          \
  TIMED(id, if (al) launch_k(k_hist<PASS, true>, fgrid, dim3(TPB), shm, stream, pdl, X, G, d, cs, s.sel, hist,    \
                             s.maxkey, only, s.tickets, s.flags);                                                  \
            else launch_k(k_hist<PASS, false>, fgrid, dim3(TPB), shm, stream, pdl, X, G, d, cs, s.sel, hist,      \
                          s.maxkey, only, s.tickets, s.flags))
#define P1_ARGS                                                                                               \
  X, G, Y, d, cs, s.sel, s.partial, s.cntpart, s.list, s.lcount, s.list_row, segcap, s.maxkey, s.rowflag,     \
      s.diffflag, s.flags, s.fhist, s.tickets
#define PASS1_CASE(N)                                                                                               \
  case N:                                                                                                           \
    if (qinline) {                                                                                                  \
      if (al) launch_k(k_pass1<N, true, 2>, sgrid, dim3(TPB), 0, stream, pdl, P1_ARGS);                             \
      else launch_k(k_pass1<N, false, 2>, sgrid, dim3(TPB), 0, stream, pdl, P1_ARGS);                               \
    } else if (al) {                                                                                                \
      if (cs.nquant) launch_k(k_pass1<N, true, 1>, sgrid, dim3(TPB), 0, stream, pdl, P1_ARGS);                      \
      else launch_k(k_pass1<N, true, 0>, sgrid, dim3(TPB), 0, stream, pdl, P1_ARGS);                                \
    } else {                                                                                                        \
      launch_k(k_pass1<N, false, 1>, sgrid, dim3(TPB), 0, stream, pdl, P1_ARGS);                                    \
    }                                                                                                               \
    break;

  if (single) {
    // 1. brackets for every Top-K threshold from a sample of the row (the last CTA of a row derives them)
    // windows of `win` granules, one granule sampled per window: at least 8192 granules (131072
    // elements) where the row has that many, at most every 64th granule
    const long long ngran = (d + SAMP_G - 1) / SAMP_G;
    long long win = ngran / 8192;
    if (win < 1) win = 1;
    if (win > 64) win = 64;
    const long long nwin = (ngran + win - 1) / win;
    long long sgx = (SMS + rows - 1) / rows;          // about one CTA per SM over all rows
    const long long per_cta = 49152 / SAMP_G;         // 16-bit per-CTA counters: fewer than 65536 elements each
    if (sgx < (nwin + per_cta - 1) / per_cta) sgx = (nwin + per_cta - 1) / per_cta;
    const long long quads = SAMP_TPB / 4;
    if (sgx > (nwin + quads - 1) / quads) sgx = (nwin + quads - 1) / quads;
    const dim3 samp_grid((unsigned)sgx, rows);
    // every element sampled and few quantisers: the sample yields the row maximum and the streaming pass the
    // quantisers' errors, so that no further pass over X and G is needed for them
    qinline = cs.nquant > 0 && cs.nquant <= P1_NQ && win == 1;
    u32* samp_max = qinline ? s.maxkey : nullptr;
    prof_begin(pf, KID_SAMPLE, stream);
    if (row_sampler) {
      if (al) launch_k(k_sample_row<true>, dim3(rows), dim3(SAMP_TPB), RS_BINS * 4, stream, pdl, X, G, d, cs, s.sel, s.tickets, s.maxkey, s.csdev, s.rowflag, s.diffflag, s.flcnt, s.cntpart, s.fhist);
      else launch_k(k_sample_row<false>, dim3(rows), dim3(SAMP_TPB), RS_BINS * 4, stream, pdl, X, G, d, cs, s.sel, s.tickets, s.maxkey, s.csdev, s.rowflag, s.diffflag, s.flcnt, s.cntpart, s.fhist);
    } else if (al) launch_k(k_sample<true>, samp_grid, dim3(SAMP_TPB), SBINS * 2, stream, pdl, X, G, d, nwin, win, s.shist, cs, s.sel, s.tickets, samp_max, s.csdev);
    else launch_k(k_sample<false>, samp_grid, dim3(SAMP_TPB), SBINS * 2, stream, pdl, X, G, d, nwin, win, s.shist, cs, s.sel, s.tickets, samp_max, s.csdev);
    prof_end(pf, stream);
    ++launches;
    // 2. the one pass over X, G, Y
    const u32 segcap = (u32)(s.list_row / nblk);
    prof_begin(pf, KID_PASS1, stream);
    switch (cs.nsel) {
      PASS1_CASE(1) PASS1_CASE(2) PASS1_CASE(3) PASS1_CASE(4)
      PASS1_CASE(5) PASS1_CASE(6) PASS1_CASE(7) PASS1_CASE(8)
    }
    prof_end(pf, stream);
    ++launches;
    // 3. exact selection among the listed keys by the digits of key - lo: two passes, each finished by its
    //    last CTA; the third only does work for brackets wider than 2^22 key values
    tol = 1.3 * (4.0 * FLUSH_TILES + 2.0) * 5.9604644775390625e-08;  // binary32 chains of 4*FLUSH_TILES terms
    long long lgx = (SMS * 4 + rows - 1) / rows;       // one wave of CTAs over all rows, each walking its share of the segments
    if (lgx > LIST_BLK) lgx = LIST_BLK;
    if (lgx > nblk) lgx = nblk;
    const dim3 lgrid((unsigned)lgx, rows);
    // the three-level list passes serve rows with a crowded threshold bin only; their work is the key lists
    // (about 1 % of a row), so a few CTAs per row do, and the usual launch that finds nothing to do stays short
    const dim3 lhgrid((unsigned)(lgx < 16 ? lgx : 16), rows);
    TIMED(KID_LCOLLECT, launch_k(k_lcollect, lgrid, dim3(TPB), (size_t)cs.nsel * FINISH_WORDS * 4, stream, pdl, cs, nblk, s.sel, s.list, s.lcount,
                                 s.list_row, segcap, s.lepart, s.rowflag, s.fl, s.flcnt, s.tickets,
                                 (cs.nquant == 0 || qinline) ? 1 : 0, d, nblk, s.partial, s.maxkey, s.dec, s.flags, out,
                                 s.diffflag, tol, (const CsetDev*)s.csdev));
    if (cs.nquant && !qinline) TIMED_AL(KID_QUANT_ERR, k_quant_err, sgrid, 0, X, G, d, cs, s.maxkey, s.partial);
    // everything that is only sometimes needed, in one cooperative launch: rows whose first-digit bin holds too many
    // keys (three digit levels of 11, 11 and 9 bits over the lists), rows whose bracket failed (the full select),
    // levels not chosen yet, exact sums, tie counts
    SideArgs sa;
    sa.X = X; sa.G = G; sa.Y = Y; sa.d = d; sa.rows = rows; sa.nseg = nblk;
    sa.lh_gx = (int)(lgx < 16 ? lgx : 16);          // the lists are about 1 % of a row: a few CTAs per row do
    sa.f_gx = nblk_full;
    long long tgx = SMS * 2;                       // per row that needs the tie order, like the fallback grid
    if (tgx > nchunk) tgx = nchunk;
    sa.t_gx = (int)tgx;
    sa.nblk_main = nblk; sa.cs_global = (const CsetDev*)s.csdev; sa.sel = s.sel; sa.list = s.list; sa.lcount = s.lcount;
    sa.list_row = s.list_row; sa.segcap = segcap; sa.lhist1 = s.lhist1; sa.hist1 = s.hist1; sa.hist2 = s.hist2; sa.hist3 = s.hist3;
    sa.lepart = s.lepart; sa.lepart3 = s.lepart3; sa.partial = s.partial; sa.rowflag = s.rowflag; sa.flcnt = s.flcnt;
    sa.tickets = s.tickets; sa.maxkey = s.maxkey; sa.flags = s.flags; sa.diffflag = s.diffflag; sa.tiecnt = s.tiecnt;
    sa.cntpart = s.cntpart; sa.fl = s.fl; sa.limbs = s.limbs; sa.dec = s.dec; sa.nchunk = nchunk; sa.out = out; sa.tol = tol;
    int per_sm = dp->side_ctas < 4 ? dp->side_ctas : 4;
    TIMED(KID_SIDE, if (al) launch_cooperative(k_side<true>, dim3((unsigned)(per_sm * SMS)), dim3(TPB), SIDE_SHM, stream, sa);
                    else launch_cooperative(k_side<false>, dim3((unsigned)(per_sm * SMS)), dim3(TPB), SIDE_SHM, stream, sa));
  } else {
  // the full radix select: every row, or (single-pass mode) only rows whose bracket failed
  if (cs.nsel || cs.nquant) TIMED_HIST(KID_HIST1, 1, BINS1 * 4, s.hist1);
  if (cs.nsel) {
    TIMED_HIST(KID_HIST2, 2, cs.nsel * BINS2 * 4, s.hist2);
    TIMED_HIST(KID_HIST3, 3, cs.nsel * BINS3 * 4, s.hist3);
  }
  TIMED_AL(KID_ENERGY, k_energy, fgrid, 0, X, G, Y, d, cs, s.sel, s.partial, only, s.diffflag);
  if (cs.nquant) TIMED_AL(KID_QUANT_ERR, k_quant_err, sgrid, 0, X, G, d, cs, s.maxkey, s.partial);
  TIMED(KID_PICK, launch_k(k_pick, dim3(rows), dim3(TPB), 0, stream, pdl, cs, d, nblk, nblk_full, only, s.partial, s.sel, s.maxkey,
                           s.dec, s.flags, out, s.diffflag, (const u32*)nullptr, tol));
  TIMED_AL(KID_EXACT, k_exact_sums, fgrid, 0, X, G, Y, d, cs, s.sel, s.maxkey, s.dec, s.limbs, s.diffflag, d, out, s.tickets, s.flags);
  if (cs.nsel) {
    long long tgx = (SMS * 4 + rows - 1) / rows;
    if (tgx > nchunk) tgx = nchunk;
    TIMED_AL(KID_TIE, k_tiecount, dim3((unsigned)tgx, rows), 0, X, G, d, s.dec, s.tiecnt, nchunk, s.tickets);
  }
  }
  {
    // Not a programmatic dependent: launched as one, this persistent grid ran 400 us instead of 270 us on
    // 8 x 25e6 (its CTAs become resident while earlier kernels still hold part of the SMs).
    const bool pdl = false;
    // many rows of few chunks: first the kernel with one column per thread, which does the work unless a row needs
    // the general path (word 14 of the first row's ticket block, cleared with the rest, says whether it did)
    const u32* skip = nullptr;
    if (rows >= 16 && nchunk < 2 * SMS && out.kept_idx == nullptr) {
      u32* done = s.tickets + 14;
      TIMED(KID_UPDATE, launch_k(k_update_narrow, dim3((unsigned)((d + TPB - 1) / TPB)), dim3(TPB), 0, stream, false, X, G, rows, d,
                                 (const RowDec*)s.dec, out, done));
      skip = done;
    }
    if (skip) {
      // the fallback of the kernel above: as its programmatic dependent it is resident by the time that one ends, reads
      // the word and returns
      const bool pdl = pf == nullptr;
      TIMED_AL(KID_UPDATE, k_update, ugrid, 0, X, G, rows, d, s.dec, s.tiecnt, nchunk, 0, out, skip);
    } else {
      TIMED_AL(KID_UPDATE, k_update, ugrid, 0, X, G, rows, d, s.dec, s.tiecnt, nchunk, 0, out, skip);
    }
  }
#undef PASS1_CASE
#undef P1_ARGS
#undef TIMED_HIST
#undef TIMED_AL
#undef TIMED
  return cudaGetLastError() == cudaSuccess ? launches : -1;
}

// --------------------------------------------------------------------------
// small vector kernels of the loop
// --------------------------------------------------------------------------
__global__ void k_mean_rows(const float* __restrict__ G, int rows, long long d, float* __restrict__ out) {
  pdl_begin();
  const long long c = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= d) return;
  float acc = G[c];
  for (int i = 1; i < rows; ++i) acc = __fadd_rn(acc, G[(long long)i * d + c]);
  out[c] = __fdiv_rn(acc, (float)rows);
}
int launch_mean_rows(const float* G, int rows, long long d, float* out, cudaStream_t stream) {
  k_mean_rows<<<(unsigned)((d + 255) / 256), 256, 0, stream>>>(G, rows, d, out);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace adacgd
