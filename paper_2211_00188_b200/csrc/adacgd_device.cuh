// Device helpers shared by the translation units of the compression stage: small warp and CTA
// primitives, the quantiser, the level choice (Eq. 11) and the exact integer sums.  Every function is
// inline: each translation unit compiles its own copy.
#pragma once

#include "adacgd_internal.cuh"

namespace adacgd {

// --------------------------------------------------------------------------
// small helpers
// --------------------------------------------------------------------------
// Programmatic dependent launch: lets the next kernel of the stream be scheduled while this one
// runs, then waits until every kernel before this one has completed and its writes are visible.
// Called first thing by every kernel, before any access to global memory.
__device__ __forceinline__ void pdl_begin() {
  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

// The two halves on their own.  A kernel whose successor is large waits first and lets the successor in only
// afterwards (or not at all): CTAs that become resident early hold registers and shared memory while they wait.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;"); }

// Number of SMs of the device the kernel runs on.
__device__ __forceinline__ int sm_count() {
  u32 n;
  asm("mov.u32 %0, %%nsmid;" : "=r"(n));
  return (int)n;
}

// Copies a candidate set member by member with compile-time indices.  A kernel that indexes its by-value
// CsetDev parameter with run-time values (or hands its address to a function) makes every thread copy the whole
// structure to local memory; kernels that need such indexing let one thread copy the parameter to shared memory
// with this function and work on that copy.
__device__ __forceinline__ void cs_copy_static(CsetDev& dst, const CsetDev& src) {
  dst.m = src.m; dst.zeta = src.zeta; dst.nsel = src.nsel; dst.nquant = src.nquant;
#pragma unroll
  for (int k = 0; k < MAXC; ++k) {
    dst.kind[k] = src.kind[k]; dst.param[k] = src.param[k]; dst.sel[k] = src.sel[k]; dst.qsel[k] = src.qsel[k];
    dst.pkind[k] = src.pkind[k]; dst.pparam[k] = src.pparam[k];
  }
}

__device__ __forceinline__ u32 key_of(float v) { return __float_as_uint(v) & 0x7fffffffu; }

template <bool ALIGNED>
__device__ __forceinline__ void load4(const float* __restrict__ row, long long c0, long long d, float (&o)[4]) {
  if (ALIGNED) {
    float4 t = *reinterpret_cast<const float4*>(row + c0);
    o[0] = t.x; o[1] = t.y; o[2] = t.z; o[3] = t.w;
  } else {
#pragma unroll
    for (int k = 0; k < 4; ++k) o[k] = (c0 + k < d) ? row[c0 + k] : 0.f;
  }
}

template <bool ALIGNED>
__device__ __forceinline__ void store4(float* __restrict__ row, long long c0, long long d, const float (&o)[4]) {
  if (ALIGNED) {
    *reinterpret_cast<float4*>(row + c0) = make_float4(o[0], o[1], o[2], o[3]);
  } else {
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (c0 + k < d) row[c0 + k] = o[k];
  }
}

__device__ __forceinline__ u32 warp_sum_u32(u32 v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Exclusive prefix sum of one u32 per thread over the CTA (NT threads); also returns the total.
template <int NT = TPB>
__device__ __forceinline__ u32 block_excl_scan(u32 v, u32* total) {
  __shared__ u32 wsum[NT / 32];
  __shared__ u32 wtot;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  u32 inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    u32 t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  __syncthreads();  // protects wsum against the previous call
  if (lane == 31) wsum[wid] = inc;
  __syncthreads();
  if (wid == 0) {
    u32 w = (lane < NT / 32) ? wsum[lane] : 0;
    u32 winc = w;
#pragma unroll
    for (int o = 1; o < NT / 32; o <<= 1) {
      u32 t = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += t;
    }
    if (lane < NT / 32) wsum[lane] = winc - w;
    if (lane == NT / 32 - 1) wtot = winc;
  }
  __syncthreads();
  if (total) *total = wtot;
  return wsum[wid] + inc - v;
}

// Finds, in a histogram of nb bins ordered by key, the bin that holds the krem-th
// largest key: out[0] = bin, out[1] = number of keys in higher bins.  All TPB threads call.
inline __device__ void block_find_kth_desc(const u32* __restrict__ hist, int nb, u32 krem, u32* out) {
  const int per = nb / TPB;  // 8 or 2
  u32 loc[8];
  u32 sum = 0;
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    loc[k] = (k < per) ? __ldcg(&hist[nb - 1 - (threadIdx.x * per + k)]) : 0;
    sum += loc[k];
  }
  u32 excl = block_excl_scan(sum, nullptr);
  if (krem > excl && krem <= excl + sum) {
    u32 run = excl;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      if (k < per) {
        if (krem <= run + loc[k]) {
          out[0] = nb - 1 - (threadIdx.x * per + k);
          out[1] = run;
          break;
        }
        run += loc[k];
      }
    }
  }
  __syncthreads();
}

// True in exactly one CTA of the row: the one that finishes last.  Every CTA calls it after its
// global writes; the caller may then read what the other CTAs of the row wrote.  No waiting.
__device__ __forceinline__ bool last_cta_of_row(u32* ticket, u32 n_ctas) {
  __shared__ u32 is_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) is_last = (atomicAdd(ticket, 1u) == n_ctas - 1u) ? 1u : 0u;
  __syncthreads();
  if (is_last) __threadfence();
  return is_last != 0;
}


__device__ __forceinline__ float quant_value(float v, float L, float inv, float step) {
  const float code = fminf(L, rintf(__fmul_rn(fabsf(v), inv)));
  return copysignf(__fmul_rn(code, step), v);
}

// --------------------------------------------------------------------------
// level choice (Eq. 11)
// --------------------------------------------------------------------------
// Bits of the message of a level (the paper counts communication but prints no formula; this is the
// library's reading): skip 0; Top-K with K < d: K values of 32 bits with an index of ceil(log2 d) bits
// each; K >= d: d values; a b-bit quantiser: the 32-bit scale and b bits per entry.  Host and device.
inline __host__ __device__ uint64_t level_bits(const CsetDev& cs, int level, long long d) {
  if (level == 0) return 0;
  const int c = level - 1;
  if (cs.kind[c] == ADACGD_TOPK) {
    if (cs.param[c] >= d) return 32ull * (uint64_t)d;
    int idx_bits = 0;
    while (idx_bits < 63 && (1ll << idx_bits) < d) ++idx_bits;   // ceil(log2 d)
    if (idx_bits < 1) idx_bits = 1;
    return (uint64_t)cs.param[c] * (uint64_t)(32 + idx_bits);
  }
  return 32ull + (uint64_t)cs.param[c] * (uint64_t)d;
}

// Fills the decision record of a row once its level is known.
inline __device__ void finalize_row(const CsetDev& cs, int row, int level, long long d, const SelRow* sel,
                             const u32* maxkey, RowDec* dec, const CompressOut& out, const double* e,
                             double D) {
  RowDec r;
  r.level = level; r.mode = 0; r.T = 0; r.q = 0; r.need_tie = 0; r.need_exact = 0;
  r.qL = r.qinv = r.qstep = 0.f; r.cut = 0xffffffffu;
  if (level > 0) {
    const int c = level - 1;
    if (cs.kind[c] == ADACGD_TOPK) {
      if (cs.param[c] >= d) {
        r.mode = 2;
      } else {
        int j = 0;
        for (int t = 0; t < cs.nsel; ++t) if (cs.sel[t] == c) j = t;
        r.mode = 1; r.T = sel[row].T[j]; r.q = sel[row].q[j];
        r.need_tie = (sel[row].tiemode[j] == 2u) ? 1 : 0;
        r.cut = (sel[row].tiemode[j] == 1u) ? sel[row].cut[j] : 0xffffffffu;
      }
    } else {
      r.mode = 3;
      const float s = __uint_as_float(maxkey[row]);
      r.qL = (float)((1 << ((int)cs.param[c] - 1)) - 1);
      if (s > 0.f) { r.qinv = __fdiv_rn(r.qL, s); r.qstep = __fdiv_rn(s, r.qL); }
    }
  }
  dec[row] = r;
  if (out.level) out.level[row] = level;
  if (out.bits) out.bits[row] = level_bits(cs, level, d);
  if (out.D) out.D[row] = D;
  if (out.err)
    for (int j = 0; j <= cs.m; ++j) out.err[(long long)row * (cs.m + 1) + j] = e[j];
}

// Chooses the level of one row from its sums (Eq. 10 and 11); run by a whole CTA of NT threads.
// The per-CTA partial sums of the streaming pass are added in a fixed order: thread t takes
// blocks t, t + NT, ..., then lanes, then warps.  D, ||v||^2 and the Top-K slots hold nblk partial
// sums per row, the quantiser slots nblk_q (their pass may run on another grid).
template <int NT = TPB>
inline __device__ void pick_row(const CsetDev& cs, long long d, int row, int nblk, int nblk_q, const double* __restrict__ partial,
                         const SelRow* __restrict__ sel, const u32* __restrict__ maxkey,
                         RowDec* __restrict__ dec, u32* __restrict__ flags, const CompressOut& out,
                         const u32* __restrict__ diffflag, double tol) {
  __shared__ double ps[NSLOT][NT / 32];
  __shared__ double p_extra[MAXC];
  __shared__ u32 p_T[MAXC], p_ntie[MAXC], p_q[MAXC], p_max, p_diff;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const int nslot = 2 + cs.m;
  // what the deciding thread needs from the selection records is fetched by several threads at once
  if (threadIdx.x < cs.nsel) {
    const int j = threadIdx.x;
    p_T[j] = __ldcg(&sel[row].T[j]); p_ntie[j] = __ldcg(&sel[row].ntie[j]);
    p_q[j] = __ldcg(&sel[row].q[j]); p_extra[j] = __ldcg(&sel[row].extraE[j]);
  }
  if (threadIdx.x == 32) { p_max = __ldcg(&maxkey[row]); p_diff = __ldcg(&diffflag[row]); }
  double a[NSLOT];
#pragma unroll
  for (int s = 0; s < NSLOT; ++s) a[s] = 0.0;
  const double* p = partial + (long long)row * MAX_BLK_PER_ROW * NSLOT;
  u32 qmask = 0;   // slots written by the quantiser pass
  for (int j = 0; j < cs.nquant; ++j) qmask |= 1u << (2 + cs.qsel[j]);
  const int nblk_max = nblk > nblk_q ? nblk : nblk_q;
  for (int b = threadIdx.x; b < nblk_max; b += NT) {
#pragma unroll
    for (int s = 0; s < NSLOT; ++s)
      if (s < nslot && b < (((qmask >> s) & 1u) ? nblk_q : nblk)) a[s] += __ldcg(&p[(long long)b * NSLOT + s]);
  }
#pragma unroll
  for (int s = 0; s < NSLOT; ++s) {
    const double v = warp_sum_f64(a[s]);
    if (lane == 0) ps[s][wid] = v;
  }
  __syncthreads();
  if (threadIdx.x != 0) return;
  double sum[NSLOT];
#pragma unroll
  for (int s = 0; s < NSLOT; ++s) {
    double t = 0.0;
    for (int w = 0; w < NT / 32; ++w) t += ps[s][w];
    sum[s] = t;
  }
  const double D = sum[0];
  double e[MAXC + 1];
  e[0] = sum[1];
  for (int c = 0; c < cs.m; ++c) {
    if (cs.kind[c] == ADACGD_TOPK) {
      if (cs.param[c] >= d) { e[c + 1] = 0.0; continue; }
      int j = 0;
      for (int t = 0; t < cs.nsel; ++t) if (cs.sel[t] == c) j = t;
      const double tv = (double)__uint_as_float(p_T[j]);
      e[c + 1] = (sum[2 + c] + p_extra[j]) + (double)(p_ntie[j] - p_q[j]) * (tv * tv);
    } else {
      e[c + 1] = sum[2 + c];
    }
  }
  const u32 diff = p_diff;
  if (p_max >= 0x7f800000u || (diff & 0x80000000u)) {  // Inf/NaN in X - G or X - Y: estimator kept
    atomicOr(&flags[0], 1u);
    finalize_row(cs, row, 0, d, sel, maxkey, dec, out, e, D);
    return;
  }
  // `tol` bounds the relative error of every sum above (non-negative terms).  A sum is only
  // trusted inside [2^-90, inf): below, binary32 squares may have underflowed; above, a chain
  // overflowed (or X - Y is not finite, which the exact pass tells).
  const double tiny = 8.0e-28;
  const bool d_ok = (D >= tiny && D <= 1.7e308);
  const bool e0_ok = (e[0] >= tiny && e[0] <= 1.7e308);
  int level = cs.m;
  bool unsure = false;
  for (int j = 0; j < cs.m; ++j) {   // levels 0 .. m-1 carry a trigger (Eq. 9); level m is the "otherwise"
    const double E = e[j];
    const int kind = cs.pkind[j];
    const double par = (double)cs.pparam[j];
    const bool by_def = (j > 0 && cs.kind[j - 1] == ADACGD_TOPK && cs.param[j - 1] >= d);  // identity: error 0
    const bool e_ok = (E >= tiny && E <= 1.7e308);
    int verdict;  // 1 true, 0 false, -1 unsure
    if (kind == ADACGD_PRED_NEVER) verdict = 0;
    else if (kind == ADACGD_PRED_ALWAYS) verdict = 1;
    else if (by_def) verdict = 1;                     // 0 <= any right side
    else if (!(D <= 1.7e308)) verdict = -1;           // overflowed chain or non-finite X - Y: the exact pass tells which
    else if (kind == ADACGD_PRED_LAZY && j == 0 && (diff & 0x7fffffffu) == 0 && d_ok)
      verdict = (par >= 1.0) ? 1 : 0;                 // |X-G| == |X-Y| entry by entry, so ||v||^2 == D > 0 exactly
    else if (kind == ADACGD_PRED_RELATIVE && j == 0 && e0_ok)
      verdict = (par >= 1.0) ? 1 : 0;                 // ||v||^2 against itself
    else if (!e_ok) verdict = -1;
    else if (par == 0.0) verdict = 0;                 // E > 0 for certain, right side is 0
    else {
      double rhs, rtol;
      bool r_ok;
      if (kind == ADACGD_PRED_LAZY) { rhs = par * D; rtol = tol; r_ok = d_ok; }
      else if (kind == ADACGD_PRED_RELATIVE) { rhs = par * e[0]; rtol = tol; r_ok = e0_ok; }
      else { rhs = par; rtol = 0.0; r_ok = true; }    // absolute tolerance: the right side is exact
      if (!r_ok) verdict = -1;
      else if (E * (1.0 + tol) < rhs * (1.0 - rtol)) verdict = 1;
      else if (E * (1.0 - tol) > rhs * (1.0 + rtol)) verdict = 0;
      else verdict = -1;
    }
    if (verdict == 1) { level = j; break; }
    if (verdict < 0) { unsure = true; break; }
  }
  if (unsure) {
    RowDec r;
    r.level = -1; r.mode = 0; r.T = 0; r.q = 0; r.need_tie = 0; r.need_exact = 1;
    r.qL = r.qinv = r.qstep = 0.f; r.cut = 0xffffffffu;
    dec[row] = r;
    atomicAdd(&flags[1], 1u);
    return;
  }
  finalize_row(cs, row, level, d, sel, maxkey, dec, out, e, D);
}


// --------------------------------------------------------------------------
// exact re-evaluation of a row whose comparison could not be certified
// --------------------------------------------------------------------------
// A square of a binary32 value is mant^2 * 2^(2*eff-2) units of 2^-298; it is added as
// three 32-bit pieces into 64-bit limbs (radix 2^32, carries resolved at the end).
__device__ __forceinline__ void sq_pieces(float w, int* k, u32 (&p)[3]) {
  const u32 b = key_of(w);
  const u32 ex = b >> 23, fr = b & 0x7fffffu;
  const u64 m = ex ? (u64)(fr | 0x800000u) : (u64)fr;
  const int off = 2 * (int)(ex ? ex : 1u) - 2;
  const unsigned __int128 t = (unsigned __int128)(m * m) << (off & 31);
  *k = off >> 5;
  p[0] = (u32)t; p[1] = (u32)(t >> 32); p[2] = (u32)(t >> 64);
}
__device__ __forceinline__ void limb_add(u64* limbs, int k, const u32 (&p)[3]) {
  if (p[0]) atomicAdd(&limbs[k], (u64)p[0]);
  if (p[1]) atomicAdd(&limbs[k + 1], (u64)p[1]);
  if (p[2]) atomicAdd(&limbs[k + 2], (u64)p[2]);
}

// Normalised radix-2^32 digits -> nearest binary64 (ties to even); value = digits * 2^-298.
inline __device__ double digits_to_double(const u32* dig) {
  int t = NLIMB - 1;
  while (t >= 0 && dig[t] == 0) --t;
  if (t < 0) return 0.0;
  const u32 hi = dig[t], mid = (t >= 1) ? dig[t - 1] : 0u, lo = (t >= 2) ? dig[t - 2] : 0u;
  bool sticky = false;
  for (int i = 0; i < t - 2; ++i) sticky |= (dig[i] != 0);
  const unsigned __int128 W = ((unsigned __int128)hi << 64) | ((unsigned __int128)mid << 32) | lo;
  const int nb = 32 - __clz(hi);         // significant bits of hi
  const int sh = nb + 11;                // keep 53 of the 64+nb bits
  u64 mant = (u64)(W >> sh);
  const bool rnd = (W >> (sh - 1)) & 1;
  sticky |= (W & (((unsigned __int128)1 << (sh - 1)) - 1)) != 0;
  if (rnd && (sticky || (mant & 1))) ++mant;
  return ldexp((double)mant, sh + 32 * (t - 2) - 298);
}

// The exact value of energy slot s of a row (0: D, 1: ||v||^2, 2 + c: candidate c): carries resolved, the
// dropped threshold-equal keys of a Top-K candidate added, rounded once to binary64.
template <bool SHARED_LIMBS = false>
inline __device__ double exact_slot_value(const CsetDev& cs, int row, long long d, const u64* row_limbs,
                                          const SelRow* __restrict__ sel, int s) {
  if (s >= 2 && cs.kind[s - 2] == ADACGD_TOPK && cs.param[s - 2] >= d) return 0.0;   // identity: no error
  u32 dig[NLIMB];
  const u64* l = row_limbs + s * NLIMB;
  unsigned __int128 tie = 0;
  int tk = 0;
  if (s >= 2 && cs.kind[s - 2] == ADACGD_TOPK) {
    int j = 0;
    for (int t = 0; t < cs.nsel; ++t) if (cs.sel[t] == s - 2) j = t;
    const u32 T = sel[row].T[j];
    const u32 ex = T >> 23, fr = T & 0x7fffffu;
    const u64 m = ex ? (u64)(fr | 0x800000u) : (u64)fr;
    const int off = 2 * (int)(ex ? ex : 1u) - 2;
    tie = ((unsigned __int128)(m * m) * (u64)(sel[row].ntie[j] - sel[row].q[j])) << (off & 31);
    tk = off >> 5;
  }
  u64 carry = 0;
  for (int k = 0; k < NLIMB; ++k) {
    u64 add = 0;
    if (k >= tk && k < tk + 4) add = (u64)(u32)(tie >> (32 * (k - tk)));
    const unsigned __int128 tsum = (unsigned __int128)(SHARED_LIMBS ? l[k] : __ldcg(&l[k])) + carry + add;
    dig[k] = (u32)tsum;
    carry = (u64)(tsum >> 32);
  }
  return digits_to_double(dig);
}

// The decision of a row from its exact sums val[0 .. 1 + m] (Eq. 10 and 11 with no rounding left to doubt).
inline __device__ void decide_exact_row(const CsetDev& cs, int row, long long d, const double* val,
                                        const SelRow* __restrict__ sel, const u32* __restrict__ maxkey,
                                        RowDec* __restrict__ dec, const CompressOut& out,
                                        const u32* __restrict__ diffflag, u32* __restrict__ flags) {
  if (__ldcg(&diffflag[row]) & 0x80000000u) {  // X - Y is not finite
    double zero[NSLOT];
    for (int s = 0; s < NSLOT; ++s) zero[s] = 0.0;
    atomicOr(&flags[0], 1u);
    finalize_row(cs, row, 0, d, sel, maxkey, dec, out, zero + 1, 0.0);
    return;
  }
  const double D = val[0];
  int level = cs.m;
  for (int j = 0; j < cs.m; ++j) {
    const double par = (double)cs.pparam[j];
    bool holds;
    switch (cs.pkind[j]) {
      case ADACGD_PRED_LAZY: holds = val[1 + j] <= par * D; break;            // Eq. 10
      case ADACGD_PRED_RELATIVE: holds = val[1 + j] <= par * val[1]; break;
      case ADACGD_PRED_ABSOLUTE: holds = val[1 + j] <= par; break;
      case ADACGD_PRED_ALWAYS: holds = true; break;
      default: holds = false; break;
    }
    if (holds) { level = j; break; }
  }
  finalize_row(cs, row, level, d, sel, maxkey, dec, out, val + 1, D);
}

// Run by one thread of the last CTA of the exact pass: carries, rounds and decides the row.
// `row_limbs`: the row's NSLOT x NLIMB accumulators in global memory.
inline __device__ void pick_exact_row(const CsetDev& cs, int row, long long d, const u64* row_limbs,
                               const SelRow* __restrict__ sel, const u32* __restrict__ maxkey,
                               RowDec* __restrict__ dec, const CompressOut& out,
                               const u32* __restrict__ diffflag, u32* __restrict__ flags) {
  double val[NSLOT];
  for (int s = 0; s < NSLOT; ++s) val[s] = (s < 2 + cs.m) ? exact_slot_value<false>(cs, row, d, row_limbs, sel, s) : 0.0;
  decide_exact_row(cs, row, d, val, sel, maxkey, dec, out, diffflag, flags);
}

// --------------------------------------------------------------------------
// host-side launch helpers
// --------------------------------------------------------------------------
inline bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

// Launches a kernel, optionally as a programmatic dependent of the kernel before it on the stream:
// its CTAs may be scheduled before that kernel has finished and wait in pdl_begin().
template <typename... KArgs, typename... Args>
inline void launch_k(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t shm, cudaStream_t stream, bool pdl,
                     Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = shm; cfg.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at; cfg.numAttrs = pdl ? 1 : 0;
  cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

// Launches a kernel whose CTAs synchronise across the grid: the launch fails unless all of them can be resident
// at once, so the grid is sized from the occupancy the runtime reports.
template <typename... KArgs, typename... Args>
inline void launch_cooperative(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t shm, cudaStream_t stream,
                               Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = shm; cfg.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeCooperative;
  at[0].val.cooperative = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

}  // namespace adacgd
