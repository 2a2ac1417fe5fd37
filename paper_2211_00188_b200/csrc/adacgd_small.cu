// Stages a2-a4 for short rows in one launch (one CTA per row) and the mean over the rows.
#include "adacgd_device.cuh"

namespace adacgd {

// --------------------------------------------------------------------------
// short rows: stages a2-a4 and the mean in one launch
// --------------------------------------------------------------------------
// One CTA per row, the row's difference vector v = X - G kept in shared memory: three radix passes
// (11 + 11 + 9 bits, all Top-K candidates at once), tail energies and quantiser errors in binary64,
// the index cut of threshold-equal keys, the level choice (pick_row, with the exact integer sums
// when a comparison cannot be certified) and the update of the row; the mean over the rows follows in
// k_small_mean.  Serves problems too small to keep the multi-kernel path busy.
// Finds, in a shared-memory histogram of nb bins (a multiple of 32) ordered by key, the bin that holds
// the krem-th largest key; one warp calls, every lane gets (bin, number of keys in higher bins).
__device__ __forceinline__ void warp_find_kth_desc(const u32* hist, int nb, u32 krem, u32* bin, u32* above) {
  const int lane = threadIdx.x & 31;
  const int per = nb / 32;                              // this lane: descending positions per*lane .. per*lane + per - 1
  u32 sum = 0;
  for (int k = 0; k < per; ++k) sum += hist[nb - 1 - (per * lane + k)];
  u32 inc = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const u32 t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  const u32 excl = inc - sum;
  const bool mine = krem > excl && krem <= excl + sum;   // true in exactly one lane when 1 <= krem <= total
  u32 fb = 0, fa = 0;
  if (mine) {
    u32 run = excl;
    for (int k = 0; k < per; ++k) {
      const u32 v = hist[nb - 1 - (per * lane + k)];
      if (krem <= run + v) { fb = (u32)(nb - 1 - (per * lane + k)); fa = run; break; }
      run += v;
    }
  }
  const u32 who = __ballot_sync(0xffffffffu, mine);
  const int src = who ? (__ffs(who) - 1) : 0;
  *bin = __shfl_sync(0xffffffffu, fb, src);
  *above = __shfl_sync(0xffffffffu, fa, src);
}

constexpr int SMALL_LIST = 4096;
#ifndef SMALL_NT_LONG_N
#define SMALL_NT_LONG_N 512
#endif
#ifndef SMALL_LONG_ROW_N
#define SMALL_LONG_ROW_N 512
#endif
constexpr int SMALL_NT_LONG = SMALL_NT_LONG_N;   // threads per CTA for rows of at least SMALL_LONG_ROW elements
constexpr int SMALL_LONG_ROW = SMALL_LONG_ROW_N;
// NT threads per CTA: 256, or 512 for rows of at least SMALL_LONG_ROW elements (c2, 20 rows of 8000: 113 -> 94 us for the
// two calls of an iteration; 1024 threads leave 64 registers per thread and measured 98 us).
template <bool ALIGNED, int NT>
__global__ void __launch_bounds__(NT) k_small_rows(const float* __restrict__ X, float* G, const float* __restrict__ Y,
                                                    int rows, long long d, CsetDev cs_param, SelRow* sel, RowDec* dec,
                                                    double* partial, u32* maxkey, u32* diffflag, u32* flags,
                                                    CompressOut out, double tol, u32* mean_ticket) {
  // mean_ticket != nullptr: the rows are so short that the CTA that finishes last also takes the mean over them
  // (summed in row order, one division), instead of a kernel of its own
  pdl_begin();
  __shared__ CsetDev cs;   // the kernel indexes the set with run-time values: a shared copy instead of a local one per thread
  if (threadIdx.x == 0) cs_copy_static(cs, cs_param);
  __syncthreads();
  extern __shared__ __align__(16) unsigned char small_smem[];
  const int dn = (int)d;
  float* vs = reinterpret_cast<float*>(small_smem);                       // [d rounded up to 4]
  u32* tab = reinterpret_cast<u32*>(small_smem) + ((dn + 3) / 4) * 4;     // max(BINS1, nsel * BINS2) words
  u32* cl = tab + (cs.nsel > 1 ? cs.nsel : 1) * BINS2;                           // SMALL_LIST keys sharing a first digit with a threshold
  __shared__ double redd[NSLOT][NT / 32];
  __shared__ u32 redu[3][NT / 32];
  __shared__ u32 s_b1[MAXC], s_ab1[MAXC], s_p2[MAXC], s_ab2[MAXC], s_T[MAXC], s_above[MAXC], s_ntie[MAXC], s_q[MAXC], s_cut[MAXC];
  __shared__ u64 lsh[NSLOT * NLIMB];
  __shared__ u32 s_ncl;
  const int row = blockIdx.x;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const int nsel = cs.nsel;
  const float* xr = X + (long long)row * d;
  float* gr = G + (long long)row * d;
  const float* yr = Y + (long long)row * d;

  // ---- v into shared memory; D, ||v||^2, row maximum, |X-G| against |X-Y|
  double aD = 0.0, aE = 0.0;
  u32 mx = 0, mxw = 0, dfl = 0;
  constexpr int SB = 4;   // tiles of NT * 4 columns requested at once: the row is short, its latency is what counts
  for (int base = threadIdx.x * 4; base < dn; base += SB * NT * 4) {
    float x[SB][4], g[SB][4], y[SB][4];
#pragma unroll
    for (int u = 0; u < SB; ++u) {
      const int c0 = base + u * NT * 4;
      if (c0 < dn) {
        load4<ALIGNED>(xr, c0, d, x[u]);
        load4<ALIGNED>(gr, c0, d, g[u]);
        load4<ALIGNED>(yr, c0, d, y[u]);
      }
    }
#pragma unroll
    for (int u = 0; u < SB; ++u) {
      const int c0 = base + u * NT * 4;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (c0 + k >= dn) break;
        const float v = __fsub_rn(x[u][k], g[u][k]);
        const float w = __fsub_rn(x[u][k], y[u][k]);
        vs[c0 + k] = v;
        const double dv = (double)v, dw = (double)w;
        aD = __dadd_rn(aD, __dmul_rn(dw, dw));
        aE = __dadd_rn(aE, __dmul_rn(dv, dv));
        mx = max(mx, key_of(v));
        mxw = max(mxw, key_of(w));
        dfl |= __float_as_uint(v) ^ __float_as_uint(w);
      }
    }
  }
  aD = warp_sum_f64(aD); aE = warp_sum_f64(aE);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    mxw = max(mxw, __shfl_xor_sync(0xffffffffu, mxw, o));
    dfl |= __shfl_xor_sync(0xffffffffu, dfl, o);
  }
  if (lane == 0) { redd[0][wid] = aD; redd[1][wid] = aE; redu[0][wid] = mx; redu[1][wid] = mxw; redu[2][wid] = dfl; }
  __syncthreads();
  mx = 0; mxw = 0; dfl = 0;
  for (int w = 0; w < NT / 32; ++w) { mx = max(mx, redu[0][w]); mxw = max(mxw, redu[1][w]); dfl |= redu[2][w]; }
  const float smax = __uint_as_float(mx);

  // ---- radix select, all candidates at once
  if (nsel) {
    for (int i = threadIdx.x; i < BINS1; i += NT) tab[i] = 0;
    __syncthreads();
#pragma unroll 4
    for (int i = threadIdx.x; i < dn; i += NT) atomicAdd(&tab[key_of(vs[i]) >> 20], 1u);
    __syncthreads();
    if (wid < nsel) {   // one warp per candidate
      u32 bin, above;
      warp_find_kth_desc(tab, BINS1, (u32)cs.param[cs.sel[wid]], &bin, &above);
      if (lane == 0) { s_b1[wid] = bin; s_ab1[wid] = above; }
    }
    __syncthreads();
    // The keys that share a first digit with some threshold (usually a few per cent of the row) are
    // compacted once, with warp votes; the second and third digit are then histogrammed from that list.
    // A list that does not fit sends the two passes over the whole row instead.
    for (int i = threadIdx.x; i < nsel * BINS2; i += NT) tab[i] = 0;
    if (threadIdx.x == 0) s_ncl = 0;
    __syncthreads();
    for (int i0 = 0; i0 < dn; i0 += NT) {
      const int i = i0 + threadIdx.x;
      const u32 key = (i < dn) ? key_of(vs[i]) : 0xffffffffu;
      bool hit = false;
      for (int j = 0; j < nsel; ++j) hit = hit || ((key >> 20) == s_b1[j]);
      const u32 m = __ballot_sync(0xffffffffu, hit);
      if (m) {
        u32 base = 0;
        if (lane == 0) base = atomicAdd(&s_ncl, (u32)__popc(m));
        base = __shfl_sync(0xffffffffu, base, 0);
        const u32 pos = base + (u32)__popc(m & ((1u << lane) - 1u));
        if (hit && pos < (u32)SMALL_LIST) cl[pos] = key;
      }
    }
    __syncthreads();
    const u32 ncl = s_ncl;
    const bool listed = ncl <= (u32)SMALL_LIST;
    const int nscan = listed ? (int)ncl : dn;
    for (int i = threadIdx.x; i < nscan; i += NT) {
      const u32 key = listed ? cl[i] : key_of(vs[i]);
      for (int j = 0; j < nsel; ++j)
        if ((key >> 20) == s_b1[j]) atomicAdd(&tab[j * BINS2 + ((key >> 9) & 0x7ffu)], 1u);
    }
    __syncthreads();
    if (wid < nsel) {
      u32 bin, above;
      warp_find_kth_desc(tab + wid * BINS2, BINS2, (u32)cs.param[cs.sel[wid]] - s_ab1[wid], &bin, &above);
      if (lane == 0) { s_p2[wid] = (s_b1[wid] << 11) | bin; s_ab2[wid] = s_ab1[wid] + above; }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < nsel * BINS3; i += NT) tab[i] = 0;
    __syncthreads();
    for (int i = threadIdx.x; i < nscan; i += NT) {
      const u32 key = listed ? cl[i] : key_of(vs[i]);
      for (int j = 0; j < nsel; ++j)
        if ((key >> 9) == s_p2[j]) atomicAdd(&tab[j * BINS3 + (key & 0x1ffu)], 1u);
    }
    __syncthreads();
    if (wid < nsel) {
      const int j = wid;
      const u32 K = (u32)cs.param[cs.sel[j]];
      u32 bin, above;
      warp_find_kth_desc(tab + j * BINS3, BINS3, K - s_ab2[j], &bin, &above);
      if (lane == 0) {
        s_T[j] = (s_p2[j] << 9) | bin;
        s_above[j] = s_ab2[j] + above;
        s_ntie[j] = tab[j * BINS3 + bin];
        s_q[j] = K - s_above[j];
        s_cut[j] = 0xffffffffu;
      }
    }
    __syncthreads();
    // of the keys equal to a threshold the q with the lowest indices are kept: index of the q-th
    for (int j = 0; j < nsel; ++j) {
      if (s_q[j] >= s_ntie[j]) continue;
      const u32 T = s_T[j], q = s_q[j];
      const int per = (dn + NT - 1) / NT;
      const int i0 = threadIdx.x * per, i1 = (i0 + per < dn) ? i0 + per : dn;
      u32 cnt = 0;
      for (int i = i0; i < i1; ++i) cnt += (key_of(vs[i]) == T) ? 1u : 0u;
      const u32 ex = block_excl_scan<NT>(cnt, nullptr);
      if (ex < q && q <= ex + cnt) {
        u32 seen = ex;
        for (int i = i0; i < i1; ++i)
          if (key_of(vs[i]) == T && ++seen == q) { s_cut[j] = (u32)i; break; }
      }
      __syncthreads();
    }
  }

  // ---- tail energies of the Top-K candidates, errors of the quantisers (binary64, exact terms)
  double aB[MAXC], aQ[MAXC];
  float qL[MAXC], qinv[MAXC], qstep[MAXC];
#pragma unroll
  for (int j = 0; j < MAXC; ++j) {
    aB[j] = 0.0; aQ[j] = 0.0; qL[j] = qinv[j] = qstep[j] = 0.f;
    if (j < cs.nquant) {
      qL[j] = (float)((1 << ((int)cs.param[cs.qsel[j]] - 1)) - 1);
      if (smax > 0.f) { qinv[j] = __fdiv_rn(qL[j], smax); qstep[j] = __fdiv_rn(smax, qL[j]); }
    }
  }
#pragma unroll 2
  for (int i = threadIdx.x; i < dn; i += NT) {
    const float v = vs[i];
    const u32 key = key_of(v);
    const double dv = (double)v;
    const double sq = __dmul_rn(dv, dv);
#pragma unroll
    for (int j = 0; j < MAXC; ++j) {
      if (j < nsel && key < s_T[j]) aB[j] = __dadd_rn(aB[j], sq);
      if (j < cs.nquant) {
        const double r = (double)__fsub_rn(v, quant_value(v, qL[j], qinv[j], qstep[j]));
        aQ[j] = __dadd_rn(aQ[j], __dmul_rn(r, r));
      }
    }
  }
#pragma unroll
  for (int j = 0; j < MAXC; ++j) {
    if (j < nsel) { const double t = warp_sum_f64(aB[j]); if (lane == 0) redd[2 + cs.sel[j]][wid] = t; }
    if (j < cs.nquant) { const double t = warp_sum_f64(aQ[j]); if (lane == 0) redd[2 + cs.qsel[j]][wid] = t; }
  }
  __syncthreads();
  // ---- the row's records, in the form the level choice reads them
  if (threadIdx.x < NSLOT) {
    const int sl = threadIdx.x;
    bool used = (sl < 2);
    for (int j = 0; j < nsel; ++j) used |= (sl == 2 + cs.sel[j]);
    for (int j = 0; j < cs.nquant; ++j) used |= (sl == 2 + cs.qsel[j]);
    double acc = 0.0;
    if (used)
      for (int w = 0; w < NT / 32; ++w) acc += redd[sl][w];
    partial[(long long)row * MAX_BLK_PER_ROW * NSLOT + sl] = acc;
  }
  if (threadIdx.x >= 32 && threadIdx.x < 32 + nsel) {
    const int j = threadIdx.x - 32;
    SelRow* sr = sel + row;
    sr->T[j] = s_T[j]; sr->above[j] = s_above[j]; sr->ntie[j] = s_ntie[j]; sr->q[j] = s_q[j];
    sr->extraE[j] = 0.0; sr->tiemode[j] = (s_q[j] < s_ntie[j]) ? 1u : 0u; sr->cut[j] = s_cut[j];
  }
  if (threadIdx.x == 64) {
    maxkey[row] = mx;
    diffflag[row] = ((mxw >= 0x7f800000u) ? 0x80000000u : 0u) | (dfl & 0x7fffffffu);
  }
  __syncthreads();
  pick_row<NT>(cs, d, row, 1, 1, partial, sel, maxkey, dec, flags, out, diffflag, tol);
  __syncthreads();
  if (__ldcg(&dec[row].need_exact)) {
    // the comparison could not be certified: exact integer sums of the row, then the decision from them
    for (int i = threadIdx.x; i < NSLOT * NLIMB; i += NT) lsh[i] = 0;
    __syncthreads();
    // A square is mant^2 * 2^off units of 2^-298.  Squares whose offset lies within 64 bits below the
    // largest one of the row are added in per-thread 128-bit integers anchored at bit `wb` (at most 128
    // terms of at most 113 bits each); the few that lie lower go straight to the shared limbs.
    const u32 kmax = max(mx, mxw);
    const int off_max = 2 * (int)((kmax >> 23) ? (kmax >> 23) : 1u) - 2;
    const int wb = off_max > 64 ? off_max - 64 : 0;
    unsigned __int128 accD = 0, accE = 0, accC[MAXC];
#pragma unroll
    for (int c = 0; c < MAXC; ++c) accC[c] = 0;
    // square of a finite value as a 128-bit integer anchored at bit wb; false if it lies below the window
    auto sq_term = [&](float val, unsigned __int128* term) -> bool {
      const u32 bkey = key_of(val);
      const u32 ex = bkey >> 23, fr = bkey & 0x7fffffu;
      const u64 m = ex ? (u64)(fr | 0x800000u) : (u64)fr;
      const int off = 2 * (int)(ex ? ex : 1u) - 2;
      *term = (off >= wb) ? (unsigned __int128)(m * m) << (off - wb) : (unsigned __int128)0;
      return off >= wb || m == 0;
    };
    auto slow_add = [&](int slot, float val) {   // rare: more than 2^32 times smaller than the row's largest entry
      int kk; u32 p[3];
      sq_pieces(val, &kk, p);
      limb_add(lsh + slot * NLIMB, kk, p);
    };
    // D needs X - Y again: four loads of each in flight per thread
    for (int base = threadIdx.x; base < dn; base += 4 * NT) {
      float xw[4], yw[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = base + u * NT;
        xw[u] = (i < dn) ? xr[i] : 0.f;
        yw[u] = (i < dn) ? yr[i] : 0.f;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (base + u * NT >= dn) break;
        const float w = __fsub_rn(xw[u], yw[u]);
        if (key_of(w) >= 0x7f800000u) { atomicOr(&diffflag[row], 0x80000000u); continue; }
        unsigned __int128 tw;
        if (sq_term(w, &tw)) accD += tw; else slow_add(0, w);
      }
    }
    for (int i = threadIdx.x; i < dn; i += NT) {
      const float v = vs[i];
      if (key_of(v) >= 0x7f800000u) { atomicOr(&diffflag[row], 0x80000000u); continue; }
      unsigned __int128 tv;
      const bool v_in = sq_term(v, &tv);
      if (v_in) accE += tv; else slow_add(1, v);
      const u32 key = key_of(v);
#pragma unroll
      for (int j = 0; j < MAXC; ++j)
        if (j < nsel && key < s_T[j] && v_in) accC[j] += tv;
      if (!v_in)
        for (int j = 0; j < nsel; ++j)
          if (key < s_T[j]) slow_add(2 + cs.sel[j], v);
      for (int j = 0; j < cs.nquant; ++j) {
        const float r = __fsub_rn(v, quant_value(v, qL[j], qinv[j], qstep[j]));
        unsigned __int128 tr;
        if (sq_term(r, &tr)) {
#pragma unroll
          for (int c = 0; c < MAXC; ++c)
            if (c == MAXC - 1 - j) accC[c] += tr;
        } else slow_add(2 + cs.qsel[j], r);
      }
    }
    // The per-thread integers are added up as four 32-bit pieces each: over the warp with shuffles, over the
    // warps through `wacc` (64-bit shared atomics are compare-and-swap loops: with every thread of the CTA on
    // the same few words they would take hundreds of microseconds), and only the totals go into the limbs.
    __shared__ u64 wacc[NT / 32][NSLOT][4];
    auto stash = [&](unsigned __int128 acc, int slot) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        u64 piece = (u64)(u32)(acc >> (32 * i));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) piece += __shfl_xor_sync(0xffffffffu, piece, o);
        if (lane == 0) wacc[wid][slot][i] = piece;
      }
    };
    for (int i = threadIdx.x; i < (NT / 32) * NSLOT * 4; i += NT) (&wacc[0][0][0])[i] = 0;
    __syncthreads();
    stash(accD, 0);
    stash(accE, 1);
#pragma unroll
    for (int j = 0; j < MAXC; ++j) {
      if (j < nsel) stash(accC[j], 2 + cs.sel[j]);
      if (j < cs.nquant) stash(accC[MAXC - 1 - j], 2 + cs.qsel[j]);
    }
    __syncthreads();
    if (threadIdx.x < NSLOT * 4) {
      const int slot = threadIdx.x >> 2, i = threadIdx.x & 3;
      u64 tot = 0;                                     // < 2^32 * 256 threads = 2^40
      for (int w = 0; w < NT / 32; ++w) tot += wacc[w][slot][i];
      const int k0 = (wb >> 5) + i, sh = wb & 31;
      const u64 lo = (tot & 0xffffffffull) << sh, hi = (tot >> 32) << sh;      // weights 2^(32 k0) and 2^(32 (k0 + 1))
      if (lo & 0xffffffffull) atomicAdd(&lsh[slot * NLIMB + k0], lo & 0xffffffffull);
      if ((lo >> 32) + (hi & 0xffffffffull)) atomicAdd(&lsh[slot * NLIMB + k0 + 1], (lo >> 32) + (hi & 0xffffffffull));
      if (hi >> 32) atomicAdd(&lsh[slot * NLIMB + k0 + 2], hi >> 32);
    }
    __syncthreads();
    // one thread per energy slot resolves its carries and rounds; one thread decides
    __shared__ double xval[NSLOT];
    if (threadIdx.x < NSLOT)
      xval[threadIdx.x] = (threadIdx.x < 2 + cs.m) ? exact_slot_value<true>(cs, row, d, lsh, sel, threadIdx.x) : 0.0;
    __syncthreads();
    if (threadIdx.x == 0) decide_exact_row(cs, row, d, xval, sel, maxkey, dec, out, diffflag, flags);
    __syncthreads();
  }

  // ---- the update of the row (Eq. 7 at the chosen level)
  const int mode = __ldcg(&dec[row].mode);
  if (mode != 0) {
    const u32 T = __ldcg(&dec[row].T), cut = __ldcg(&dec[row].cut);
    const float L = __ldcg(&dec[row].qL), inv = __ldcg(&dec[row].qinv), step = __ldcg(&dec[row].qstep);
    for (int base = threadIdx.x * 4; base < dn; base += SB * NT * 4) {
      float gq[SB][4];
#pragma unroll
      for (int u = 0; u < SB; ++u)
        if (base + u * NT * 4 < dn) load4<ALIGNED>(gr, base + u * NT * 4, d, gq[u]);
#pragma unroll
      for (int u = 0; u < SB; ++u) {
        const int c0 = base + u * NT * 4;
        if (c0 >= dn) break;
        bool any = false;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          if (c0 + k >= dn) break;
          const float v = vs[c0 + k];
          const u32 key = key_of(v);
          bool kept = true;
          float add = v;
          if (mode == 1) kept = (key > T) || (key == T && (u32)(c0 + k) <= cut);
          else if (mode == 3) add = quant_value(v, L, inv, step);
          if (kept) {
            gq[u][k] = __fadd_rn(gq[u][k], add);
            any = true;
            if (out.kept_idx && mode != 3) {
              const long long pos = (long long)atomicAdd((u64*)&out.kept_cnt[row], 1ull);
              if (pos < out.kept_stride) out.kept_idx[(long long)row * out.kept_stride + pos] = c0 + k;
            }
          }
        }
        if (any) store4<ALIGNED>(gr, c0, d, gq[u]);
      }
    }
  }
  if (mean_ticket == nullptr) return;
  __shared__ u32 mean_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    mean_last = (atomicAdd(mean_ticket, 1u) == gridDim.x - 1u) ? 1u : 0u;
    if (mean_last) *mean_ticket = 0u;   // ready for the next call
  }
  __syncthreads();
  if (!mean_last) return;
  __threadfence();
  const float nf = (float)rows;
  for (int c = threadIdx.x; c < dn; c += NT) {
    float acc = -0.f;                    // -0 + g == g bit for bit
    for (int i = 0; i < rows; ++i) acc = __fadd_rn(acc, __ldcg(G + (long long)i * d + c));
    out.mean_out[c] = __fdiv_rn(acc, nf);
  }
}

// The mean over short rows (summed in row order, one division): a thread owns four columns and
// requests eight rows at once.
template <bool ALIGNED>
__global__ void __launch_bounds__(TPB) k_small_mean(const float* G, int rows, long long d, float* __restrict__ mean_out) {
  pdl_begin();
  const int dn = (int)d;
  const int c0 = (blockIdx.x * TPB + threadIdx.x) * 4;
  if (c0 >= dn) return;
  const float nf = (float)rows;
  float acc[4] = {-0.f, -0.f, -0.f, -0.f};
  for (int i0 = 0; i0 < rows; i0 += 8) {
    float g[8][4];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = i0 + u;
#pragma unroll
      for (int k = 0; k < 4; ++k) g[u][k] = 0.f;
      if (i < rows) {
        const float* src = G + (long long)i * d + c0;
        if (ALIGNED) {
          const float4 t = __ldcg(reinterpret_cast<const float4*>(src));
          g[u][0] = t.x; g[u][1] = t.y; g[u][2] = t.z; g[u][3] = t.w;
        } else {
#pragma unroll
          for (int k = 0; k < 4; ++k)
            if (c0 + k < dn) g[u][k] = __ldcg(src + k);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      if (i0 + u >= rows) break;
#pragma unroll
      for (int k = 0; k < 4; ++k) acc[k] = __fadd_rn(acc[k], g[u][k]);
    }
  }
#pragma unroll
  for (int k = 0; k < 4; ++k)
    if (c0 + k < dn) mean_out[c0 + k] = __fdiv_rn(acc[k], nf);
}


// The row and the tables of up to MAXC candidates exceed the default 48 KB of dynamic shared memory.
void set_small_kernel_attributes() {
  const int bytes = 4 * (SMALL_DMAX + MAXC * BINS2 + SMALL_LIST);
  cudaFuncSetAttribute(k_small_rows<true, TPB>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  cudaFuncSetAttribute(k_small_rows<false, TPB>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  cudaFuncSetAttribute(k_small_rows<true, SMALL_NT_LONG>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  cudaFuncSetAttribute(k_small_rows<false, SMALL_NT_LONG>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}

// Enqueues k_small_rows and, if a mean is wanted, k_small_mean; returns the number of launches (< 0: CUDA error).
int launch_small_rows(const Scratch& s, const CsetDev& cs, const float* X, float* G, const float* Y, int rows,
                      long long d, const CompressOut& out, cudaStream_t stream, bool pdl) {
  if (!current_device()) return -1;   // also sets the shared-memory limits at the first use of a device
  Prof* pf = s.prof;
  int launches = 0;
  const size_t shm = 4 * ((size_t)((d + 3) / 4) * 4 + (size_t)(cs.nsel > 1 ? cs.nsel : 1) * BINS2 + SMALL_LIST);
  const double tol64 = 4.0 * ((double)d + 16.0) * 1.1102230246251565e-16;  // binary64 sums of <= d exact terms
  const bool al4 = (d % 4 == 0) && aligned16(X) && aligned16(G) && aligned16(Y);
  prof_begin(pf, KID_SMALL, stream);
  // a few thousand entries in all: the last CTA takes the mean as well (the ticket lives in the status words'
  // block, word 8, zero between calls)
  const bool tiny_mean = out.mean_out != nullptr && (long long)rows * d <= 16384;
  u32* mean_ticket = tiny_mean ? s.flags + 8 : nullptr;
#define SMALL_LAUNCH(AL, NT)                                                                                          \
  launch_k(k_small_rows<AL, NT>, dim3(rows), dim3(NT), shm, stream, pdl, X, G, Y, rows, d, cs, s.sel, s.dec, s.partial, \
           s.maxkey, s.diffflag, s.flags, out, tol64, mean_ticket)
  if (d >= SMALL_LONG_ROW) { if (al4) SMALL_LAUNCH(true, SMALL_NT_LONG); else SMALL_LAUNCH(false, SMALL_NT_LONG); }
  else { if (al4) SMALL_LAUNCH(true, TPB); else SMALL_LAUNCH(false, TPB); }
#undef SMALL_LAUNCH
  prof_end(pf, stream);
  ++launches;
  if (out.mean_out && !tiny_mean) {
    const dim3 mgrid((unsigned)((d + TPB * 4 - 1) / (TPB * 4)));
    prof_begin(pf, KID_SMALL, stream);
    if (al4 && aligned16(out.mean_out)) launch_k(k_small_mean<true>, mgrid, dim3(TPB), 0, stream, pdl, (const float*)G, rows, d, out.mean_out);
    else launch_k(k_small_mean<false>, mgrid, dim3(TPB), 0, stream, pdl, (const float*)G, rows, d, out.mean_out);
    prof_end(pf, stream);
    ++launches;
  }
  return cudaGetLastError() == cudaSuccess ? launches : -1;
}

}  // namespace adacgd
