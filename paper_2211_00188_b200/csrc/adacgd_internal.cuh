// Internal declarations shared by the translation units of libadacgd.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "adacgd.h"

namespace adacgd {

typedef uint16_t u16;
typedef uint32_t u32;
typedef unsigned long long u64;

constexpr int TPB = 256;            // threads per CTA of the streaming kernels
constexpr int MAXC = ADACGD_MAX_CANDS;
constexpr int NSLOT = 2 + MAXC;     // energy slots: D, ||v||^2, then one per candidate
constexpr int NLIMB = 20;           // 32-bit digits of the exact accumulator (covers 2^-298 .. 2^342)
constexpr int BINS1 = 2048;         // key bits [30:20]
constexpr int BINS2 = 2048;         // key bits [19:9]
constexpr int BINS3 = 512;          // key bits [8:0]
constexpr int UPD_COLS = TPB * 4;   // columns per CTA of the update kernel (also the tie-order chunk)
constexpr int MAX_BLK_PER_ROW = 2048;
constexpr int SBINS = 65536;        // sample histogram: key bits [30:15]
constexpr int LIST_BLK = 256;       // CTAs per row of the passes over the candidate lists
constexpr int NTICKET = 16;         // per-row words: completion counters 0 sample, 1-3 list levels, 4-6 full passes, 7 exact, 8 ties,
                                    // 11 streaming pass, 12 collection pass; flags 9 = level already picked, 10 = a third list
                                    // level is needed, 13 = the row takes the three-level list passes
constexpr int LB1 = 256;            // bins of the first digit of key - lo histogrammed by the streaming pass
constexpr int FINAL_CAP = 2048;     // entries kept per bracket for ranking threshold-equal keys by index
constexpr int FLUSH_TILES = 16;     // binary32 chains are folded into binary64 every 16 tiles (64 terms)

// Optional per-kernel timing with CUDA events on the launching stream.
enum KernelId {
  KID_MEMSET = 0, KID_HIST1, KID_HIST2, KID_HIST3, KID_SCAN, KID_ENERGY, KID_QUANT_ERR, KID_PICK,
  KID_EXACT, KID_TIE, KID_UPDATE, KID_GRAD_FWD, KID_GRAD_BWD, KID_GRAD_REDUCE, KID_LOSS, KID_AXPY,
  KID_LOG, KID_SAMPLE, KID_BRACKET, KID_PASS1, KID_LHIST, KID_LCOLLECT, KID_SMALL, KID_CSR_FWD, KID_CSC_BWD, KID_CSR_RES, KID_DELTA, KID_INC, KID_INC_FINISH, KID_SIDE,
  KID_COUNT
};
struct Prof {
  int cap, used;
  cudaEvent_t* beg;
  cudaEvent_t* end;
  int* id;
};
inline void prof_begin(Prof* p, int id, cudaStream_t s) {
  if (p && p->used < p->cap) { p->id[p->used] = id; cudaEventRecord(p->beg[p->used], s); }
}
inline void prof_end(Prof* p, cudaStream_t s) {
  if (p && p->used < p->cap) { cudaEventRecord(p->end[p->used], s); ++p->used; }
}

// What the launch code needs to know about the current device.  The first call on a device also raises
// the dynamic shared memory limit of the kernels that need more than the default (the limit is a
// per-device attribute).  Returns nullptr when there is no usable current device.
struct DevProps {
  int ordinal;
  int sms;       // streaming multiprocessors: grids are sized in multiples of it
  int side_ctas; // CTAs of the cooperative side-path kernel that fit on one SM
};
const DevProps* current_device();
void set_compress_kernel_attributes();   // adacgd_compress.cu
void set_small_kernel_attributes();      // adacgd_small.cu

// Candidate set as the kernels see it (passed by value).
struct CsetDev {
  int m;                 // candidates
  float zeta;
  int pkind[MAXC];       // trigger of level j = 0 .. m-1 (level 0 = skip): ADACGD_PRED_*
  float pparam[MAXC];    // its parameter
  int kind[MAXC];
  long long param[MAXC]; // K or bits
  int nsel;              // Top-K candidates with K < d: they need a threshold
  int sel[MAXC];         // their candidate indices, K ascending
  int nquant;
  int qsel[MAXC];
};

// Result of the selection for one row: per selecting candidate (index in CsetDev::sel)
struct SelRow {
  u32 b1[MAXC], above1[MAXC];   // pass 1: bin of key[30:20], #keys in higher bins
  u32 p2[MAXC], above2[MAXC];   // pass 2: key[30:9] prefix, #keys with a higher prefix
  u32 T[MAXC];                  // threshold key: the K-th largest |v| bit pattern
  u32 above[MAXC];              // #keys  > T
  u32 ntie[MAXC];               // #keys == T
  u32 q[MAXC];                  // how many of the ties are kept (lowest indices first)
  // single-pass path: bracket [lo, hi) of key values that must contain T, from a sample
  u32 lo[MAXC], hi[MAXC];
  u32 above_hi[MAXC];           // #keys >= hi
  double extraE[MAXC];          // energy of listed keys in [lo, T)
  // which of the keys equal to T are kept: 0 all of them, 1 those with index <= cut, 2 the q lowest
  // indices as ranked by the chunk-prefix pass (k_tiecount / k_tiescan)
  u32 tiemode[MAXC], cut[MAXC];
  u32 sh1[MAXC], sh2[MAXC];     // digit shifts of key - lo inside the bracket
  // first digit (8 bits) of key - lo as histogrammed by the streaming pass: bin holding the K-th
  // largest key, #keys above that bin, #keys inside it
  u32 fb1[MAXC], fabove1[MAXC], fc1[MAXC];
};

// Decision for one row, consumed by the update kernel.
struct RowDec {
  int level;       // 0 = skip, j = j-th candidate
  int mode;        // 0 none, 1 Top-K with threshold, 2 identity (K >= d), 3 quantiser
  u32 T, q;
  int need_tie;    // q < ntie: ties must be ranked by index
  int need_exact;  // the fast comparison could not be certified
  float qL, qinv, qstep;
  u32 cut;         // threshold-equal keys are kept up to this index (need_tie == 0)
};

struct Scratch {
  // carved from the caller's workspace by carve_scratch(); all device pointers
  u32* hist1;      // [rows][BINS1]
  u32* hist2;      // [rows][MAXC][BINS2]
  u32* hist3;      // [rows][MAXC][BINS3]
  u32* maxkey;     // [rows]
  u64* limbs;      // [rows][NSLOT][NLIMB] exact accumulators
  u32* flags;      // [4]: 0 nonfinite seen, 1 #exact rechecks
  CsetDev* csdev;  // the call's candidate set, for code that indexes it with run-time values
  void* zero_begin; size_t zero_bytes;  // region cleared at the start of every call
  size_t zero_rare;                     // its first part: tables that in the single-pass route only k_side uses (and clears)
  SelRow* sel;     // [rows]
  RowDec* dec;     // [rows]
  double* partial; // [rows][MAX_BLK_PER_ROW][NSLOT]
  double* energy;  // [rows][NSLOT]
  u32* tiecnt;     // [rows][nchunk]  (exclusive prefix after the scan)
  // single-pass path (null when the scratch was carved without it)
  u32* shist;      // [rows][SBINS] sample histogram
  u32* lhist1;     // [rows][MAXC][BINS1] first digit of the listed keys, per bracket (three-level passes)
  u32* fhist;      // [rows][MAXC][LB1] first digit as histogrammed by the streaming pass
  u64* list;       // [rows][list_row] (key << 32 | index), one segment of segcap entries per CTA
  u32* lcount;     // [rows][MAX_BLK_PER_ROW] entries per segment
  u32* cntpart;    // [rows][MAXC] keys >= hi of each bracket, added up by the CTAs of the streaming pass
  double* lepart;  // [rows][LIST_BLK][MAXC] per-CTA energies of listed keys below the chosen first digit
  double* lepart3; // same, below the chosen second digit
  u64* fl;         // [rows][MAXC][FINAL_CAP] listed keys sharing the threshold's 22-bit prefix
  u32* flcnt;      // [rows][MAXC]
  u32* tickets;    // [rows][NTICKET]
  u32* rowflag;    // [rows] 1: the row must take the full radix select (bracket missed or list overflow)
  u32* diffflag;   // [rows] nonzero: some |X-G| differs from |X-Y|
  long long list_row;
  int rows_cap; long long d_cap; long long nchunk_cap;
  Prof* prof;      // host pointer, may be null
};

size_t scratch_bytes(int rows, long long d, bool single_pass);
void carve_scratch(Scratch* s, void* base, int rows, long long d, bool single_pass);

// Validates and converts a host candidate set. Returns ADACGD_OK / error and a message.
adacgd_status make_cset(const adacgd_cset* in, long long d, CsetDev* out, const char** msg);

struct CompressOut {
  float* mean_out; int32_t* level; uint64_t* bits; double* err; double* D;
  int32_t* kept_idx; long long kept_stride; long long* kept_cnt;
};

// Enqueues stages a2-a4 (+ mean) on `stream`; returns the number of kernels launched (<0: CUDA error).
int launch_compress(const Scratch& s, const CsetDev& cs, const float* X, float* G, const float* Y,
                    int rows, long long d, const CompressOut& out, cudaStream_t stream);

// Short rows (d <= SMALL_DMAX): stages a2-a4 in one launch, one CTA per row, then the mean.
constexpr int SMALL_DMAX = 32768;
int launch_small_rows(const Scratch& s, const CsetDev& cs, const float* X, float* G, const float* Y, int rows,
                      long long d, const CompressOut& out, cudaStream_t stream, bool pdl);

// ---- gradient stage (a1) ----
struct GradScratch {
  float* r;         // [n][m_rows] residuals scaled by 1/m
  float* part;      // [split][n][d] partial column sums (split > 1 only)
  double* losspart; // [n][loss_blocks] loss of the sample rows of every CTA of the forward kernel
  double* regpart;  // [n][loss_blocks] regulariser of every CTA's share of x
  double* loss;     // [1]
  u32* loss_ticket; // [1 + n] completion counts of the forward kernel: grid rows done, then CTAs done per grid row (reset by the last)
  u32* bwd_tickets; // [n][column tiles] completion counts of the backward kernel's row slices
  size_t ticket_bytes;
  int split; int loss_blocks;
  // CSR layout: transposed copy built at init (column-major over all workers: column c of worker i
  // is "row" i*d + c)
  long long* csc_ptr;   // [n*d + 1]
  int* csc_row;         // [nnz] sample row inside the worker
  u16* csc_row16;       // the same in 16 bits (span kernel: at most 8192 samples per worker)
  u16* csr_col16;       // blocked forward kernel: column index inside its column block, regrouped like fwd_val
  float* fwd_val;       // values regrouped block-major, every (block, row) span padded to a multiple of four
  float* csc_val;       // [nnz]
  // column-blocked forward: the entries of sample row g whose column lies in block b are the groups of four
  // [csr_split[b*rows + g], csr_split[b*rows + g + 1]) of fwd_val / csr_col16; zpart[b*rows + g] is that block's
  // share of a_g . x
  int nb, blk;          // column blocks and columns per block (nb = 0: plain warp-per-row kernel)
  long long* csr_split; // [nb * n*m_rows + 1]
  float* zpart;         // [nb][n*m_rows]
  // span backward: column pointers relative to the worker's first entry
  int ccols;            // 1: contiguous spans per warp; 0: one thread per column on csc_ptr
  long long* wbase;     // [n+1] first transposed entry of every worker
  u32* ptr32;           // [n][d+1]
  // incremental forward (dense layout, ADACGD_FLAG_INCREMENTAL_FORWARD): z_i = A_i x and u_i = A_i g are kept
  // between iterations and moved along by the entries of g that changed
  int inc;              // 1: the buffers below exist
  float* AT;            // [n][d][m_rows] column-major copy of the features
  float* z;             // [n][m_rows]  A_i x
  float* u;             // [n][m_rows]  A_i g_prev
  float* g_prev;        // [d] the g that u belongs to
  u32* dl_count;        // [inc_chunks] changed entries of g per chunk of INC_CHUNK columns
  int* dl_idx;          // [inc_chunks][INC_CHUNK] their columns, ascending
  float* dl_val;        // [inc_chunks][INC_CHUNK] g - g_prev there
  float* ipart;         // [n][inc_chunks][m_rows] a chunk's contribution to u_i
  u64* inc_cols;        // [1] columns gathered by incremental passes since init
  u32* dl_flag;         // [2] route of the iteration (1: gathered columns, 0: full forward), completion ticket of the scan
  int inc_chunks;
  Prof* prof;
};
constexpr int INC_CHUNK = 512;
size_t grad_scratch_bytes(const adacgd_problem& p, int flags);
void carve_grad_scratch(GradScratch* g, void* base, const adacgd_problem& p, int flags);
int launch_gradient(const adacgd_problem& p, const GradScratch& g, const float* x, float* grads,
                    cudaStream_t stream);
// Incremental variant of stage a1 (the caller has already moved x): u += A (g - g_prev), z -= gamma u, then the
// residuals from z and the backward pass.  `refresh`: z = A x and u = A g are recomputed in full instead.
int launch_gradient_incremental(const adacgd_problem& p, const GradScratch& g, const float* x, const float* gvec,
                                float gamma, bool refresh, float* grads, cudaStream_t stream);
int build_transposed_features(const adacgd_problem& p, const GradScratch& g, cudaStream_t stream);
const char* build_csc(const adacgd_problem& p, GradScratch* g, cudaStream_t stream);

int launch_mean_rows(const float* G, int rows, long long d, float* out, cudaStream_t stream);

// Stores the message that adacgd_last_error(NULL) returns on this thread.
void set_thread_error(const char* msg);

}  // namespace adacgd
