// adacgd_compress_noalloc: the compression step on a scratch array compiled into the library.
#include "adacgd_device.cuh"

// --------------------------------------------------------------------------
// compression without any device allocation
// --------------------------------------------------------------------------
namespace adacgd {

// Scratch of adacgd_compress_noalloc.  It is part of the library image: every GPU that
// loads libadacgd holds these 2 MiB until the process exits, whether or not the entry
// point is ever called.
constexpr size_t NOALLOC_SCRATCH_BYTES = 2u << 20;
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_SCRATCH_BYTES];

constexpr int NOALLOC_MAX_DEVICES = 64;
static void* g_noalloc_base[NOALLOC_MAX_DEVICES] = {nullptr};

// In host code `g_noalloc_scratch` is only a handle; the address a kernel may use has to be
// asked for, per device, with that device current.
static adacgd_status noalloc_base(void** base) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NOALLOC_MAX_DEVICES) {
    set_thread_error("adacgd_compress_noalloc: no current CUDA device (or device ordinal above 63)");
    return ADACGD_ERR_CUDA;
  }
  if (!g_noalloc_base[dev]) {
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess || !p) {
      set_thread_error("adacgd_compress_noalloc: cudaGetSymbolAddress failed for the built-in scratch");
      return ADACGD_ERR_CUDA;
    }
    g_noalloc_base[dev] = p;
  }
  *base = g_noalloc_base[dev];
  return ADACGD_OK;
}

}  // namespace adacgd

extern "C" adacgd_status adacgd_compress_noalloc(const float* X_dev, float* G_dev, const float* Y_dev,
                                                 int32_t rows, int64_t d, const adacgd_cset* cset,
                                                 float* mean_out_dev, int32_t* level_dev, uint64_t* bits_dev,
                                                 void* cuda_stream) {
  using namespace adacgd;
  if (!X_dev || !G_dev || !Y_dev) {
    set_thread_error("adacgd_compress_noalloc: X, G, Y must be non-NULL");
    return ADACGD_ERR_INVALID_ARG;
  }
  if (rows < 1 || rows > ADACGD_NOALLOC_MAX_ROWS || d < 1 || d > ADACGD_NOALLOC_MAX_D ||
      scratch_bytes(rows, d, false) > NOALLOC_SCRATCH_BYTES) {
    set_thread_error("adacgd_compress_noalloc: shape exceeds the built-in scratch "
                     "(rows <= ADACGD_NOALLOC_MAX_ROWS = 4, d <= ADACGD_NOALLOC_MAX_D = 4194304); "
                     "use adacgd_init + adacgd_compress with a caller-owned workspace");
    return ADACGD_ERR_INVALID_ARG;
  }
  const char* msg = "";
  CsetDev cs;
  const adacgd_status st = make_cset(cset, d, &cs, &msg);
  if (st != ADACGD_OK) {
    set_thread_error(msg);
    return st;
  }
  void* base = nullptr;
  const adacgd_status sb = noalloc_base(&base);
  if (sb != ADACGD_OK) return sb;
  Scratch s;
  carve_scratch(&s, base, rows, d, false);
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  // the array keeps whatever the previous call left: the status words start from zero here,
  // the histograms and accumulators are cleared by launch_compress itself
  if (cudaMemsetAsync(s.flags, 0, 64, stream) != cudaSuccess) {
    set_thread_error("adacgd_compress_noalloc: cudaMemsetAsync failed");
    return ADACGD_ERR_CUDA;
  }
  CompressOut o;
  memset(&o, 0, sizeof(o));
  o.mean_out = mean_out_dev;
  o.level = level_dev;
  o.bits = bits_dev;
  if (launch_compress(s, cs, X_dev, G_dev, Y_dev, rows, d, o, stream) < 0) {
    set_thread_error("adacgd_compress_noalloc: kernel launch failed");
    return ADACGD_ERR_CUDA;
  }
  return ADACGD_OK;
}
