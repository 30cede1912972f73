// fpt_w4a4_linear_static: the W4A4 linear for callers that cannot hand over a workspace.
//
// fpt_w4a4_linear needs scratch in device memory (the packed activation codes, one float per
// token and the status block) and asks the caller to allocate it.  Some callers have no way to
// do that: a plug-in that an inference runtime calls with nothing but input and output
// pointers, a serving loop whose memory pool was sized and frozen at start-up, code that runs
// where a device allocation would synchronise the whole GPU.  For them the same three steps run
// here on a scratch area that is part of the library image itself: a file-scope __device__
// array.  Every GPU that loads the library carries that array until the process exits, so it is
// kept modest (FPT_STATIC_SCRATCH_BYTES), and problems that do not fit are refused.
//
// Host code must not pass the array's name to a kernel: on the host the symbol is only a handle.
// Its device address is looked up once per device with cudaGetSymbolAddress (with that device
// current) and cached; kernels get that address.
#include <mutex>

#include "fpt_internal.cuh"

namespace fpt {

constexpr size_t kStaticScratchBytes = FPT_STATIC_SCRATCH_BYTES;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

static std::mutex g_scratch_mutex;
static unsigned char* g_scratch_addr[kMaxDevices] = {};

// Device address of the scratch array on the current device (looked up on first use).
static int static_scratch(unsigned char** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return FPT_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return FPT_ERR_CUDA;
    g_scratch_addr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_scratch_addr[dev];
  return FPT_OK;
}

}  // namespace fpt

using namespace fpt;

extern "C" int fpt_w4a4_linear_static(void* stream, const void* X, int M, int K, const uint8_t* Wq, const void* sw,
                                      int scale_dtype, const int32_t* wsum, int N, const fpt_qparams* act_qp,
                                      int flags, float eps, const float* s_in, int post_mode, const float* post,
                                      void* Y, float* s_out) {
  if (!act_qp) return FPT_ERR_BAD_ARG;
  if (act_qp->bits != 4) return FPT_ERR_UNSUPPORTED;       // the 8-bit route of fpt_w4a4_linear is not offered here
  int rc = linear4_check(X, Wq, sw, scale_dtype, wsum, Y, act_qp, M, N, K, flags, s_in, post_mode, post);
  if (rc) return rc;
  // the same carving as fpt_w4a4_linear's workspace, inside the built-in array
  if (fpt_workspace_bytes(FPT_OP_LINEAR, M, N, K) > kStaticScratchBytes) return FPT_ERR_WORKSPACE;

  unsigned char* base = nullptr;
  rc = static_scratch(&base);
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  // the array keeps whatever the last call left: the control block (status word, tile counters)
  // has to start at zero
  if (cudaMemsetAsync(base, 0, kStatusBytes, st) != cudaSuccess) return FPT_ERR_CUDA;
  return linear4_run(st, X, M, K, Wq, sw, scale_dtype, wsum, N, act_qp, flags, eps, s_in, post_mode, post, Y, s_out, base);
}
