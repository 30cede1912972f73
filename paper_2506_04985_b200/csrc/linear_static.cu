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
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

static std::mutex g_scratch_mutex;
static unsigned char* g_scratch_addr[kMaxDevices] = {};

static inline size_t up256s(size_t x) { return (x + 255) & ~(size_t)255; }

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
  if (!X || !Wq || !sw || !Y || !act_qp) return FPT_ERR_BAD_ARG;
  if (act_qp->bits != 4) return FPT_ERR_UNSUPPORTED;
  if (!(act_qp->scale > 0.0f)) return FPT_ERR_BAD_ARG;
  if (!act_qp->symmetric && (act_qp->zero_point < 0 || act_qp->zero_point > 15 || !wsum)) return FPT_ERR_BAD_ARG;
  if (M <= 0 || N <= 0 || K <= 0) return FPT_ERR_BAD_ARG;
  if (K % 128 != 0 || K > 65535 || N % 8 != 0) return FPT_ERR_UNSUPPORTED;
  if (flags & ~(FPT_RMSNORM | FPT_SCALE_INPUT)) return FPT_ERR_UNSUPPORTED;
  if ((flags & FPT_SCALE_INPUT) && !s_in) return FPT_ERR_BAD_ARG;
  if (post_mode < FPT_POST_NONE || post_mode > FPT_POST_VECTOR) return FPT_ERR_BAD_ARG;
  if (post_mode == FPT_POST_VECTOR && !post) return FPT_ERR_BAD_ARG;
  if (scale_dtype != FPT_DTYPE_F32 && scale_dtype != FPT_DTYPE_F16) return FPT_ERR_BAD_ARG;
  if (((uintptr_t)X | (uintptr_t)Wq | (uintptr_t)Y) & 15) return FPT_ERR_ALIGNMENT;
  // control block | matmul scratch (decode sizes only) | packed codes [M, K/2] | one float per token
  const size_t codes = up256s((size_t)M * (size_t)K / 2);
  const size_t gemm_ws = kStatusBytes + gemm_scratch_bytes(M);
  const size_t need = gemm_ws + codes + up256s((size_t)M * 4);
  if (need > kStaticScratchBytes) return FPT_ERR_WORKSPACE;     // the built-in scratch is too small for M x K

  unsigned char* base = nullptr;
  int rc = static_scratch(&base);
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  // the array keeps whatever the last call left: the control block (status word, tile counters)
  // has to start at zero
  if (cudaMemsetAsync(base, 0, kStatusBytes, st) != cudaSuccess) return FPT_ERR_CUDA;
  uint8_t* Xq = base + gemm_ws;
  float* post_inv = reinterpret_cast<float*>(Xq + codes);
  if (act_quant_launch(st, X, M, K, K, act_qp, flags, eps, nullptr, s_in, Xq, s_out,
                       post_mode == FPT_POST_INVERSE_OF_PRE ? post_inv : nullptr, nullptr) != cudaSuccess)
    return FPT_ERR_CUDA;
  const float* pv = post_mode == FPT_POST_NONE ? nullptr : post_mode == FPT_POST_VECTOR ? post : post_inv;
  GemmParams P{};
  P.M = M; P.N = N; P.K = K;
  P.sw = sw; P.scale_dtype = scale_dtype;
  P.wsum = act_qp->symmetric ? nullptr : wsum;
  P.zero_point = act_qp->symmetric ? 0 : act_qp->zero_point;
  P.a_unsigned = act_qp->symmetric ? 0 : 1;
  P.act_scale = act_qp->scale;
  P.post = pv;
  P.Y = reinterpret_cast<__nv_bfloat16*>(Y);
  P.status = reinterpret_cast<uint32_t*>(base);
  P.scratch = base + kStatusBytes;
  return gemm_launch(st, Xq, Wq, P);
}
