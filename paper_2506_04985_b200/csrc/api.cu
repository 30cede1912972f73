// C-ABI entry points that compose the kernels: argument checks, workspace carving,
// launches.  No device memory is allocated here; everything lives in caller buffers.
#include "fpt_internal.cuh"

namespace fpt {

static inline size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }

static int check_qp(const fpt_qparams* qp) {
  if (!qp) return FPT_ERR_BAD_ARG;
  if (qp->bits != 4) return FPT_ERR_UNSUPPORTED;
  if (!(qp->scale > 0.0f)) return FPT_ERR_BAD_ARG;
  if (!qp->symmetric && (qp->zero_point < 0 || qp->zero_point > 15)) return FPT_ERR_BAD_ARG;
  return FPT_OK;
}

// bf16 buffer between the two matmuls of the MLP block: nothing when the gate||up matmul's epilogue
// quantises the products itself (more than 128 tokens, no online transform), the products [M, d_ff]
// when the transform needs whole rows of them, gate||up [M, 2 d_ff] on the unfused route.
static size_t mlp_gu_bytes(int M, int d_ff, bool hadamard) {
  if (M > 128) return hadamard ? (size_t)M * (size_t)d_ff * 2 : 0;
  return (size_t)M * 2 * (size_t)d_ff * 2;
}

static int check_gemm_shape(int M, int N, int K) {
  if (M <= 0 || N <= 0 || K <= 0) return FPT_ERR_BAD_ARG;
  if (K % 128 != 0 || K > 65535 || N % 8 != 0) return FPT_ERR_UNSUPPORTED;
  return FPT_OK;
}

static int g_programmatic_launch = 1;
int programmatic_launch_enabled() { return g_programmatic_launch; }

// The 4-bit static linear behind fpt_w4a4_linear and fpt_w4a4_linear_static: one set of argument
// checks and one carving of the workspace (control block | matmul scratch | codes | one float per token).
int linear4_check(const void* X, const uint8_t* Wq, const void* sw, int scale_dtype, const int32_t* wsum, const void* Y,
                  const fpt_qparams* act_qp, int M, int N, int K, int flags, const float* s_in, int post_mode,
                  const float* post) {
  if (!X || !Wq || !sw || !Y) return FPT_ERR_BAD_ARG;
  int rc = check_qp(act_qp);
  if (rc) return rc;
  rc = check_gemm_shape(M, N, K);
  if (rc) return rc;
  if (scale_dtype != FPT_DTYPE_F32 && scale_dtype != FPT_DTYPE_F16) return FPT_ERR_BAD_ARG;
  if (flags & ~(FPT_RMSNORM | FPT_SCALE_INPUT)) return FPT_ERR_UNSUPPORTED;
  if ((flags & FPT_SCALE_INPUT) && !s_in) return FPT_ERR_BAD_ARG;
  if (post_mode < FPT_POST_NONE || post_mode > FPT_POST_VECTOR) return FPT_ERR_BAD_ARG;
  if (post_mode == FPT_POST_VECTOR && !post) return FPT_ERR_BAD_ARG;
  if (!act_qp->symmetric && !wsum) return FPT_ERR_BAD_ARG;
  if (((uintptr_t)X | (uintptr_t)Wq | (uintptr_t)Y | (uintptr_t)sw | (uintptr_t)wsum) & 15) return FPT_ERR_ALIGNMENT;
  return FPT_OK;
}

int linear4_run(cudaStream_t st, const void* X, int M, int K, const uint8_t* Wq, const void* sw, int scale_dtype,
                const int32_t* wsum, int N, const fpt_qparams* act_qp, int flags, float eps, const float* s_in,
                int post_mode, const float* post, void* Y, float* s_out, uint8_t* ws) {
  const size_t gemm_ws = kStatusBytes + gemm_scratch_bytes(M);      // control block + matmul scratch
  uint8_t* Xq = ws + gemm_ws;
  float* post_inv = reinterpret_cast<float*>(Xq + up256((size_t)M * K / 2));
  if (act_quant_launch(st, X, M, K, K, act_qp, flags, eps, nullptr, s_in, Xq, s_out,
                       post_mode == FPT_POST_INVERSE_OF_PRE ? post_inv : nullptr, nullptr) != cudaSuccess)
    return FPT_ERR_CUDA;
  GemmParams P{};
  P.M = M; P.N = N; P.K = K;
  P.sw = sw; P.scale_dtype = scale_dtype;
  P.wsum = act_qp->symmetric ? nullptr : wsum;
  P.zero_point = act_qp->symmetric ? 0 : act_qp->zero_point;
  P.a_unsigned = act_qp->symmetric ? 0 : 1;
  P.act_scale = act_qp->scale;
  P.post = post_mode == FPT_POST_NONE ? nullptr : post_mode == FPT_POST_VECTOR ? post : post_inv;
  P.Y = reinterpret_cast<__nv_bfloat16*>(Y);
  P.status = reinterpret_cast<uint32_t*>(ws);
  P.scratch = ws + kStatusBytes;
  return gemm_launch(st, Xq, Wq, P);
}

}  // namespace fpt

using namespace fpt;

extern "C" int fpt_version(void) { return 101; }

extern "C" int fpt_set_programmatic_launch(int enabled) {
  const int old = g_programmatic_launch;
  g_programmatic_launch = enabled ? 1 : 0;
  return old;
}

extern "C" const char* fpt_strerror(int code) {
  switch (code) {
    case FPT_OK: return "ok";
    case FPT_ERR_BAD_ARG: return "bad argument";
    case FPT_ERR_UNSUPPORTED: return "unsupported size, bit-width or combination of flags";
    case FPT_ERR_ALIGNMENT: return "misaligned pointer or leading dimension";
    case FPT_ERR_WORKSPACE: return "workspace missing or too small";
    case FPT_ERR_CUDA: return "CUDA call failed";
    case FPT_ERR_TIMEOUT: return "a device-side wait gave up";
    default: return "unknown error code";
  }
}

extern "C" size_t fpt_workspace_bytes(int op, int M, int N, int K) {
  if (M <= 0 || N <= 0 || K <= 0) return 0;
  const size_t m = (size_t)M;
  switch (op) {
    case FPT_OP_GEMM:
      return kStatusBytes + gemm_scratch_bytes(M);
    case FPT_OP_LINEAR:
      return kStatusBytes + gemm_scratch_bytes(M) + up256(m * (size_t)K / 2) + up256(m * 4);
    case FPT_OP_GEMM_A8:
      return kStatusBytes + gemm_scratch_bytes(M) + gemm_a8_scratch_bytes(M, N, K);
    case FPT_OP_LINEAR_A8:
      return kStatusBytes + gemm_scratch_bytes(M) + gemm_a8_scratch_bytes(M, N, K) + up256(m * (size_t)K) + up256(m * 4);
    case FPT_OP_MLP:
    case FPT_OP_MLP_HADAMARD: {   // N = d_ff, K = d
      const size_t dff = (size_t)N, d = (size_t)K;
      return kStatusBytes + gemm_scratch_bytes(M) + up256(m * d / 2) + 2 * up256(m * 4) +
             up256(mlp_gu_bytes(M, N, op == FPT_OP_MLP_HADAMARD)) + up256(m * dff / 2);
    }
    default:
      return 0;
  }
}

extern "C" int fpt_reset_status(void* stream, void* workspace) {
  if (!workspace) return FPT_ERR_BAD_ARG;
  return cudaMemsetAsync(workspace, 0, kStatusBytes, (cudaStream_t)stream) == cudaSuccess ? FPT_OK : FPT_ERR_CUDA;
}

extern "C" int fpt_check_status(void* stream, void* workspace) {
  if (!workspace) return FPT_ERR_BAD_ARG;
  uint32_t word = 0;
  if (cudaMemcpyAsync(&word, workspace, 4, cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess)
    return FPT_ERR_CUDA;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return FPT_ERR_CUDA;
  return word == 0 ? FPT_OK : FPT_ERR_TIMEOUT;
}

extern "C" int fpt_w4a4_gemm(void* stream, const uint8_t* Xq, const uint8_t* Wq, int M, int N, int K, const void* sw,
                             int scale_dtype, const int32_t* wsum, float act_scale, int act_symmetric,
                             int act_zero_point, const float* post, const void* residual, const float* res_scale,
                             void* Y, int32_t* acc_out, void* workspace, size_t workspace_bytes) {
  if (!Xq || !Wq || !sw || (!Y && !acc_out)) return FPT_ERR_BAD_ARG;
  int rc = check_gemm_shape(M, N, K);
  if (rc) return rc;
  if (scale_dtype != FPT_DTYPE_F32 && scale_dtype != FPT_DTYPE_F16) return FPT_ERR_BAD_ARG;
  if (!(act_scale > 0.0f)) return FPT_ERR_BAD_ARG;
  if (!act_symmetric && (!wsum || act_zero_point < 0 || act_zero_point > 15)) return FPT_ERR_BAD_ARG;
  if (((uintptr_t)Xq | (uintptr_t)Wq | (uintptr_t)Y | (uintptr_t)acc_out | (uintptr_t)residual | (uintptr_t)workspace |
       (uintptr_t)sw | (uintptr_t)wsum) & 15)
    return FPT_ERR_ALIGNMENT;
  if (!workspace || workspace_bytes < fpt_workspace_bytes(FPT_OP_GEMM, M, N, K)) return FPT_ERR_WORKSPACE;
  GemmParams P{};
  P.M = M; P.N = N; P.K = K;
  P.sw = sw; P.scale_dtype = scale_dtype;
  P.wsum = act_symmetric ? nullptr : wsum;
  P.zero_point = act_symmetric ? 0 : act_zero_point;
  P.a_unsigned = act_symmetric ? 0 : 1;
  P.act_scale = act_scale;
  P.post = post;
  P.residual = reinterpret_cast<const __nv_bfloat16*>(residual);
  P.res_scale = res_scale;
  P.Y = reinterpret_cast<__nv_bfloat16*>(Y);
  P.acc_out = acc_out;
  P.status = reinterpret_cast<uint32_t*>(workspace);
  P.scratch = reinterpret_cast<uint8_t*>(workspace) + kStatusBytes;
  return gemm_launch((cudaStream_t)stream, Xq, Wq, P);
}

extern "C" int fpt_w4a4_linear(void* stream, const void* X, int M, int K, const uint8_t* Wq, const void* sw,
                               int scale_dtype, const int32_t* wsum, int N, const fpt_qparams* act_qp, int flags,
                               float eps, const float* s_in, int post_mode, const float* post, void* Y, float* s_out,
                               void* workspace, size_t workspace_bytes) {
  if (!X || !Wq || !sw || !Y) return FPT_ERR_BAD_ARG;
  const bool a8 = act_qp && act_qp->bits == 8;
  int rc = a8 ? ((act_qp->symmetric && act_qp->scale > 0.0f) ? FPT_OK : FPT_ERR_UNSUPPORTED) : check_qp(act_qp);
  if (rc) return rc;
  rc = check_gemm_shape(M, N, K);
  if (rc) return rc;
  if (flags & ~(FPT_RMSNORM | FPT_SCALE_INPUT)) return FPT_ERR_UNSUPPORTED;
  if ((flags & FPT_SCALE_INPUT) && !s_in) return FPT_ERR_BAD_ARG;
  if (post_mode < FPT_POST_NONE || post_mode > FPT_POST_VECTOR) return FPT_ERR_BAD_ARG;
  if (post_mode == FPT_POST_VECTOR && !post) return FPT_ERR_BAD_ARG;
  if (a8) {
    if (((uintptr_t)X | (uintptr_t)Wq | (uintptr_t)Y | (uintptr_t)workspace) & 15) return FPT_ERR_ALIGNMENT;
    if (!workspace || workspace_bytes < fpt_workspace_bytes(FPT_OP_LINEAR_A8, M, N, K)) return FPT_ERR_WORKSPACE;
    const size_t gemm_ws8 = fpt_workspace_bytes(FPT_OP_GEMM_A8, M, N, K);
    int8_t* Xq8 = reinterpret_cast<int8_t*>(workspace) + gemm_ws8;
    float* pinv = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(Xq8) + up256((size_t)M * K));
    if (act_quant_dyn_launch((cudaStream_t)stream, X, M, K, K, 8, 0, act_qp->scale, flags, eps, s_in, post_mode, post,
                             Xq8, s_out, post_mode == FPT_POST_INVERSE_OF_PRE ? pinv : nullptr, nullptr,
                             nullptr) != cudaSuccess)
      return FPT_ERR_CUDA;
    const float* pv8 = post_mode == FPT_POST_NONE ? nullptr : post_mode == FPT_POST_VECTOR ? post : pinv;
    return fpt_w4a8_gemm(stream, Xq8, Wq, M, N, K, sw, scale_dtype, act_qp->scale, pv8, nullptr, nullptr, Y, nullptr,
                         workspace, gemm_ws8);
  }
  rc = linear4_check(X, Wq, sw, scale_dtype, wsum, Y, act_qp, M, N, K, flags, s_in, post_mode, post);
  if (rc) return rc;
  if ((uintptr_t)workspace & 15) return FPT_ERR_ALIGNMENT;
  if (!workspace || workspace_bytes < fpt_workspace_bytes(FPT_OP_LINEAR, M, N, K)) return FPT_ERR_WORKSPACE;
  return linear4_run((cudaStream_t)stream, X, M, K, Wq, sw, scale_dtype, wsum, N, act_qp, flags, eps, s_in, post_mode,
                     post, Y, s_out, reinterpret_cast<uint8_t*>(workspace));
}

extern "C" int fpt_decoder_mlp(void* stream, const void* X, int M, int d, int d_ff, const uint8_t* Wgu_q,
                               const void* sw_gu, const uint8_t* Wd_q, const void* sw_d, int scale_dtype,
                               const fpt_qparams* qp_in, const fpt_qparams* qp_mid, float eps, const float* s_prev,
                               float* s_out, int add_residual, int mid_hadamard, void* Y, void* workspace,
                               size_t workspace_bytes) {
  if (!X || !Wgu_q || !sw_gu || !Wd_q || !sw_d || !Y) return FPT_ERR_BAD_ARG;
  int rc = check_qp(qp_in);
  if (rc) return rc;
  rc = check_qp(qp_mid);
  if (rc) return rc;
  if (!qp_in->symmetric || !qp_mid->symmetric) return FPT_ERR_UNSUPPORTED;
  if (M <= 0 || d <= 0 || d_ff <= 0) return FPT_ERR_BAD_ARG;
  if (d % 128 != 0 || d_ff % 128 != 0 || d_ff > 32768 || d > 65535) return FPT_ERR_UNSUPPORTED;
  if (scale_dtype != FPT_DTYPE_F32 && scale_dtype != FPT_DTYPE_F16) return FPT_ERR_BAD_ARG;
  if (mid_hadamard && (hadamard_block(d_ff) < 256 || hadamard_block(d_ff) > 4096)) return FPT_ERR_UNSUPPORTED;
  if (((uintptr_t)X | (uintptr_t)Wgu_q | (uintptr_t)Wd_q | (uintptr_t)Y | (uintptr_t)workspace) & 15)
    return FPT_ERR_ALIGNMENT;
  if (!workspace ||
      workspace_bytes < fpt_workspace_bytes(mid_hadamard ? FPT_OP_MLP_HADAMARD : FPT_OP_MLP, M, d_ff, d))
    return FPT_ERR_WORKSPACE;
  const size_t m = (size_t)M;
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  const size_t gemm_ws = kStatusBytes + gemm_scratch_bytes(M);      // control block + matmul scratch
  uint8_t* Xq = ws + gemm_ws;
  float* sn_ws = reinterpret_cast<float*>(Xq + up256(m * d / 2));
  float* r_ws = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(sn_ws) + up256(m * 4));
  uint8_t* GU = reinterpret_cast<uint8_t*>(r_ws) + up256(m * 4);
  uint8_t* Mq = GU + up256(mlp_gu_bytes(M, d_ff, mid_hadamard != 0));
  float* sn = s_out ? s_out : sn_ws;
  cudaStream_t st = (cudaStream_t)stream;

  // X~ = RMSNorm(X) on the grid qp_in; S_n = S_{n-1} * r
  if (act_quant_launch(st, X, M, d, d, qp_in, FPT_RMSNORM, eps, nullptr, s_prev, Xq, sn, nullptr, r_ws) != cudaSuccess)
    return FPT_ERR_CUDA;
  if (M > 128) {
    // gate || up in one matmul whose epilogue forms m = bf16(silu(g) * u) and quantises m * S_n:
    // the static grid and S_n are known before the matmul starts, so g and u never reach memory
    GemmParams P{};
    P.M = M; P.N = 2 * d_ff; P.K = d;
    P.sw = sw_gu; P.scale_dtype = scale_dtype;
    P.act_scale = qp_in->scale;
    if (mid_hadamard) {          // the products leave as bf16 [M, d_ff]; the transform needs whole rows of them
      P.swiglu_bf16 = 1;
      P.Y = reinterpret_cast<__nv_bfloat16*>(GU);
    } else {
      P.Mq = Mq; P.mid_scale = sn;
      P.mid_inv_delta = 1.0f / qp_mid->scale;
      P.mid_qmax_minus_z = 7; P.mid_flip = 0x77777777u;
    }
    P.status = reinterpret_cast<uint32_t*>(workspace);
    P.scratch = ws + kStatusBytes;
    rc = gemm_pair_launch(st, Xq, Wgu_q, P);
    if (rc) return rc;
    if (mid_hadamard &&
        hadamard_quant_launch(st, GU, M, d_ff, d_ff, qp_mid, 0, sn, Mq) != cudaSuccess)
      return FPT_ERR_CUDA;
  } else if (mid_hadamard) {
    rc = fpt_w4a4_gemm(stream, Xq, Wgu_q, M, 2 * d_ff, d, sw_gu, scale_dtype, nullptr, qp_in->scale, 1, 0, nullptr,
                       nullptr, nullptr, GU, nullptr, workspace, gemm_ws);
    if (rc) return rc;
    if (hadamard_quant_launch(st, GU, M, d_ff, 2 * d_ff, qp_mid, 1, sn, Mq) != cudaSuccess) return FPT_ERR_CUDA;
  } else {
    // gate || up in one matmul over the interleaved weight
    rc = fpt_w4a4_gemm(stream, Xq, Wgu_q, M, 2 * d_ff, d, sw_gu, scale_dtype, nullptr, qp_in->scale, 1, 0, nullptr,
                       nullptr, nullptr, GU, nullptr, workspace, gemm_ws);
    if (rc) return rc;
    // m = bf16(silu(g) * u), quantised after the multiply by S_n
    if (act_quant_launch(st, GU, M, d_ff, 2 * d_ff, qp_mid, FPT_SILU_MUL | FPT_GU_INTERLEAVED | FPT_SCALE_INPUT, 0.0f,
                         nullptr, sn, Mq, nullptr, nullptr, nullptr) != cudaSuccess)
      return FPT_ERR_CUDA;
  }
  // down projection; the normalised residual X * r joins before the final rounding
  return fpt_w4a4_gemm(stream, Mq, Wd_q, M, d, d_ff, sw_d, scale_dtype, nullptr, qp_mid->scale, 1, 0, nullptr,
                       add_residual ? X : nullptr, add_residual ? r_ws : nullptr, Y, nullptr, workspace, gemm_ws);
}

extern "C" int fpt_decoder_attn_qkv(void* stream, const void* X, int M, int d, const uint8_t* Wqkv_q, const void* sw_qkv,
                                    int scale_dtype, const int32_t* wsum_qkv, int n_qkv, const fpt_qparams* qp_in,
                                    float eps, const float* s_prev, float* s_out, float* r_out, void* QKV,
                                    void* workspace, size_t workspace_bytes) {
  if (!X || !Wqkv_q || !sw_qkv || !QKV || !s_out || !r_out) return FPT_ERR_BAD_ARG;
  int rc = check_qp(qp_in);
  if (rc) return rc;
  rc = check_gemm_shape(M, n_qkv, d);
  if (rc) return rc;
  if (!qp_in->symmetric && !wsum_qkv) return FPT_ERR_BAD_ARG;
  if (((uintptr_t)X | (uintptr_t)Wqkv_q | (uintptr_t)QKV | (uintptr_t)workspace) & 15) return FPT_ERR_ALIGNMENT;
  if (!workspace || workspace_bytes < fpt_workspace_bytes(FPT_OP_LINEAR, M, n_qkv, d)) return FPT_ERR_WORKSPACE;
  const size_t gemm_ws = kStatusBytes + gemm_scratch_bytes(M);
  uint8_t* Xq = reinterpret_cast<uint8_t*>(workspace) + gemm_ws;
  // X~ = RMSNorm(X) on the grid qp_in; S_n = S_{n-1} * r; r kept for the residual
  if (act_quant_launch((cudaStream_t)stream, X, M, d, d, qp_in, FPT_RMSNORM, eps, nullptr, s_prev, Xq, s_out, nullptr,
                       r_out) != cudaSuccess)
    return FPT_ERR_CUDA;
  return fpt_w4a4_gemm(stream, Xq, Wqkv_q, M, n_qkv, d, sw_qkv, scale_dtype, wsum_qkv, qp_in->scale, qp_in->symmetric,
                       qp_in->zero_point, nullptr, nullptr, nullptr, QKV, nullptr, workspace, gemm_ws);
}

extern "C" int fpt_decoder_attn_out(void* stream, const void* A, int M, int k_o, const uint8_t* Wo_q, const void* sw_o,
                                    int scale_dtype, const int32_t* wsum_o, int d, const fpt_qparams* qp_ap,
                                    const float* s_n, const void* X, const float* r, void* Y, void* workspace,
                                    size_t workspace_bytes) {
  if (!A || !Wo_q || !sw_o || !Y || !s_n) return FPT_ERR_BAD_ARG;
  if (X && !r) return FPT_ERR_BAD_ARG;
  int rc = check_qp(qp_ap);
  if (rc) return rc;
  rc = check_gemm_shape(M, d, k_o);
  if (rc) return rc;
  if (!qp_ap->symmetric && !wsum_o) return FPT_ERR_BAD_ARG;
  if (((uintptr_t)A | (uintptr_t)Wo_q | (uintptr_t)Y | (uintptr_t)X | (uintptr_t)workspace) & 15) return FPT_ERR_ALIGNMENT;
  if (!workspace || workspace_bytes < fpt_workspace_bytes(FPT_OP_LINEAR, M, d, k_o)) return FPT_ERR_WORKSPACE;
  const size_t gemm_ws = kStatusBytes + gemm_scratch_bytes(M);
  uint8_t* Aq = reinterpret_cast<uint8_t*>(workspace) + gemm_ws;
  // the sequence scaler at the attention output: the grid sees A * S_n
  if (act_quant_launch((cudaStream_t)stream, A, M, k_o, k_o, qp_ap, FPT_SCALE_INPUT, 0.0f, nullptr, s_n, Aq, nullptr,
                       nullptr, nullptr) != cudaSuccess)
    return FPT_ERR_CUDA;
  // output projection; the normalised residual X * r joins before the final rounding
  return fpt_w4a4_gemm(stream, Aq, Wo_q, M, d, k_o, sw_o, scale_dtype, wsum_o, qp_ap->scale, qp_ap->symmetric,
                       qp_ap->zero_point, nullptr, X, X ? r : nullptr, Y, nullptr, workspace, gemm_ws);
}

extern "C" int fpt_w4a4_linear_dynamic(void* stream, const void* X, int M, int K, const uint8_t* Wq, const void* sw,
                                       int scale_dtype, int N, int bits, int flags, float eps, const float* s_in,
                                       int post_mode, const float* post, void* Y, float* s_out, void* workspace,
                                       size_t workspace_bytes) {
  if (!X || !Wq || !sw || !Y) return FPT_ERR_BAD_ARG;
  if (bits != 4 && bits != 8) return FPT_ERR_UNSUPPORTED;
  int rc = check_gemm_shape(M, N, K);
  if (rc) return rc;
  if (flags & ~(FPT_RMSNORM | FPT_SCALE_INPUT)) return FPT_ERR_UNSUPPORTED;
  if ((flags & FPT_SCALE_INPUT) && !s_in) return FPT_ERR_BAD_ARG;
  if (post_mode < FPT_POST_NONE || post_mode > FPT_POST_VECTOR) return FPT_ERR_BAD_ARG;
  if (post_mode == FPT_POST_VECTOR && !post) return FPT_ERR_BAD_ARG;
  if (((uintptr_t)X | (uintptr_t)Wq | (uintptr_t)Y | (uintptr_t)workspace) & 15) return FPT_ERR_ALIGNMENT;
  if (bits == 8) {
    if (!workspace || workspace_bytes < fpt_workspace_bytes(FPT_OP_LINEAR_A8, M, N, K)) return FPT_ERR_WORKSPACE;
    const size_t gemm_ws8 = fpt_workspace_bytes(FPT_OP_GEMM_A8, M, N, K);
    int8_t* Xq8 = reinterpret_cast<int8_t*>(workspace) + gemm_ws8;
    float* c8 = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(Xq8) + up256((size_t)M * K));
    if (act_quant_dyn_launch((cudaStream_t)stream, X, M, K, K, 8, 1, 1.0f, flags, eps, s_in, post_mode, post, Xq8, s_out,
                             c8, nullptr, nullptr) != cudaSuccess)
      return FPT_ERR_CUDA;
    return fpt_w4a8_gemm(stream, Xq8, Wq, M, N, K, sw, scale_dtype, 1.0f, c8, nullptr, nullptr, Y, nullptr, workspace,
                         gemm_ws8);
  }
  if (!workspace || workspace_bytes < fpt_workspace_bytes(FPT_OP_LINEAR, M, N, K)) return FPT_ERR_WORKSPACE;
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  const size_t gemm_ws = kStatusBytes + gemm_scratch_bytes(M);
  uint8_t* Xq = ws + gemm_ws;
  float* c_t = reinterpret_cast<float*>(Xq + up256((size_t)M * K / 2));
  // per-token grid; the factor the epilogue needs (D_t, times whatever the post mode asks for) per token
  if (act_quant_dyn_launch((cudaStream_t)stream, X, M, K, K, 4, 1, 1.0f, flags, eps, s_in, post_mode, post, Xq, s_out,
                           c_t, nullptr, nullptr) != cudaSuccess)
    return FPT_ERR_CUDA;
  return fpt_w4a4_gemm(stream, Xq, Wq, M, N, K, sw, scale_dtype, nullptr, 1.0f, 1, 0, c_t, nullptr, nullptr, Y, nullptr,
                       workspace, gemm_ws);
}
