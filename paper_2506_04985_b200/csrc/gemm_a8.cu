// Steps (2)+(3) with 8-bit activation codes and 4-bit weights (the W4A8 setting of Sec. 4,
// Table "4-8-8"): the same exact integer matmul and scale-factor epilogue (App. B, App. J).
//
// More than 16 tokens and 128 outputs: the CTA-pair kernel with the activation tile loaded as int8 (no
// widening on that side); up to 16 tokens: the register kernel reading int8 codes.  What is left (17 to 128
// tokens with at most 128 outputs, or more tokens with few outputs) takes a route that needs no kernel of its own: an int8 code is
// a = 16 h + l with h = a >> 4 in [-8, 7] and l = a & 15 in [0, 15], so
//   sum_k a w = 16 sum_k h w + sum_k l w,
// two 4-bit matmuls (one signed, one unsigned activation operand) through the existing kernels,
// their int32 results combined exactly before the scale factors.  Twice the matmul work: meant
// for the small shapes, where the time is launch- or weight-stream-bound anyway.
#include "fpt_internal.cuh"

namespace fpt {

static inline size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }

static bool a8_uses_pair(int M, int N) { return M > 16 && N > 128; }
static bool a8_native(int M, int N) { return M <= 16 || a8_uses_pair(M, N); }       // a kernel takes int8 activations as they are

size_t gemm_a8_scratch_bytes(int M, int N, int K) {
  if (a8_native(M, N)) return 0;
  return 2 * up256((size_t)M * K / 2) + 2 * up256((size_t)M * N * 4);
}

// int8 [M, K] -> packed high nibbles (two's complement, the signed part) and packed low nibbles (unsigned).
__global__ void __launch_bounds__(256) split_a8_kernel(const uint4* __restrict__ A, uint2* __restrict__ H,
                                                       uint2* __restrict__ Lo, size_t chunks) {
  const size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= chunks) return;
  const uint4 a = A[i];
  const uint32_t w[4] = {a.x, a.y, a.z, a.w};
  uint32_t h[4], l[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const uint32_t hn = (w[j] >> 4) & 0x0F0F0F0Fu, ln = w[j] & 0x0F0F0F0Fu;
    h[j] = hn | (hn >> 4);          // bytes 0 and 2 hold code pairs (even k low, odd k high)
    l[j] = ln | (ln >> 4);
  }
  H[i] = make_uint2(__byte_perm(h[0], h[1], 0x6420), __byte_perm(h[2], h[3], 0x6420));
  Lo[i] = make_uint2(__byte_perm(l[0], l[1], 0x6420), __byte_perm(l[2], l[3], 0x6420));
}

struct CombineParams {
  const int32_t* acc_h; const int32_t* acc_l;
  const void* sw; int scale_dtype;
  float act_scale; const float* post;
  const __nv_bfloat16* residual; const float* res_scale;
  __nv_bfloat16* Y; int32_t* acc_out;
  int M, N;
};

// acc = 16 acc_h + acc_l; y = bf16(((float)acc * sw[n]) * c_t [+ res * res_scale]); 8 outputs per thread.
__global__ void __launch_bounds__(256) combine_a8_kernel(const CombineParams P) {
  const size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;          // group of 8 columns
  const size_t groups = (size_t)P.M * (size_t)(P.N / 8);
  if (i >= groups) return;
  const int t = (int)(i / (size_t)(P.N / 8)), n0 = (int)(i % (size_t)(P.N / 8)) * 8;
  const size_t off = (size_t)t * P.N + n0;
  const int4 h0 = *reinterpret_cast<const int4*>(P.acc_h + off), h1 = *reinterpret_cast<const int4*>(P.acc_h + off + 4);
  const int4 l0 = *reinterpret_cast<const int4*>(P.acc_l + off), l1 = *reinterpret_cast<const int4*>(P.acc_l + off + 4);
  const int acc[8] = {16 * h0.x + l0.x, 16 * h0.y + l0.y, 16 * h0.z + l0.z, 16 * h0.w + l0.w,
                      16 * h1.x + l1.x, 16 * h1.y + l1.y, 16 * h1.z + l1.z, 16 * h1.w + l1.w};
  if (P.acc_out) {
    *reinterpret_cast<int4*>(P.acc_out + off) = make_int4(acc[0], acc[1], acc[2], acc[3]);
    *reinterpret_cast<int4*>(P.acc_out + off + 4) = make_int4(acc[4], acc[5], acc[6], acc[7]);
  }
  if (!P.Y) return;
  const float c = P.post ? __fmul_rn(P.act_scale, __ldg(P.post + t)) : P.act_scale;
  const float rs = P.res_scale ? __ldg(P.res_scale + t) : 1.0f;
  uint32_t o[4];
#pragma unroll
  for (int j = 0; j < 8; j += 2) {
    float y[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      y[e] = __fmul_rn(__fmul_rn((float)acc[j + e], load_scale(P.sw, P.scale_dtype, n0 + j + e)), c);
      if (P.residual) y[e] = __fadd_rn(y[e], __fmul_rn(__bfloat162float(P.residual[off + j + e]), rs));
    }
    o[j / 2] = f32_to_bf16_bits(y[0]) | (f32_to_bf16_bits(y[1]) << 16);
  }
  *reinterpret_cast<uint4*>(P.Y + off) = make_uint4(o[0], o[1], o[2], o[3]);
}

}  // namespace fpt

using namespace fpt;

extern "C" int fpt_w4a8_gemm(void* stream, const int8_t* Xq8, const uint8_t* Wq, int M, int N, int K, const void* sw,
                             int scale_dtype, float act_scale, const float* post, const void* residual,
                             const float* res_scale, void* Y, int32_t* acc_out, void* workspace,
                             size_t workspace_bytes) {
  if (!Xq8 || !Wq || !sw || (!Y && !acc_out)) return FPT_ERR_BAD_ARG;
  if (M <= 0 || N <= 0 || K <= 0) return FPT_ERR_BAD_ARG;
  if (K % 128 != 0 || N % 8 != 0) return FPT_ERR_UNSUPPORTED;
  if (K > 16384) return FPT_ERR_UNSUPPORTED;               // keeps (float)acc exact: |acc| <= 1024 K < 2^24
  if (scale_dtype != FPT_DTYPE_F32 && scale_dtype != FPT_DTYPE_F16) return FPT_ERR_BAD_ARG;
  if (!(act_scale > 0.0f)) return FPT_ERR_BAD_ARG;
  if (((uintptr_t)Xq8 | (uintptr_t)Wq | (uintptr_t)Y | (uintptr_t)acc_out | (uintptr_t)residual | (uintptr_t)workspace |
       (uintptr_t)sw) & 15)
    return FPT_ERR_ALIGNMENT;
  if (!workspace || workspace_bytes < fpt_workspace_bytes(FPT_OP_GEMM_A8, M, N, K)) return FPT_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  GemmParams P{};
  P.M = M; P.N = N; P.K = K;
  P.sw = sw; P.scale_dtype = scale_dtype;
  P.status = reinterpret_cast<uint32_t*>(workspace);
  P.scratch = ws + kStatusBytes;
  if (a8_native(M, N)) {
    P.a_bits = 8;
    P.act_scale = act_scale; P.post = post;
    P.residual = reinterpret_cast<const __nv_bfloat16*>(residual); P.res_scale = res_scale;
    P.Y = reinterpret_cast<__nv_bfloat16*>(Y); P.acc_out = acc_out;
    if (M <= 16) return gemm_decode_small_launch(st, reinterpret_cast<const uint8_t*>(Xq8), Wq, P);
    return gemm_pair_launch(st, reinterpret_cast<const uint8_t*>(Xq8), Wq, P);
  }
  // a = 16 h + l through two 4-bit matmuls
  uint8_t* Hq = ws + kStatusBytes + gemm_scratch_bytes(M);
  uint8_t* Lq = Hq + up256((size_t)M * K / 2);
  int32_t* acc_h = reinterpret_cast<int32_t*>(Lq + up256((size_t)M * K / 2));
  int32_t* acc_l = reinterpret_cast<int32_t*>(reinterpret_cast<uint8_t*>(acc_h) + up256((size_t)M * N * 4));
  const size_t chunks = (size_t)M * K / 16;
  split_a8_kernel<<<(unsigned)((chunks + 255) / 256), 256, 0, st>>>(reinterpret_cast<const uint4*>(Xq8),
                                                                     reinterpret_cast<uint2*>(Hq),
                                                                     reinterpret_cast<uint2*>(Lq), chunks);
  if (cudaGetLastError() != cudaSuccess) return FPT_ERR_CUDA;
  P.act_scale = 1.0f;
  P.acc_out = acc_h;
  int rc = gemm_launch(st, Hq, Wq, P);
  if (rc) return rc;
  P.acc_out = acc_l;
  P.a_unsigned = 1;                       // unsigned nibbles, zero point 0: no row-sum correction needed
  rc = gemm_launch(st, Lq, Wq, P);
  if (rc) return rc;
  CombineParams C;
  C.acc_h = acc_h; C.acc_l = acc_l; C.sw = sw; C.scale_dtype = scale_dtype;
  C.act_scale = act_scale; C.post = post;
  C.residual = reinterpret_cast<const __nv_bfloat16*>(residual); C.res_scale = res_scale;
  C.Y = reinterpret_cast<__nv_bfloat16*>(Y); C.acc_out = acc_out;
  C.M = M; C.N = N;
  const size_t groups = (size_t)M * (N / 8);
  combine_a8_kernel<<<(unsigned)((groups + 255) / 256), 256, 0, st>>>(C);
  return cudaGetLastError() == cudaSuccess ? FPT_OK : FPT_ERR_CUDA;
}
