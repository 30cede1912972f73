// The activation quantiser's two other forms: the dynamic variant (App. B "Dynamic quantization":
// per token, the extreme values are reduced over the row and the resulting scale factor is applied
// to every value -- the reduce-broadcast the paper's static set-up avoids) and 8-bit codes (the
// W4A8 setting of Sec. 4).  Same per-token multiplier p_t as the static step (Sec. 3.1.3).
//
// One CTA per token, the row held in registers across both reductions (sum of squares for the
// RMSNorm factor, largest magnitude for the grid), so the dynamic form reads the row once, like
// the static one; what it adds is the second block-wide reduction.
#include "fpt_internal.cuh"
#include "quant_math.cuh"

namespace fpt {

struct DynQuantParams {
  const uint4* X;        // [M, ldx] bf16
  const float* s_in;     // [M] or nullptr
  const float* post;     // [M] or nullptr: FPT_POST_VECTOR factor
  void*        Xq;       // 4 bits: [M, K/2] packed; 8 bits: [M, K] int8
  float*       s_out;    // [M] or nullptr          S_n
  float*       c_out;    // [M] or nullptr          dynamic: the epilogue's per-token factor; static: 1 / p_t
  float*       delta_out;// [M] or nullptr          dynamic: D_t
  float*       r_out;    // [M] or nullptr          r_t
  int M, K, ldx;
  int flags, post_mode, dynamic;
  float eps;
  float inv_delta;       // static: 1 / D rounded once on the host
};

// Largest bf16 magnitude pattern of a chunk, per 16-bit half (patterns order like magnitudes; Inf and
// NaN are the largest).
__device__ __forceinline__ uint32_t max_mag(const uint4& v, uint32_t acc) {
  acc = __vmaxu2(acc, v.x & 0x7FFF7FFFu);
  acc = __vmaxu2(acc, v.y & 0x7FFF7FFFu);
  acc = __vmaxu2(acc, v.z & 0x7FFF7FFFu);
  acc = __vmaxu2(acc, v.w & 0x7FFF7FFFu);
  return acc;
}

// clamp(rne((x * p) * inv), -128, 127), a NaN to -128; four codes per word.
__device__ __forceinline__ uint32_t quant8_pair(uint32_t w, float p, float inv, uint32_t prev) {
  const float u0 = __fmul_rn(__fmul_rn(bf16lo_to_f32(w), p), inv);
  const float u1 = __fmul_rn(__fmul_rn(bf16hi_to_f32(w), p), inv);
  int q0 = max(-128, min(127, __float2int_rn(u0)));      // the conversion saturates; NaN converts to 0
  int q1 = max(-128, min(127, __float2int_rn(u1)));
  if (u0 != u0) q0 = -128;
  if (u1 != u1) q1 = -128;
  return (prev >> 16) | ((uint32_t)(q0 & 0xFF) << 16) | ((uint32_t)(q1 & 0xFF) << 24);
}
__device__ __forceinline__ uint2 quant8_chunk(const uint4& v, float p, float inv) {
  uint2 o;
  o.x = quant8_pair(v.y, p, inv, quant8_pair(v.x, p, inv, 0u));
  o.y = quant8_pair(v.w, p, inv, quant8_pair(v.z, p, inv, 0u));
  return o;
}

template <int T, int V, int BITS>
__global__ void __launch_bounds__(T, V <= 4 ? 2048 / T : 1) act_quant_dyn_kernel(const DynQuantParams P) {
  __shared__ double warp_part[T / 32];
  __shared__ uint32_t warp_max[T / 32];
  __shared__ float bcast;
  __shared__ uint32_t bmax;
  pdl_wait();                                    // X may come from the kernel before this one
  pdl_launch_dependents();
  const int t = blockIdx.x, tid = threadIdx.x;
  const int chunks = P.K >> 3;
  const size_t row = (size_t)t * (size_t)(P.ldx >> 3);
  uint4 v[V];
#pragma unroll
  for (int i = 0; i < V; ++i) {
    const int c = i * T + tid;
    if (c < chunks) v[i] = __ldg(P.X + row + c);
  }
  // the two reductions; the sum of squares follows the static kernel step by step
  uint32_t mx = 0;
  double acc = 0.0;
#pragma unroll
  for (int i = 0; i < V; ++i)
    if (i * T + tid < chunks) { mx = max_mag(v[i], mx); if (P.flags & FPT_RMSNORM) acc = sumsq(v[i], acc); }
  mx = max(mx & 0xFFFFu, mx >> 16);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    acc += __shfl_xor_sync(0xffffffffu, acc, o);
  }
  if ((tid & 31) == 0) { warp_part[tid >> 5] = acc; warp_max[tid >> 5] = mx; }
  __syncthreads();
  if (tid == 0) {
    double s = 0.0; uint32_t m = 0;
#pragma unroll
    for (int w = 0; w < T / 32; ++w) { s += warp_part[w]; m = max(m, warp_max[w]); }
    bcast = (float)s; bmax = m;
  }
  __syncthreads();
  const uint32_t amax_bits = bmax;
  float r = 1.0f;
  if (P.flags & FPT_RMSNORM) {
    if (!(bcast <= 3.4028234e38f)) {               // Inf / NaN in the row (or a genuine overflow): by the definition
      __syncthreads();
      acc = 0.0;
#pragma unroll
      for (int i = 0; i < V; ++i)
        if (i * T + tid < chunks) acc = sumsq_exact(v[i], acc);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
      if ((tid & 31) == 0) warp_part[tid >> 5] = acc;
    }
    __syncthreads();
    if (tid == 0) {
      double s = 0.0;
#pragma unroll
      for (int w = 0; w < T / 32; ++w) s += warp_part[w];
      const float ss = (float)s;                                        // one rounding to float32
      const float ms = __fdiv_rn(ss, (float)P.K);
      const float rho = __fsqrt_rn(__fadd_rn(ms, P.eps));
      bcast = __fdiv_rn(1.0f, rho);
    }
    __syncthreads();
    r = bcast;
  }
  const float s = P.s_in ? __ldg(P.s_in + t) : 1.0f;
  const float rs = P.s_in ? __fmul_rn(r, s) : r;
  const float p = (P.flags & FPT_SCALE_INPUT) ? rs : r;
  constexpr float kQmax = BITS == 8 ? 127.0f : 7.0f;
  float delta = 1.0f, inv = P.inv_delta;
  if (P.dynamic) {
    // max_k |x * p| = |max_k |x| * p|: rounding is monotone, so the largest input gives the largest product
    const float m = fabsf(__fmul_rn(__uint_as_float(amax_bits << 16), p));
    if (m > 0.0f && m <= 3.4028234e38f) delta = __fdiv_rn(m, kQmax);     // zero, Inf and NaN rows: D_t = 1
    inv = __fdiv_rn(1.0f, delta);
  }
  if (tid == 0) {
    if (P.s_out) P.s_out[t] = rs;
    if (P.r_out) P.r_out[t] = r;
    if (P.delta_out) P.delta_out[t] = delta;
    if (P.c_out) {
      const float pinv = __fdiv_rn(1.0f, p);
      if (!P.dynamic) P.c_out[t] = pinv;
      else P.c_out[t] = P.post_mode == FPT_POST_NONE ? delta
                      : P.post_mode == FPT_POST_INVERSE_OF_PRE ? __fmul_rn(delta, pinv)
                                                              : __fmul_rn(delta, __ldg(P.post + t));
    }
  }
  if (BITS == 4) {
    uint32_t* out = reinterpret_cast<uint32_t*>(P.Xq) + (size_t)t * (size_t)chunks;
    const QuantConsts qc = quant_consts(p, inv, 7, 0x77777777u);
#pragma unroll
    for (int i = 0; i < V; ++i) {
      const int c = i * T + tid;
      if (c < chunks) out[c] = quant_word(v[i], qc);
    }
  } else {
    uint2* out = reinterpret_cast<uint2*>(P.Xq) + (size_t)t * (size_t)chunks;
#pragma unroll
    for (int i = 0; i < V; ++i) {
      const int c = i * T + tid;
      if (c < chunks) out[c] = quant8_chunk(v[i], p, inv);
    }
  }
}

template <int T, int V>
static cudaError_t launch(const DynQuantParams& P, int bits, cudaStream_t st) {
  if (bits == 8) return launch_kernel(act_quant_dyn_kernel<T, V, 8>, dim3(P.M), dim3(T), 0, st, true, P);
  return launch_kernel(act_quant_dyn_kernel<T, V, 4>, dim3(P.M), dim3(T), 0, st, true, P);
}

// bits 4: dynamic only (the static 4-bit grid has its own kernels); bits 8: static (dynamic = 0,
// qp_scale = D) or dynamic.  All arguments already validated.
cudaError_t act_quant_dyn_launch(cudaStream_t st, const void* X, int M, int K, int ldx, int bits, int dynamic,
                                 float qp_scale, int flags, float eps, const float* s_in, int post_mode,
                                 const float* post, void* Xq, float* s_out, float* c_out, float* delta_out,
                                 float* r_out) {
  DynQuantParams P;
  P.X = reinterpret_cast<const uint4*>(X);
  P.s_in = s_in; P.post = post; P.Xq = Xq;
  P.s_out = s_out; P.c_out = c_out; P.delta_out = delta_out; P.r_out = r_out;
  P.M = M; P.K = K; P.ldx = ldx;
  P.flags = flags; P.post_mode = post_mode; P.dynamic = dynamic;
  P.eps = eps;
  P.inv_delta = dynamic ? 1.0f : 1.0f / qp_scale;
  const int chunks = K / 8;
  if (chunks <= 128)        return launch<128, 1>(P, bits, st);
  else if (chunks <= 256)   return launch<128, 2>(P, bits, st);
  else if (chunks <= 512)   return launch<128, 4>(P, bits, st);
  else if (chunks <= 1024)  return launch<256, 4>(P, bits, st);
  else if (chunks <= 2048)  return launch<512, 4>(P, bits, st);
  else if (chunks <= 4096)  return launch<512, 8>(P, bits, st);
  else if (chunks <= 8192)  return launch<1024, 8>(P, bits, st);
  return cudaErrorInvalidValue;
}

}  // namespace fpt

extern "C" int fpt_act_quant_dynamic(void* stream, const void* X, int M, int K, int ldx, int bits, int flags,
                                     float eps, const float* s_in, void* Xq, float* s_out, float* delta_out) {
  if (!X || !Xq || !delta_out || M <= 0 || K <= 0) return FPT_ERR_BAD_ARG;
  if (bits != 4 && bits != 8) return FPT_ERR_UNSUPPORTED;
  if (K % 32 != 0 || K > 65536) return FPT_ERR_UNSUPPORTED;
  if (flags & ~(FPT_RMSNORM | FPT_SCALE_INPUT)) return FPT_ERR_UNSUPPORTED;
  if ((flags & FPT_SCALE_INPUT) && !s_in) return FPT_ERR_BAD_ARG;
  if (ldx < K || ldx % 8 != 0) return FPT_ERR_ALIGNMENT;
  if (((uintptr_t)X | (uintptr_t)Xq) & 15) return FPT_ERR_ALIGNMENT;
  cudaError_t e = fpt::act_quant_dyn_launch((cudaStream_t)stream, X, M, K, ldx, bits, 1, 1.0f, flags, eps, s_in,
                                            FPT_POST_NONE, nullptr, Xq, s_out, nullptr, delta_out, nullptr);
  return e == cudaSuccess ? FPT_OK : FPT_ERR_CUDA;
}
