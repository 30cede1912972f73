// Step (1) of the path: RMSNorm-derived per-token scale + static INT4 quantise + pack
// (Sec. 3.1.3, Eq. 6-7; App. B "Static quantization"), and the SiLU*mul variant that
// feeds the down projection.  Memory-bound: one CTA per token, the row is read once
// with 128-bit loads, kept in registers across the reduction, and written as packed
// nibbles.
#include "fpt_internal.cuh"

namespace fpt {

struct ActQuantParams {
  const uint4* X;      // [M, ldx] bf16
  const uint4* X2;     // SILU_MUL second operand (same layout) or nullptr
  const float* s_in;   // [M] or nullptr
  uint32_t*    Xq;     // [M, K/2] bytes, written as 32-bit words (8 codes each)
  float*       s_out;  // [M] or nullptr          S_n
  float*       post_inv;  // [M] or nullptr       1 / p_t
  float*       r_out;  // [M] or nullptr          r_t
  int M, K, ldx;       // elements
  int flags;
  float eps;
  float inv_delta;     // 1 / D, rounded once on the host
  float lo, hi;        // qmin - z, qmax - z
  float magic;         // 1.5 * 2^23 + z
};

// 2^f on [-0.5, 0.5]: degree-6 Taylor coefficients (ln 2)^k / k!, rounded to float32.
__device__ __forceinline__ float exp2_spec(float t) {
  t = fminf(fmaxf(t, -126.0f), 126.0f);
  const float n = rintf(t);
  const float f = __fsub_rn(t, n);
  float a = 0x1.430912p-13f;                               // (ln2)^6 / 720
  a = __fadd_rn(__fmul_rn(a, f), 0x1.5d87fep-10f);         // (ln2)^5 / 120
  a = __fadd_rn(__fmul_rn(a, f), 0x1.3b2ab6p-7f);          // (ln2)^4 / 24
  a = __fadd_rn(__fmul_rn(a, f), 0x1.c6b08ep-5f);          // (ln2)^3 / 6
  a = __fadd_rn(__fmul_rn(a, f), 0x1.ebfbep-3f);           // (ln2)^2 / 2
  a = __fadd_rn(__fmul_rn(a, f), 0x1.62e43p-1f);           // ln2
  a = __fadd_rn(__fmul_rn(a, f), 1.0f);
  const float two_n = __int_as_float(((int)n + 127) << 23);
  return __fmul_rn(a, two_n);
}

__device__ __forceinline__ float silu_spec(float g) {
  const float e = exp2_spec(__fmul_rn(-g, 0x1.715476p+0f));   // log2(e)
  return __fdiv_rn(g, __fadd_rn(1.0f, e));
}

// bf16(silu(g) * u) for a packed pair of bf16 values.
__device__ __forceinline__ uint32_t silu_mul_pair(uint32_t g, uint32_t u) {
  const float lo = __fmul_rn(silu_spec(bf16lo_to_f32(g)), bf16lo_to_f32(u));
  const float hi = __fmul_rn(silu_spec(bf16hi_to_f32(g)), bf16hi_to_f32(u));
  return f32_to_bf16_bits(lo) | (f32_to_bf16_bits(hi) << 16);
}

__device__ __forceinline__ uint32_t quant_nibble(float x, float p, const ActQuantParams& P) {
  float u = __fmul_rn(__fmul_rn(x, p), P.inv_delta);
  u = fminf(fmaxf(u, P.lo), P.hi);                           // NaN -> lo
  return __float_as_uint(__fadd_rn(u, P.magic)) & 0xFu;      // rne(u) + z in the low mantissa bits
}

__device__ __forceinline__ uint32_t quant_word(const uint4& v, float p, const ActQuantParams& P) {
  uint32_t w;
  w  = quant_nibble(bf16lo_to_f32(v.x), p, P);
  w |= quant_nibble(bf16hi_to_f32(v.x), p, P) << 4;
  w |= quant_nibble(bf16lo_to_f32(v.y), p, P) << 8;
  w |= quant_nibble(bf16hi_to_f32(v.y), p, P) << 12;
  w |= quant_nibble(bf16lo_to_f32(v.z), p, P) << 16;
  w |= quant_nibble(bf16hi_to_f32(v.z), p, P) << 20;
  w |= quant_nibble(bf16lo_to_f32(v.w), p, P) << 24;
  w |= quant_nibble(bf16hi_to_f32(v.w), p, P) << 28;
  return w;
}

__device__ __forceinline__ double sumsq(const uint4& v, double acc) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float a = bf16lo_to_f32(w[i]), b = bf16hi_to_f32(w[i]);
    acc += (double)__fmul_rn(a, a);            // the square of a bf16 value is exact in float32
    acc += (double)__fmul_rn(b, b);
  }
  return acc;
}

// T threads per token, up to V 16-byte chunks (8 elements) per thread held in registers.
template <int T, int V>
__global__ void __launch_bounds__(T) act_quant_kernel(const ActQuantParams P) {
  __shared__ double warp_part[T / 32];
  __shared__ float  bcast;
  const int t = blockIdx.x;
  const int tid = threadIdx.x;
  const int chunks = P.K >> 3;                   // 16-byte chunks per row
  const size_t row = (size_t)t * (size_t)(P.ldx >> 3);
  const bool silu = (P.flags & FPT_SILU_MUL) != 0;
  const bool inter = (P.flags & FPT_GU_INTERLEAVED) != 0;

  uint4 v[V];
#pragma unroll
  for (int i = 0; i < V; ++i) {
    const int c = i * T + tid;
    if (c < chunks) {
      if (!silu) {
        v[i] = __ldg(P.X + row + c);
      } else {
        // gate column of logical chunk c: groups of 16 chunks (128 columns), gate then up
        const int gc = inter ? ((c >> 4) << 5) + (c & 15) : c;
        const uint4 g = __ldg(P.X + row + gc);
        const uint4 u = inter ? __ldg(P.X + row + gc + 16) : __ldg(P.X2 + row + c);
        v[i].x = silu_mul_pair(g.x, u.x);
        v[i].y = silu_mul_pair(g.y, u.y);
        v[i].z = silu_mul_pair(g.z, u.z);
        v[i].w = silu_mul_pair(g.w, u.w);
      }
    }
  }

  float r = 1.0f;
  if (P.flags & FPT_RMSNORM) {
    double acc = 0.0;
#pragma unroll
    for (int i = 0; i < V; ++i)
      if (i * T + tid < chunks) acc = sumsq(v[i], acc);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if ((tid & 31) == 0) warp_part[tid >> 5] = acc;
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
  if (tid == 0) {
    if (P.s_out) P.s_out[t] = rs;
    if (P.post_inv) P.post_inv[t] = __fdiv_rn(1.0f, p);
    if (P.r_out) P.r_out[t] = r;
  }
  uint32_t* out = P.Xq + (size_t)t * (size_t)chunks;
#pragma unroll
  for (int i = 0; i < V; ++i) {
    const int c = i * T + tid;
    if (c < chunks) out[c] = quant_word(v[i], p, P);
  }
}

template <int T, int V>
static cudaError_t launch(const ActQuantParams& P, cudaStream_t st) {
  act_quant_kernel<T, V><<<P.M, T, 0, st>>>(P);
  return cudaGetLastError();
}

// Internal entry shared by the public functions (also fills post_inv / r_out for the
// composed calls).  All arguments already validated.
cudaError_t act_quant_launch(cudaStream_t st, const void* X, int M, int K, int ldx, const fpt_qparams* qp,
                             int flags, float eps, const void* X2, const float* s_in, uint8_t* Xq,
                             float* s_out, float* post_inv, float* r_out) {
  ActQuantParams P;
  P.X = reinterpret_cast<const uint4*>(X);
  P.X2 = reinterpret_cast<const uint4*>(X2);
  P.s_in = s_in;
  P.Xq = reinterpret_cast<uint32_t*>(Xq);
  P.s_out = s_out;
  P.post_inv = post_inv;
  P.r_out = r_out;
  P.M = M; P.K = K; P.ldx = ldx;
  P.flags = flags;
  P.eps = eps;
  P.inv_delta = 1.0f / qp->scale;
  const int z = qp->symmetric ? 0 : qp->zero_point;
  const int qmin = qp->symmetric ? -8 : 0, qmax = qp->symmetric ? 7 : 15;
  P.lo = (float)(qmin - z);
  P.hi = (float)(qmax - z);
  P.magic = 12582912.0f + (float)z;
  const int chunks = K / 8;
  if (chunks <= 128)        return launch<128, 1>(P, st);
  else if (chunks <= 256)   return launch<128, 2>(P, st);
  else if (chunks <= 512)   return launch<256, 2>(P, st);
  else if (chunks <= 1024)  return launch<256, 4>(P, st);
  else if (chunks <= 2048)  return launch<512, 4>(P, st);
  else if (chunks <= 4096)  return launch<512, 8>(P, st);
  else if (chunks <= 8192)  return launch<1024, 8>(P, st);
  return cudaErrorInvalidValue;
}

}  // namespace fpt

extern "C" int fpt_act_quant(void* stream, const void* X, int M, int K, int ldx, const fpt_qparams* qp,
                             int flags, float eps, const void* X2, const float* s_in, uint8_t* Xq,
                             float* s_out) {
  if (!X || !qp || !Xq || M <= 0 || K <= 0) return FPT_ERR_BAD_ARG;
  if (qp->bits != 4) return FPT_ERR_UNSUPPORTED;
  if (!(qp->scale > 0.0f)) return FPT_ERR_BAD_ARG;
  if (!qp->symmetric && (qp->zero_point < 0 || qp->zero_point > 15)) return FPT_ERR_BAD_ARG;
  if (K % 32 != 0 || K > 65536) return FPT_ERR_UNSUPPORTED;
  const bool silu = flags & FPT_SILU_MUL, inter = flags & FPT_GU_INTERLEAVED;
  if (flags & ~(FPT_RMSNORM | FPT_SCALE_INPUT | FPT_SILU_MUL | FPT_GU_INTERLEAVED)) return FPT_ERR_BAD_ARG;
  if (inter && !silu) return FPT_ERR_BAD_ARG;
  if (silu && (flags & FPT_RMSNORM)) return FPT_ERR_UNSUPPORTED;
  if (silu && !inter && !X2) return FPT_ERR_BAD_ARG;
  if (inter && K % 128 != 0) return FPT_ERR_UNSUPPORTED;
  if ((flags & FPT_SCALE_INPUT) && !s_in) return FPT_ERR_BAD_ARG;
  const int need_ld = inter ? 2 * K : K;
  if (ldx < need_ld || ldx % 8 != 0) return FPT_ERR_ALIGNMENT;
  if (((uintptr_t)X | (uintptr_t)Xq | (uintptr_t)X2) & 15) return FPT_ERR_ALIGNMENT;
  cudaError_t e = fpt::act_quant_launch((cudaStream_t)stream, X, M, K, ldx, qp, flags, eps, X2, s_in, Xq,
                                        s_out, nullptr, nullptr);
  return e == cudaSuccess ? FPT_OK : FPT_ERR_CUDA;
}
