// Offline weight quantiser: per-output-channel symmetric INT4 grid, round-to-nearest,
// min-max or L_p range setting (Sec. 4 "Quantization Setup"; App. D "Quantizer range
// setting"), packed two codes per byte (App. J).  Not on the timed path: one CTA per row.
#include "fpt_common.cuh"

namespace fpt {

constexpr int kWqThreads = 256;

template <typename T> __device__ __forceinline__ float wload(const T* p, size_t i);
template <> __device__ __forceinline__ float wload<__nv_bfloat16>(const __nv_bfloat16* p, size_t i) { return __bfloat162float(p[i]); }
template <> __device__ __forceinline__ float wload<float>(const float* p, size_t i) { return p[i]; }

__device__ __forceinline__ float store_round(float d, int scale_dtype) {
  return scale_dtype == FPT_DTYPE_F16 ? __half2float(__float2half_rn(d)) : d;
}

__device__ __forceinline__ int quant_code(float w, float d) {
  float u = rintf(__fdiv_rn(w, d));
  u = fminf(fmaxf(u, -8.0f), 7.0f);              // NaN -> -8
  return (int)u;
}

template <typename V>
__device__ __forceinline__ V block_reduce(V v, V* scratch, bool is_max) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const V other = __shfl_xor_sync(0xffffffffu, v, o);
    v = is_max ? (other > v ? other : v) : v + other;
  }
  __syncthreads();                                // scratch may still be read from the last call
  if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
  __syncthreads();
  V r = scratch[0];
  for (int w = 1; w < kWqThreads / 32; ++w) r = is_max ? (scratch[w] > r ? scratch[w] : r) : r + scratch[w];
  return r;
}

template <typename T>
__global__ void __launch_bounds__(kWqThreads) weight_quant_kernel(const T* __restrict__ W, int N, int K, int range_mode,
                                                                  float p, int scale_dtype, uint8_t* __restrict__ Wq,
                                                                  void* __restrict__ sw, int32_t* __restrict__ wsum) {
  __shared__ double scratch_d[kWqThreads / 32];
  __shared__ float scratch_f[kWqThreads / 32];
  __shared__ int scratch_i[kWqThreads / 32];
  const int n = blockIdx.x;
  const size_t base = (size_t)n * (size_t)K;
  const int tid = threadIdx.x;

  float a = 0.0f;
  for (int k = tid; k < K; k += kWqThreads) a = fmaxf(a, fabsf(wload(W, base + k)));
  a = block_reduce<float>(a, scratch_f, true);

  float delta = store_round(__fdiv_rn(a, 7.0f), scale_dtype);
  if (a == 0.0f || delta == 0.0f) delta = 1.0f;
  if (range_mode == FPT_RANGE_LP) {
    double best = 1.0 / 0.0;   // +inf
    for (int i = 20; i <= 100; ++i) {
      const float frac = __fdiv_rn((float)i, 100.0f);
      float d = store_round(__fdiv_rn(__fmul_rn(a, frac), 7.0f), scale_dtype);
      if (a == 0.0f || d == 0.0f) d = 1.0f;
      double err = 0.0;
      for (int k = tid; k < K; k += kWqThreads) {
        const float w = wload(W, base + k);
        const double e = fabs((double)w - (double)d * (double)quant_code(w, d));
        err += pow(e, (double)p);
      }
      err = block_reduce<double>(err, scratch_d, false);
      if (err <= best) { best = err; delta = d; }
    }
  }
  if (tid == 0) {
    if (scale_dtype == FPT_DTYPE_F16) reinterpret_cast<__half*>(sw)[n] = __float2half_rn(delta);
    else reinterpret_cast<float*>(sw)[n] = delta;
  }
  int sum = 0;
  uint8_t* out = Wq + (size_t)n * (size_t)(K / 2);
  for (int j = tid; j < K / 2; j += kWqThreads) {
    const int q0 = quant_code(wload(W, base + 2 * j), delta);
    const int q1 = quant_code(wload(W, base + 2 * j + 1), delta);
    sum += q0 + q1;
    out[j] = (uint8_t)((q0 & 0xF) | ((q1 & 0xF) << 4));
  }
  if (wsum) {
    sum = block_reduce<int>(sum, scratch_i, false);
    if (tid == 0) wsum[n] = sum;
  }
}

}  // namespace fpt

extern "C" int fpt_quantize_weights(void* stream, const void* W, int w_dtype, int N, int K, const fpt_qparams* qp,
                                    int range_mode, float p, int scale_dtype, uint8_t* Wq, void* sw, int32_t* wsum) {
  if (!W || !qp || !Wq || !sw || N <= 0 || K <= 0) return FPT_ERR_BAD_ARG;
  if (qp->bits != 4 || !qp->symmetric) return FPT_ERR_UNSUPPORTED;
  if (K % 32 != 0) return FPT_ERR_UNSUPPORTED;
  if (w_dtype != FPT_DTYPE_BF16 && w_dtype != FPT_DTYPE_F32) return FPT_ERR_BAD_ARG;
  if (scale_dtype != FPT_DTYPE_F32 && scale_dtype != FPT_DTYPE_F16) return FPT_ERR_BAD_ARG;
  if (range_mode != FPT_RANGE_MINMAX && range_mode != FPT_RANGE_LP) return FPT_ERR_BAD_ARG;
  if (range_mode == FPT_RANGE_LP && !(p > 0.0f)) return FPT_ERR_BAD_ARG;
  if (((uintptr_t)W | (uintptr_t)Wq | (uintptr_t)sw) & 15) return FPT_ERR_ALIGNMENT;
  cudaStream_t st = (cudaStream_t)stream;
  if (w_dtype == FPT_DTYPE_BF16)
    fpt::weight_quant_kernel<__nv_bfloat16><<<N, fpt::kWqThreads, 0, st>>>(
        reinterpret_cast<const __nv_bfloat16*>(W), N, K, range_mode, p, scale_dtype, Wq, sw, wsum);
  else
    fpt::weight_quant_kernel<float><<<N, fpt::kWqThreads, 0, st>>>(reinterpret_cast<const float*>(W), N, K,
                                                                    range_mode, p, scale_dtype, Wq, sw, wsum);
  return cudaGetLastError() == cudaSuccess ? FPT_OK : FPT_ERR_CUDA;
}

extern "C" int fpt_interleave_gate_up(void* stream, const uint8_t* Wg_q, const uint8_t* Wu_q, const void* sw_g,
                                      const void* sw_u, int scale_dtype, int d_ff, int K, uint8_t* Wgu_q,
                                      void* sw_gu) {
  if (!Wg_q || !Wu_q || !sw_g || !sw_u || !Wgu_q || !sw_gu || d_ff <= 0 || K <= 0) return FPT_ERR_BAD_ARG;
  if (d_ff % 64 != 0 || K % 32 != 0) return FPT_ERR_UNSUPPORTED;
  if (scale_dtype != FPT_DTYPE_F32 && scale_dtype != FPT_DTYPE_F16) return FPT_ERR_BAD_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t row = (size_t)K / 2, grp = 64 * row;           // bytes of 64 packed rows
  const size_t sgrp = 64 * (scale_dtype == FPT_DTYPE_F16 ? 2 : 4);
  const size_t groups = (size_t)d_ff / 64;
  cudaError_t e;
  e = cudaMemcpy2DAsync(Wgu_q, 2 * grp, Wg_q, grp, grp, groups, cudaMemcpyDeviceToDevice, st);
  if (e == cudaSuccess) e = cudaMemcpy2DAsync(Wgu_q + grp, 2 * grp, Wu_q, grp, grp, groups, cudaMemcpyDeviceToDevice, st);
  if (e == cudaSuccess) e = cudaMemcpy2DAsync(sw_gu, 2 * sgrp, sw_g, sgrp, sgrp, groups, cudaMemcpyDeviceToDevice, st);
  if (e == cudaSuccess)
    e = cudaMemcpy2DAsync((char*)sw_gu + sgrp, 2 * sgrp, sw_u, sgrp, sgrp, groups, cudaMemcpyDeviceToDevice, st);
  return e == cudaSuccess ? FPT_OK : FPT_ERR_CUDA;
}
