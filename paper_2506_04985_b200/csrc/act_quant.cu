// Step (1) of the path: RMSNorm-derived per-token scale + static INT4 quantise + pack
// (Sec. 3.1.3, Eq. 6-7; App. B "Static quantization"), and the SiLU*mul variant that
// feeds the down projection.  Memory-bound: one CTA per token, the row is read once
// with 128-bit loads, kept in registers across the reduction, and written as packed
// nibbles.
#include "fpt_internal.cuh"
#include "quant_math.cuh"

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
  int   qmax_minus_z;  // upper end of the grid minus the zero point
  uint32_t flip;       // see quant_word
};

// T threads per token, up to V 16-byte chunks (8 elements) per thread held in registers.
template <int T, int V>
__global__ void __launch_bounds__(T, V <= 4 ? 2048 / T : 1) act_quant_kernel(const ActQuantParams P) {
  __shared__ double warp_part[T / 32];
  __shared__ float  bcast;
  pdl_wait();                                    // X may come from the kernel before this one
  pdl_launch_dependents();
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
        // gate column of logical chunk c: groups of 8 chunks (64 columns), gate then up
        const int gc = inter ? ((c >> 3) << 4) + (c & 7) : c;
        const uint4 g = __ldg(P.X + row + gc);
        const uint4 u = inter ? __ldg(P.X + row + gc + 8) : __ldg(P.X2 + row + c);
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
      bcast = (float)s;
    }
    __syncthreads();
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
  if (tid == 0) {
    if (P.s_out) P.s_out[t] = rs;
    if (P.post_inv) P.post_inv[t] = __fdiv_rn(1.0f, p);
    if (P.r_out) P.r_out[t] = r;
  }
  uint32_t* out = P.Xq + (size_t)t * (size_t)chunks;
  const QuantConsts qc = quant_consts(p, P.inv_delta, P.qmax_minus_z, P.flip);
#pragma unroll
  for (int i = 0; i < V; ++i) {
    const int c = i * T + tid;
    if (c < chunks) out[c] = quant_word(v[i], qc);
  }
}

// One warp per token for rows of up to 256 * V elements: the row lives in registers, the
// reduction is a warp shuffle, no shared memory and no block-wide barrier.  W warps per CTA.
template <int V, int W>
__global__ void __launch_bounds__(W * 32) act_quant_warp_kernel(const ActQuantParams P) {
  pdl_wait();
  pdl_launch_dependents();
  const int lane = threadIdx.x & 31;
  const int t = blockIdx.x * W + (threadIdx.x >> 5);
  if (t >= P.M) return;
  const int chunks = P.K >> 3;
  const uint4* row = P.X + (size_t)t * (size_t)(P.ldx >> 3);
  uint4 v[V];
#pragma unroll
  for (int i = 0; i < V; ++i) {
    const int c = i * 32 + lane;
    if (c < chunks) v[i] = __ldg(row + c);
  }
  float r = 1.0f;
  if (P.flags & FPT_RMSNORM) {
    double acc0 = 0.0, acc1 = 0.0;                 // two chains: the float64 adds are latency-bound otherwise
#pragma unroll
    for (int i = 0; i < V; ++i)
      if (i * 32 + lane < chunks) { if (i & 1) acc1 = sumsq(v[i], acc1); else acc0 = sumsq(v[i], acc0); }
    double acc = acc0 + acc1;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (!((float)acc <= 3.4028234e38f)) {          // Inf / NaN in the row (or a genuine overflow): by the definition
      acc0 = 0.0;
#pragma unroll
      for (int i = 0; i < V; ++i)
        if (i * 32 + lane < chunks) acc0 = sumsq_exact(v[i], acc0);
      acc = acc0;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    }
    const float ss = (float)acc;                   // one rounding to float32 (every lane holds the same sum)
    const float ms = __fdiv_rn(ss, (float)P.K);
    const float rho = __fsqrt_rn(__fadd_rn(ms, P.eps));
    r = __fdiv_rn(1.0f, rho);
  }
  const float s = P.s_in ? __ldg(P.s_in + t) : 1.0f;
  const float rs = P.s_in ? __fmul_rn(r, s) : r;
  const float p = (P.flags & FPT_SCALE_INPUT) ? rs : r;
  if (lane == 0) {
    if (P.s_out) P.s_out[t] = rs;
    if (P.post_inv) P.post_inv[t] = __fdiv_rn(1.0f, p);
    if (P.r_out) P.r_out[t] = r;
  }
  uint32_t* out = P.Xq + (size_t)t * (size_t)chunks;
  const QuantConsts qc = quant_consts(p, P.inv_delta, P.qmax_minus_z, P.flip);
#pragma unroll
  for (int i = 0; i < V; ++i) {
    const int c = i * 32 + lane;
    if (c < chunks) out[c] = quant_word(v[i], qc);
  }
}

// Persistent streaming version of the same: one CTA per SM, W warps, each warp walks over its
// tokens with its own row buffer(s) in shared memory, filled by a bulk copy; while one warp waits
// for its next row the others compute, so the HBM stream and the arithmetic overlap.  The row is read from
// shared memory twice (sum of squares, then quantise); nothing is held in registers.
// A wait on a row that does not arrive within about two seconds makes the warp stop (its
// remaining tokens stay unwritten); nothing can be reported from here, the entry point has no
// status word.
__global__ void __launch_bounds__(1024) act_quant_stream_kernel(const ActQuantParams P, int W, int NB, uint32_t row_bytes) {
  extern __shared__ __align__(128) uint8_t smem_aq[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint8_t* buf0 = smem_aq + (size_t)(warp * NB) * row_bytes;
  const uint32_t bars = smem_u32(smem_aq + (size_t)(W * NB) * row_bytes) + (uint32_t)warp * 16u;
  if (lane == 0) { mbar_init(bars, 1); mbar_init(bars + 8, 1); }
  fence_mbar_init();
  __syncthreads();
  pdl_wait();
  pdl_launch_dependents();
  const int chunks = P.K >> 3;
  const long long stride = (long long)gridDim.x * W;
  const long long first = (long long)warp * gridDim.x + blockIdx.x;
  const uint8_t* X = reinterpret_cast<const uint8_t*>(P.X);
  const size_t ld_bytes = (size_t)P.ldx * 2;
  if (lane == 0) {
    for (int b = 0; b < NB; ++b) {
      const long long t = first + b * stride;
      if (t < P.M) {
        mbar_arrive_expect_tx(bars + 8 * b, row_bytes);
        bulk_load_1d(smem_u32(buf0 + (size_t)b * row_bytes), X + (size_t)t * ld_bytes, row_bytes, bars + 8 * b);
      }
    }
  }
  int it = 0;
  for (long long t = first; t < P.M; t += stride, ++it) {
    const int b = NB == 2 ? (it & 1) : 0; const uint32_t ph = (NB == 2 ? (it >> 1) : it) & 1;
    {
      const uint64_t t0 = globaltimer_ns();
      bool ok = true;
      while (!mbar_try_wait(bars + 8 * b, ph)) {
        if (globaltimer_ns() - t0 > kWaitLimitNs) { ok = false; break; }
      }
      if (!__all_sync(0xffffffffu, ok)) return;
    }
    const uint4* row = reinterpret_cast<const uint4*>(buf0 + (size_t)b * row_bytes);
    float r = 1.0f;
    if (P.flags & FPT_RMSNORM) {
      double acc0 = 0.0, acc1 = 0.0;
      int c = lane;
      for (; c + 32 < chunks; c += 64) { acc0 = sumsq(row[c], acc0); acc1 = sumsq(row[c + 32], acc1); }
      if (c < chunks) acc0 = sumsq(row[c], acc0);
      double acc = acc0 + acc1;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
      if (!((float)acc <= 3.4028234e38f)) {        // Inf / NaN in the row (or a genuine overflow): by the definition
        acc = 0.0;
        for (int c2 = lane; c2 < chunks; c2 += 32) acc = sumsq_exact(row[c2], acc);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
      }
      const float ss = (float)acc;                 // one rounding to float32
      const float ms = __fdiv_rn(ss, (float)P.K);
      const float rho = __fsqrt_rn(__fadd_rn(ms, P.eps));
      r = __fdiv_rn(1.0f, rho);
    }
    const float s = P.s_in ? __ldg(P.s_in + t) : 1.0f;
    const float rs = P.s_in ? __fmul_rn(r, s) : r;
    const float p = (P.flags & FPT_SCALE_INPUT) ? rs : r;
    if (lane == 0) {
      if (P.s_out) P.s_out[t] = rs;
      if (P.post_inv) P.post_inv[t] = __fdiv_rn(1.0f, p);
      if (P.r_out) P.r_out[t] = r;
    }
    uint32_t* out = P.Xq + (size_t)t * (size_t)chunks;
    const QuantConsts qc = quant_consts(p, P.inv_delta, P.qmax_minus_z, P.flip);
#pragma unroll 4
    for (int c = lane; c < chunks; c += 32) out[c] = quant_word(row[c], qc);
    __syncwarp();                                  // every lane is done with the buffer
    const long long tn = t + NB * stride;
    if (lane == 0 && tn < P.M) {
      fence_proxy_async_smem();                    // our reads of the buffer come before the copy's writes
      mbar_arrive_expect_tx(bars + 8 * b, row_bytes);
      bulk_load_1d(smem_u32(buf0 + (size_t)b * row_bytes), X + (size_t)tn * ld_bytes, row_bytes, bars + 8 * b);
    }
  }
}

static cudaError_t launch_stream(const ActQuantParams& P, cudaStream_t st) {
  static PerDeviceInt attr_set;
  if (!ensure_smem_attr(attr_set, act_quant_stream_kernel, 220 * 1024)) return cudaErrorInvalidValue;
  const int sms = device_sm_count();
  // as many warps as row buffers fit (each warp needs at least one); two buffers per warp when
  // 32 warps leave room for them
  const uint32_t row_bytes = (uint32_t)P.K * 2;
  const int fit = (int)((200u * 1024u) / row_bytes);
  const int NB = fit >= 64 ? 2 : 1;
  int wmax = fit / NB;
  if (wmax > 32) wmax = 32;
  const int grid = P.M < sms ? P.M : sms;
  // warps per CTA: of the counts that fit, the one that leaves the fewest idle slots in the last
  // round of tokens (a CTA gets about M / grid tokens, its warps take them in turns)
  const int per_cta = (P.M + grid - 1) / grid;
  int W = wmax; double best = 0.0;
  for (int w = wmax; w >= 4 && 10 * w >= 7 * wmax; --w) {       // fewer warps also means less latency hiding
    const int rounds = (per_cta + w - 1) / w;
    const double eff = (double)per_cta / ((double)w * rounds);
    if (eff > best + 0.1) { best = eff; W = w; }
  }
  const size_t smem = (size_t)W * NB * row_bytes + (size_t)W * 16;
  return launch_kernel(act_quant_stream_kernel, dim3(grid), dim3(W * 32), smem, st, true, P, W, NB, row_bytes);
}

template <int V, int W>
static cudaError_t launch_warp(const ActQuantParams& P, cudaStream_t st) {
  return launch_kernel(act_quant_warp_kernel<V, W>, dim3((P.M + W - 1) / W), dim3(W * 32), 0, st, true, P);
}

template <int T, int V>
static cudaError_t launch(const ActQuantParams& P, cudaStream_t st) {
  return launch_kernel(act_quant_kernel<T, V>, dim3(P.M), dim3(T), 0, st, true, P);
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
  const int qmax = qp->symmetric ? 7 : 15;
  P.qmax_minus_z = qmax - z;
  P.flip = qp->symmetric ? 0x77777777u : 0xFFFFFFFFu;
  const int chunks = K / 8;
  // Many tokens: long rows do best with one CTA per token and many CTAs per SM (measured: 2048 x 8192 in
  // 13 us against 19 us for the streaming kernel); short rows with the persistent streaming kernel
  // (16384 x 2048: 20 us against 23 us).
  if (!(flags & FPT_SILU_MUL) && M >= 512) {
    if (chunks >= 128 && chunks < 512) return launch_stream(P, st);
    if (chunks == 512) return launch<128, 4>(P, st);
    if (chunks > 512 && chunks <= 1024) return launch<256, 4>(P, st);
    if (chunks > 1024 && chunks <= 2048) return launch<512, 4>(P, st);
  }
  if (!(flags & FPT_SILU_MUL)) {
    if (chunks <= 64)        return launch_warp<2, 4>(P, st);
    else if (chunks <= 128)  return launch_warp<4, 4>(P, st);
    else if (chunks <= 256)  return launch_warp<8, 4>(P, st);
    else if (chunks <= 512)  return launch_warp<16, 4>(P, st);
    else if (chunks <= 1024) return launch_warp<32, 4>(P, st);
  }
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
  if (qp->bits == 8) {          // int8 codes [M, K] on the symmetric grid (W4A8); Xq then has K bytes per row
    if (!qp->symmetric || (flags & ~(FPT_RMSNORM | FPT_SCALE_INPUT))) return FPT_ERR_UNSUPPORTED;
    if (!(qp->scale > 0.0f) || ((flags & FPT_SCALE_INPUT) && !s_in)) return FPT_ERR_BAD_ARG;
    if (K % 32 != 0 || K > 65536) return FPT_ERR_UNSUPPORTED;
    if (ldx < K || ldx % 8 != 0 || (((uintptr_t)X | (uintptr_t)Xq) & 15)) return FPT_ERR_ALIGNMENT;
    cudaError_t e8 = fpt::act_quant_dyn_launch((cudaStream_t)stream, X, M, K, ldx, 8, 0, qp->scale, flags, eps, s_in,
                                               FPT_POST_NONE, nullptr, Xq, s_out, nullptr, nullptr, nullptr);
    return e8 == cudaSuccess ? FPT_OK : FPT_ERR_CUDA;
  }
  if (qp->bits != 4) return FPT_ERR_UNSUPPORTED;
  if (!(qp->scale > 0.0f)) return FPT_ERR_BAD_ARG;
  if (!qp->symmetric && (qp->zero_point < 0 || qp->zero_point > 15)) return FPT_ERR_BAD_ARG;
  if (K % 32 != 0 || K > 65536) return FPT_ERR_UNSUPPORTED;
  const bool silu = flags & FPT_SILU_MUL, inter = flags & FPT_GU_INTERLEAVED;
  if (flags & ~(FPT_RMSNORM | FPT_SCALE_INPUT | FPT_SILU_MUL | FPT_GU_INTERLEAVED)) return FPT_ERR_BAD_ARG;
  if (inter && !silu) return FPT_ERR_BAD_ARG;
  if (silu && (flags & FPT_RMSNORM)) return FPT_ERR_UNSUPPORTED;
  if (silu && !inter && !X2) return FPT_ERR_BAD_ARG;
  if (inter && K % 64 != 0) return FPT_ERR_UNSUPPORTED;
  if ((flags & FPT_SCALE_INPUT) && !s_in) return FPT_ERR_BAD_ARG;
  const int need_ld = inter ? 2 * K : K;
  if (ldx < need_ld || ldx % 8 != 0) return FPT_ERR_ALIGNMENT;
  if (((uintptr_t)X | (uintptr_t)Xq | (uintptr_t)X2) & 15) return FPT_ERR_ALIGNMENT;
  cudaError_t e = fpt::act_quant_launch((cudaStream_t)stream, X, M, K, ldx, qp, flags, eps, X2, s_in, Xq,
                                        s_out, nullptr, nullptr);
  return e == cudaSuccess ? FPT_OK : FPT_ERR_CUDA;
}
