// Online block-wise Hadamard transform at the down-projection input, fused with the per-token
// scale and the static INT4 quantiser (Sec. 3.1, last paragraph; App. A transform table:
// H_n = n^(-1/2) (x) [[1, 1], [1, -1]]; App. D "Hadamard non-powers of 2": groups of a
// power-of-two size, never zero padding).  Optionally the SwiGLU product is formed on the way in.
//
// One warp per (token, group of 256 * C channels).  A lane holds C chunks of 8 consecutive
// channels, chunk c of lane l being channels ((c * 32 + l) * 8 ...) of the group, so that loads
// and stores are fully coalesced.  The butterflies run in ascending distance, which is the order
// the result is defined in (each add / subtract rounded to float32): distances 1, 2, 4 inside a
// chunk, 8 ... 128 between lanes (shuffles), 256 ... inside the lane across its chunks; one
// multiply by float32(n^(-1/2)) follows, then (h * S_n) * (1/D) and the grid.
#include "fpt_internal.cuh"
#include "quant_math.cuh"

namespace fpt {

struct HadQuantParams {
  const uint4* X;        // [M, ldx] bf16: the products m, or gate||up in 64-column groups
  const float* s_in;     // [M] S_n or nullptr (1)
  uint32_t* Xq;          // [M, K/2] bytes as 32-bit words
  int M, K, ldx;         // K = channels after the product (d_ff)
  int silu_inter;        // 1: X holds gate||up (2K columns), m = bf16(silu(g) * u) is formed here
  float norm;            // float32(block^(-1/2))
  float inv_delta;
  int qmax_minus_z;
  uint32_t flip;
};

template <int C>
__global__ void __launch_bounds__(256) hadamard_quant_kernel(const HadQuantParams P) {
  constexpr int kBlock = 256 * C;
  pdl_wait();                                    // the products come from the matmul before this kernel
  pdl_launch_dependents();
  const int lane = threadIdx.x & 31;
  const int groups = P.K / kBlock;
  const long long wid = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (wid >= (long long)P.M * groups) return;
  const int t = (int)(wid / groups), grp = (int)(wid % groups);
  const uint4* row = P.X + (size_t)t * (size_t)(P.ldx >> 3);
  float x[C][8];
#pragma unroll
  for (int c = 0; c < C; ++c) {
    const int chunk = grp * (kBlock / 8) + c * 32 + lane;          // 16-byte chunk of the row of products
    uint4 v;
    if (P.silu_inter) {
      const int gc = ((chunk >> 3) << 4) + (chunk & 7);             // gate chunk; its up chunk is 8 further
      const uint4 g = __ldg(row + gc), u = __ldg(row + gc + 8);
      v.x = silu_mul_pair(g.x, u.x); v.y = silu_mul_pair(g.y, u.y);
      v.z = silu_mul_pair(g.z, u.z); v.w = silu_mul_pair(g.w, u.w);
    } else {
      v = __ldg(row + chunk);
    }
    x[c][0] = bf16lo_to_f32(v.x); x[c][1] = bf16hi_to_f32(v.x);
    x[c][2] = bf16lo_to_f32(v.y); x[c][3] = bf16hi_to_f32(v.y);
    x[c][4] = bf16lo_to_f32(v.z); x[c][5] = bf16hi_to_f32(v.z);
    x[c][6] = bf16lo_to_f32(v.w); x[c][7] = bf16hi_to_f32(v.w);
  }
  // distances 1, 2, 4: inside a chunk
#pragma unroll
  for (int s = 1; s < 8; s <<= 1)
#pragma unroll
    for (int c = 0; c < C; ++c)
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if ((i & s) == 0) {
          const float a = x[c][i], b = x[c][i + s];
          x[c][i] = __fadd_rn(a, b);
          x[c][i + s] = __fsub_rn(a, b);
        }
  // distances 8 ... 128: between lanes; the lane with the bit clear holds a and keeps a + b
#pragma unroll
  for (int m = 1; m < 32; m <<= 1) {
    const bool upper = (lane & m) != 0;
#pragma unroll
    for (int c = 0; c < C; ++c)
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float other = __shfl_xor_sync(0xffffffffu, x[c][i], m);
        x[c][i] = upper ? __fsub_rn(other, x[c][i]) : __fadd_rn(x[c][i], other);
      }
  }
  // distances 256 ...: between the chunks of a lane
#pragma unroll
  for (int s = 1; s < C; s <<= 1)
#pragma unroll
    for (int c = 0; c < C; ++c)
      if ((c & s) == 0)
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float a = x[c][i], b = x[c + s][i];
          x[c][i] = __fadd_rn(a, b);
          x[c + s][i] = __fsub_rn(a, b);
        }
  const float p = P.s_in ? __ldg(P.s_in + t) : 1.0f;
  const QuantConsts qc = quant_consts(p, P.inv_delta, P.qmax_minus_z, P.flip);
  uint32_t* out = P.Xq + (size_t)t * (size_t)(P.K >> 3) + grp * (kBlock / 8);
#pragma unroll
  for (int c = 0; c < C; ++c) {
#pragma unroll
    for (int i = 0; i < 8; ++i) x[c][i] = __fmul_rn(x[c][i], P.norm);
    out[c * 32 + lane] = quant_word_f32(x[c], qc);
  }
}

template <int C>
static cudaError_t launch_had(const HadQuantParams& P, cudaStream_t st) {
  const long long warps = (long long)P.M * (P.K / (256 * C));
  return launch_kernel(hadamard_quant_kernel<C>, dim3((unsigned)((warps + 7) / 8)), dim3(256), 0, st, true, P);
}

int hadamard_block(int K) { return K & (-K); }

// Validated arguments only.
cudaError_t hadamard_quant_launch(cudaStream_t st, const void* X, int M, int K, int ldx, const fpt_qparams* qp,
                                  int silu_inter, const float* s_in, uint8_t* Xq) {
  HadQuantParams P;
  P.X = reinterpret_cast<const uint4*>(X);
  P.s_in = s_in;
  P.Xq = reinterpret_cast<uint32_t*>(Xq);
  P.M = M; P.K = K; P.ldx = ldx;
  P.silu_inter = silu_inter;
  const int block = hadamard_block(K);
  P.norm = (float)(1.0 / sqrt((double)block));
  P.inv_delta = 1.0f / qp->scale;
  const int z = qp->symmetric ? 0 : qp->zero_point;
  P.qmax_minus_z = (qp->symmetric ? 7 : 15) - z;
  P.flip = qp->symmetric ? 0x77777777u : 0xFFFFFFFFu;
  switch (block) {
    case 256: return launch_had<1>(P, st);
    case 512: return launch_had<2>(P, st);
    case 1024: return launch_had<4>(P, st);
    case 2048: return launch_had<8>(P, st);
    case 4096: return launch_had<16>(P, st);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace fpt

extern "C" int fpt_hadamard_quant(void* stream, const void* X, int M, int K, int ldx, const fpt_qparams* qp, int flags,
                                  const float* s_in, uint8_t* Xq) {
  if (!X || !qp || !Xq || M <= 0 || K <= 0) return FPT_ERR_BAD_ARG;
  if (qp->bits != 4) return FPT_ERR_UNSUPPORTED;
  if (!(qp->scale > 0.0f)) return FPT_ERR_BAD_ARG;
  if (!qp->symmetric && (qp->zero_point < 0 || qp->zero_point > 15)) return FPT_ERR_BAD_ARG;
  if (flags & ~(FPT_SILU_MUL | FPT_GU_INTERLEAVED | FPT_SCALE_INPUT)) return FPT_ERR_BAD_ARG;
  const bool silu = flags & FPT_SILU_MUL, inter = flags & FPT_GU_INTERLEAVED;
  if (silu != inter) return FPT_ERR_UNSUPPORTED;                 // the product is formed from the interleaved layout only
  if ((flags & FPT_SCALE_INPUT) && !s_in) return FPT_ERR_BAD_ARG;
  const int block = fpt::hadamard_block(K);
  if (block < 256 || block > 4096) return FPT_ERR_UNSUPPORTED;
  const int need_ld = inter ? 2 * K : K;
  if (ldx < need_ld || ldx % 8 != 0) return FPT_ERR_ALIGNMENT;
  if (((uintptr_t)X | (uintptr_t)Xq) & 15) return FPT_ERR_ALIGNMENT;
  cudaError_t e = fpt::hadamard_quant_launch((cudaStream_t)stream, X, M, K, ldx, qp, inter ? 1 : 0,
                                             (flags & FPT_SCALE_INPUT) ? s_in : nullptr, Xq);
  return e == cudaSuccess ? FPT_OK : FPT_ERR_CUDA;
}
