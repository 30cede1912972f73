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

// The same transform for groups of 2048 channels (d_ff = 14336 = 7 x 2048) with the lane-crossing
// stages taken off the shuffle unit: a lane first holds 64 CONSECUTIVE channels (brought in by
// coalesced loads and redistributed through shared memory), so the stages of distance 1 ... 32 are
// butterflies between its own registers; one transpose through shared memory (16 wide stores and
// 32 loads per lane instead of 320 shuffles) then gives it channels
// {64 l + 2 lane, 64 l + 2 lane + 1 : l = 0..31}, and the stages of distance 64 ... 1024 are again
// between its own registers, two channels per packed instruction.  The order of the stages and the
// operands of every add and subtract are those of the definition, so the codes are the same.
// The codes return through the same shared-memory tile (a byte of two codes per lane and l) so that
// the packed row leaves in full 128-byte lines.
constexpr int kTrStride = 68;                        // floats per transposed row: 16-byte stores of 8 lanes hit 8 bank groups
constexpr int kTrWarp = 32 * kTrStride;              // floats per warp

// kTwo: groups of 4096 channels, two warps per group: each warp does the above for its half, then the
// halves meet in the last stage (distance 2048) through the same tile -- warp 0 keeps a + b, warp 1 a - b.
template <bool kSilu, bool kTwo = false>
__global__ void __launch_bounds__(256, 3) hadamard2048_quant_kernel(const HadQuantParams P) {
  extern __shared__ __align__(16) float tr_all[];
  pdl_wait();                                    // the products come from the matmul before this kernel
  pdl_launch_dependents();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int groups = P.K >> (kTwo ? 12 : 11);
  const int half = kTwo ? (warp & 1) : 0;        // which 2048 channels of a 4096-channel group
  const long long wid = kTwo ? (long long)blockIdx.x * 4 + (warp >> 1) : (long long)blockIdx.x * 8 + warp;
  if (wid >= (long long)P.M * groups) return;    // (both warps of a group leave together; no CTA-wide barrier)
  const int t = (int)(wid / groups);
  const int grp = (int)(wid % groups) * (kTwo ? 2 : 1) + half;     // in units of 2048 channels
  const uint4* row = P.X + (size_t)t * (size_t)(P.ldx >> 3);
  float* tr = tr_all + warp * kTrWarp;
  // The group's 256 chunks of 8 channels arrive in fully coalesced loads (lane l takes chunks
  // 32 j + l) and are parked in the tile; then every lane picks up ITS 64 consecutive channels
  // (chunks 8 l ... 8 l + 7).  Chunk c sits at row c / 8, position (c % 8) ^ (row % 8): both the
  // stores and the loads of a quarter warp then cover all eight 16-byte bank groups.
  uint4* stage = reinterpret_cast<uint4*>(tr);
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int c = 32 * j + lane;                 // chunk of the group
    uint4 v;
    if (kSilu) {
      // products chunk grp * 256 + c: its gate chunk, the up chunk 8 further
      const int pc = grp * 256 + c;
      const uint4* g = row + ((pc >> 3) << 4) + (pc & 7);
      const uint4 gv = __ldg(g), uv = __ldg(g + 8);
      v.x = silu_mul_pair(gv.x, uv.x); v.y = silu_mul_pair(gv.y, uv.y);
      v.z = silu_mul_pair(gv.z, uv.z); v.w = silu_mul_pair(gv.w, uv.w);
    } else {
      v = __ldg(row + grp * 256 + c);
    }
    const int r = c >> 3;
    stage[r * 8 + ((c & 7) ^ (r & 7))] = v;
  }
  __syncwarp();
  float x[64];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const uint4 v = stage[lane * 8 + (j ^ (lane & 7))];
    x[8 * j + 0] = bf16lo_to_f32(v.x); x[8 * j + 1] = bf16hi_to_f32(v.x);
    x[8 * j + 2] = bf16lo_to_f32(v.y); x[8 * j + 3] = bf16hi_to_f32(v.y);
    x[8 * j + 4] = bf16lo_to_f32(v.z); x[8 * j + 5] = bf16hi_to_f32(v.z);
    x[8 * j + 6] = bf16lo_to_f32(v.w); x[8 * j + 7] = bf16hi_to_f32(v.w);
  }
  __syncwarp();                                  // the tile is reused for the transpose below
  // distance 1
#pragma unroll
  for (int i = 0; i < 64; i += 2) {
    const float a = x[i], b = x[i + 1];
    x[i] = __fadd_rn(a, b);
    x[i + 1] = __fsub_rn(a, b);
  }
  // distances 2 ... 32, two butterflies per instruction
#pragma unroll
  for (int s = 2; s < 64; s <<= 1)
#pragma unroll
    for (int i = 0; i < 64; i += 2)
      if ((i & s) == 0) {
        const uint64_t a = pack_f32x2(x[i], x[i + 1]), b = pack_f32x2(x[i + s], x[i + s + 1]);
        unpack_f32x2(add_f32x2(a, b), x[i], x[i + 1]);
        unpack_f32x2(sub_f32x2(a, b), x[i + s], x[i + s + 1]);
      }
  // transpose: row `lane` of the tile <- this lane's 64 values; then column pair `lane` of every row
#pragma unroll
  for (int j = 0; j < 16; ++j)
    *reinterpret_cast<float4*>(tr + lane * kTrStride + 4 * j) = make_float4(x[4 * j], x[4 * j + 1], x[4 * j + 2], x[4 * j + 3]);
  __syncwarp();
#pragma unroll
  for (int l = 0; l < 32; ++l) {
    const float2 v = *reinterpret_cast<const float2*>(tr + l * kTrStride + 2 * lane);
    x[2 * l] = v.x; x[2 * l + 1] = v.y;          // channels 64 l + 2 lane, 64 l + 2 lane + 1
  }
  // distances 64 ... 1024: between rows l and l + d
#pragma unroll
  for (int d = 1; d < 32; d <<= 1)
#pragma unroll
    for (int l = 0; l < 32; ++l)
      if ((l & d) == 0) {
        const uint64_t a = pack_f32x2(x[2 * l], x[2 * l + 1]), b = pack_f32x2(x[2 * (l + d)], x[2 * (l + d) + 1]);
        unpack_f32x2(add_f32x2(a, b), x[2 * l], x[2 * l + 1]);
        unpack_f32x2(sub_f32x2(a, b), x[2 * (l + d)], x[2 * (l + d) + 1]);
      }
  if constexpr (kTwo) {
    // distance 2048: channel c of the first half with channel c of the second.  Each warp parks its
    // 64 values per lane in its own tile (word 32 j + lane), the pair meets at a named barrier, reads
    // the partner's values, and meets again before the tiles are reused for the codes.
    __syncwarp();                                // every lane has read the transposed tile
#pragma unroll
    for (int j = 0; j < 64; ++j) tr[32 * j + lane] = x[j];
    named_bar_sync(1 + (warp >> 1), 64);
    const float* other = tr_all + (warp ^ 1) * kTrWarp;
#pragma unroll
    for (int j = 0; j < 64; ++j) {
      const float y = other[32 * j + lane];
      x[j] = half ? __fsub_rn(y, x[j]) : __fadd_rn(x[j], y);
    }
    named_bar_sync(1 + (warp >> 1), 64);
  }
  const float p = P.s_in ? __ldg(P.s_in + t) : 1.0f;
  const QuantConsts qc = quant_consts(p, P.inv_delta, P.qmax_minus_z, P.flip);
  __syncwarp();                                  // every lane has read the tile before it is overwritten
  uint8_t* bytes = reinterpret_cast<uint8_t*>(tr);
  const uint64_t norm2 = pack_f32x2(P.norm, P.norm);
#pragma unroll
  for (int l = 0; l < 32; ++l)                   // h = x * norm, then the quantiser: two codes per byte
    bytes[l * 36 + lane] = (uint8_t)((quant_pair_f32_pre(pack_f32x2(x[2 * l], x[2 * l + 1]), norm2, qc, 0u) ^ qc.flip) & 0xFFu);
  __syncwarp();
  uint32_t* out = P.Xq + (size_t)t * (size_t)(P.K >> 3) + grp * 256;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int w = i * 32 + lane;                 // word w: codes of channels 8 w ... 8 w + 7 = row w / 8, bytes 4 (w % 8) ...
    out[w] = *reinterpret_cast<const uint32_t*>(bytes + (w >> 3) * 36 + 4 * (w & 7));
  }
}

template <bool kSilu, bool kTwo>
static cudaError_t launch_had_tr(const HadQuantParams& P, cudaStream_t st) {
  const long long warps = (long long)P.M * (P.K / 2048);          // 8 per CTA either way
  const size_t smem = (size_t)8 * kTrWarp * sizeof(float);
  static PerDeviceInt attr;
  if (!ensure_smem_attr(attr, hadamard2048_quant_kernel<kSilu, kTwo>, (int)smem)) return cudaErrorInvalidValue;
  return launch_kernel(hadamard2048_quant_kernel<kSilu, kTwo>, dim3((unsigned)((warps + 7) / 8)), dim3(256), smem, st, true, P);
}

static cudaError_t launch_had2048(const HadQuantParams& P, cudaStream_t st) {
  return P.silu_inter ? launch_had_tr<true, false>(P, st) : launch_had_tr<false, false>(P, st);
}
static cudaError_t launch_had4096(const HadQuantParams& P, cudaStream_t st) {
  return P.silu_inter ? launch_had_tr<true, true>(P, st) : launch_had_tr<false, true>(P, st);
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
    case 2048: return launch_had2048(P, st);
    case 4096: return launch_had4096(P, st);
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
