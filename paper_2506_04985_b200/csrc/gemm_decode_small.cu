// Steps (2)+(3) of the path for at most 16 tokens: the same exact INT32 matmul (App. J "Setup")
// and scale-factor epilogue (App. B "Static quantization"), where the only cost that matters is
// reading the packed weights once from HBM -- and, for a transfer of a few microseconds, how
// soon after launch the first byte is requested and how soon after the last byte the kernel ends.
//
// So this kernel has no staging at all: one CTA per 16 weight rows, its warps take alternate
// 64-byte column blocks of those rows, every lane loads 16 packed bytes of two rows straight
// into registers (four lanes cover 64 contiguous bytes of a row), widens the nibbles to int8
// (code * 16, as everywhere) and feeds them to mma.sync m16n8k32 with the tokens as the N side.
// Any fixed permutation of k inside a block is harmless as long as both operands use it: the
// activation fragment is the same 16 bytes of the token's row widened by the same function.
// The activations (a few KB) are read through L1 by every warp.  Warps add their partial
// accumulators through shared memory -- integers, so the order does not matter.
//
// The tensor-memory kernel of gemm_decode.cu keeps the sizes from 17 to 64 tokens: with four or
// eight token groups this form was measured 1.5 to 2.5 times slower than that kernel (registers,
// re-widening the activations per group, legacy-MMA issue rate).
#include "fpt_internal.cuh"

namespace fpt {
namespace decode_small {

constexpr int kRows = 16;                  // weight rows per CTA = M of the MMA

struct Params {
  GemmParams g;
  int ntiles;                              // token groups of 8: 1 or 2
  int kblocks;                             // 64-byte packed blocks per row: K / 128
};

// C[16x8] += A[16x32] * B[32x8], int8 operands (B signed or unsigned), int32 accumulators.
template <bool kBUnsigned>
__device__ __forceinline__ void mma_16x8x32(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                            uint32_t b0, uint32_t b1) {
  if (kBUnsigned)
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  else
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// int8 activation codes (one byte each): 32 codes of a token in the byte order the widening gives the
// weights (16 even-k codes, then 16 odd-k codes), not multiplied by 16.
__device__ __forceinline__ void gather_i8(const uint4& lo, const uint4& hi, uint32_t* out) {
  const uint32_t a[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
#pragma unroll
  for (int w = 0; w < 4; ++w) {
    out[w] = __byte_perm(a[2 * w], a[2 * w + 1], 0x6420);
    out[4 + w] = __byte_perm(a[2 * w], a[2 * w + 1], 0x7531);
  }
}

// kA8: Xq holds int8 codes [M, K] instead of packed 4-bit codes [M, K/2] (signed, kBUnsigned = false).
// U: 64-byte blocks in flight per warp; kMinCtas: CTAs per SM the register allocation must allow.
template <int NW, int NT, bool kBUnsigned, bool kA8 = false, int U = 4, int kMinCtas = 768 / (NW * 32)>
__global__ void __launch_bounds__(NW * 32, kMinCtas) gemm_w4a4_decode_small_kernel(const uint8_t* __restrict__ Xq,
                                                                          const uint8_t* __restrict__ Wq, const Params D) {
  __shared__ int part[NW][kRows][8 * NT];
  pdl_wait();                      // the activation codes come from the kernel before this one
  pdl_launch_dependents();
  const GemmParams& P = D.g;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int n0 = blockIdx.x * kRows;
  const size_t row_bytes = (size_t)P.K / 2;
  // rows past the end of the matrix and tokens past M are read from a valid row and masked to zero
  const int ra = n0 + g, rb = n0 + g + 8;
  const bool ra_ok = ra < P.N, rb_ok = rb < P.N;
  const uint8_t* wa = Wq + (size_t)(ra_ok ? ra : 0) * row_bytes + 16 * t;
  const uint8_t* wb = Wq + (size_t)(rb_ok ? rb : 0) * row_bytes + 16 * t;
  const uint8_t* xr[NT];
  bool x_ok[NT];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    const int tok = nt * 8 + g;
    x_ok[nt] = tok < P.M;
    xr[nt] = Xq + (size_t)(x_ok[nt] ? tok : 0) * row_bytes * (kA8 ? 2 : 1) + (kA8 ? 32 : 16) * t;
  }
  int acc[NT][4];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[nt][j] = 0;
  // what the epilogue needs from global memory, requested now so that it has arrived by then
  // (output o = weight row o % 16 of token o / 16; a thread finishes outputs tid, tid + blockDim, ...)
  constexpr int kOut = kRows * 8 * NT, kPer = (kOut + NW * 32 - 1) / (NW * 32);
  float o_sw[kPer], o_ct[kPer], o_rs[kPer], o_res[kPer];
  int o_zw[kPer];
  bool o_ok[kPer];
#pragma unroll
  for (int q = 0; q < kPer; ++q) {
    const int o = threadIdx.x + q * NW * 32;
    const int o_n = n0 + o % kRows, o_tok = o / kRows;
    o_ok[q] = o < kOut && o_n < P.N && o_tok < P.M;
    o_sw[q] = 0.0f; o_ct[q] = P.act_scale; o_rs[q] = 1.0f; o_res[q] = 0.0f; o_zw[q] = 0;
    if (o_ok[q]) {
      o_sw[q] = load_scale(P.sw, P.scale_dtype, o_n);
      if (P.wsum) o_zw[q] = P.zero_point * __ldg(P.wsum + o_n);
      if (P.post) o_ct[q] = __fmul_rn(P.act_scale, __ldg(P.post + o_tok));
      if (P.residual) {
        o_res[q] = __bfloat162float(P.residual[(size_t)o_tok * P.N + o_n]);
        if (P.res_scale) o_rs[q] = __ldg(P.res_scale + o_tok);
      }
    }
  }

  const uint4 zero = make_uint4(0, 0, 0, 0);
  for (int b0 = warp; b0 < D.kblocks; b0 += NW * U) {
    uint4 pa[U], pb[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int b = b0 + u * NW;
      if (b < D.kblocks) {
        pa[u] = __ldcs(reinterpret_cast<const uint4*>(wa + (size_t)b * 64));      // streamed once: evict first
        pb[u] = __ldcs(reinterpret_cast<const uint4*>(wb + (size_t)b * 64));
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int b = b0 + u * NW;
      if (b < D.kblocks) {
        uint32_t a[8], c[8];
        widen(ra_ok ? pa[u] : zero, a);
        widen(rb_ok ? pb[u] : zero, c);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          uint32_t x[8];
          if constexpr (kA8) {
            const uint4 p0 = __ldg(reinterpret_cast<const uint4*>(xr[nt] + (size_t)b * 128));
            const uint4 p1 = __ldg(reinterpret_cast<const uint4*>(xr[nt] + (size_t)b * 128 + 16));
            gather_i8(x_ok[nt] ? p0 : zero, x_ok[nt] ? p1 : zero, x);
          } else {
            const uint4 px = __ldg(reinterpret_cast<const uint4*>(xr[nt] + (size_t)b * 64));
            widen(x_ok[nt] ? px : zero, x);
          }
#pragma unroll
          for (int j = 0; j < 4; ++j)
            mma_16x8x32<kBUnsigned>(acc[nt], a[2 * j], c[2 * j], a[2 * j + 1], c[2 * j + 1], x[2 * j], x[2 * j + 1]);
        }
      }
    }
  }
  // accumulator fragment: c0 (row g, token 2t), c1 (row g, token 2t+1), c2 / c3 the same for row g + 8
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    part[warp][g][nt * 8 + 2 * t] = acc[nt][0];
    part[warp][g][nt * 8 + 2 * t + 1] = acc[nt][1];
    part[warp][g + 8][nt * 8 + 2 * t] = acc[nt][2];
    part[warp][g + 8][nt * 8 + 2 * t + 1] = acc[nt][3];
  }
  __syncthreads();
  // consecutive threads take consecutive weight rows of one token
#pragma unroll
  for (int q = 0; q < kPer; ++q) {
    if (!o_ok[q]) continue;
    const int o = threadIdx.x + q * NW * 32;
    const int o_r = o % kRows, o_tok = o / kRows;
    int s = 0;
#pragma unroll
    for (int w = 0; w < NW; ++w) s += part[w][o_r][o_tok];
    const int a = (s >> (kA8 ? 4 : 8)) - o_zw[q];
    const size_t idx = (size_t)o_tok * P.N + n0 + o_r;
    if (P.acc_out) P.acc_out[idx] = a;
    if (P.Y) {
      float y = __fmul_rn(__fmul_rn((float)a, o_sw[q]), o_ct[q]);
      if (P.residual) y = __fadd_rn(y, __fmul_rn(o_res[q], o_rs[q]));
      P.Y[idx] = __float2bfloat16_rn(y);
    }
  }
}

template <int NW, int NT, int U = 4, int kMinCtas = 768 / (NW * 32)>
static int launch(cudaStream_t st, const uint8_t* Xq, const uint8_t* Wq, const Params& D) {
  const int grid = (D.g.N + kRows - 1) / kRows;
  cudaError_t e;
  if (D.g.a_bits == 8)
    e = launch_kernel(gemm_w4a4_decode_small_kernel<NW, NT, false, true>, dim3(grid), dim3(NW * 32), 0, st, true, Xq, Wq, D);
  else if (D.g.a_unsigned)
    e = launch_kernel(gemm_w4a4_decode_small_kernel<NW, NT, true, false, U, kMinCtas>, dim3(grid), dim3(NW * 32), 0, st, true, Xq, Wq, D);
  else
    e = launch_kernel(gemm_w4a4_decode_small_kernel<NW, NT, false, false, U, kMinCtas>, dim3(grid), dim3(NW * 32), 0, st, true, Xq, Wq, D);
  return e == cudaSuccess ? FPT_OK : FPT_ERR_CUDA;
}

}  // namespace decode_small

// Xq [M <= 16, K/2], Wq [N, K/2]; needs no scratch.
int gemm_decode_small_launch(cudaStream_t st, const uint8_t* Xq, const uint8_t* Wq, const GemmParams& P) {
  using namespace decode_small;
  Params D;
  D.g = P;
  D.ntiles = (P.M + 7) / 8;
  D.kblocks = P.K / 128;
  // few row strips (a short, wide matrix): more warps per strip, so that enough loads are in flight; two such
  // CTAs per SM (at most 64 registers, two blocks in flight per warp), so that 256 strips are all resident at
  // once instead of 148 and then 108 (4096 x 14336: 10.8 -> 8.2 us at one token; 8192 x 28672: 33.7 -> 26.2 us)
  const bool wide = (P.N + kRows - 1) / kRows < 600;
  if (D.ntiles == 1) return wide ? launch<16, 1, 2, 2>(st, Xq, Wq, D) : launch<8, 1>(st, Xq, Wq, D);
  return wide ? launch<16, 2, 2, 2>(st, Xq, Wq, D) : launch<8, 2>(st, Xq, Wq, D);
}

}  // namespace fpt
