// Steps (2)+(3) of the path: packed-INT4 x packed-INT4 matmul with an exact INT32
// accumulator (App. J "Setup") and the floating-point scale factors applied after it
// (App. B "Static quantization").
//
// Persistent, warp-specialised kernel, one CTA per SM:
//   warp 0      TMA producer: packed nibble tiles (64 bytes per row and k-block) global -> shared
//   warps 6..   converters:   nibbles -> int8 (code * 16) written in the 128-byte-swizzled K-major
//                             layout the tensor core reads
//   warp 1      MMA issuer:   tcgen05.mma kind::i8 into one of two TMEM accumulators
//   warps 2..5  epilogue:     tcgen05.ld, >> 8, scales, bf16, global stores (overlaps the next tile)
//
// Both operands are expanded as code*16 (a nibble moved to the top of its byte is the
// two's complement int8 of 16*code), so the accumulator holds 256 * sum(qa*qw); the
// epilogue shifts it back, exactly.  |256*acc| <= 256*128*K < 2^31 for K <= 65535.
// The 8 codes of a packed 32-bit word are split into the four even and the four odd
// ones; activations and weights use the same split, so the dot product is unchanged.
#include <cuda.h>

#include "fpt_internal.cuh"

namespace fpt {

constexpr int BM = 128;             // rows of the MMA "A" operand per tile
constexpr int BK = 128;             // codes per k-block: 64 packed bytes, 128 int8 bytes per row
constexpr int PK_ROW = BK / 2;
constexpr int I8_ROW = BK;
constexpr int kEpiWarps = 4;
constexpr int kFirstConvWarp = 2 + kEpiWarps;

template <int BN, int NI8, int NPK>
struct SmemLayout {
  static constexpr int kI8Stage = (BM + BN) * I8_ROW;
  static constexpr int kPkStage = (BM + BN) * PK_ROW;
  static constexpr int kI8Off = 0;
  static constexpr int kPkOff = kI8Off + NI8 * kI8Stage;
  static constexpr int kSwOff = kPkOff + NPK * kPkStage;             // 2 x BN floats
  static constexpr int kWsumOff = kSwOff + 2 * BN * 4;               // 2 x BN ints
  static constexpr int kBarOff = kWsumOff + 2 * BN * 4;
  static constexpr int kNumBars = 2 * NPK + 2 * NI8 + 6;
  static constexpr int kMiscOff = kBarOff + kNumBars * 8;            // tmem ptr, abort flag
  static constexpr int kBytes = kMiscOff + 16;
  static constexpr int kAlloc = kBytes + 1024;                       // slack to align the base to 1024
};

__device__ __forceinline__ void expand_nibbles(const uint4& p, uint4& even, uint4& odd) {
  uint32_t w[8];
  widen(p, w);
  even = make_uint4(w[0], w[1], w[2], w[3]);
  odd = make_uint4(w[4], w[5], w[6], w[7]);
}

template <int BN, int NI8, int NPK, int NCONV>
__global__ void __launch_bounds__((kFirstConvWarp + NCONV) * 32, 1)
gemm_w4a4_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const GemmParams P) {
  using L = SmemLayout<BN, NI8, NPK>;
  constexpr uint32_t kTmemCols = (2 * BN <= 32) ? 32 : (2 * BN <= 64) ? 64 : (2 * BN <= 128) ? 128
                                 : (2 * BN <= 256) ? 256 : 512;
  extern __shared__ uint8_t smem_raw[];
  // aligned to 1024 bytes by an offset on the shared-memory array itself (a round trip through an
  // integer would leave a generic pointer: generic loads and stores, and no way for the compiler to
  // tell shared from global accesses apart)
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bar0 = sbase + L::kBarOff;
  auto pk_full = [&](int s) { return bar0 + 8u * s; };
  auto pk_empty = [&](int s) { return bar0 + 8u * (NPK + s); };
  auto i8_full = [&](int s) { return bar0 + 8u * (2 * NPK + s); };
  auto i8_empty = [&](int s) { return bar0 + 8u * (2 * NPK + NI8 + s); };
  auto acc_full = [&](int s) { return bar0 + 8u * (2 * NPK + 2 * NI8 + s); };
  auto acc_empty = [&](int s) { return bar0 + 8u * (2 * NPK + 2 * NI8 + 2 + s); };
  auto sw_full = [&](int s) { return bar0 + 8u * (2 * NPK + 2 * NI8 + 4 + s); };
  volatile uint32_t* misc = reinterpret_cast<volatile uint32_t*>(smem + L::kMiscOff);
  volatile uint32_t* abort_flag = misc + 1;
  float* sw_s = reinterpret_cast<float*>(smem + L::kSwOff);
  int* wsum_s = reinterpret_cast<int*>(smem + L::kWsumOff);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < NPK; ++s) { mbar_init(pk_full(s), 1); mbar_init(pk_empty(s), NCONV); }
    for (int s = 0; s < NI8; ++s) { mbar_init(i8_full(s), NCONV); mbar_init(i8_empty(s), 1); }
    for (int s = 0; s < 2; ++s) {
      mbar_init(acc_full(s), 1);
      mbar_init(acc_empty(s), kEpiWarps);
      mbar_init(sw_full(s), kEpiWarps);
    }
    misc[1] = 0;
    fence_mbar_init();
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmB);
  }
  if (warp == 1) {
    tmem_alloc(sbase + L::kMiscOff, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = misc[0];
  pdl_wait();                      // nothing above touched memory another kernel may write
  pdl_launch_dependents();

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int s = 0; uint32_t ph = 0;
      uint32_t armed = 0, armed_par = 0;          // per stage: a copy was issued / parity of its phase
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < P.num_tiles; tile += gridDim.x) {
        const int m0 = (tile % P.tiles_m) * BM, n0 = (tile / P.tiles_m) * BN;
        for (int kb = 0; kb < P.kblocks; ++kb) {
          if (!mbar_wait(pk_empty(s), ph ^ 1u, abort_flag, P.status, 1)) { ok = false; break; }
          mbar_arrive_expect_tx(pk_full(s), L::kPkStage);
          const uint32_t dst = sbase + L::kPkOff + s * L::kPkStage;
          tma_load_2d(dst, &tmA, pk_full(s), kb * PK_ROW, m0);
          tma_load_2d(dst + BM * PK_ROW, &tmB, pk_full(s), kb * PK_ROW, n0);
          armed |= 1u << s;
          armed_par = (armed_par & ~(1u << s)) | (ph << s);
          if (++s == NPK) { s = 0; ph ^= 1u; }
        }
      }
      if (!ok) {
        // bounded wait for the copies still in flight before this CTA's shared memory goes away
        const uint64_t t0 = globaltimer_ns();
        for (int q = 0; q < NPK; ++q)
          if (armed & (1u << q))
            while (!mbar_try_wait(pk_full(q), (armed_par >> q) & 1u) && globaltimer_ns() - t0 < 2000000ull) {}
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_i8(BM, BN, !P.a_unsigned, true);
      int s = 0; uint32_t ph = 0; int it = 0;
      for (int tile = blockIdx.x; tile < P.num_tiles; tile += gridDim.x, ++it) {
        const int as = it & 1; const uint32_t aph = (it >> 1) & 1;
        if (!mbar_wait(acc_empty(as), aph ^ 1u, abort_flag, P.status, 2)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + as * BN;
        bool ok = true;
        for (int kb = 0; kb < P.kblocks; ++kb) {
          if (!mbar_wait(i8_full(s), ph, abort_flag, P.status, 3)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = sbase + L::kI8Off + s * L::kI8Stage;
          const uint64_t adesc = umma_desc_kmajor_sw128(a_addr);
          const uint64_t bdesc = umma_desc_kmajor_sw128(a_addr + BM * I8_ROW);
#pragma unroll
          for (int kk = 0; kk < BK / 32; ++kk)
            umma_i8(d_tmem, adesc + 2u * kk, bdesc + 2u * kk, idesc, (kb | kk) != 0);
          umma_commit(i8_empty(s));
          if (++s == NI8) { s = 0; ph ^= 1u; }
        }
        if (!ok) break;
        umma_commit(acc_full(as));
      }
    }
  } else if (warp < kFirstConvWarp) {
    // ------------------------------------------------------------------ epilogue
    const int quad = warp & 3;                      // TMEM lane quadrant this warp may read
    const int etid = (warp - 2) * 32 + lane;
    int it = 0;
    for (int tile = blockIdx.x; tile < P.num_tiles; tile += gridDim.x, ++it) {
      const int as = it & 1; const uint32_t aph = (it >> 1) & 1;
      const int m0 = (tile % P.tiles_m) * BM, n0 = (tile / P.tiles_m) * BN;
      for (int j = etid; j < BN; j += kEpiWarps * 32) {
        const int n = n0 + j;
        sw_s[as * BN + j] = n < P.N ? load_scale(P.sw, P.scale_dtype, n) : 0.0f;
        wsum_s[as * BN + j] = (P.wsum && n < P.N) ? P.zero_point * P.wsum[n] : 0;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(sw_full(as));
      if (!mbar_wait(sw_full(as), aph, abort_flag, P.status, 7)) break;
      if (!mbar_wait(acc_full(as), aph, abort_flag, P.status, 4)) break;
      tc_fence_after();
      const int row = m0 + quad * 32 + lane;
      const bool row_ok = row < P.M;
      float c = P.act_scale, rs = 1.0f;
      if (row_ok && P.post) c = __fmul_rn(P.act_scale, __ldg(P.post + row));
      if (row_ok && P.res_scale) rs = __ldg(P.res_scale + row);
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + as * BN;
      const size_t rowoff = (size_t)row * (size_t)P.N;
#pragma unroll 1
      for (int ch = 0; ch < BN / 32; ++ch) {
        uint32_t v[32];
        tmem_ld_32x32(taddr + ch * 32, v);
        tmem_wait_ld();
        const int col0 = n0 + ch * 32;
        if (row_ok) {
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            const int col = col0 + g * 8;
            if (col < P.N) {
              int a[8];
#pragma unroll
              for (int j = 0; j < 8; ++j)
                a[j] = (((int)v[g * 8 + j]) >> 8) - wsum_s[as * BN + ch * 32 + g * 8 + j];
              if (P.acc_out) {
                int4* o = reinterpret_cast<int4*>(P.acc_out + rowoff + col);
                o[0] = make_int4(a[0], a[1], a[2], a[3]);
                o[1] = make_int4(a[4], a[5], a[6], a[7]);
              }
              if (P.Y) {
                float y[8];
#pragma unroll
                for (int j = 0; j < 8; ++j)
                  y[j] = __fmul_rn(__fmul_rn((float)a[j], sw_s[as * BN + ch * 32 + g * 8 + j]), c);
                if (P.residual) {
                  const uint4 r4 = __ldg(reinterpret_cast<const uint4*>(P.residual + rowoff + col));
                  const uint32_t rw[4] = {r4.x, r4.y, r4.z, r4.w};
#pragma unroll
                  for (int j = 0; j < 4; ++j) {
                    y[2 * j]     = __fadd_rn(y[2 * j],     __fmul_rn(bf16lo_to_f32(rw[j]), rs));
                    y[2 * j + 1] = __fadd_rn(y[2 * j + 1], __fmul_rn(bf16hi_to_f32(rw[j]), rs));
                  }
                }
                uint4 o;
                o.x = f32_to_bf16_bits(y[0]) | (f32_to_bf16_bits(y[1]) << 16);
                o.y = f32_to_bf16_bits(y[2]) | (f32_to_bf16_bits(y[3]) << 16);
                o.z = f32_to_bf16_bits(y[4]) | (f32_to_bf16_bits(y[5]) << 16);
                o.w = f32_to_bf16_bits(y[6]) | (f32_to_bf16_bits(y[7]) << 16);
                *reinterpret_cast<uint4*>(P.Y + rowoff + col) = o;
              }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty(as));
    }
  } else {
    // ------------------------------------------------------------------ converters
    constexpr int kThreads = NCONV * 32;
    constexpr int kChunks = (BM + BN) * (PK_ROW / 16);
    static_assert(kChunks % kThreads == 0, "converter threads must tile the packed stage");
    const int ctid = threadIdx.x - kFirstConvWarp * 32;
    int ps = 0, is = 0; uint32_t pph = 0, iph = 0;
    bool ok = true;
    for (int tile = blockIdx.x; ok && tile < P.num_tiles; tile += gridDim.x) {
      for (int kb = 0; kb < P.kblocks; ++kb) {
        if (!mbar_wait(pk_full(ps), pph, abort_flag, P.status, 5) ||
            !mbar_wait(i8_empty(is), iph ^ 1u, abort_flag, P.status, 6)) { ok = false; break; }
        const uint4* src = reinterpret_cast<const uint4*>(smem + L::kPkOff + ps * L::kPkStage);
        uint8_t* dst = smem + L::kI8Off + is * L::kI8Stage;
#pragma unroll
        for (int i = 0; i < kChunks / kThreads; ++i) {
          const int id = i * kThreads + ctid;           // 16-byte chunk: row id/4, packed chunk id%4
          const int r = id >> 2, c = id & 3;
          const uint4 p = src[id];
          uint4 even, odd;
          expand_nibbles(p, even, odd);
          uint8_t* rowp = dst + r * I8_ROW;
          *reinterpret_cast<uint4*>(rowp + (((2 * c) ^ (r & 7)) << 4)) = even;
          *reinterpret_cast<uint4*>(rowp + (((2 * c + 1) ^ (r & 7)) << 4)) = odd;
        }
        fence_proxy_async_smem();       // generic-proxy writes -> visible to the tensor core's async proxy
        __syncwarp();
        if (lane == 0) { mbar_arrive(i8_full(is)); mbar_arrive(pk_empty(ps)); }
        if (++ps == NPK) { ps = 0; pph ^= 1u; }
        if (++is == NI8) { is = 0; iph ^= 1u; }
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------
// Tensor map over a packed [rows, K/2]-byte matrix; one box = box_rows rows of one k-block.
static bool make_packed_map(CUtensorMap* m, const void* base, int rows, int K, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)(K / 2), (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)(K / 2)};
  const cuuint32_t box[2] = {(cuuint32_t)PK_ROW, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static int num_sms() { return device_sm_count(); }

template <int BN, int NI8, int NPK, int NCONV>
static int launch_gemm(cudaStream_t st, const uint8_t* Xq, const uint8_t* Wq, GemmParams P) {
  using L = SmemLayout<BN, NI8, NPK>;
  auto kern = gemm_w4a4_kernel<BN, NI8, NPK, NCONV>;
  static PerDeviceInt attr_set;
  if (!ensure_smem_attr(attr_set, kern, L::kAlloc)) return FPT_ERR_CUDA;
  CUtensorMap tmA, tmB;
  if (!make_packed_map(&tmA, Xq, P.M, P.K, BM) || !make_packed_map(&tmB, Wq, P.N, P.K, BN)) return FPT_ERR_CUDA;
  P.tiles_m = (P.M + BM - 1) / BM;
  P.num_tiles = P.tiles_m * ((P.N + BN - 1) / BN);
  P.kblocks = P.K / BK;
  const int grid = P.num_tiles < num_sms() ? P.num_tiles : num_sms();
  return launch_kernel(kern, dim3(grid), dim3((kFirstConvWarp + NCONV) * 32), L::kAlloc, st, true, tmA, tmB, P) ==
                 cudaSuccess
             ? FPT_OK
             : FPT_ERR_CUDA;
}

int gemm_launch(cudaStream_t st, const uint8_t* Xq, const uint8_t* Wq, const GemmParams& P) {
  if (P.M <= 16) return gemm_decode_small_launch(st, Xq, Wq, P);
  if (P.M <= 64 && P.scratch) return gemm_decode_launch(st, Xq, Wq, P, P.scratch);
  if (P.M > 128 && P.N > 128) return gemm_pair_launch(st, Xq, Wq, P);
  if (P.M > 64 && P.N > 128) {
    // 65..128 tokens: the CTA-pair kernel (half of its 256 activation rows empty) still beats the
    // one-CTA kernel per k-block (measured 0.5 against 0.68 us), unless it needs more rounds of tiles
    const int sms = num_sms(), pairs = sms >= 2 ? sms / 2 : 1;
    const int rounds_1 = ((P.N + 255) / 256 + sms - 1) / sms;
    const int rounds_2 = ((P.N + 207) / 208 + pairs - 1) / pairs;
    if (rounds_2 * 3 < rounds_1 * 4) return gemm_pair_launch(st, Xq, Wq, P);
  }
  if (P.N <= 64) return launch_gemm<64, 4, 4, 8>(st, Xq, Wq, P);
  if (P.N <= 128) return launch_gemm<128, 4, 4, 8>(st, Xq, Wq, P);
  return launch_gemm<256, 3, 3, 8>(st, Xq, Wq, P);
}

}  // namespace fpt
