// Steps (2)+(3) of the path for prefill sizes: packed-INT4 x packed-INT4 matmul with an exact
// INT32 accumulator (App. J "Setup") and the floating-point scale factors applied after it
// (App. B "Static quantization"), on CTA pairs.
//
// Why this shape: the shared-memory data pipe of an SM moves 128 bytes per cycle and is shared
// by ld/st.shared, TMA writes and the tensor core's operand reads.  Widening nibbles to int8 in
// shared memory for both operands of a 1-CTA tile needs 1152 of those transfers per 128-code
// k-block against 512 cycles of MMA.  Here
//   * two CTAs form one 256 x 256 tile (tcgen05.mma.cta_group::2): each CTA widens and feeds only
//     its own 128 weight rows, and its tensor core reads only those;
//   * the activation operand is widened in registers and written to TENSOR memory (tcgen05.st);
//     the MMA takes it from there, so it is never stored to or read from shared memory as int8.
// Per k-block and CTA: TMA in 16 KB, converter loads 16 KB, int8 weight stores 16 KB, tensor-core
// reads 16 KB = 512 transfers for 512 MMA cycles.
//
// Roles per CTA (20 warps):
//   warp 0        TMA producer: packed tiles (128 rows x 64 bytes of each operand per k-block)
//   warp 1        tensor-memory owner; in the leader CTA (rank 0) also the MMA issuer
//   warps 4..11   converters, two groups of four warps that take the k-blocks in turns: a group widens
//                 the CTA's activation rows (shared -> registers -> tcgen05.st, one row per thread) and,
//                 while that store completes, its weight rows (-> 128-byte-swizzled K-major int8 tile)
//   warps 12..19  epilogue: tcgen05.ld, >> 8, scales, bf16 into a swizzled shared-memory tile; the
//                 accumulator is released as soon as it has been read, the tile leaves by TMA store;
//                 a residual tile is fetched by TMA into the same slabs while the tile's matmul runs
// Both operands are widened as code*16 (see gemm_w4a4.cu), so the accumulator holds 256 * sum.
// Variants (template parameters): the two fused SwiGLU epilogues, int8 activation codes (the
// activation tile then needs no widening and the shift is 4), output tiles of 208..256 columns.
#include <cuda.h>

#include "fpt_internal.cuh"
#include "quant_math.cuh"

namespace fpt {
namespace pair {

constexpr int TM = 256, TN = 256;          // output tile of a CTA pair
constexpr int HR = 128;                    // rows of each operand a CTA owns
constexpr int BK = 128;                    // codes per k-block
constexpr int PK_ROW = BK / 2;             // packed bytes per row and k-block
constexpr int I8_ROW = BK;                 // int8 bytes per row and k-block
constexpr int kAccCols = 256;              // tensor-memory columns of the accumulator
constexpr int kAStageCols = BK / 4;        // 32 columns hold 128 int8 per lane
constexpr int kTmemCols = 512;
constexpr int kThreads = 640;
constexpr int kConvWarp0 = 4, kEpiWarp0 = 12, kEpiWarps = 8;
// Registers per thread: what the CTA is launched with, and what the roles trade it into (warps 0-3,
// the two converter groups, epilogue).  A CTA can only redistribute what it owns: an
// increase that the decreases do not cover would never return, so the sum is checked here.
constexpr int kRegsLaunch = 96, kRegsCtl = 48, kRegsConv = 64, kRegsEpi = 152;
static_assert(kThreads * kRegsLaunch <= 65536, "launch allocation exceeds the register file");
static_assert(128 * (kRegsCtl + 2 * kRegsConv) + 32 * kEpiWarps * kRegsEpi <= kThreads * kRegsLaunch,
              "the warpgroups ask for more registers than the CTA was launched with: setmaxnreg.inc would never return");

// NS: stages of widened operands (int8 weight tile in shared memory + activation columns in
// tensor memory); NPK: stages of packed tiles in flight from TMA.
// kA8: the activation operand arrives as int8 codes (one byte each, 128-byte rows per k-block)
// instead of packed 4-bit codes.
template <int NS, int NPK, bool kA8 = false>
struct Smem {
  static_assert(kAccCols + NS * kAStageCols <= kTmemCols, "operand stages must fit beside the accumulator");
  static constexpr int kB8Stage = HR * I8_ROW;                      // 16 KB
  static constexpr int kPkOp = HR * PK_ROW;                         // 8 KB: a packed weight tile
  static constexpr int kPkOpA = kA8 ? HR * I8_ROW : HR * PK_ROW;    // the activation tile of a stage
  static constexpr int kB8Off = 0;
  static constexpr int kPkAOff = kB8Off + NS * kB8Stage;
  static constexpr int kPkBOff = kPkAOff + NPK * kPkOpA;
  static constexpr int kStgOff = kPkBOff + NPK * kPkOp;             // bf16 output tile: 4 slabs of 128 rows x 64 columns
  static constexpr int kStgSlab = HR * 128;                         // 16 KB, 128-byte rows, 128-byte swizzle
  static constexpr int kScaleOff = kStgOff + 4 * kStgSlab;          // 2 x 256 floats (sw) + 2 x 256 ints (z * wsum)
  static constexpr int kBarOff = kScaleOff + 2 * TN * 4 * 2;
  static constexpr int kNumBars = 2 * NPK + 2 * NS + 2 + 2 + 2 + 2 + 2;
  static constexpr int kMiscOff = kBarOff + kNumBars * 8;           // tmem base, abort flag
  static constexpr int kBytes = kMiscOff + 16;
  static constexpr int kAlloc = kBytes + 1024;                      // slack to align the base to 1024
  static_assert(kAlloc <= 232448, "exceeds the shared memory of one CTA");
};

// kFuse: 0 plain scale-factor epilogue; 1 SwiGLU product + quantiser (codes out); 2 SwiGLU product
// (bf16 out).  Separate instantiations keep the plain epilogue's register budget free of the others.
template <int NS, int NPK, int kFuse, bool kA8 = false, int kTN = TN>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
gemm_w4a4_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                      const __grid_constant__ CUtensorMap tmY, const __grid_constant__ CUtensorMap tmYt,
                      const __grid_constant__ CUtensorMap tmR, const __grid_constant__ CUtensorMap tmRt,
                      const GemmParams P) {
  using L = Smem<NS, NPK, kA8>;
  static_assert(!kA8 || kFuse == 0, "8-bit activations: plain epilogue only");
  extern __shared__ uint8_t smem_raw[];
  // aligned to 1024 bytes by an offset on the shared-memory array itself (a round trip through an
  // integer would leave a generic pointer: generic loads and stores, and no way for the compiler to
  // tell shared from global accesses apart)
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bar0 = sbase + L::kBarOff;
  auto pk_full = [&](int s) { return bar0 + 8u * s; };
  auto pk_empty = [&](int s) { return bar0 + 8u * (NPK + s); };
  auto op_full = [&](int s) { return bar0 + 8u * (2 * NPK + s); };             // waited on in the leader CTA
  auto op_empty = [&](int s) { return bar0 + 8u * (2 * NPK + NS + s); };
  const uint32_t acc_full = bar0 + 8u * (2 * NPK + 2 * NS);
  const uint32_t acc_empty = acc_full + 8u;                                    // waited on in the leader CTA
  auto sc_full = [&](int b) { return acc_full + 16u + 8u * b; };               // scales of a tile are in shared memory
  auto stg_full = [&](int h) { return acc_full + 32u + 8u * h; };              // a 128-column half of the tile is staged
  auto stg_empty = [&](int h) { return acc_full + 48u + 8u * h; };             // ... and has been read by its TMA store
  auto res_full = [&](int h) { return acc_full + 64u + 8u * h; };              // the residual of a half has arrived in the staging slabs
  volatile uint32_t* misc = reinterpret_cast<volatile uint32_t*>(smem + L::kMiscOff);
  volatile uint32_t* abort_flag = misc + 1;

  // the parameter block is read once, here (not inside the role loops)
  uint32_t* const status_w = P.status;
  const int kblocks = P.kblocks, num_tiles = P.num_tiles, tiles_m = P.tiles_m;
  const int n_cols = P.N, m_rows = P.M;
  int32_t* const acc_out_p = P.acc_out;
  const __nv_bfloat16* const residual_p = P.residual;
  __nv_bfloat16* const y_out_p = P.Y;
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();             // 0 = leader
  const int pair_id = blockIdx.x >> 1;
  const int num_pairs = gridDim.x >> 1;
  // Width of the output tile.  The plain epilogue also exists for 208, 224 and 240 columns: the host
  // picks the width that wastes the least of the last round of tiles (the kernel is bound by the
  // tensor pipe, so a narrower tile takes proportionally less time).  The fused epilogues need 256.
  static_assert(kTN == TN || (kFuse == 0 && kTN >= 208 && kTN % 16 == 0), "tile width");
  constexpr int tn = kTN;
  constexpr int hb = tn >> 1;                          // weight rows of the tile this CTA holds

  if (threadIdx.x == 0) {
    for (int s = 0; s < NPK; ++s) { mbar_init(pk_full(s), 1); mbar_init(pk_empty(s), 4); }      // the four warps of a group
    for (int s = 0; s < NS; ++s) { mbar_init(op_full(s), 8); mbar_init(op_empty(s), 1); }        // ... in both CTAs
    mbar_init(acc_full, 1);
    mbar_init(acc_empty, 2 * kEpiWarps);
    for (int b = 0; b < 2; ++b) { mbar_init(sc_full(b), kEpiWarps); mbar_init(stg_full(b), 4); mbar_init(stg_empty(b), 1); mbar_init(res_full(b), 1); }
    misc[1] = 0;
    fence_mbar_init();
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmB);
    if (y_out_p || kFuse == 1) { prefetch_tmap(&tmY); if (tn < TN) prefetch_tmap(&tmYt); }
  }
  if (warp == 1) {
    tmem_alloc_pair(sbase + L::kMiscOff, kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  cluster_sync_all();                                  // barriers of both CTAs exist before any remote arrive
  tc_fence_after();
  const uint32_t tmem_base = misc[0];
  // everything above touched only this CTA pair's own shared and tensor memory; the operands, the
  // per-token vectors and the outputs may belong to the kernel before this one
  pdl_wait();
  pdl_launch_dependents();

  // Registers: the epilogue wants the 128 accumulators of its row in registers at once, the other
  // roles need few; the warpgroups trade.  A CTA can only redistribute what it was launched with
  // (640 x 96 registers): 128 x (48 + 64 + 64) + 256 x 152 = 61440 <= 61440, so the request of the
  // epilogue groups is always met once the three other groups have given theirs back.  Each role
  // branch starts with its own re-allocation (the compiler budgets registers per branch).
  if (warp < kConvWarp0) {
    reg_dec<kRegsCtl>();
    if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int s = 0; uint32_t ph = 0;
      uint32_t armed = 0, armed_par = 0;
      bool ok = true;
      for (int tile = pair_id; ok && tile < num_tiles; tile += num_pairs) {
        const int m0 = (tile % tiles_m) * TM + (int)rank * HR;
        const int n0 = (tile / tiles_m) * tn + (int)rank * hb;
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(pk_empty(s), ph ^ 1u, abort_flag, status_w, 1)) { ok = false; break; }
          mbar_arrive_expect_tx(pk_full(s), L::kPkOpA + (uint32_t)hb * PK_ROW);
          tma_load_2d(sbase + L::kPkAOff + s * L::kPkOpA, &tmA, pk_full(s), kb * (kA8 ? I8_ROW : PK_ROW), m0);
          tma_load_2d(sbase + L::kPkBOff + s * L::kPkOp, &tmB, pk_full(s), kb * PK_ROW, n0);
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
    // ------------------------------------------------------------------ MMA issuer (leader CTA only)
    if (rank == 0 && lane == 0) {
      const uint32_t idesc = umma_idesc_i8(TM, tn, !P.a_unsigned, true);
      int s = 0; uint32_t ph = 0; int it = 0;
      for (int tile = pair_id; tile < num_tiles; tile += num_pairs, ++it) {
        if (!mbar_wait_cluster(acc_empty, (it & 1) ^ 1u, abort_flag, status_w, 2)) break;
        tc_fence_after();
        bool ok = true;
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait_cluster(op_full(s), ph, abort_flag, status_w, 3)) { ok = false; break; }
          tc_fence_after();
          const uint64_t bdesc = umma_desc_kmajor_sw128(sbase + L::kB8Off + s * L::kB8Stage);
          const uint32_t a_tmem = tmem_base + kAccCols + s * kAStageCols;
#pragma unroll
          for (int kk = 0; kk < BK / 32; ++kk)
            umma_i8_ts_pair(tmem_base, a_tmem + 8u * kk, bdesc + 2u * kk, idesc, (kb | kk) != 0);
          umma_commit_pair(op_empty(s), 3);
          if (++s == NS) { s = 0; ph ^= 1u; }
        }
        if (!ok) break;
        umma_commit_pair(acc_full, 3);
      }
    }
    }
  } else if (warp < kEpiWarp0) {
    // ------------------------------------------------------------------ converters
    // Two groups of four warps (4..7 and 8..11) take the k-blocks in turns, and a group widens a whole
    // k-block: the CTA's 128 activation rows into tensor memory (one row per thread; warp % 4 selects
    // the tensor-memory lanes the warp may touch) and the CTA's weight rows into the int8 tile in shared
    // memory.  For one warp a k-block is a chain of long latencies (shared loads, the tensor-memory store
    // and its wait, the proxy fence) that does not shrink with the tile; alternating groups give every
    // chain two k-block periods.
    reg_dec<kRegsConv>();
    const int grp = (warp - kConvWarp0) >> 2;
    const int quad = warp & 3;                           // the TMEM lanes this warp may touch
    const int r = quad * 32 + lane;                      // activation row of the CTA's 128; also this thread's chunk column
    const uint32_t swz = (uint32_t)((r >> 1) & 3);       // SWIZZLE_64B: 16-byte chunk index ^= (row / 2) % 4
    const uint32_t op_full_leader = map_to_cta(op_full(0), 0);
    int ps = 0, s = 0; uint32_t pph = 0, ph = 0;
    uint32_t gk = 0;                                     // k-blocks since the start of the kernel
    bool ok = true;
    for (int tile = pair_id; ok && tile < num_tiles; tile += num_pairs) {
      for (int kb = 0; kb < kblocks; ++kb, ++gk) {
        if ((int)(gk & 1u) == grp) {
          if (!mbar_wait(pk_full(ps), pph, abort_flag, status_w, 5)) { ok = false; break; }
          uint32_t v[32];
          if constexpr (kA8) {
            // int8 codes, 128-byte rows under the 128-byte swizzle.  The weight side orders the 32 codes
            // of a group as 16 even-k then 16 odd-k bytes (that is how the nibbles fall apart); the
            // activation bytes are put into the same order.
            const uint8_t* src = smem + L::kPkAOff + ps * L::kPkOpA + r * I8_ROW;
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              const uint4 c0 = *reinterpret_cast<const uint4*>(src + (((uint32_t)(2 * g) ^ (uint32_t)(r & 7)) << 4));
              const uint4 c1 = *reinterpret_cast<const uint4*>(src + (((uint32_t)(2 * g + 1) ^ (uint32_t)(r & 7)) << 4));
              const uint32_t a[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
#pragma unroll
              for (int w = 0; w < 4; ++w) {
                v[8 * g + w] = __byte_perm(a[2 * w], a[2 * w + 1], 0x6420);
                v[8 * g + 4 + w] = __byte_perm(a[2 * w], a[2 * w + 1], 0x7531);
              }
            }
          } else {
            const uint8_t* src = smem + L::kPkAOff + ps * L::kPkOpA + r * PK_ROW;
            uint4 c[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) c[j] = *reinterpret_cast<const uint4*>(src + (((uint32_t)j ^ swz) << 4));
#pragma unroll
            for (int j = 0; j < 4; ++j) widen(c[j], v + 8 * j);
          }
          // the packed weight tile: 16-byte chunk i * 128 + r is row (i * 128 + r) / 4, chunk r % 4
          const uint4* srcb = reinterpret_cast<const uint4*>(smem + L::kPkBOff + ps * L::kPkOp);
          uint4 cb[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) cb[i] = srcb[i * 128 + r];
          if (!mbar_wait(op_empty(s), ph ^ 1u, abort_flag, status_w, 6)) { ok = false; break; }
          tc_fence_after();
          tmem_st_32x32(tmem_base + ((uint32_t)(quad * 32) << 16) + kAccCols + s * kAStageCols, v);
          // while the tensor-memory store completes: the weight rows
          uint8_t* dst = smem + L::kB8Off + s * L::kB8Stage;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int br = (i * 128 + r) >> 2, ch = r & 3;
            if (i == 3 && br >= hb) continue;            // a narrower tile has fewer weight rows
            uint32_t w[8];
            widen(cb[i], w);
            uint8_t* rowp = dst + br * I8_ROW;
            *reinterpret_cast<uint4*>(rowp + (((2 * ch) ^ (br & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
            *reinterpret_cast<uint4*>(rowp + (((2 * ch + 1) ^ (br & 7)) << 4)) = make_uint4(w[4], w[5], w[6], w[7]);
          }
          tmem_wait_st();
          tc_fence_before();
          // One fence for both hand-overs: the widened tile becomes visible to the tensor core's async
          // proxy, and the reads of the packed tiles (consumed by the stores above) are ordered before
          // the TMA writes that re-fill them.  The packed tiles go back to TMA only here: handing them
          // back right after the loads, with nothing depending on them yet, let the next TMA write
          // overtake reads still in flight (seen as wrong weight rows, rarely, under load).
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) { mbar_arrive(pk_empty(ps)); mbar_arrive_cluster(op_full_leader + 8u * s); }
        }
        if (++ps == NPK) { ps = 0; pph ^= 1u; }
        if (++s == NS) { s = 0; ph ^= 1u; }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    reg_inc<kRegsEpi>();
    const int quad = warp & 3;                           // TMEM lane quadrant this warp may read
    const int half = (warp - kEpiWarp0) >> 2;            // which 128 of the 256 columns
    const int etid = (warp - kEpiWarp0) * 32 + lane;     // 0..255: the tile column whose scale this thread fetches
    const uint32_t acc_empty_leader = map_to_cta(acc_empty, 0);
    float* sw_s = reinterpret_cast<float*>(smem + L::kScaleOff);
    int* zw_s = reinterpret_cast<int*>(smem + L::kScaleOff + 2 * TN * 4);
    const int r = quad * 32 + lane;                      // row of the CTA's 128
    constexpr int kShift = kA8 ? 4 : 8;                  // both operands carry a factor 16, int8 activations none
    // |acc| < 2^22: int -> float by the exponent trick.  With 4-bit activation codes that holds for every K
    // the entry points accept (64 * 65408 < 2^22), so the conversion instruction is never even emitted.
    const bool magic_ok = kA8 ? P.K < 4096 : true;
    const bool issuer = quad == 0 && lane == 0;          // issues the TMA stores (and residual loads) of its half
    const bool use_res = kFuse == 0 && residual_p != nullptr && y_out_p != nullptr;
    const bool has_z = P.wsum != nullptr;                // asymmetric activation grid: row-sum correction
    int it = 0;
    int res_armed = 0, res_seen = 0;                     // residual loads issued / seen to arrive (tiles, 1-based)
    for (int tile = pair_id; tile < num_tiles; tile += num_pairs, ++it) {
      const int b = it & 1; const uint32_t bph = (it >> 1) & 1;
      const int m0 = (tile % tiles_m) * TM + (int)rank * HR;
      const int nt = (tile / tiles_m) * tn;            // first column of the tile
      const int n_end = nt + tn < n_cols ? nt + tn : n_cols;   // one past the tile's last valid column
      // scale factors of the tile's columns -> shared memory, while the matmul of the tile runs
      {
        const int n = nt + etid;
        sw_s[b * TN + etid] = n < n_end ? load_scale(P.sw, P.scale_dtype, n) : 0.0f;
        zw_s[b * TN + etid] = (P.wsum && n < n_end) ? P.zero_point * __ldg(P.wsum + n) : 0;
      }
      const int row = m0 + r;
      const bool row_ok = row < m_rows;
      float c = P.act_scale, rs = 1.0f;
      if (row_ok && P.post) c = __fmul_rn(P.act_scale, __ldg(P.post + row));
      if (row_ok && P.res_scale) rs = __ldg(P.res_scale + row);
      const float sn = (kFuse == 1 && row_ok) ? __ldg(P.mid_scale + row) : 0.0f;
      __syncwarp();
      if (lane == 0) mbar_arrive(sc_full(b));
      if (!mbar_wait(sc_full(b), bph, abort_flag, status_w, 9)) break;
      // the staging half must have been read by the TMA store of the previous tile
      if ((y_out_p || kFuse == 1) && !mbar_wait(stg_empty(half), (it & 1) ^ 1u, abort_flag, status_w, 10)) break;
      if constexpr (kFuse == 0) {
        // The residual tile of this half travels by TMA into the staging slabs, in the layout the output
        // will have there, while the matmul of the tile still runs; each thread later reads the 16 bytes
        // it is about to overwrite.  (Read straight from global memory, one row per thread, these loads
        // were uncoalesced and made the epilogue the slow side.)
        if (use_res && issuer) {
          const uint32_t s0 = sbase + L::kStgOff + (half * 2) * L::kStgSlab;
          const uint32_t second = (tn < TN && half == 1) ? (uint32_t)HR * (uint32_t)(tn - 192) * 2u : (uint32_t)L::kStgSlab;
          mbar_arrive_expect_tx(res_full(half), (uint32_t)L::kStgSlab + second);
          tma_load_2d(s0, &tmR, res_full(half), nt + half * 128, m0);
          tma_load_2d(s0 + L::kStgSlab, (tn < TN && half == 1) ? &tmRt : &tmR, res_full(half), nt + half * 128 + 64, m0);
          res_armed = it + 1;
        }
      }
      if (!mbar_wait(acc_full, it & 1, abort_flag, status_w, 4)) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + half * 128;
      const size_t rowoff = (size_t)row * (size_t)n_cols;
      const float* sws = sw_s + b * TN + half * 128;
      const int* zws = zw_s + b * TN + half * 128;
      // all 128 accumulators of this thread's row -> registers, then the accumulator is free again
      uint32_t v[128];
      tmem_ld_32x64(taddr, v);                           // each load and its wait in one statement
      tmem_ld_32x64(taddr + 64, v + 64);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(acc_empty_leader);
      if constexpr (kFuse != 0) {
        // v[0..63]: gate accumulators of 64 features, v[64..127]: their up accumulators.
        // g, u = bf16 outputs of the two linears; m = bf16(silu(g) * u); code = grid(m * S_n).
        const QuantConsts qc = quant_consts(sn, P.mid_inv_delta, P.mid_qmax_minus_z, P.mid_flip);
        uint32_t codes[8];
#pragma unroll
        for (int j8 = 0; j8 < 8; ++j8) {
          uint32_t mw[4];
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) {
            const int f = j8 * 8 + jj * 2;
            uint32_t gw = 0, uw = 0;
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              const int ag = ((int)v[f + e]) >> 8, au = ((int)v[64 + f + e]) >> 8;
              const float gf = magic_ok ? __fsub_rn(__int_as_float(0x4B400000 + ag), 12582912.0f) : (float)ag;
              const float uf = magic_ok ? __fsub_rn(__int_as_float(0x4B400000 + au), 12582912.0f) : (float)au;
              gw |= f32_to_bf16_bits(__fmul_rn(__fmul_rn(gf, sws[f + e]), c)) << (16 * e);
              uw |= f32_to_bf16_bits(__fmul_rn(__fmul_rn(uf, sws[64 + f + e]), c)) << (16 * e);
            }
            mw[jj] = silu_mul_pair(gw, uw);
          }
          if constexpr (kFuse == 1) {
            codes[j8] = quant_word(make_uint4(mw[0], mw[1], mw[2], mw[3]), qc);
          } else {                                         // the products themselves: 128-byte rows, 128-byte swizzle
            uint8_t* slab = smem + L::kStgOff + (half * 2) * L::kStgSlab + r * 128;
            *reinterpret_cast<uint4*>(slab + ((j8 ^ (r & 7)) << 4)) = make_uint4(mw[0], mw[1], mw[2], mw[3]);
          }
        }
        if constexpr (kFuse == 1) {
          uint4* stg = reinterpret_cast<uint4*>(smem + L::kStgOff + (half * 2) * L::kStgSlab + r * 32);
          stg[0] = make_uint4(codes[0], codes[1], codes[2], codes[3]);
          stg[1] = make_uint4(codes[4], codes[5], codes[6], codes[7]);
        }
      } else {
      if (use_res && !mbar_wait(res_full(half), it & 1, abort_flag, status_w, 12)) break;
      res_seen = it + 1;
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        uint8_t* slab = smem + L::kStgOff + (half * 2 + (ch >> 1)) * L::kStgSlab + r * 128;
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          const int col = nt + half * 128 + ch * 32 + g * 8;
          // the eight scale factors (and row-sum corrections) of the group as 16-byte shared loads:
          // every lane reads the same words, one word per load was a wavefront of the contended
          // shared-memory pipe each
          const float4 sa = *reinterpret_cast<const float4*>(sws + ch * 32 + g * 8);
          const float4 sb = *reinterpret_cast<const float4*>(sws + ch * 32 + g * 8 + 4);
          const float sg[8] = {sa.x, sa.y, sa.z, sa.w, sb.x, sb.y, sb.z, sb.w};
          int zg[8] = {0, 0, 0, 0, 0, 0, 0, 0};
          if (has_z) {
            const int4 za = *reinterpret_cast<const int4*>(zws + ch * 32 + g * 8);
            const int4 zb = *reinterpret_cast<const int4*>(zws + ch * 32 + g * 8 + 4);
            zg[0] = za.x; zg[1] = za.y; zg[2] = za.z; zg[3] = za.w; zg[4] = zb.x; zg[5] = zb.y; zg[6] = zb.z; zg[7] = zb.w;
          }
          int a[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) a[j] = (((int)v[ch * 32 + g * 8 + j]) >> kShift) - zg[j];
          if (acc_out_p && row_ok && col < n_end) {
            int4* o = reinterpret_cast<int4*>(acc_out_p + rowoff + col);
            o[0] = make_int4(a[0], a[1], a[2], a[3]);
            o[1] = make_int4(a[4], a[5], a[6], a[7]);
          }
          if (y_out_p) {
            float y[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              // exact int -> float: 1.5 * 2^23 + a has a in its low mantissa bits
              const float af = magic_ok ? __fsub_rn(__int_as_float(0x4B400000 + a[j]), 12582912.0f) : (float)a[j];
              y[j] = __fmul_rn(__fmul_rn(af, sg[j]), c);
            }
            // where these 8 outputs go in the staging slabs (and where their residual waits)
            const int chunk = (ch & 1) * 4 + g;          // 16-byte chunk of the slab row; 128-byte swizzle
            uint4* dst = reinterpret_cast<uint4*>(slab + ((chunk ^ (r & 7)) << 4));
            bool in_tile = true;
            if (tn < TN && half == 1 && ch >= 2) {
              // last slab of a narrower tile: tn - 192 columns, dense rows, no swizzle (its own tensor map)
              constexpr int tail_bytes = (tn - 192) * 2;
              in_tile = chunk * 16 < tail_bytes;
              dst = reinterpret_cast<uint4*>(smem + L::kStgOff + 3 * L::kStgSlab + r * tail_bytes + chunk * 16);
            }
            if (use_res && in_tile) {                    // rows and columns outside the matrix arrive as zeros
              const uint4 r4 = *dst;
              const uint32_t rw[4] = {r4.x, r4.y, r4.z, r4.w};
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                y[2 * j]     = __fadd_rn(y[2 * j],     __fmul_rn(bf16lo_to_f32(rw[j]), rs));
                y[2 * j + 1] = __fadd_rn(y[2 * j + 1], __fmul_rn(bf16hi_to_f32(rw[j]), rs));
              }
            }
            uint4 o;                                     // two roundings to bf16 per instruction
            o.x = f32x2_to_bf16x2_bits(y[0], y[1]);
            o.y = f32x2_to_bf16x2_bits(y[2], y[3]);
            o.z = f32x2_to_bf16x2_bits(y[4], y[5]);
            o.w = f32x2_to_bf16x2_bits(y[6], y[7]);
            if (in_tile) *dst = o;
          }
        }
      }
      }
      if (y_out_p || kFuse == 1) {
        fence_proxy_async_smem();                        // staged tile -> visible to the TMA engine
        __syncwarp();
        if (lane == 0) mbar_arrive(stg_full(half));
        if (issuer) {
          if (!mbar_wait(stg_full(half), it & 1, abort_flag, status_w, 11)) break;
          const uint32_t s0 = sbase + L::kStgOff + (half * 2) * L::kStgSlab;
          if constexpr (kFuse == 1) {
            tma_store_2d(&tmY, s0, nt / 4 + half * 32, m0);            // 128 rows x 32 bytes of packed codes
          } else if constexpr (kFuse == 2) {
            tma_store_2d(&tmY, s0, nt / 2 + half * 64, m0);            // 128 rows x 64 products
          } else {
            tma_store_2d(&tmY, s0, nt + half * 128, m0);
            tma_store_2d((tn < TN && half == 1) ? &tmYt : &tmY, s0 + L::kStgSlab, nt + half * 128 + 64, m0);
          }
          tma_store_commit();
          tma_store_wait_read();
          mbar_arrive(stg_empty(half));
        }
        __syncwarp();
      }
    }
    if (issuer) tma_store_wait_read();
    if (issuer && res_armed > res_seen) {
      // left the loop on a timeout with a residual load still in flight: bounded wait before the
      // shared memory it writes to goes away
      const uint64_t t0 = globaltimer_ns();
      while (!mbar_try_wait(res_full(half), (uint32_t)(res_armed - 1) & 1u) && globaltimer_ns() - t0 < 2000000ull) {}
    }
  }

  // ------------------------------------------------------------------ teardown
  // Neither CTA may leave (or free tensor memory) while its peer can still arrive on its
  // barriers or the pair's MMAs can still read its shared / tensor memory.
  __syncwarp();
  tc_fence_before();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

// ------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------
// Tensor map over a packed [rows, K/2]-byte matrix; one box = 128 rows of one k-block (64 bytes each).
static bool make_map(CUtensorMap* m, const void* base, int rows, int K, CUtensorMapSwizzle swz, int box_rows = HR) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)(K / 2), (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)(K / 2)};
  const cuuint32_t box[2] = {(cuuint32_t)PK_ROW, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor map over an int8 [rows, K]-byte matrix; one box = 128 rows of one k-block (128 bytes each).
static bool make_map_i8(CUtensorMap* m, const void* base, int rows, int K) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)K};
  const cuuint32_t box[2] = {(cuuint32_t)I8_ROW, (cuuint32_t)HR};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor map over the bf16 output [M, N]; one box = 128 rows x 64 columns, 128-byte swizzle in shared memory.
// (box_cols < 64: the narrow last slab of a tile that is less than 256 columns wide; dense rows, no swizzle.)
static bool make_out_map(CUtensorMap* m, const void* base, int M, int N, int box_cols = 64) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)M};
  const cuuint64_t strides[1] = {(cuuint64_t)N * 2};
  const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)HR};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, box_cols == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
            CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tile width for the plain epilogue: tiles are dealt out in rounds of `pairs`, a tile's time is
// proportional to its width (tensor-pipe bound), so the width with the smallest rounds x width wins;
// among equal costs the widest (fewest tiles, least activation traffic).
static int choose_tn(int M, int N, int pairs) {
  const int tiles_m = (M + TM - 1) / TM;
  int best = TN;
  long long best_cost = -1;
  for (int tn = TN; tn >= 208; tn -= 16) {
    const long long tiles = (long long)tiles_m * ((N + tn - 1) / tn);
    const long long cost = ((tiles + pairs - 1) / pairs) * tn;
    if (best_cost < 0 || cost * 100 < best_cost * 98) { best_cost = cost; best = tn; }
  }
  return best;
}

// Tensor map over the packed codes [M, N/4 bytes] the fused SwiGLU epilogue writes; one box = 128 rows x 32 bytes.
static bool make_codes_map(CUtensorMap* m, const void* base, int M, int row_bytes) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)M};
  const cuuint64_t strides[1] = {(cuuint64_t)row_bytes};
  const cuuint32_t box[2] = {32, (cuuint32_t)HR};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int NS, int NPK, int kFuse, bool kA8 = false, int kTN = TN>
static int launch(cudaStream_t st, const uint8_t* Xq, const uint8_t* Wq, GemmParams P) {
  using L = Smem<NS, NPK, kA8>;
  auto kern = gemm_w4a4_pair_kernel<NS, NPK, kFuse, kA8, kTN>;
  static PerDeviceInt pairs_cache;          // co-resident CTA pairs on the current device
  const int max_pairs = pairs_cache.get([&] {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kAlloc) != cudaSuccess) return 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = L::kAlloc;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n <= 0) {
      cudaGetLastError();
      n = device_sm_count() / 2;
    }
    return n > 0 ? n : 1;
  });
  if (max_pairs <= 0) return FPT_ERR_CUDA;
  CUtensorMap tmA, tmB, tmY, tmYt;
  if (!(kA8 ? make_map_i8(&tmA, Xq, P.M, P.K) : make_map(&tmA, Xq, P.M, P.K, CU_TENSOR_MAP_SWIZZLE_64B)) ||
      !make_map(&tmB, Wq, P.N, P.K, CU_TENSOR_MAP_SWIZZLE_NONE, kTN / 2))
    return FPT_ERR_CUDA;
  if (P.Mq) { if (!make_codes_map(&tmY, P.Mq, P.M, P.N / 4)) return FPT_ERR_CUDA; }
  else if (P.Y) { if (!make_out_map(&tmY, P.Y, P.M, P.swiglu_bf16 ? P.N / 2 : P.N)) return FPT_ERR_CUDA; }
  else tmY = tmA;                                                                  // unused without an output tile
  tmYt = tmY;
  if (kTN < TN && P.Y && !make_out_map(&tmYt, P.Y, P.M, P.N, kTN - 192)) return FPT_ERR_CUDA;
  CUtensorMap tmR = tmY, tmRt = tmYt;                                              // unused without a residual
  if (kFuse == 0 && P.Y && P.residual) {
    if (!make_out_map(&tmR, P.residual, P.M, P.N)) return FPT_ERR_CUDA;
    tmRt = tmR;
    if (kTN < TN && !make_out_map(&tmRt, P.residual, P.M, P.N, kTN - 192)) return FPT_ERR_CUDA;
  }
  P.tiles_m = (P.M + TM - 1) / TM;
  P.num_tiles = P.tiles_m * ((P.N + kTN - 1) / kTN);
  P.kblocks = P.K / BK;
  const int pairs = P.num_tiles < max_pairs ? P.num_tiles : max_pairs;
  return launch_kernel(kern, dim3(2 * pairs), dim3(kThreads), L::kAlloc, st, true, tmA, tmB, tmY, tmYt, tmR, tmRt, P) ==
                 cudaSuccess
             ? FPT_OK
             : FPT_ERR_CUDA;
}

}  // namespace pair

static int device_pairs() { const int sms = device_sm_count(); return sms >= 2 ? sms / 2 : 1; }

int gemm_pair_launch(cudaStream_t st, const uint8_t* Xq, const uint8_t* Wq, const GemmParams& P) {
  if (P.Mq) return pair::launch<4, 5, 1>(st, Xq, Wq, P);
  if (P.swiglu_bf16) return pair::launch<4, 5, 2>(st, Xq, Wq, P);
  const int tn = pair::choose_tn(P.M, P.N, device_pairs());
  if (P.a_bits == 8) {                                                        // Xq: int8 [M, K]
    switch (tn) {
      case 240: return pair::launch<4, 3, 0, true, 240>(st, Xq, Wq, P);
      case 224: return pair::launch<4, 3, 0, true, 224>(st, Xq, Wq, P);
      case 208: return pair::launch<4, 3, 0, true, 208>(st, Xq, Wq, P);
      default:  return pair::launch<4, 3, 0, true, 256>(st, Xq, Wq, P);
    }
  }
  switch (tn) {
    case 240: return pair::launch<4, 5, 0, false, 240>(st, Xq, Wq, P);
    case 224: return pair::launch<4, 5, 0, false, 224>(st, Xq, Wq, P);
    case 208: return pair::launch<4, 5, 0, false, 208>(st, Xq, Wq, P);
    default:  return pair::launch<4, 5, 0, false, 256>(st, Xq, Wq, P);
  }
}

}  // namespace fpt
