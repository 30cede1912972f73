// Steps (2)+(3) of the path at decode sizes (at most 64 tokens): the packed INT4 weights are
// streamed once from HBM, which is the whole cost; the arithmetic is the same exact INT32
// matmul (App. J "Setup") and scale-factor epilogue (App. B "Static quantization").
//
// The operands swap sides: 128 WEIGHT rows are the M side of the MMA and the (padded) tokens
// are its N side, so one tcgen05.mma of shape 128 x {16,32,64} x 32 consumes 128 x 32 weight
// codes.  Weights are widened nibble -> int8 in registers and written to tensor memory
// (tcgen05.st), the MMA reads them from there; only the few token rows are widened into a
// shared-memory tile.  Nothing of the weight stream is ever stored to shared memory twice.
//
// Work is split stream-K style: the T = (N/128) * (K/256) weight k-blocks are cut into equal
// contiguous ranges, one per CTA (one CTA per SM), so every SM streams the same number of bytes
// whatever the shape.  A range that covers part of a tile leaves its raw int32 partial sums in
// a scratch slot; the last CTA to arrive at a tile (an atomic counter per tile and lane
// quadrant) adds the slots up -- integer addition, so the result does not depend on the order
// -- and runs the epilogue.  No CTA ever waits for another.
// Where every tile is cut into the same 2, 4 or 8 ranges (few tiles, long rows), the CTAs of a tile are
// launched as one thread-block cluster instead: each leaves its partial sums in its OWN shared
// memory, the cluster synchronises once, and every CTA then adds up and finishes its share of the
// tokens by reading the others' shared memory directly -- no trip through L2, no atomics, and the
// final epilogue is spread over all CTAs of the tile.  (A cluster barrier does wait for the peers,
// but they are co-scheduled by construction and all reach it.)
//
// Roles (24 warps): warp 0 TMA producer, warp 1 MMA issuer and tensor-memory owner (warps 2-3 idle),
// warps 4-7 token converters (with 64 tokens their tile is half as many bytes as the weights': two
// warps were the slowest stage of the pipeline), warps 8-19 weight converters (three groups of four
// warps, each group taking every third k-block: the chain load -> widen -> tcgen05.st -> wait -> arrive
// is long, and one tcgen05.mma of 128 rows x 32 codes takes about 100 cycles whatever its width, so
// several k-blocks in conversion are what keeps the tensor core's queue from running dry),
// warps 20-23 epilogue.
// Registers are traded between the warpgroups (setmaxnreg): the epilogue holds 64 accumulators per thread.
#include <cuda.h>

#include "fpt_internal.cuh"

namespace fpt {
namespace decode {

constexpr int HR = 128;                    // weight rows per tile
constexpr int BK = 256;                    // codes per k-block: 128 packed bytes per row, one full cache line
constexpr int PK_ROW = BK / 2;
constexpr int I8_ROW = 128;                // the widened token tile is two 128-byte-swizzled halves of 128 codes
constexpr int NS = 6;                      // widened stages: 6 x 64 tensor-memory columns + 6 token tiles
constexpr int NPK = 4;                     // packed stages in flight from TMA
constexpr int kGroups = 3;                 // weight-converter groups
constexpr int kTokWarps = 4;               // token-converter warps
constexpr int kMaxTok = 64;
constexpr int kAccCols = 64;               // per accumulator buffer (two of them)
constexpr int kAStage0 = 2 * kAccCols;
constexpr int kTmemCols = 512;
constexpr int kConvBWarp0 = 4, kConvAWarp0 = kConvBWarp0 + kTokWarps, kEpiWarp0 = kConvAWarp0 + 4 * kGroups;
constexpr int kThreads = 32 * (kEpiWarp0 + 4);
// registers per thread after the trade: warps 0-3, each converter group, the epilogue group
constexpr int kRegsLaunch = (65536 / kThreads) / 8 * 8, kRegsCtl = 64, kRegsTok = 64, kRegsConv = 64, kRegsEpi = 152;
static_assert(kTokWarps == 4, "the token converters are one warpgroup");
static_assert(kThreads * kRegsLaunch <= 65536, "launch allocation exceeds the register file");
static_assert(128 * (kRegsCtl + kRegsTok + kGroups * kRegsConv + kRegsEpi) <= kThreads * kRegsLaunch,
              "the warpgroups ask for more registers than the CTA was launched with: setmaxnreg.inc would never return");
static_assert(2 * kAccCols + NS * (BK / 4) <= kTmemCols, "operand stages must fit beside the two accumulators");

struct Smem {
  static constexpr int kB8Half = kMaxTok * I8_ROW;                  // 8 KB: 64 token rows x 128 codes as int8
  static constexpr int kB8Stage = 2 * kB8Half;                      // 16 KB: widened token tile
  static constexpr int kPkW = HR * PK_ROW;                          // 16 KB: packed weights of one k-block
  static constexpr int kPkX = kMaxTok * PK_ROW;                     // 8 KB: packed tokens of one k-block
  static constexpr int kB8Off = 0;
  static constexpr int kPkWOff = kB8Off + NS * kB8Stage;
  static constexpr int kPkXOff = kPkWOff + NPK * kPkW;
  static constexpr int kVecOff = kPkXOff + NPK * kPkX;              // c_t and residual scale per token: 2 x 64 floats
  static constexpr int kBarOff = kVecOff + 2 * kMaxTok * 4;
  static constexpr int kNumBars = 2 * NPK + 2 * NS + 4;
  static constexpr int kMiscOff = kBarOff + kNumBars * 8;
  static constexpr int kBytes = kMiscOff + 16;
  static constexpr int kAlloc = kBytes + 1024;
  static_assert(kAlloc <= 232448, "exceeds the shared memory of one CTA");
};

struct DecodeParams {
  GemmParams g;            // M = tokens, N = weight rows, K
  int npad;                // tokens padded to the MMA N: 16, 32 or 64
  int tiles;               // N / 128 rounded up
  int kblocks;             // K / 256 rounded up (a half block at the end reads zeros past the row)
  long long total;         // tiles * kblocks
  int per, rem;            // total = per * CTAs + rem: CTA c takes per k-blocks, the first rem CTAs one more
  int whole_tiles;         // 1: ranges end on tile boundaries (no partial sums, no counters)
  int cluster;             // > 1: every tile is cut into this many equal ranges and the CTAs of a range set form a
                           // thread-block cluster: partial sums are exchanged through distributed shared memory
  int32_t* slots;          // [gridDim.x][2][npad][128] raw int32 partial sums
  uint32_t* counters;      // [tiles][4], zero between launches
};

// First weight k-block (global index) of CTA c's range.
__device__ __forceinline__ long long range_start(const DecodeParams& D, int c, int nctas) {
  if (D.whole_tiles) return (long long)D.kblocks * (long long)((unsigned)(D.tiles * c) / (unsigned)nctas);
  return (long long)c * D.per + (c < D.rem ? c : D.rem);          // no division: this runs inside the epilogue
}

__global__ void __launch_bounds__(kThreads, 1)
gemm_w4a4_decode_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
                        const DecodeParams D) {
  using L = Smem;
  const GemmParams& P = D.g;
  extern __shared__ uint8_t smem_raw[];
  // aligned to 1024 bytes by an offset on the shared-memory array itself (a round trip through an
  // integer would leave a generic pointer: generic loads and stores, and no way for the compiler to
  // tell shared from global accesses apart)
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bar0 = sbase + L::kBarOff;
  auto pk_full = [&](int s) { return bar0 + 8u * s; };
  auto pk_empty = [&](int s) { return bar0 + 8u * (NPK + s); };
  auto op_full = [&](int s) { return bar0 + 8u * (2 * NPK + s); };
  auto op_empty = [&](int s) { return bar0 + 8u * (2 * NPK + NS + s); };
  auto acc_full = [&](int b) { return bar0 + 8u * (2 * NPK + 2 * NS + b); };
  auto acc_empty = [&](int b) { return bar0 + 8u * (2 * NPK + 2 * NS + 2 + b); };
  volatile uint32_t* misc = reinterpret_cast<volatile uint32_t*>(smem + L::kMiscOff);
  volatile uint32_t* abort_flag = misc + 1;
  float* c_s = reinterpret_cast<float*>(smem + L::kVecOff);        // act_scale * post[t]
  float* rs_s = c_s + kMaxTok;                                      // residual scale per token

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int nctas = gridDim.x;
  const long long g_begin = range_start(D, blockIdx.x, nctas);
  const long long g_end = range_start(D, blockIdx.x + 1, nctas);
  const uint32_t pkx_bytes = (uint32_t)D.npad * PK_ROW;

  if (threadIdx.x == 0) {
    for (int s = 0; s < NPK; ++s) { mbar_init(pk_full(s), 1); mbar_init(pk_empty(s), kTokWarps + 4); }
    for (int s = 0; s < NS; ++s) { mbar_init(op_full(s), kTokWarps + 4); mbar_init(op_empty(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_empty(b), 4); }
    misc[1] = 0;
    fence_mbar_init();
    prefetch_tmap(&tmW);
    prefetch_tmap(&tmX);
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

  // Registers: the epilogue wants the 64 accumulators of its row in registers at once, the other roles
  // need few; the warpgroups trade (see the static_assert above: the requests are covered).
  if (warp < kConvBWarp0) reg_dec<kRegsCtl>();
  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int s = 0; uint32_t ph = 0;
      uint32_t armed = 0, armed_par = 0;
      bool ok = true;
      for (long long g = g_begin; g < g_end; ++g) {
        const int tile = (int)(g / D.kblocks), kb = (int)(g % D.kblocks);
        if (!mbar_wait(pk_empty(s), ph ^ 1u, abort_flag, P.status, 1)) { ok = false; break; }
        mbar_arrive_expect_tx(pk_full(s), L::kPkW + pkx_bytes);
        tma_load_2d(sbase + L::kPkWOff + s * L::kPkW, &tmW, pk_full(s), kb * PK_ROW, tile * HR);
        tma_load_2d(sbase + L::kPkXOff + s * L::kPkX, &tmX, pk_full(s), kb * PK_ROW, 0);
        armed |= 1u << s;
        armed_par = (armed_par & ~(1u << s)) | (ph << s);
        if (++s == NPK) { s = 0; ph ^= 1u; }
      }
      if (!ok) {
        const uint64_t t0 = globaltimer_ns();
        for (int q = 0; q < NPK; ++q)
          if (armed & (1u << q))
            while (!mbar_try_wait(pk_full(q), (armed_par >> q) & 1u) && globaltimer_ns() - t0 < 2000000ull) {}
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_i8(HR, D.npad, true, !P.a_unsigned);
      int s = 0; uint32_t ph = 0; int seg = 0;
      long long g = g_begin;
      bool ok = true;
      while (ok && g < g_end) {
        const int kb0 = (int)(g % D.kblocks);
        const long long left = g_end - g;
        const int kb1 = (D.kblocks - kb0) < left ? D.kblocks : kb0 + (int)left;
        const int b = seg & 1; const uint32_t bph = (seg >> 1) & 1;
        if (!mbar_wait(acc_empty(b), bph ^ 1u, abort_flag, P.status, 2)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + b * kAccCols;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(op_full(s), ph, abort_flag, P.status, 3)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_tmem = tmem_base + kAStage0 + s * (BK / 4);
#pragma unroll
          for (int kk = 0; kk < BK / 32; ++kk) {
            const uint64_t bdesc = umma_desc_kmajor_sw128(sbase + L::kB8Off + s * L::kB8Stage + (kk >> 2) * L::kB8Half);
            umma_i8_ts(d_tmem, a_tmem + 8u * kk, bdesc + 2u * (kk & 3), idesc, (kb != kb0) || kk != 0);
          }
          umma_commit(op_empty(s));
          if (++s == NS) { s = 0; ph ^= 1u; }
        }
        if (!ok) break;
        umma_commit(acc_full(b));
        g += kb1 - kb0;
        ++seg;
      }
    }
  } else if (warp < kConvBWarp0) {
    // (warps 2-3: nothing to do)
  } else if (warp < kConvAWarp0) {
    // ------------------------------------------------------------------ token converters -> shared int8 tile
    reg_dec<kRegsTok>();
    constexpr int kTokThreads = kTokWarps * 32;
    const int ctid = threadIdx.x - kConvBWarp0 * 32;     // 0..127
    const int per_thread = D.npad * 8 / kTokThreads;     // 16-byte chunks per thread: 1, 2 or 4
    int ps = 0, s = 0; uint32_t pph = 0, ph = 0;
    for (long long g = g_begin; g < g_end; ++g) {
      if (!mbar_wait(pk_full(ps), pph, abort_flag, P.status, 7)) break;
      const uint4* src = reinterpret_cast<const uint4*>(smem + L::kPkXOff + ps * L::kPkX);
      uint4 c[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) if (i < per_thread) c[i] = src[i * kTokThreads + ctid];
      if (!mbar_wait(op_empty(s), ph ^ 1u, abort_flag, P.status, 8)) break;
      uint8_t* dst = smem + L::kB8Off + s * L::kB8Stage;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (i < per_thread) {
          const int id = i * kTokThreads + ctid;         // 16-byte packed chunk: row id/8, chunk id%8
          const int r = id >> 3, ch = id & 3;            // chunks 0-3: first 128 codes, 4-7: second half
          uint32_t w[8];
          widen(c[i], w);
          uint8_t* rowp = dst + ((id >> 2) & 1) * L::kB8Half + r * I8_ROW;
          *reinterpret_cast<uint4*>(rowp + (((2 * ch) ^ (r & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
          *reinterpret_cast<uint4*>(rowp + (((2 * ch + 1) ^ (r & 7)) << 4)) = make_uint4(w[4], w[5], w[6], w[7]);
        }
      }
      // One fence for both hand-overs: the widened tile becomes visible to the tensor core's async
      // proxy, and the reads of the packed tile -- consumed by the stores above -- are ordered before
      // the TMA write that re-fills it.  (A packed tile handed back right after its loads, before
      // anything depends on them, can be overwritten while the loads are still in flight.)
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) { mbar_arrive(pk_empty(ps)); mbar_arrive(op_full(s)); }
      if (++ps == NPK) { ps = 0; pph ^= 1u; }
      if (++s == NS) { s = 0; ph ^= 1u; }
    }
  } else if (warp < kEpiWarp0) {
    // ------------------------------------------------------------------ weight converters -> tensor memory
    reg_dec<kRegsConv>();
    const int quad = warp & 3;                           // TMEM lanes this warp may touch
    const int grp = (warp - kConvAWarp0) >> 2;           // takes the k-blocks whose running index is grp modulo kGroups
    const int r = quad * 32 + lane;
    const uint32_t swz = (uint32_t)(r & 7);              // SWIZZLE_128B of the packed weight tile
    const int n_local = (int)(g_end - g_begin);          // k-blocks of this CTA
    for (int kc = grp; kc < n_local; kc += kGroups) {    // kc: running k-block index of this CTA
      const int ps = kc % NPK; const uint32_t pph = (uint32_t)((kc / NPK) & 1);
      const int s = kc % NS;   const uint32_t ph = (uint32_t)((kc / NS) & 1);
      if (!mbar_wait(pk_full(ps), pph, abort_flag, P.status, 5)) break;
      const uint8_t* src = smem + L::kPkWOff + ps * L::kPkW + r * PK_ROW;
      const uint32_t a_tmem = tmem_base + ((uint32_t)(quad * 32) << 16) + kAStage0 + s * (BK / 4);
      bool ok = true;
      // the row's 256 codes in two halves of 128 (32 tensor-memory columns each): fewer live registers
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        uint4 c[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) c[j] = *reinterpret_cast<const uint4*>(src + (((uint32_t)(4 * h + j) ^ swz) << 4));
        uint32_t v[32];
#pragma unroll
        for (int j = 0; j < 4; ++j) widen(c[j], v + 8 * j);
        if (h == 0) {
          if (!mbar_wait(op_empty(s), ph ^ 1u, abort_flag, P.status, 6)) { ok = false; break; }
          tc_fence_after();
        }
        tmem_st_32x32(a_tmem + 32 * h, v);
      }
      if (!ok) break;
      tmem_wait_st();
      tc_fence_before();
      fence_proxy_async_smem();      // reads of the packed tile (consumed above) before the TMA write that re-fills it
      __syncwarp();
      if (lane == 0) { mbar_arrive(pk_empty(ps)); mbar_arrive(op_full(s)); }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    reg_inc<kRegsEpi>();
    const int quad = warp & 3;
    const int npad = D.npad;
    {
      // per-token factors of the epilogue, shared by the four epilogue warps
      const int t = threadIdx.x - kEpiWarp0 * 32;
      if (t < kMaxTok) {
        c_s[t] = (t < P.M && P.post) ? __fmul_rn(P.act_scale, __ldg(P.post + t)) : P.act_scale;
        rs_s[t] = (t < P.M && P.res_scale) ? __ldg(P.res_scale + t) : 1.0f;
      }
      named_bar_sync(1, 128);
    }
    int seg = 0;
    long long g = g_begin;
    while (g < g_end) {
      const int tile = (int)(g / D.kblocks), kb0 = (int)(g % D.kblocks);
      const long long left = g_end - g;
      const int kb1 = (D.kblocks - kb0) < left ? D.kblocks : kb0 + (int)left;
      const bool whole = kb0 == 0 && kb1 == D.kblocks;
      const int b = seg & 1; const uint32_t bph = (seg >> 1) & 1;
      const int n = tile * HR + quad * 32 + lane;        // weight row = output feature of this thread
      const bool n_ok = n < P.N;
      // per-row constants, fetched while the matmul of the segment runs
      const float swn = n_ok ? load_scale(P.sw, P.scale_dtype, n) : 0.0f;
      const int zw = (P.wsum && n_ok) ? P.zero_point * __ldg(P.wsum + n) : 0;
      if (!mbar_wait(acc_full(b), bph, abort_flag, P.status, 4)) break;
      tc_fence_after();
      uint32_t v[kMaxTok];
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + b * kAccCols;
      {
        uint32_t t16[16];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          if (q * 16 < npad) {
            tmem_ld_32x16(taddr + q * 16, t16);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 16; ++j) v[q * 16 + j] = t16[j];
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty(b));

      bool finalize = whole;
      if (!whole && D.cluster > 1) {
        // raw partial sums -> this CTA's shared memory (the packed weight ring is free: every stage has been
        // consumed once the accumulator is complete); finished after the cluster barrier below
        int32_t* red = reinterpret_cast<int32_t*>(smem + L::kPkWOff) + quad * 32 + lane;
#pragma unroll
        for (int t = 0; t < kMaxTok; ++t) if (t < npad) red[t * HR] = (int32_t)v[t];
      } else if (!whole) {
        // raw partial sums -> this CTA's slot; the last contributor of the tile adds all slots up
        const int my_slot = (g == g_begin) ? 0 : 1;
        int32_t* slot = D.slots + ((size_t)(blockIdx.x * 2 + my_slot) * npad) * HR + quad * 32 + lane;
#pragma unroll
        for (int t = 0; t < kMaxTok; ++t) if (t < npad) slot[(size_t)t * HR] = (int32_t)v[t];
        __threadfence();
        __syncwarp();
        // contributors of this tile: every CTA whose range meets [tile*KB, (tile+1)*KB)
        const long long t_begin = (long long)tile * D.kblocks, t_end = t_begin + D.kblocks;
        int c_first = blockIdx.x, c_last = blockIdx.x;
        while (c_first > 0 && range_start(D, c_first, nctas) > t_begin) --c_first;
        while (c_last + 1 < nctas && range_start(D, c_last + 1, nctas) < t_end) ++c_last;
        const uint32_t expected = (uint32_t)(c_last - c_first + 1);
        uint32_t old = 0;
        if (lane == 0) old = atomicAdd(D.counters + tile * 4 + quad, 1u);
        old = __shfl_sync(0xffffffffu, old, 0);
        if (old == expected - 1) {
          __threadfence();
#pragma unroll
          for (int t = 0; t < kMaxTok; ++t) v[t] = 0;
          // (sixteen loads in flight per batch: the four epilogue warps are alone on the SM by now, so
          // nothing else hides the latency of a dependent chain)
          for (int c = c_first; c <= c_last; ++c) {
            const int cs = (range_start(D, c, nctas) >= t_begin) ? 0 : 1;
            const int32_t* src = D.slots + ((size_t)(c * 2 + cs) * npad) * HR + quad * 32 + lane;
#pragma unroll
            for (int t0 = 0; t0 < kMaxTok; t0 += 16) {
              if (t0 < npad) {
                uint32_t w[16];
#pragma unroll
                for (int t = 0; t < 16; ++t) w[t] = (uint32_t)__ldcg(src + (size_t)(t0 + t) * HR);
#pragma unroll
                for (int t = 0; t < 16; ++t) v[t0 + t] += w[t];
              }
            }
          }
          if (lane == 0) D.counters[tile * 4 + quad] = 0;      // ready for the next launch
          finalize = true;
        }
      }
      if (finalize && n_ok) {
        // (everything the loop needs from the parameter block is read once, here)
        const int m_tok = P.M;
        const size_t ldy = (size_t)P.N;
        int32_t* const acc_out = P.acc_out ? P.acc_out + n : nullptr;
        __nv_bfloat16* const yp = P.Y ? P.Y + n : nullptr;
        const __nv_bfloat16* const resp = P.residual ? P.residual + n : nullptr;
        if (yp && !acc_out && !resp) {
          // the usual case, straight-line: sixteen outputs computed, then sixteen stores
#pragma unroll
          for (int t0 = 0; t0 < kMaxTok; t0 += 16) {
            if (t0 < m_tok) {
              __nv_bfloat16 y[16];
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                const float4 c4 = *reinterpret_cast<const float4*>(c_s + t0 + 4 * q);
                const float cc[4] = {c4.x, c4.y, c4.z, c4.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  const int a = (((int)v[t0 + 4 * q + j]) >> 8) - zw;
                  y[4 * q + j] = __float2bfloat16_rn(__fmul_rn(__fmul_rn((float)a, swn), cc[j]));
                }
              }
              __nv_bfloat16* o = yp + (size_t)t0 * ldy;
#pragma unroll
              for (int t = 0; t < 16; ++t) if (t0 + t < m_tok) o[(size_t)t * ldy] = y[t];
            }
          }
        } else {
#pragma unroll
          for (int t = 0; t < kMaxTok; ++t) {
            if (t < m_tok) {
              const int a = (((int)v[t]) >> 8) - zw;
              if (acc_out) acc_out[(size_t)t * ldy] = a;
              if (yp) {
                float y = __fmul_rn(__fmul_rn((float)a, swn), c_s[t]);
                if (resp) y = __fadd_rn(y, __fmul_rn(__bfloat162float(resp[(size_t)t * ldy]), rs_s[t]));
                yp[(size_t)t * ldy] = __float2bfloat16_rn(y);
              }
            }
          }
        }
      }
      g += kb1 - kb0;
      ++seg;
    }
  }

  if (D.cluster > 1) {
    // ---------------------------------------------------------------- split tiles: exchange inside the cluster
    __syncwarp();
    cluster_sync_all();                                  // every CTA's partial sums are in its shared memory
    {
      // Every thread of the CTA takes part (the other roles are done): this CTA finishes tokens
      // [rank * tp, (rank + 1) * tp) of the tile, one (token, weight row) output per thread and pass,
      // adding the partial sums of all CTAs of the cluster straight from their shared memory.
      const uint32_t rank = cluster_ctarank(), csize = cluster_nctarank();
      const int tp = D.npad / (int)csize;
      const int t_lo = (int)rank * tp;
      const int tile = (int)(g_begin / D.kblocks);
      const int m_tok = P.M;
      const size_t ldy = (size_t)P.N;
      const uint32_t red0 = sbase + L::kPkWOff;
      uint32_t peer[8];
#pragma unroll
      for (int c = 0; c < 8; ++c) peer[c] = map_to_cta(red0, (uint32_t)c < csize ? (uint32_t)c : 0u);
      for (int idx = threadIdx.x; idx < tp * HR; idx += kThreads) {
        const int tok = t_lo + idx / HR, nl = idx % HR;
        const int n = tile * HR + nl;
        const uint32_t off = 4u * (uint32_t)(tok * HR + nl);
        uint32_t w[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) w[c] = (uint32_t)c < csize ? ld_shared_cluster_u32(peer[c] + off) : 0u;
        const int sum = (int)(((w[0] + w[1]) + (w[2] + w[3])) + ((w[4] + w[5]) + (w[6] + w[7])));
        if (n < P.N && tok < m_tok) {
          const int zw = P.wsum ? P.zero_point * __ldg(P.wsum + n) : 0;
          const int a = (sum >> 8) - zw;
          if (P.acc_out) P.acc_out[(size_t)tok * ldy + n] = a;
          if (P.Y) {
            const float ct = P.post ? __fmul_rn(P.act_scale, __ldg(P.post + tok)) : P.act_scale;
            float y = __fmul_rn(__fmul_rn((float)a, load_scale(P.sw, P.scale_dtype, n)), ct);
            if (P.residual) {
              const float rs = P.res_scale ? __ldg(P.res_scale + tok) : 1.0f;
              y = __fadd_rn(y, __fmul_rn(__bfloat162float(P.residual[(size_t)tok * ldy + n]), rs));
            }
            P.Y[(size_t)tok * ldy + n] = __float2bfloat16_rn(y);
          }
        }
      }
    }
    __syncwarp();
    cluster_sync_all();                                  // nobody leaves while a peer may still read its shared memory
  }
  // ------------------------------------------------------------------ teardown
  __syncwarp();
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
static bool make_map(CUtensorMap* m, const void* base, int rows, int K, int box_rows, CUtensorMapSwizzle swz) {
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

static int num_sms() { return device_sm_count(); }

}  // namespace decode

int decode_npad(int M) { return M <= 16 ? 16 : M <= 32 ? 32 : 64; }

size_t gemm_decode_scratch_bytes(int M) {
  return (size_t)kDecodeMaxCtas * 2 * (size_t)decode_npad(M) * decode::HR * sizeof(int32_t);
}

// Xq [M <= 64, K/2], Wq [N, K/2]; `scratch` holds gemm_decode_scratch_bytes(M) bytes; the counters
// live in the workspace's control block behind the status word.
int gemm_decode_launch(cudaStream_t st, const uint8_t* Xq, const uint8_t* Wq, const GemmParams& P, void* scratch) {
  using namespace decode;
  static PerDeviceInt attr_set;
  if (!ensure_smem_attr(attr_set, gemm_w4a4_decode_kernel, Smem::kAlloc)) return FPT_ERR_CUDA;
  DecodeParams D;
  D.g = P;
  D.cluster = 0;
  D.npad = decode_npad(P.M);
  D.tiles = (P.N + HR - 1) / HR;
  D.kblocks = (P.K + BK - 1) / BK;
  D.total = (long long)D.tiles * D.kblocks;
  D.whole_tiles = D.tiles * 4 > kDecodeMaxCounters ? 1 : 0;
  D.slots = reinterpret_cast<int32_t*>(scratch);
  D.counters = P.status + kCounterWord0;
  CUtensorMap tmW, tmX;
  if (!make_map(&tmW, Wq, P.N, P.K, HR, CU_TENSOR_MAP_SWIZZLE_128B) ||
      !make_map(&tmX, Xq, P.M, P.K, D.npad, CU_TENSOR_MAP_SWIZZLE_NONE))
    return FPT_ERR_CUDA;
  // Number of CTAs (= equal ranges of the weight stream).  With fewer tiles than SMs each tile is
  // cut into the same number of ranges, so that range ends fall on tile ends (fewest partial sums);
  // with more tiles than SMs every SM gets the same share and ranges end where they end.
  const int sms = num_sms() < kDecodeMaxCtas ? num_sms() : kDecodeMaxCtas;
  int ctas = sms;
  if (D.tiles <= sms) {
    int split = sms / D.tiles;
    const int max_split = D.kblocks / 2 > 0 ? D.kblocks / 2 : 1;      // at least 2 k-blocks (512 codes) per range
    if (split > max_split) split = max_split;
    ctas = D.tiles * split;
    // a power-of-two split up to 8 that keeps at least 85 % of those CTAs: the ranges of a tile become one cluster
    int pw = 1;
    while (pw * 2 <= split && pw * 2 <= 8) pw *= 2;
    D.cluster = (pw > 1 && !D.whole_tiles && pw * 100 >= split * 85 && D.kblocks % pw == 0 && D.npad % pw == 0) ? pw : 0;
    if (D.cluster) ctas = D.tiles * pw;
    // (112 tiles stay on 112 SMs: cutting them into 148 equal ranges was measured slower, 19.4 against
    // 14.4 us at 64 tokens -- the partial sums of a split tile are 32 KB per range)
  }
  const long long units = D.whole_tiles ? D.tiles : D.total;
  if (units < ctas) ctas = (int)units;
  D.per = (int)(D.total / ctas);
  D.rem = (int)(D.total % ctas);
  if (D.cluster > 1) {
    // the clusters must fit: with one CTA per SM a cluster needs that many free SMs in one GPC
    static PerDeviceInt fits[4];                          // cluster sizes 2, 4, 8 -> index 1, 2, 3
    const int idx = D.cluster == 2 ? 1 : D.cluster == 4 ? 2 : 3;
    const int cl = D.cluster;
    const int ok = fits[idx].get([&] {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(cl, 1, 1);
      cfg.blockDim = dim3(kThreads, 1, 1);
      cfg.dynamicSmemBytes = Smem::kAlloc;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = (unsigned)cl; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr; cfg.numAttrs = 1;
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, gemm_w4a4_decode_kernel, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
      return n > 0 ? n + 1 : 1;                           // 1: does not fit (cached as such)
    }) - 1;
    if (ok * D.cluster < ctas) D.cluster = 0;             // not all clusters resident at once: use the slots instead
  }
  const cudaError_t e = D.cluster > 1
      ? launch_kernel_cluster(gemm_w4a4_decode_kernel, dim3(ctas), dim3(kThreads), Smem::kAlloc, st, true, D.cluster, tmW, tmX, D)
      : launch_kernel(gemm_w4a4_decode_kernel, dim3(ctas), dim3(kThreads), Smem::kAlloc, st, true, tmW, tmX, D);
  return e == cudaSuccess ? FPT_OK : FPT_ERR_CUDA;
}

}  // namespace fpt
