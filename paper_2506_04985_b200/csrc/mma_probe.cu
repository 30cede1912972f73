// Measurement aid (no counterpart in the paper): how fast this GPU's tensor cores run the 8-bit
// integer tcgen05.mma that step (2) of the path is built on, with every data movement taken away.
// One thread per CTA (per CTA pair) issues `iters` groups of four K = 32 instructions on operand
// tiles that stay where they are (pseudo-random bytes, so that the data toggles as real codes do),
// rotating over `n_acc` accumulators; the kernel ends when the last instruction has completed.
// The rate it reaches is the ceiling the matmul kernels are compared with, and its dependence on
// the instruction shape (rows, columns, accumulators in rotation, A operand in tensor or shared
// memory) is what the decode-size kernels are designed around.
#include "fpt_internal.cuh"

namespace fpt {
namespace probe {

constexpr int kThreads = 128;
constexpr int kATile = 128 * 128;                  // 128 rows x 128 bytes, 128-byte swizzle
constexpr int kBTile = 256 * 128;                  // up to 256 rows x 128 bytes
constexpr int kBarOff = kATile + kBTile;
constexpr int kBytes = kBarOff + 64;
constexpr int kAlloc = kBytes + 1024;
constexpr int kTmemCols = 512;
constexpr int kAStageCol = 480;                    // 32 columns hold 128 int8 per lane

struct Params {
  int n;                   // columns of one instruction (multiple of 16, 16..256)
  int n_acc;               // accumulators in rotation: n_acc * n <= 448 columns
  int a_in_tmem;           // A operand from tensor memory (else from shared memory)
  int iters;               // groups of four instructions
  uint32_t* status;
  unsigned long long* cycles;   // [CTAs] clock64 ticks from the first issue to the last completion (leaders only)
};

template <bool kPair>
__global__ void __launch_bounds__(kThreads, 1) mma_probe_kernel(const Params P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bar = sbase + kBarOff;
  volatile uint32_t* misc = reinterpret_cast<volatile uint32_t*>(smem + kBarOff + 16);
  volatile uint32_t* abort_flag = misc + 1;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = kPair ? cluster_ctarank() : 0u;

  // operand tiles: bytes from a counter hash (the values do not matter, their toggling does)
  for (int i = threadIdx.x; i < (kATile + kBTile) / 4; i += kThreads) {
    uint32_t h = (uint32_t)i * 2654435761u + blockIdx.x * 40503u;
    h ^= h >> 15; h *= 2246822519u; h ^= h >> 13;
    reinterpret_cast<uint32_t*>(smem)[i] = h & 0xF0F0F0F0u;        // code * 16, as the kernels feed them
  }
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    misc[1] = 0;
    fence_mbar_init();
  }
  fence_proxy_async_smem();
  if (warp == 0) {
    if (kPair) { tmem_alloc_pair(sbase + kBarOff + 16, kTmemCols); tmem_relinquish_pair(); }
    else { tmem_alloc(sbase + kBarOff + 16, kTmemCols); tmem_relinquish(); }
  }
  tc_fence_before();
  if (kPair) cluster_sync_all(); else __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = misc[0];
  {
    // A operand in tensor memory: every lane gets 128 bytes
    uint32_t v[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      uint32_t h = (uint32_t)(threadIdx.x * 32 + j) * 2246822519u + 12345u;
      h ^= h >> 13; h *= 2654435761u; h ^= h >> 16;
      v[j] = h & 0xF0F0F0F0u;
    }
    tmem_st_32x32(tmem_base + ((uint32_t)(warp * 32) << 16) + kAStageCol, v);
    tmem_wait_st();
  }
  tc_fence_before();
  if (kPair) cluster_sync_all(); else __syncthreads();
  tc_fence_after();

  if (warp == 0 && lane == 0 && rank == 0) {
    const uint32_t idesc = umma_idesc_i8(kPair ? 256 : 128, P.n, true, true);
    const uint64_t adesc = umma_desc_kmajor_sw128(sbase);
    const uint64_t bdesc = umma_desc_kmajor_sw128(sbase + kATile);
    const uint32_t a_tmem = tmem_base + kAStageCol;
    const int n = P.n, n_acc = P.n_acc, iters = P.iters;
    const bool a_tm = P.a_in_tmem != 0;
    int acc = 0;
    const long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        const uint32_t d = tmem_base + (uint32_t)(acc * n);
        if (kPair) {
          if (a_tm) umma_i8_ts_pair(d, a_tmem + 8u * kk, bdesc + 2u * kk, idesc, 1u);
          else umma_i8_pair(d, adesc + 2u * kk, bdesc + 2u * kk, idesc, 1u);
        } else {
          if (a_tm) umma_i8_ts(d, a_tmem + 8u * kk, bdesc + 2u * kk, idesc, 1u);
          else umma_i8(d, adesc + 2u * kk, bdesc + 2u * kk, idesc, 1u);
        }
        if (++acc == n_acc) acc = 0;
      }
    }
    if (kPair) umma_commit_pair(bar, 1); else umma_commit(bar);
    mbar_wait(bar, 0, abort_flag, P.status, 1);
    const long long t1 = clock64();
    if (P.cycles) P.cycles[kPair ? blockIdx.x >> 1 : blockIdx.x] = (unsigned long long)(t1 - t0);
  }
  __syncwarp();
  tc_fence_before();
  if (kPair) cluster_sync_all(); else __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    if (kPair) tmem_dealloc_pair(tmem_base, kTmemCols); else tmem_dealloc(tmem_base, kTmemCols);
  }
}

// Self-test of the bounded wait every kernel of the library relies on: one thread waits on an
// mbarrier on which nothing ever arrives, with a limit of `limit_ns`; the wait must give up, record
// where in the status word, and the kernel must end normally.
__global__ void __launch_bounds__(32, 1) wait_timeout_kernel(uint32_t* status, unsigned long long limit_ns, uint32_t* gave_up) {
  __shared__ __align__(8) unsigned long long bar_mem;
  __shared__ uint32_t abort_flag;
  const uint32_t bar = smem_u32(&bar_mem);
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(bar, 1);
    fence_mbar_init();
  }
  __syncwarp();
  if (threadIdx.x == 0) {
    const bool ok = mbar_wait_limit(bar, 0, &abort_flag, status, 14, limit_ns);
    if (gave_up) *gave_up = ok ? 0u : 1u;
    mbar_inval(bar);
  }
}

}  // namespace probe
}  // namespace fpt

using namespace fpt;

extern "C" int fpt_selftest_wait_timeout(void* stream, void* workspace, unsigned int limit_us, unsigned int* gave_up) {
  if (!workspace || limit_us == 0 || limit_us > 100000u) return FPT_ERR_BAD_ARG;
  if ((uintptr_t)workspace & 15) return FPT_ERR_ALIGNMENT;
  probe::wait_timeout_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(reinterpret_cast<uint32_t*>(workspace),
                                                                (unsigned long long)limit_us * 1000ull, gave_up);
  return cudaGetLastError() == cudaSuccess ? FPT_OK : FPT_ERR_CUDA;
}

extern "C" int fpt_probe_mma(void* stream, int pair, int n, int n_acc, int a_in_tmem, int iters, int ctas,
                             unsigned long long* cycles, void* workspace) {
  using namespace probe;
  if (!workspace || iters <= 0 || ctas <= 0) return FPT_ERR_BAD_ARG;
  if (n < 16 || n > 256 || n % 16 != 0 || n_acc < 1 || n_acc * n > kAStageCol) return FPT_ERR_UNSUPPORTED;
  if (pair && (ctas & 1)) return FPT_ERR_BAD_ARG;
  if ((uintptr_t)workspace & 15) return FPT_ERR_ALIGNMENT;
  Params P;
  P.n = n; P.n_acc = n_acc; P.a_in_tmem = a_in_tmem; P.iters = iters;
  P.status = reinterpret_cast<uint32_t*>(workspace);
  P.cycles = cycles;
  cudaStream_t st = (cudaStream_t)stream;
  if (pair) {
    if (cudaFuncSetAttribute(mma_probe_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAlloc) != cudaSuccess)
      return FPT_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ctas, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = kAlloc;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, mma_probe_kernel<true>, P) != cudaSuccess) return FPT_ERR_CUDA;
  } else {
    if (cudaFuncSetAttribute(mma_probe_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAlloc) != cudaSuccess)
      return FPT_ERR_CUDA;
    mma_probe_kernel<false><<<ctas, kThreads, kAlloc, st>>>(P);
  }
  return cudaGetLastError() == cudaSuccess ? FPT_OK : FPT_ERR_CUDA;
}
