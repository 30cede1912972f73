// Host-side helpers shared by the launchers: per-device caches (SM count, one-time kernel
// attributes) and the driver entry point that encodes tensor maps.  Everything that depends on
// the GPU is keyed by the current device and guarded by a mutex: a process may drive several
// GPUs, from several threads.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

#include <mutex>

namespace fpt {

constexpr int kMaxDevices = 64;

// Current device index, or -1 (no device, or an index beyond kMaxDevices).
inline int current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
  return dev;
}

// One integer per device, computed on first use on that device.  `compute` returns the value
// (> 0) or a value <= 0 for "failed, try again next time".
struct PerDeviceInt {
  std::mutex mu;
  int v[kMaxDevices] = {};
  template <class F>
  int get(F compute) {
    const int dev = current_device();
    if (dev < 0) return 0;
    std::lock_guard<std::mutex> lock(mu);
    if (v[dev] <= 0) v[dev] = compute();
    return v[dev];
  }
};

// Number of SMs of the current device (at least 1).
inline int device_sm_count() {
  static PerDeviceInt cache;
  const int n = cache.get([] {
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    return sms;
  });
  return n > 0 ? n : 1;
}

// Raises the dynamic shared-memory limit of `kern` once per device.  `cache` is one object per kernel
// (a function-local static of the launcher).
template <class K>
inline bool ensure_smem_attr(PerDeviceInt& cache, K kern, int bytes) {
  return cache.get([&] {
    return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) == cudaSuccess ? 1 : 0;
  }) > 0;
}

// Whether kernels are launched with the programmatic-serialisation attribute (fpt_set_programmatic_launch).
int programmatic_launch_enabled();

// Launches `kern` on `st`; with `pdl` (and the library-wide switch on) the launch carries the
// programmatic-serialisation attribute: the kernel may start before the previous kernel of the stream
// has finished and orders itself behind it with pdl_wait().  Only kernels that call pdl_wait() before
// their first access to memory another kernel may have written are launched this way.
// `cluster` > 1: the grid is launched in thread-block clusters of that many CTAs along x.
template <class... KArgs, class... Args>
inline cudaError_t launch_kernel_cluster(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                         bool pdl, int cluster, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  int n = 0;
  if (cluster > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = (unsigned)cluster; attr[n].val.clusterDim.y = 1; attr[n].val.clusterDim.z = 1;
    ++n;
  }
  if (pdl && programmatic_launch_enabled()) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  cfg.attrs = n ? attr : nullptr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

template <class... KArgs, class... Args>
inline cudaError_t launch_kernel(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool pdl,
                                 Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  int n = 0;
  if (pdl && programmatic_launch_enabled()) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  cfg.attrs = n ? attr : nullptr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// cuTensorMapEncodeTiled through the runtime (the library does not link libcuda); the entry point is the
// same for every device of the process.
inline EncodeTiledFn encode_fn() {
  static const EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      return reinterpret_cast<EncodeTiledFn>(p);
    return static_cast<EncodeTiledFn>(nullptr);
  }();
  return fn;
}

}  // namespace fpt
