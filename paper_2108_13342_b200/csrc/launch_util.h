// Kernel launch with programmatic dependent launch: a block's kernel may start while the
// previous kernel on the stream is still draining, and blocks at pdl_wait() until that kernel
// has completed and its writes are visible.  Every kernel of this library calls pdl_wait()
// before its first global-memory access, so the result equals plain stream order; only the
// launch latency and the prologue (index set-up, barrier and tensor-memory set-up) overlap
// the predecessor's tail.  Works in plain streams and under stream capture.
#pragma once
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>
#include <cstdlib>

namespace dnnf {

// Function attributes (the opt-in to more than 48 KB of dynamic shared memory) are per device: one flag per
// device ordinal and kernel instantiation, so that a second GPU used by the same process is configured too.
struct PerDeviceOnce {
  std::atomic<uint64_t> mask{0};
  bool first_use() {
    int d = 0;
    if (cudaGetDevice(&d) != cudaSuccess) return true;
    const uint64_t bit = 1ull << (d & 63);
    return !(mask.fetch_or(bit) & bit);
  }
};

// Number of SMs of the current device; 148 (B200) where no device can be asked, e.g. planning on a host without a GPU.
inline int sm_count() {
  static std::atomic<int> cached{0};
  int n = cached.load();
  if (n > 0) return n;
  int d = 0, v = 0;
  if (cudaGetDevice(&d) == cudaSuccess && cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, d) == cudaSuccess && v > 0) n = v;
  else { cudaGetLastError(); n = 148; }
  cached.store(n);
  return n;
}

__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <class... KArgs, class... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
#ifdef DNNF_DEV_SWITCHES
  static const bool pdl_off = getenv("DNNF_NO_PDL") != nullptr;
#else
  constexpr bool pdl_off = false;
#endif
  attr[0].val.programmaticStreamSerializationAllowed = pdl_off ? 0 : 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(std::forward<Args>(args))...);
}

}  // namespace dnnf
