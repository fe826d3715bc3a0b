// Launch helper: programmatic dependent launch for the step's kernel chain.
//
// Every kernel of the library begins with pdl_wait() (griddepcontrol.wait: returns once the
// preceding kernel of the stream has completed and its writes are visible) followed by
// pdl_launch_dependents(), and every launch carries the programmatic-stream-serialization
// attribute.  The next kernel's CTAs may therefore become resident, and run their private
// set-up (barrier init, TMEM allocation, tensor-map prefetch), while the current kernel is
// still draining; they touch global memory only after the wait.  Because each kernel releases
// its dependents only after its own wait has returned, at most one kernel runs ahead.
// pdl_switch() holds the process-wide on/off state (marche_set_tuning; on by default).
#pragma once

#include <cuda_runtime.h>

#include <utility>

namespace marche {

inline bool& pdl_switch() {
  static bool on = true;
  return on;
}

// Raises a kernel's dynamic shared-memory limit to at least `bytes` on the current device.  The
// attribute belongs to the device's context, so what has been set is remembered per device
// (`cache`: one zero-initialised array per kernel instantiation at the call site).
constexpr int kMaxDevices = 64;
template <typename Kernel>
cudaError_t ensure_dynamic_smem(Kernel kernel, size_t bytes, size_t (&cache)[kMaxDevices]) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (bytes <= cache[dev]) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess) cache[dev] = bytes;
  return e;
}

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  int n = 0;
  if (pdl_switch()) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(std::forward<Args>(args))...);
}

}  // namespace marche
