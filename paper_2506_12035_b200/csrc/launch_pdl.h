// Launch helper: programmatic dependent launch for the step's kernel chain.
//
// Every kernel of the library begins with pdl_wait() (griddepcontrol.wait: returns once the
// preceding kernel of the stream has completed and its writes are visible) followed by
// pdl_launch_dependents(), and every launch carries the programmatic-stream-serialization
// attribute.  The next kernel's CTAs may therefore become resident, and run their private
// set-up (barrier init, TMEM allocation, tensor-map prefetch), while the current kernel is
// still draining; they touch global memory only after the wait.  Because each kernel releases
// its dependents only after its own wait has returned, at most one kernel runs ahead.
// MARCHE_PDL=0 turns the attribute off (plain stream order).
#pragma once

#include <cuda_runtime.h>

#include <cstdlib>
#include <utility>

namespace marche {

inline bool pdl_enabled() {
  static int on = -1;
  if (on < 0) {
    const char* e = getenv("MARCHE_PDL");
    on = (e && e[0] == '0') ? 0 : 1;
  }
  return on == 1;
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

// cluster_x > 1 additionally launches the grid in clusters of that many consecutive CTAs (used only
// to co-schedule CTAs that stream neighbouring bytes of the same DRAM pages; no cluster-level
// synchronisation or shared memory is involved).
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl_cluster(int cluster_x, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                               cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  int n = 0;
  if (pdl_enabled()) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  if (cluster_x > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = (unsigned)cluster_x;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(std::forward<Args>(args))...);
}

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  return launch_pdl_cluster(1, kernel, grid, block, smem, st, std::forward<Args>(args)...);
}

}  // namespace marche
