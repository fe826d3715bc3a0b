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

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(std::forward<Args>(args))...);
}

}  // namespace marche
