// Diagnostic kernel behind marche_debug_bounded_wait: exercises the give-up path of the bounded
// mbarrier wait that every TMA / tcgen05 kernel of the library relies on (sm100_ptx.cuh, mbar_wait).
// One thread waits on a barrier that nothing ever arrives on; once the cycle limit has passed the
// wait returns false, the thread writes a code into the status word and the kernel ends normally.
// Nothing traps, faults or spins without a bound; the context stays usable.
#include "kernels.h"
#include "launch_pdl.h"
#include "sm100_ptx.cuh"

namespace marche {

namespace {

enum { ST_PROBE = 0x61 };

__global__ void __launch_bounds__(32)
bounded_wait_probe_kernel(long long limit_cycles, int* __restrict__ status) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    ptx::mbar_init(ptx::smem_u32(&bar), 1);
    abort_flag = 0;
    ptx::fence_barrier_init();
  }
  __syncwarp();
  pdl_sync();
  if (threadIdx.x == 0) {
    if (!ptx::mbar_wait(ptx::smem_u32(&bar), 0u, &abort_flag, limit_cycles)) *(volatile int*)status = ST_PROBE;
  }
}

}  // namespace

cudaError_t launch_bounded_wait_probe(long long limit_cycles, int* status, cudaStream_t st) {
  return launch_pdl(bounded_wait_probe_kernel, dim3(1), dim3(32), 0, st, limit_cycles, status);
}

}  // namespace marche
