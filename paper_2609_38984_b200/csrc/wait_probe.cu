// Two diagnostic kernels: the self-test of the failure-reporting path of the device-side waits, and an empty kernel
// whose launch is the latency floor that the latency-bound stages (selection) are reported against.
//
// Every wait in the library's kernels (attention roles on their mbarriers, the bulk-copy ring of pack and scatter) goes
// through mbar_wait_bounded and, when its limit runs out, raises the timeout bit of the status word and lets the
// kernel return.  This kernel makes that happen on purpose in the only harmless way: one warp initialises a barrier
// that expects one arrival, nobody ever arrives, and the warp waits with a caller-given limit (microseconds), after
// which it reports and returns.  Nothing is left waiting and the context stays usable.
#include "swam_internal.cuh"

namespace swam {
namespace {

__global__ void __launch_bounds__(32) wait_probe_kernel(int* status, unsigned long long limit_cycles) {
  __shared__ __align__(8) unsigned long long bar;
  const uint32_t bar_a = (uint32_t)__cvta_generic_to_shared(&bar);
  if (threadIdx.x == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_a) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  const bool ok = mbar_wait_bounded(bar_a, 0, limit_cycles, nullptr);
  const bool any_timeout = __any_sync(0xffffffffu, !ok);
  if (threadIdx.x == 0) {
    if (any_timeout) atomicOr(status, ST_TIMEOUT);
    asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(bar_a) : "memory");
  }
}

__global__ void __launch_bounds__(32) noop_kernel() {}

}  // namespace

cudaError_t launch_noop(cudaStream_t st, int* launches) {
  ++*launches;
  noop_kernel<<<1, 32, 0, st>>>();
  return cudaGetLastError();
}

cudaError_t launch_wait_probe(int* status, unsigned long long limit_cycles, cudaStream_t st, int* launches) {
  ++*launches;
  wait_probe_kernel<<<1, 32, 0, st>>>(status, limit_cycles);
  return cudaGetLastError();
}

}  // namespace swam
