// Failure-path probe for the bounded device-side waits.
//
// Every barrier wait of the tensor-core kernels goes through tc::mbar_wait, which gives up after a
// limit of SM cycles, records a code in the context's status word and lets the kernel return.
// In a healthy run no such wait ever runs out, so that path would never execute in a test.  This
// kernel makes it run without harming anything: one warp initialises a barrier that nothing will
// ever complete, waits on it through the same mbar_wait with a short limit, and returns when the
// limit has passed.  No trap, no fault, no unbounded loop: the context stays usable.
#include "tt_internal.h"
#include "tc_ptx.cuh"

namespace tt {
namespace {

__global__ void __launch_bounds__(32) wait_probe_kernel(int32_t* status, long long limit_cycles, int code) {
  __shared__ __align__(8) uint64_t s_bar;
  __shared__ int s_abort;
  if (threadIdx.x == 0) {
    tc::mbar_init(tc::smem_u32(&s_bar), 1);
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  // parity 0 of a freshly initialised barrier is the phase that has not completed yet
  bool ok = true;
  if (threadIdx.x == 0) ok = tc::mbar_wait(tc::smem_u32(&s_bar), 0u, &s_abort, status, code, limit_cycles);
  ok = __all_sync(0xffffffffu, ok);
  (void)ok;   // expired: the status word holds `code`; nothing is in flight, so there is nothing to drain
}

}  // namespace

cudaError_t launch_wait_probe(int32_t* status, long long limit_cycles, int code, cudaStream_t s) {
  wait_probe_kernel<<<1, 32, 0, s>>>(status, limit_cycles, code);
  return cudaGetLastError();
}

}  // namespace tt
