// Self-test of the failure path that every bounded device-side wait of the library shares.
//
// The tensor-core kernels never spin without a limit: a wait on an mbarrier (or on another CTA's
// counter) that does not complete within its time limit gives up, raises the CTA's abort flag, records
// GSHARD_ERR_TIMEOUT in the status word of the workspace, waits a bounded time for copies in
// flight, releases its tensor memory and returns, so that the context stays usable.  In a healthy
// run no wait ever gives up, which would leave that path untested; the kernel below walks it on
// purpose and harmlessly: one CTA allocates tensor memory, initialises an mbarrier that nothing
// will ever arrive at, waits on it with a short limit, and leaves through the same teardown
// sequence as the GEMM kernels.  Nothing faults, traps or hangs; the launch takes about the limit.
#include "kernels.cuh"
#include "sm100_ptx.cuh"

namespace gshard {
namespace {

__global__ void __launch_bounds__(64, 1) wait_timeout_probe_kernel(int* status, uint64_t limit_ns) {
  __shared__ uint64_t bar;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag_mem;
  volatile int* abort_flag = &abort_flag_mem;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    *abort_flag = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 1) {
    ptx::tmem_alloc(&tmem_slot, 32);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = tmem_slot;

  bool ok = true;
  if (warp == 0) {
    // a producer-style single-lane wait: phase 0 of the barrier never completes
    if (lane == 0) ok = ptx::mbar_wait(&bar, 0u, abort_flag, limit_ns);
  } else {
    // an epilogue-style whole-warp wait on the same barrier
    ok = ptx::mbar_wait_warp(&bar, 0u, abort_flag, lane, limit_ns);
  }

  // ------------------------------ teardown (as in the GEMM kernels) ---------------------------
  if (!ok) {
    *abort_flag = 1;
    set_device_status(status, GSHARD_ERR_TIMEOUT);
    const uint64_t t0 = ptx::globaltimer_ns();
    while (ptx::globaltimer_ns() - t0 < 20000ull) { __nanosleep(1000); }
  }
  __syncwarp();
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, 32);
  }
}

}  // namespace
}  // namespace gshard

extern "C" int gshard_moe_debug_wait_timeout(void* workspace, uint32_t limit_us, void* cuda_stream) {
  using namespace gshard;
  launch_counter().n = 0;
  if (workspace == nullptr || reinterpret_cast<uintptr_t>(workspace) % kAlign) return GSHARD_ERR_INVALID_ARG;
  if (limit_us == 0 || limit_us > 1000) return GSHARD_ERR_INVALID_ARG;    // at most a millisecond
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return GSHARD_ERR_CUDA; }
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return GSHARD_ERR_CUDA;
  if (major != 10) return GSHARD_ERR_ARCH;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int* status = static_cast<int*>(workspace);      // the status word is the first word of a workspace
  if (cudaMemsetAsync(status, 0, sizeof(int), st) != cudaSuccess) return GSHARD_ERR_CUDA;
  wait_timeout_probe_kernel<<<1, 64, 0, st>>>(status, (uint64_t)limit_us * 1000ull);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? GSHARD_OK : GSHARD_ERR_CUDA;
}
