// moga_selftest_wait_timeout: runs the kernels' bounded mbarrier wait to its limit, on purpose
// and in isolation, so that the time-out path (status word, detail word, abort flag, orderly
// exit) is exercised without starving a barrier inside a real kernel.
//
// One CTA of 64 threads, one mbarrier that nothing ever arrives on.  Warp 0 waits on it with
// the caller's limit (capped at 100 ms) through the same helper the attention and router
// kernels use; when the limit passes it records MOGA_ERR_TIMEOUT in the workspace header.
// Warp 1 waits on the same barrier with a much longer limit and leaves through the abort
// flag warp 0 set, the way the other roles of a real kernel leave.  The kernel then returns
// normally: the context stays usable and nothing faults.
#include "moga_internal.cuh"
#include "sm100_ptx.cuh"

namespace moga {
namespace {

using namespace sm100;

constexpr uint32_t kSelftestWhere = 0x7e;   // "where" tag of the detail word for this kernel

__global__ void __launch_bounds__(64, 1)
wait_timeout_selftest_kernel(uint32_t* header, uint64_t limit_ns) {
  __shared__ __align__(8) uint64_t barrier_word;
  __shared__ uint32_t abort_word;
  const uint32_t bar = smem_u32(&barrier_word);
  volatile uint32_t* abort_flag = &abort_word;
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    abort_word = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5;
  const uint64_t t0 = global_timer_ns();
  // warp 0: the wait that runs out; warp 1: a wait that is released by the abort flag
  const WaitResult res = mbar_wait_bounded(bar, 0u, abort_flag, warp == 0 ? limit_ns : 40ull * limit_ns + 1000000ull);
  const uint64_t waited = global_timer_ns() - t0;
  if (res == kWaitExpired && warp == 0)
    report_status(header, MOGA_ERR_TIMEOUT, (kSelftestWhere << 24) | ((uint32_t)blockIdx.x << 8) | 0u);
  if (threadIdx.x == 0) {           // how long the expiring wait took, for the caller to check
    header[2] = (uint32_t)waited;
    header[3] = (uint32_t)(waited >> 32);
  }
  if (threadIdx.x == 32) header[4] = (uint32_t)res;   // how the second role left (kWaitAborted expected)
}

}  // namespace
}  // namespace moga

extern "C" moga_status moga_selftest_wait_timeout(void* ws, size_t ws_bytes, uint64_t limit_ns, void* stream) {
  if (ws == nullptr || ws_bytes < 256 || (reinterpret_cast<uintptr_t>(ws) & (moga::kWsAlign - 1)))
    return MOGA_ERR_WORKSPACE;
  if (limit_ns == 0 || limit_ns > 100000000ull) return MOGA_ERR_INVALID_ARG;   // at most 100 ms
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  MOGA_CUDA_OK(cudaMemsetAsync(ws, 0, 256, cs));
  moga::wait_timeout_selftest_kernel<<<1, 64, 0, cs>>>(static_cast<uint32_t*>(ws), limit_ns);
  MOGA_CUDA_OK(cudaGetLastError());
  return MOGA_OK;
}
