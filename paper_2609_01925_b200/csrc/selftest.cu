// Self-test of the failure-reporting path that every kernel of the library shares: a bounded mbarrier wait
// that runs out, the shared abort flag that ends the other roles' waits, the status word, and the host-side
// poll.  The kernel waits on a barrier that nothing ever arrives at, so the wait is certain to give up; it
// then returns by itself.  Nothing faults, traps or spins without a bound.
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace crisp {
using namespace sm100;

namespace {
constexpr long long kSelftestMaxLimitNs = 10ll * 1000ll * 1000ll;  // 10 ms

// Warp 0 waits with the short limit the caller chose; warp 1 waits with the library's normal limit and must
// be released early by warp 0's abort flag.  out[0], out[1]: how long each warp waited, in nanoseconds.
__global__ void __launch_bounds__(64) bounded_wait_selftest_kernel(int* status, unsigned long long* out,
                                                                   unsigned long long limit_ns) {
  __shared__ uint64_t never;
  __shared__ int abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(&never, 1);
    fence_mbar_init();
  }
  __syncthreads();
  if (lane == 0) {
    const unsigned long long t0 = global_timer_ns();
    const bool ok = warp == 0 ? mbar_wait_limit(&never, 0, &abort_flag, limit_ns) : mbar_wait(&never, 0, &abort_flag);
    out[warp] = global_timer_ns() - t0;
    if (ok) out[warp] = ~0ull;  // cannot happen: nothing arrives at the barrier
  }
  __syncthreads();
  if (threadIdx.x == 0 && abort_flag) atomicExch(status, CRISP_ERR_DEVICE_TIMEOUT);
}
}  // namespace

int launch_selftest_bounded_wait(void* ws, long long limit_ns, cudaStream_t stream) {
  if (limit_ns < 1 || limit_ns > kSelftestMaxLimitNs) return CRISP_ERR_INVALID_ARG;
  CRISP_CUDA_TRY(cudaMemsetAsync(ws, 0, kWsHeader, stream), "selftest: clear status");
  auto* out = reinterpret_cast<unsigned long long*>(static_cast<uint8_t*>(ws) + 64);
  bounded_wait_selftest_kernel<<<1, 64, 0, stream>>>(static_cast<int*>(ws), out, static_cast<unsigned long long>(limit_ns));
  CRISP_CUDA_TRY(cudaGetLastError(), "selftest: launch");
  return CRISP_OK;
}

}  // namespace crisp
