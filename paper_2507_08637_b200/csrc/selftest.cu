// Self-test of the bounded-wait error path shared by the tensor-core kernels: one CTA waits, with a short
// limit, on an mbarrier that is one arrival short, so the wait runs out; the kernel must record the
// code in the status word, raise its abort flag, let the other role skip its work and return normally.
#include "common.cuh"
#include "tc_common.cuh"

namespace wersa {
using namespace tc;

namespace {

constexpr int kErrSelfTest = 99;

// 64 threads: warp 0 waits on `never` (expects two arrivals, gets one), warp 1 waits on `handoff`, which
// warp 0 would only signal after its own wait had succeeded -- it leaves through the abort flag instead.
__global__ void __launch_bounds__(64) k_selftest_wait(int* __restrict__ status, unsigned long long limit_ns,
                                                      int* __restrict__ observed) {
  __shared__ uint64_t never, handoff;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&never, 2);
    mbar_init(&handoff, 1);
    abort_flag = 0;
    fence_mbar_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) mbar_arrive(&never);   // one of the two arrivals the phase needs
  volatile int* af = &abort_flag;
  const int warp = threadIdx.x >> 5;
  bool ok;
  if (warp == 0) {
    ok = __all_sync(0xffffffffu, mbar_wait(&never, 0, af, status, kErrSelfTest, limit_ns));
    if (ok && threadIdx.x == 0) mbar_arrive(&handoff);
  } else {
    // a generous limit of its own: this role must leave because the CTA is aborting, not by its own clock
    ok = __all_sync(0xffffffffu, mbar_wait(&handoff, 0, af, status, kErrSelfTest + 1, 1000ull * limit_ns));
  }
  __syncthreads();
  if (threadIdx.x == 0) observed[0] = abort_flag;
  if ((threadIdx.x & 31) == 0) observed[1 + warp] = ok ? 1 : 0;
}

}  // namespace

cudaError_t launch_selftest_wait(const Ws& w, unsigned long long limit_ns, int* observed, cudaStream_t st) {
  k_selftest_wait<<<1, 64, 0, st>>>(w.status, limit_ns, observed);
  return cudaGetLastError();
}

}  // namespace wersa
