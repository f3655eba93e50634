// Self-test of the bounded barrier wait that the TMA kernels use: one small CTA waits, with a
// probe bound of 2^10 (about a millisecond), on a barrier that nobody ever arrives at.  The wait
// must give up, leave RECACHE_DEV_TIMEOUT (and where) in the status words, make the other
// threads' waits return at once, take the same drain as the real kernels and end normally, so that
// the context stays usable.  Nothing here hangs or faults: the wait is bounded by construction.
#include "common.cuh"

namespace {

constexpr uint32_t SELFTEST_PROBES = 1u << 10;

__global__ void __launch_bounds__(64) wait_selftest_kernel(int32_t* status, int32_t* report) {
  __shared__ __align__(8) uint64_t barrier_word;
  __shared__ int abort_word;
  const uint32_t bar = (uint32_t)__cvta_generic_to_shared(&barrier_word);
  volatile int* abort_flag = &abort_word;
  if (threadIdx.x == 0) {
    abort_word = 0;
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(1u) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const long long t0 = clock64();
  // warp 0 runs into the bound; warp 1 starts later and must be released by the abort flag
  if (threadIdx.x >= 32) { while (clock64() - t0 < 20000ll) { } }
  rc_mbar_wait<SELFTEST_PROBES, RC_WHERE_SELFTEST>(bar, 0u, abort_flag, status);
  const long long t1 = clock64();
  if (*abort_flag) rc_timeout_drain();
  __syncthreads();
  if (threadIdx.x == 0) {
    report[0] = *abort_flag;                                   // 1: the wait gave up
    report[1] = (int32_t)min((t1 - t0) >> 10, 0x7fffffffll);   // kilo-cycles spent waiting
  }
}

}  // namespace

cudaError_t rc_launch_wait_selftest(const recache_ctx* ctx, int32_t* report, cudaStream_t st) {
  wait_selftest_kernel<<<1, 64, 0, st>>>(ctx->status, report);
  return cudaGetLastError();
}
