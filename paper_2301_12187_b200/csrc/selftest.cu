// Self-test of the bounded waits that every tensor-core kernel of the library relies on: a tiny
// kernel waits, with the same wait routines, on an mbarrier that nothing ever completes.  The waits
// must give up after the limit, latch DC_ERR_TIMEOUT and the site of the wait in the workspace
// header, tell the other role through the abort flag, and let the kernel return normally, so that
// the context stays usable.  No copy, tensor-core instruction or tensor memory is in flight.
#include "tc_ptx.cuh"

namespace {
using namespace tc;

constexpr uint32_t kSiteWarp = 0x90000u;   // the converged-warp wait (as the MMA and epilogue warps wait)
constexpr uint32_t kSiteLane = 0x90001u;   // the single-lane wait (as the producer lane waits)

__global__ void __launch_bounds__(64, 1) k_wait_probe(DcWsHeader *ws, unsigned long long limit_ns) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ uint32_t abort_word;
  __shared__ uint32_t gave_up;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);                       // one arrival expected; none will come
    abort_word = 0;
    gave_up = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  volatile uint32_t *abort_flag = &abort_word;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp == 0) {
    if (!warp_wait(&bar, 0, abort_flag, ws, kSiteWarp, limit_ns) && lane == 0) atomicAdd(&gave_up, 1u);
  } else if (lane == 0) {
    // starts later, so it normally learns of the timeout through the abort flag
    if (!mbar_wait(&bar, 0, abort_flag, ws, kSiteLane, 4 * limit_ns)) atomicAdd(&gave_up, 1u);
  }
  __syncthreads();
  if (threadIdx.x == 0) ws->pad[0] = gave_up;   // both roles must have left their wait
}

}  // namespace

extern "C" dc_status dc_selftest_bounded_wait(void *workspace, size_t workspace_bytes, unsigned int limit_us,
                                              dc_stream stream) {
  if (!workspace) return DC_ERR_WORKSPACE;
  if (workspace_bytes < sizeof(DcWsHeader)) return DC_ERR_WORKSPACE;
  if (!dc_aligned16(workspace)) return DC_ERR_ALIGNMENT;
  if (limit_us == 0 || limit_us > 100000u) return DC_ERR_INVALID_ARG;
  k_wait_probe<<<1, 64, 0, (cudaStream_t)stream>>>((DcWsHeader *)workspace, 1000ull * limit_us);
  return cudaGetLastError() == cudaSuccess ? DC_OK : DC_ERR_CUDA;
}
