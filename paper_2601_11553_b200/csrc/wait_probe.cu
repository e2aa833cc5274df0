// percache_debug_wait_probe: lets one bounded wait run out on purpose, in the only form that is safe to run.
//
// Every mbarrier wait of the tcgen05 kernels goes through mbar_wait() (ptx.cuh): it gives up after a time limit,
// records a code in the error word with a compare-and-swap, and also gives up as soon as it sees a code another
// role recorded.  The host then reports PERCACHE_E_DEVICE_TIMEOUT and the context stays usable.  This kernel
// exercises exactly that function on a shared-memory barrier that nobody ever arrives at: no bulk copy, no tensor
// memory, nothing in flight, so nothing has to be drained when the wait returns.
//   warp 0  waits with the caller's (short) limit; its wait runs out and it records DEV_ERR_WAIT_PROBE;
//   warp 1  waits on the same barrier with a limit 1000 times longer; it must leave early, because it sees the
//           error word, not because its own limit ran out.
#include "../../include/percache.h"
#include "kernels.h"
#include "ptx.cuh"

namespace pc {
namespace {

struct WaitProbeResult {
  int err_word;
  int first_returned, second_returned;           // what mbar_wait returned (0 = gave up)
  unsigned long long first_ns, second_ns;        // how long each waiter waited
};

__global__ void __launch_bounds__(64) wait_probe_kernel(WaitProbeResult* res, unsigned long long limit_ns) {
  __shared__ __align__(8) uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    fence_mbar_init();
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) {
    const unsigned long long t0 = globaltimer_ns();
    if (warp == 0) {
      res->first_returned = mbar_wait(&bar, 0u, &res->err_word, DEV_ERR_WAIT_PROBE, limit_ns) ? 1 : 0;
      res->first_ns = globaltimer_ns() - t0;
    } else {
      res->second_returned = mbar_wait(&bar, 0u, &res->err_word, DEV_ERR_GEMM_MMA, 1000ull * limit_ns) ? 1 : 0;
      res->second_ns = globaltimer_ns() - t0;
    }
  }
  __syncthreads();
}

}  // namespace
}  // namespace pc

extern "C" int percache_debug_wait_probe(int32_t device, uint32_t limit_us, int32_t* code_out, uint64_t* waited_ns) {
  using namespace pc;
  if (limit_us == 0 || limit_us > 2000) return PERCACHE_E_INVAL;      // the second waiter's own limit stays <= 2 s
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device < 0 || device >= n_dev) { cudaGetLastError(); return PERCACHE_E_CUDA; }
  if (cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); return PERCACHE_E_CUDA; }
  WaitProbeResult* d = nullptr;
  if (cudaMalloc(reinterpret_cast<void**>(&d), sizeof(WaitProbeResult)) != cudaSuccess) { cudaGetLastError(); return PERCACHE_E_NOMEM; }
  WaitProbeResult r{};
  int rc = PERCACHE_OK;
  if (cudaMemset(d, 0, sizeof(WaitProbeResult)) != cudaSuccess) rc = PERCACHE_E_CUDA;
  if (rc == PERCACHE_OK) {
    wait_probe_kernel<<<1, 64>>>(d, 1000ull * limit_us);
    if (cudaDeviceSynchronize() != cudaSuccess || cudaGetLastError() != cudaSuccess ||
        cudaMemcpy(&r, d, sizeof(r), cudaMemcpyDeviceToHost) != cudaSuccess)
      rc = PERCACHE_E_CUDA;
  }
  cudaFree(d);
  if (rc != PERCACHE_OK) return rc;
  if (code_out) *code_out = r.err_word;
  if (waited_ns) { waited_ns[0] = r.first_ns; waited_ns[1] = r.second_ns; }
  // the same mapping percache_prefill applies to its error word
  return r.err_word != 0 ? PERCACHE_E_DEVICE_TIMEOUT : PERCACHE_OK;
}
