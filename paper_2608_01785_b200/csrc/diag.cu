// Diagnostic kernel for the bounded-wait protocol of the step's kernels.
//
// Every wait inside the kernels (on an mbarrier, or on a word another block writes) gives up after a time limit:
// the waiting thread raises its block's abort flag, records HS_ERR_TIMEOUT in the device status word, every role
// leaves its loop, the block lets copies in flight land, frees its tensor memory and returns -- nothing traps
// and the context stays usable.  hs_op_wait_probe runs exactly that sequence on purpose, with a limit given by
// the caller: one block whose threads wait on an mbarrier that nobody ever arrives on.  It is the way to see the
// protocol work without a real fault.
#include "../../include/horizonserve_ops.h"
#include "kernels.h"
#include "ptx.cuh"

namespace hs {
namespace {

constexpr int PROBE_THREADS = 96;     // three warps: a "producer", an "issuer" that owns tensor memory, a "consumer"
constexpr uint32_t PROBE_TMEM_COLS = 32;

struct ProbeParams {
  unsigned long long limit_ns;
  int* status;                        // device status word
  unsigned long long* waited_ns;      // nullable: time the first waiter spent before it gave up
};

__global__ void __launch_bounds__(PROBE_THREADS, 1) wait_probe_kernel(const ProbeParams p) {
  __shared__ __align__(8) uint64_t never;       // armed for one arrival that does not come
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_word;
  volatile int* abort_flag = &abort_word;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    mbar_init(&never, 1);
    abort_word = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(&tmem_slot, PROBE_TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_slot;

  // every role waits the way the step's kernels do: one elected thread polls with the time limit, the others
  // of the block learn of the failure through the abort flag the next time they look
  if (lane == 0) {
    const unsigned long long t0 = globaltimer_ns();
    const bool ok = mbar_wait(&never, 0, abort_flag, p.status, p.limit_ns);
    if (!ok && warp == 0 && p.waited_ns) *p.waited_ns = globaltimer_ns() - t0;
  }
  __syncwarp();
  if (*abort_flag) drain_after_abort();
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, PROBE_TMEM_COLS);
  }
}

}  // namespace
}  // namespace hs

using namespace hs;

extern "C" hs_status_t hs_op_wait_probe(uint64_t limit_ns, int32_t* status_dev, uint64_t* waited_ns_dev,
                                        void* cuda_stream) {
  if (!status_dev) return HS_ERR_INVALID_ARG;
  // the probe exists to show a wait giving up quickly: refuse limits a test should never sit through
  if (limit_ns < 1000 || limit_ns > 100000000ull) return HS_ERR_INVALID_ARG;
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return HS_ERR_CUDA;
  if (major != 10) return HS_ERR_CUDA;
  ProbeParams p{};
  p.limit_ns = limit_ns;
  p.status = status_dev;
  p.waited_ns = reinterpret_cast<unsigned long long*>(waited_ns_dev);
  wait_probe_kernel<<<1, PROBE_THREADS, 0, static_cast<cudaStream_t>(cuda_stream)>>>(p);
  return cudaGetLastError() == cudaSuccess ? HS_OK : HS_ERR_CUDA;
}
