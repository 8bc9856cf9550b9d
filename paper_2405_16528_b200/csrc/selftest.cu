// Self-test of the bounded device-side wait.  Every wait in the GEMM engine goes
// through ptx::mbar_wait, which gives up after a time limit, raises the CTA's
// abort flag and writes the status word instead of spinning forever.  The kernel
// here runs that same routine on a barrier nobody will ever arrive on, with a
// short limit, so that the give-up path can be exercised and its report checked
// on the host.  No copy, MMA or other asynchronous work is in flight: the kernel
// waits, records and returns.
#include "ptx.cuh"

namespace loqt {

__global__ void __launch_bounds__(32)
wait_timeout_selftest_kernel(uint32_t *status, uint64_t limit_ns, uint32_t *observed) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ uint32_t abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    ptx::mbar_init(smem_u32(&bar), 1);
    ptx::fence_barrier_init();
  }
  __syncthreads();
  // Phase 0 of a barrier that expects one arrival and gets none never completes.
  // Lane 0 runs into the limit; the other lanes leave through the abort flag.
  const bool done = ptx::mbar_wait(smem_u32(&bar), 0, &abort_flag, status, limit_ns);
  if (observed != nullptr) {
    if (done) atomicAdd(observed, 1u);                       // lanes whose wait (wrongly) completed
    if (threadIdx.x == 0) observed[1] = abort_flag;           // the CTA-wide abort flag
  }
}

}  // namespace loqt

using namespace loqt;

extern "C" loqt_status loqt_selftest_wait_timeout(void *ws, size_t ws_bytes, uint32_t limit_us, void *stream) {
  if (ws == nullptr || ws_bytes < 256) return LOQT_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return LOQT_ERR_ALIGNMENT;
  if (limit_us == 0 || limit_us > 100000) return LOQT_ERR_INVALID_ARG;  // at most 0.1 s
  loqt_status st;
  if ((st = check_arch()) != LOQT_OK) return st;
  uint32_t *words = static_cast<uint32_t *>(ws);
  // words[0]: the status word; words[2], words[3]: what the kernel observed
  wait_timeout_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(words, static_cast<uint64_t>(limit_us) * 1000ull,
                                                                                 words + 2);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? LOQT_OK : LOQT_ERR_CUDA;
}
