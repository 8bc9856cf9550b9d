// Process-wide helpers of the LoQT library: status strings, architecture check,
// launch counter, device status word.
#include <atomic>

#include "common.cuh"

namespace loqt {

static std::atomic<uint64_t> g_launches{0};

void count_launch(int n) { g_launches.fetch_add(static_cast<uint64_t>(n), std::memory_order_relaxed); }

loqt_status check_arch() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return LOQT_ERR_CUDA;
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return LOQT_ERR_CUDA;
  return major == 10 ? LOQT_OK : LOQT_ERR_ARCH;
}

int sm_count() {
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) != cudaSuccess) return sms;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 148;
  return sms;
}

loqt_status validate_nf4(const loqt_nf4_mat &m) {
  if (m.block != kBlock) return LOQT_ERR_UNSUPPORTED;
  if (m.codes == nullptr || m.absmax == nullptr) return LOQT_ERR_INVALID_ARG;
  if (m.rows <= 0 || m.cols <= 0 || m.ld < m.cols) return LOQT_ERR_INVALID_ARG;
  if (m.ld % kBlock != 0) return LOQT_ERR_ALIGNMENT;
  if ((reinterpret_cast<uintptr_t>(m.codes) & 15u) != 0 || (reinterpret_cast<uintptr_t>(m.absmax) & 3u) != 0)
    return LOQT_ERR_ALIGNMENT;
  return LOQT_OK;
}

}  // namespace loqt

extern "C" {

uint64_t loqt_launch_count(void) { return loqt::g_launches.load(std::memory_order_relaxed); }

const char *loqt_status_string(loqt_status st) {
  switch (st) {
    case LOQT_OK: return "ok";
    case LOQT_ERR_INVALID_ARG: return "invalid argument";
    case LOQT_ERR_ALIGNMENT: return "misaligned pointer or leading dimension";
    case LOQT_ERR_UNSUPPORTED: return "unsupported NF4 block size (must be 64) or size beyond the limit";
    case LOQT_ERR_WORKSPACE: return "workspace missing or too small";
    case LOQT_ERR_CUDA: return "CUDA call failed";
    case LOQT_ERR_TIMEOUT: return "device-side wait timed out";
    case LOQT_ERR_ARCH: return "device is not sm_100";
    case LOQT_ERR_NUMERIC: return "matrix numerically rank deficient (Cholesky pivot not positive)";
  }
  return "unknown status";
}

loqt_status loqt_device_status(const void *ws, void *stream) {
  if (ws == nullptr) return LOQT_ERR_INVALID_ARG;
  uint32_t word = 0;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(&word, ws, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return LOQT_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return LOQT_ERR_CUDA;
  if (word & loqt::kErrTimeout) return LOQT_ERR_TIMEOUT;
  return (word & loqt::kErrNumeric) ? LOQT_ERR_NUMERIC : LOQT_OK;
}

}  // extern "C"
