// Double quantisation of the NF4 block scales (paper Section 2.4: the quantisation
// state is itself quantised, following QLoRA).  The fp32 scales of a matrix, taken
// in row-major order, are centred by their mean and stored as FP8 E4M3 codes, 256
// to a block, with one fp32 second-level scale per block:
//
//   offset = mean(c2);  per block: d = c2 - offset, m = max |d|,
//   code = E4M3( (d / m) * 448 ),  c1 = m / 448;        c2' = E4M3(code) * c1 + offset
//
// (every operation rounded to fp32 on its own).  Streaming kernels: 4 bytes in and
// 1 + 1/64 bytes out per scale, i.e. 1/16 of a byte per weight.
#include "common.cuh"

namespace loqt {

constexpr int kDqThreads = 256;
constexpr int kDqMaxPartials = 1024;

// Stage 1 of the mean: block b sums its own contiguous share of the scales in
// double precision, in a fixed order (thread-strided, then a fixed tree), so that
// the result does not depend on scheduling.
__global__ void __launch_bounds__(kDqThreads)
dq_partial_sum_kernel(const float *__restrict__ c2, int64_t n, int64_t chunk, double *__restrict__ partial) {
  __shared__ double red[kDqThreads];
  const int64_t lo = static_cast<int64_t>(blockIdx.x) * chunk;
  const int64_t hi = lo + chunk < n ? lo + chunk : n;
  double acc = 0.0;
  for (int64_t i = lo + threadIdx.x; i < hi; i += kDqThreads) acc += static_cast<double>(__ldg(c2 + i));
  red[threadIdx.x] = acc;
  __syncthreads();
  for (int s = kDqThreads / 2; s > 0; s >>= 1) {
    if (threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0) partial[blockIdx.x] = red[0];
}

// Stage 2 + quantisation: every block adds the partial sums in the same fixed
// order (so all agree on the offset), then codes its 256 scales.
__global__ void __launch_bounds__(kDqThreads)
dq_quantize_kernel(const float *__restrict__ c2, int64_t n, const double *__restrict__ partial, int n_partial,
                   uint8_t *__restrict__ codes8, float *__restrict__ c1, float *__restrict__ offset_out) {
  __shared__ double red[kDqThreads];
  __shared__ float wmax[kDqThreads / 32];
  double acc = 0.0;
  for (int i = threadIdx.x; i < n_partial; i += kDqThreads) acc += partial[i];
  red[threadIdx.x] = acc;
  __syncthreads();
  for (int s = kDqThreads / 2; s > 0; s >>= 1) {
    if (threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
    __syncthreads();
  }
  const float offset = static_cast<float>(red[0] / static_cast<double>(n));
  if (blockIdx.x == 0 && threadIdx.x == 0) *offset_out = offset;

  const int64_t i = static_cast<int64_t>(blockIdx.x) * kDqBlock + threadIdx.x;
  const bool live = i < n;
  const float d = live ? __fsub_rn(__ldg(c2 + i), offset) : 0.0f;
  float m = fabsf(d);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = m;
  __syncthreads();
  m = wmax[0];
#pragma unroll
  for (int w = 1; w < kDqThreads / 32; ++w) m = fmaxf(m, wmax[w]);
  if (threadIdx.x == 0) c1[blockIdx.x] = __fdiv_rn(m, 448.0f);
  if (live) codes8[i] = m > 0.0f ? static_cast<uint8_t>(float_to_e4m3(__fmul_rn(__fdiv_rn(d, m), 448.0f))) : static_cast<uint8_t>(0);
}

__global__ void __launch_bounds__(kDqThreads)
dq_dequantize_kernel(const uint8_t *__restrict__ codes8, const float *__restrict__ c1, const float *__restrict__ offset,
                     int64_t n, float *__restrict__ c2) {
  const int64_t stride = static_cast<int64_t>(gridDim.x) * kDqThreads;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * kDqThreads + threadIdx.x; i < n; i += stride) c2[i] = dq_scale(codes8, c1, offset, i);
}

static loqt_status check_scales(const loqt_dq_scales &dq) {
  if (dq.codes8 == nullptr || dq.c1 == nullptr || dq.offset == nullptr || dq.n <= 0) return LOQT_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(dq.c1) & 3u) != 0 || (reinterpret_cast<uintptr_t>(dq.offset) & 3u) != 0) return LOQT_ERR_ALIGNMENT;
  return LOQT_OK;
}

}  // namespace loqt

using namespace loqt;

extern "C" size_t loqt_scales_workspace_bytes(void) { return 256 + kDqMaxPartials * sizeof(double); }

extern "C" loqt_status loqt_scales_double_quantize(const float *absmax, loqt_dq_scales dst, void *ws, size_t ws_bytes, void *stream) {
  loqt_status st;
  if ((st = check_scales(dst)) != LOQT_OK) return st;
  if (absmax == nullptr) return LOQT_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(absmax) & 3u) != 0) return LOQT_ERR_ALIGNMENT;
  if (ws == nullptr || ws_bytes < loqt_scales_workspace_bytes()) return LOQT_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return LOQT_ERR_ALIGNMENT;
  if ((st = check_arch()) != LOQT_OK) return st;
  const int64_t n = dst.n;
  const int64_t blocks = (n + kDqBlock - 1) / kDqBlock;
  if (blocks >= (1ll << 31)) return LOQT_ERR_UNSUPPORTED;
  cudaStream_t stm = static_cast<cudaStream_t>(stream);
  double *partial = reinterpret_cast<double *>(static_cast<uint8_t *>(ws) + 256);
  // shares of at least 4096 scales, at most kDqMaxPartials of them
  int64_t parts = (n + 4095) / 4096;
  if (parts > kDqMaxPartials) parts = kDqMaxPartials;
  const int64_t chunk = (n + parts - 1) / parts;
  parts = (n + chunk - 1) / chunk;
  dq_partial_sum_kernel<<<static_cast<int>(parts), kDqThreads, 0, stm>>>(absmax, n, chunk, partial);
  dq_quantize_kernel<<<static_cast<int>(blocks), kDqThreads, 0, stm>>>(absmax, n, partial, static_cast<int>(parts), dst.codes8, dst.c1,
                                                                     dst.offset);
  count_launch(2);
  return cudaGetLastError() == cudaSuccess ? LOQT_OK : LOQT_ERR_CUDA;
}

extern "C" loqt_status loqt_scales_double_dequantize(loqt_dq_scales src, float *absmax, void *stream) {
  loqt_status st;
  if ((st = check_scales(src)) != LOQT_OK) return st;
  if (absmax == nullptr) return LOQT_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(absmax) & 3u) != 0) return LOQT_ERR_ALIGNMENT;
  if ((st = check_arch()) != LOQT_OK) return st;
  int64_t blocks = (src.n + kDqThreads - 1) / kDqThreads;
  const int64_t cap = static_cast<int64_t>(sm_count()) * 8;
  if (blocks > cap) blocks = cap;
  dq_dequantize_kernel<<<static_cast<int>(blocks), kDqThreads, 0, static_cast<cudaStream_t>(stream)>>>(src.codes8, src.c1, src.offset,
                                                                                                        src.n, absmax);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? LOQT_OK : LOQT_ERR_CUDA;
}
