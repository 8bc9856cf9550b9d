// NF4 block quantise / dequantise streaming kernels (paper Section 5.1).
//
// Both kernels are HBM-bound: quantise moves 4 + 0.5625 bytes per element,
// dequantise 0.5625 + 2 (bf16) or + 4 (fp32).  Eight threads share one block of
// 64 weights; loads and stores are 128-bit where alignment allows.
#include "common.cuh"

namespace loqt {

constexpr int kQThreads = 256;

// ---------------------------------------------------------------------------
// quantise: fp32 [rows][ld_src] -> codes [rows][ld/2], absmax [rows][ld/64]
// ---------------------------------------------------------------------------
template <bool kVec>
__global__ void __launch_bounds__(kQThreads)
nf4_quantize_kernel(const float *__restrict__ src, int64_t ld_src, uint8_t *__restrict__ codes,
                    float *__restrict__ absmax, int rows, int cols, int ld) {
  __shared__ Nf4Tables tab;
  __shared__ __align__(16) uint8_t bins[kNf4Bins];
  nf4_tables_init(tab, threadIdx.x);
  nf4_bins_load(bins, threadIdx.x, kQThreads);
  __syncthreads();

  const int nb = ld / kBlock;
  const int64_t n_items = static_cast<int64_t>(rows) * nb;  // one item = one NF4 block
  const int l = threadIdx.x & 7;                            // lane within the 8-thread group
  const int64_t group0 = (static_cast<int64_t>(blockIdx.x) * kQThreads + threadIdx.x) >> 3;
  const int64_t stride = (static_cast<int64_t>(gridDim.x) * kQThreads) >> 3;
  // All 8 threads of a group run the same trip count, and a warp holds 4 whole
  // groups; inactive groups still take part in the shuffles.
  const int64_t trips = (n_items + stride - 1) / stride;

  for (int64_t it = 0; it < trips; ++it) {
    const int64_t item = group0 + it * stride;
    const bool live = item < n_items;
    const int row = live ? static_cast<int>(item / nb) : 0;
    const int b = live ? static_cast<int>(item - static_cast<int64_t>(row) * nb) : 0;
    const int c0 = b * kBlock;
    const float *p = src + static_cast<int64_t>(row) * ld_src + c0;
    // thread l owns elements [4l, 4l+4) and [32+4l, 32+4l+4) of the block
    float v[8];
    if (kVec && live && c0 + kBlock <= cols) {
      const float4 a = __ldg(reinterpret_cast<const float4 *>(p) + l);
      const float4 c = __ldg(reinterpret_cast<const float4 *>(p) + 8 + l);
      v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
      v[4] = c.x; v[5] = c.y; v[6] = c.z; v[7] = c.w;
    } else {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int e = (j < 4) ? (4 * l + j) : (32 + 4 * l + j - 4);
        v[j] = (live && c0 + e < cols) ? __ldg(p + e) : 0.0f;
      }
    }
    float m = 0.0f;
#pragma unroll
    for (int j = 0; j < 8; ++j) m = fmaxf(m, fabsf(v[j]));
    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 4));
    if (!live) continue;

    uint32_t w = kZeroWord;
    if (m > 0.0f) w = nf4_quantize8(tab, bins, v, nf4_divisor(m));
    uint8_t *crow = codes + static_cast<int64_t>(row) * (ld / 2) + c0 / 2;
    *reinterpret_cast<uint16_t *>(crow + 2 * l) = static_cast<uint16_t>(w & 0xffffu);
    *reinterpret_cast<uint16_t *>(crow + 16 + 2 * l) = static_cast<uint16_t>(w >> 16);
    if (l == 0) absmax[static_cast<int64_t>(row) * nb + b] = m;
  }
}

// ---------------------------------------------------------------------------
// dequantise: one thread per 8 consecutive elements (one 32-bit code word)
// ---------------------------------------------------------------------------
template <bool kBf16, bool kVec>
__global__ void __launch_bounds__(kQThreads)
nf4_dequantize_kernel(const uint8_t *__restrict__ codes, const float *__restrict__ absmax,
                      void *__restrict__ dst, int64_t ld_dst, int rows, int cols, int ld) {
  __shared__ Nf4Tables tab;
  nf4_tables_init(tab, threadIdx.x);
  __syncthreads();

  const int wpr = ld / 8;  // code words per row
  const int nb = ld / kBlock;
  const int64_t n_items = static_cast<int64_t>(rows) * wpr;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * kQThreads;
  for (int64_t item = static_cast<int64_t>(blockIdx.x) * kQThreads + threadIdx.x; item < n_items;
       item += stride) {
    const int row = static_cast<int>(item / wpr);
    const int wi = static_cast<int>(item - static_cast<int64_t>(row) * wpr);
    const int c0 = wi * 8;
    if (c0 >= cols) continue;
    const uint32_t w = __ldg(reinterpret_cast<const uint32_t *>(codes + static_cast<int64_t>(row) * (ld / 2)) + wi);
    const float M = __ldg(absmax + static_cast<int64_t>(row) * nb + (c0 >> 6));
    float v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = M * tab.level[(w >> (4 * j)) & 15u];
    const bool full = kVec && (c0 + 8 <= cols);
    if (kBf16) {
      __nv_bfloat16 *o = reinterpret_cast<__nv_bfloat16 *>(dst) + static_cast<int64_t>(row) * ld_dst + c0;
      if (full) {
        uint4 q;
        q.x = pack_bf16x2(v[0], v[1]);
        q.y = pack_bf16x2(v[2], v[3]);
        q.z = pack_bf16x2(v[4], v[5]);
        q.w = pack_bf16x2(v[6], v[7]);
        *reinterpret_cast<uint4 *>(o) = q;
      } else {
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (c0 + j < cols) o[j] = __float2bfloat16_rn(v[j]);
      }
    } else {
      float *o = reinterpret_cast<float *>(dst) + static_cast<int64_t>(row) * ld_dst + c0;
      if (full) {
        reinterpret_cast<float4 *>(o)[0] = make_float4(v[0], v[1], v[2], v[3]);
        reinterpret_cast<float4 *>(o)[1] = make_float4(v[4], v[5], v[6], v[7]);
      } else {
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (c0 + j < cols) o[j] = v[j];
      }
    }
  }
}

static int grid_for(int64_t threads_needed) {
  int64_t blocks = (threads_needed + kQThreads - 1) / kQThreads;
  const int64_t cap = static_cast<int64_t>(sm_count()) * 8;  // 8 resident CTAs of 256 threads per SM
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  return static_cast<int>(blocks);
}

}  // namespace loqt

using namespace loqt;

extern "C" loqt_status loqt_nf4_quantize(const float *src, int64_t ld_src, loqt_nf4_mat dst, void *stream) {
  loqt_status st = validate_nf4(dst);
  if (st != LOQT_OK) return st;
  if (src == nullptr || ld_src < dst.cols) return LOQT_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(src) & 3u) != 0) return LOQT_ERR_ALIGNMENT;
  if ((st = check_arch()) != LOQT_OK) return st;
  const int64_t items = static_cast<int64_t>(dst.rows) * (dst.ld / kBlock);
  const int grid = grid_for(items * 8);
  const bool vec = (reinterpret_cast<uintptr_t>(src) & 15u) == 0 && (ld_src % 4) == 0;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (vec)
    nf4_quantize_kernel<true><<<grid, kQThreads, 0, s>>>(src, ld_src, dst.codes, dst.absmax, dst.rows, dst.cols, dst.ld);
  else
    nf4_quantize_kernel<false><<<grid, kQThreads, 0, s>>>(src, ld_src, dst.codes, dst.absmax, dst.rows, dst.cols, dst.ld);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? LOQT_OK : LOQT_ERR_CUDA;
}

extern "C" loqt_status loqt_nf4_dequantize(loqt_nf4_mat src, void *dst, int64_t ld_dst, int dst_is_bf16,
                                           void *stream) {
  loqt_status st = validate_nf4(src);
  if (st != LOQT_OK) return st;
  if (dst == nullptr || ld_dst < src.cols) return LOQT_ERR_INVALID_ARG;
  const uintptr_t a = reinterpret_cast<uintptr_t>(dst);
  if ((a & (dst_is_bf16 ? 1u : 3u)) != 0) return LOQT_ERR_ALIGNMENT;
  if ((st = check_arch()) != LOQT_OK) return st;
  const int64_t items = static_cast<int64_t>(src.rows) * (src.ld / 8);
  const int grid = grid_for(items);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const bool vec = (a & 15u) == 0 && (ld_dst % (dst_is_bf16 ? 8 : 4)) == 0;
  if (dst_is_bf16) {
    if (vec) nf4_dequantize_kernel<true, true><<<grid, kQThreads, 0, s>>>(src.codes, src.absmax, dst, ld_dst, src.rows, src.cols, src.ld);
    else nf4_dequantize_kernel<true, false><<<grid, kQThreads, 0, s>>>(src.codes, src.absmax, dst, ld_dst, src.rows, src.cols, src.ld);
  } else {
    if (vec) nf4_dequantize_kernel<false, true><<<grid, kQThreads, 0, s>>>(src.codes, src.absmax, dst, ld_dst, src.rows, src.cols, src.ld);
    else nf4_dequantize_kernel<false, false><<<grid, kQThreads, 0, s>>>(src.codes, src.absmax, dst, ld_dst, src.rows, src.cols, src.ld);
  }
  count_launch();
  return cudaGetLastError() == cudaSuccess ? LOQT_OK : LOQT_ERR_CUDA;
}
