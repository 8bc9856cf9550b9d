// NF4 block quantise / requantise / dequantise streaming kernels (paper Section 5.1).
//
// All are HBM-bound: quantise moves 4 + 0.5625 bytes per element, requantise
// 4 + 2 * 0.5625, dequantise 0.5625 + 2 (bf16) or + 4 (fp32).  Loads and stores
// are 128-bit where alignment allows, and every thread keeps the next trip's
// loads in flight while it works on the current one.
#include "common.cuh"

namespace loqt {

constexpr int kQThreads = 256;

// ---------------------------------------------------------------------------
// quantise:   fp32 [rows][ld_src] -> codes [rows][ld/2], absmax [rows][ld/64]
// requantise: W_q <- q_NF4(deq32(W_q) + s * src), in place (the streaming half of
//             the two-pass merge)
// residual:   quantise `src` and also write bf16(ref - deq32(codes)) for every real
//             element (the error-compensation step: `ref` is the weight matrix
//             the quantised one should approximate, `src` what is quantised)
// Four threads share one block of 64 weights; each owns 16 consecutive elements
// (four 128-bit loads, one 64-bit store of 16 codes; the requantiser also loads
// its 16 old codes and the block's old scale).
// ---------------------------------------------------------------------------
struct QuantItem {
  uint32_t row, b;
  int c0;
  bool live;
};

enum : int { kQuantise = 0, kRequantise = 1, kQuantiseResidual = 2 };

template <bool kVec, int kMode>
__global__ void __launch_bounds__(kQThreads)
nf4_quantize_kernel(const float *__restrict__ src, int64_t ld_src, float s, uint8_t *__restrict__ codes,
                    float *__restrict__ absmax, int rows, int cols, int ld, const float *__restrict__ ref,
                    int64_t ld_ref, __nv_bfloat16 *__restrict__ resid, int64_t ld_resid) {
  constexpr bool kRequant = (kMode == kRequantise);
  __shared__ Nf4Tables tab;
  nf4_tables_init(tab, threadIdx.x);
  __syncthreads();

  const uint32_t nb = static_cast<uint32_t>(ld / kBlock);
  const uint32_t n_items = static_cast<uint32_t>(rows) * nb;  // one item = one NF4 block (host checks < 2^30)
  const uint32_t l = threadIdx.x & 3;                         // lane within the 4-thread group
  const uint32_t group0 = (blockIdx.x * kQThreads + threadIdx.x) >> 2;
  const uint32_t stride = (gridDim.x * kQThreads) >> 2;
  // All threads of a warp run the same trip count: idle groups still take part in the shuffles.
  const uint32_t trips = (n_items + stride - 1) / stride;

  auto item_of = [&](uint32_t it) {
    QuantItem q;
    const uint32_t item = group0 + it * stride;
    q.live = it < trips && item < n_items;
    q.row = q.live ? item / nb : 0;
    q.b = q.live ? item - q.row * nb : 0;
    q.c0 = static_cast<int>(q.b) * kBlock + 16 * static_cast<int>(l);
    return q;
  };
  // Issues the loads of one item: 16 source values and, for the requantiser, the
  // 16 old codes and the old scale.  Elements past `cols` read as zero.
  auto fetch = [&](const QuantItem &q, float (&v)[16], uint2 &old, float &Mold) {
    const float *p = src + static_cast<int64_t>(q.row) * ld_src + q.c0;
    old = make_uint2(kZeroWord, kZeroWord);
    Mold = 0.0f;
    if (kRequant && q.live) {
      old = *reinterpret_cast<const uint2 *>(codes + static_cast<int64_t>(q.row) * (ld / 2) + (q.c0 >> 1));
      Mold = absmax[static_cast<int64_t>(q.row) * nb + q.b];
    }
    if (kVec && q.live && q.c0 + 16 <= cols) {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float4 a = __ldg(reinterpret_cast<const float4 *>(p) + k);
        v[4 * k] = a.x; v[4 * k + 1] = a.y; v[4 * k + 2] = a.z; v[4 * k + 3] = a.w;
      }
    } else {
#pragma unroll
      for (int j = 0; j < 16; ++j) v[j] = (q.live && q.c0 + j < cols) ? __ldg(p + j) : 0.0f;
    }
  };

  QuantItem cur = item_of(0);
  float v[16], Mold;
  uint2 old;
  fetch(cur, v, old, Mold);
#pragma unroll 1
  for (uint32_t it = 0; it < trips; ++it) {
    const QuantItem nxt = item_of(it + 1);
    float vn[16], Mn;
    uint2 oldn;
    fetch(nxt, vn, oldn, Mn);  // in flight while this item is quantised

    float m = 0.0f;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      if (kRequant) {
        const uint32_t code = ((j < 8 ? old.x : old.y) >> (4 * (j & 7))) & 15u;
        v[j] = fmaf(s, v[j], Mold * tab.level[code]);
      }
      m = fmaxf(m, fabsf(v[j]));
    }
    // (requantiser: every thread of the block has read the old scale by now - the
    // shuffles need its value - so lane 0 may replace it below)
    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
    if (cur.live) {
      uint2 w = make_uint2(kZeroWord, kZeroWord);
      if (m > 0.0f) {
        const Nf4Divisor d = nf4_divisor(m);
        const float lo[8] = {v[0], v[1], v[2], v[3], v[4], v[5], v[6], v[7]};
        const float hi[8] = {v[8], v[9], v[10], v[11], v[12], v[13], v[14], v[15]};
        if (d.exact) {
          w.x = nf4_quantize8<true>(tab, lo, d);
          w.y = nf4_quantize8<true>(tab, hi, d);
        } else {
          w.x = nf4_quantize8<false>(tab, lo, d);
          w.y = nf4_quantize8<false>(tab, hi, d);
        }
      }
      *reinterpret_cast<uint2 *>(codes + static_cast<int64_t>(cur.row) * (ld / 2) + (cur.c0 >> 1)) = w;
      if (l == 0) absmax[static_cast<int64_t>(cur.row) * nb + cur.b] = m;
      if (kMode == kQuantiseResidual && cur.c0 < cols) {
        const float *rp = ref + static_cast<int64_t>(cur.row) * ld_ref + cur.c0;
        __nv_bfloat16 *dp = resid + static_cast<int64_t>(cur.row) * ld_resid + cur.c0;
        const bool full = kVec && (cur.c0 + 16 <= cols);
        float e[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const uint32_t code = ((j < 8 ? w.x : w.y) >> (4 * (j & 7))) & 15u;
          const float t = (full || cur.c0 + j < cols) ? (ref == src ? v[j] : __ldg(rp + j)) : 0.0f;
          e[j] = __fsub_rn(t, __fmul_rn(m, tab.level[code]));  // two roundings, as the definition has them
        }
        if (full) {
#pragma unroll
          for (int g = 0; g < 2; ++g) {
            uint4 pk;
            pk.x = pack_bf16x2(e[8 * g + 0], e[8 * g + 1]);
            pk.y = pack_bf16x2(e[8 * g + 2], e[8 * g + 3]);
            pk.z = pack_bf16x2(e[8 * g + 4], e[8 * g + 5]);
            pk.w = pack_bf16x2(e[8 * g + 6], e[8 * g + 7]);
            reinterpret_cast<uint4 *>(dp)[g] = pk;
          }
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (cur.c0 + j < cols) dp[j] = __float2bfloat16_rn(e[j]);
        }
      }
    }
    cur = nxt;
    old = oldn;
    Mold = Mn;
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = vn[j];
  }
}

// ---------------------------------------------------------------------------
// dequantise: one thread per 8 consecutive elements (one 32-bit word of codes,
// one 16- or 32-byte store, so that a warp's stores are contiguous), four
// independent words per trip so that enough loads are in flight.
// ---------------------------------------------------------------------------
constexpr int kDqUnroll = 4;

// Expands the code words first, first + stride, ... of one matrix.
// Doubly quantised scales of a matrix (null codes8: plain fp32 scales are used).
struct DqScales {
  const uint8_t *codes8;
  const float *c1;
  const float *offset;
};

template <bool kBf16, bool kVec, bool kDq = false>
__device__ __forceinline__ void dequantize_words(const Nf4Tables &tab, const uint8_t *__restrict__ codes,
                                                 const float *__restrict__ absmax, void *__restrict__ dst, int64_t ld_dst,
                                                 int rows, int cols, int ld, uint32_t first, uint32_t stride,
                                                 DqScales dq = DqScales{nullptr, nullptr, nullptr}) {
  const uint32_t wpr = static_cast<uint32_t>(ld / 8);  // code words per row
  const uint32_t nb = static_cast<uint32_t>(ld / kBlock);
  const uint32_t n_items = static_cast<uint32_t>(rows) * wpr;  // (host checks < 2^31)

  struct Word {
    uint32_t w, row;
    int c0;
    float M;
    bool live;
  };
  auto fetch = [&](uint32_t item) {
    Word q;
    q.live = item < n_items;
    q.row = q.live ? item / wpr : 0;
    const uint32_t h = q.live ? item - q.row * wpr : 0;
    q.c0 = static_cast<int>(h) * 8;
    q.live = q.live && q.c0 < cols;
    q.w = kZeroWord;
    q.M = 0.0f;
    if (q.live) {
      q.w = __ldg(reinterpret_cast<const uint32_t *>(codes + static_cast<int64_t>(q.row) * (ld / 2)) + h);
      const int64_t si = static_cast<int64_t>(q.row) * nb + (h >> 3);
      q.M = kDq ? dq_scale(dq.codes8, dq.c1, dq.offset, si) : __ldg(absmax + si);
    }
    return q;
  };

  Word cur[kDqUnroll];
#pragma unroll
  for (int u = 0; u < kDqUnroll; ++u) cur[u] = fetch(first + u * stride);
#pragma unroll 1
  for (uint32_t base = first; base < n_items; base += kDqUnroll * stride) {
    Word nxt[kDqUnroll];  // in flight while this trip's words are expanded
#pragma unroll
    for (int u = 0; u < kDqUnroll; ++u) nxt[u] = fetch(base + (kDqUnroll + u) * stride);
#pragma unroll
    for (int u = 0; u < kDqUnroll; ++u) {
      const Word &q = cur[u];
      if (!q.live) continue;
      float v[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) v[j] = q.M * tab.level[(q.w >> (4 * j)) & 15u];
      const bool full = kVec && (q.c0 + 8 <= cols);
      if (kBf16) {
        __nv_bfloat16 *o = reinterpret_cast<__nv_bfloat16 *>(dst) + static_cast<int64_t>(q.row) * ld_dst + q.c0;
        if (full) {
          uint4 pk;
          pk.x = pack_bf16x2(v[0], v[1]);
          pk.y = pack_bf16x2(v[2], v[3]);
          pk.z = pack_bf16x2(v[4], v[5]);
          pk.w = pack_bf16x2(v[6], v[7]);
          *reinterpret_cast<uint4 *>(o) = pk;
        } else {
#pragma unroll
          for (int j = 0; j < 8; ++j)
            if (q.c0 + j < cols) o[j] = __float2bfloat16_rn(v[j]);
        }
      } else {
        float *o = reinterpret_cast<float *>(dst) + static_cast<int64_t>(q.row) * ld_dst + q.c0;
        if (full) {
          reinterpret_cast<float4 *>(o)[0] = make_float4(v[0], v[1], v[2], v[3]);
          reinterpret_cast<float4 *>(o)[1] = make_float4(v[4], v[5], v[6], v[7]);
        } else {
#pragma unroll
          for (int j = 0; j < 8; ++j)
            if (q.c0 + j < cols) o[j] = v[j];
        }
      }
    }
#pragma unroll
    for (int u = 0; u < kDqUnroll; ++u) cur[u] = nxt[u];
  }
}

template <bool kBf16, bool kVec>
__global__ void __launch_bounds__(kQThreads)
nf4_dequantize_kernel(const uint8_t *__restrict__ codes, const float *__restrict__ absmax,
                      void *__restrict__ dst, int64_t ld_dst, int rows, int cols, int ld) {
  __shared__ Nf4Tables tab;
  nf4_tables_init(tab, threadIdx.x);
  __syncthreads();
  dequantize_words<kBf16, kVec>(tab, codes, absmax, dst, ld_dst, rows, cols, ld, blockIdx.x * kQThreads + threadIdx.x,
                                gridDim.x * kQThreads);
}

// The same with doubly quantised block scales (paper Section 2.4).
template <bool kBf16, bool kVec>
__global__ void __launch_bounds__(kQThreads)
nf4_dequantize_dq_kernel(const uint8_t *__restrict__ codes, DqScales dq, void *__restrict__ dst, int64_t ld_dst, int rows,
                         int cols, int ld) {
  __shared__ Nf4Tables tab;
  nf4_tables_init(tab, threadIdx.x);
  __syncthreads();
  dequantize_words<kBf16, kVec, true>(tab, codes, nullptr, dst, ld_dst, rows, cols, ld, blockIdx.x * kQThreads + threadIdx.x,
                                      gridDim.x * kQThreads, dq);
}

// Several matrices to bf16 in one launch (the staging step of a batched merge):
// the grid is dealt to the matrices in proportion to their sizes, blocks cta0 ..
// cta0 + ctas - 1 stride over matrix i.
struct DequantBatch {
  struct Item {
    const uint8_t *codes;
    const float *absmax;
    void *dst;
    int64_t ld_dst;
    int rows, cols, ld;
    int cta0, ctas;
  } item[kStageBatchMax];
  int count;
};

template <bool kVec>
__global__ void __launch_bounds__(kQThreads)
nf4_dequantize_batch_kernel(const __grid_constant__ DequantBatch batch) {
  __shared__ Nf4Tables tab;
  nf4_tables_init(tab, threadIdx.x);
  __syncthreads();
  int i = 0;
  while (i + 1 < batch.count && static_cast<int>(blockIdx.x) >= batch.item[i + 1].cta0) ++i;
  const DequantBatch::Item &m = batch.item[i];
  const uint32_t local = blockIdx.x - static_cast<uint32_t>(m.cta0);
  dequantize_words<true, kVec>(tab, m.codes, m.absmax, m.dst, m.ld_dst, m.rows, m.cols, m.ld, local * kQThreads + threadIdx.x,
                               static_cast<uint32_t>(m.ctas) * kQThreads);
}

// Grid of a streaming kernel: enough blocks for the work, at most as many as
// are resident at once (the kernels loop with a grid stride).
template <typename Kernel>
static int grid_for(Kernel kernel, int64_t threads_needed) {
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kQThreads, 0) != cudaSuccess || per_sm < 1) per_sm = 1;
  int64_t blocks = (threads_needed + kQThreads - 1) / kQThreads;
  const int64_t cap = static_cast<int64_t>(sm_count()) * per_sm;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  return static_cast<int>(blocks);
}

// fp32 -> bf16 (round to nearest even), row-major with leading dimensions.
__global__ void __launch_bounds__(kQThreads)
convert_f32_bf16_kernel(const float *__restrict__ src, int64_t ld_src, __nv_bfloat16 *__restrict__ dst, int64_t ld_dst,
                        int rows, int cols) {
  const int64_t total = static_cast<int64_t>(rows) * cols;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * kQThreads;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * kQThreads + threadIdx.x; i < total; i += stride) {
    const int r = static_cast<int>(i / cols);
    const int c = static_cast<int>(i - static_cast<int64_t>(r) * cols);
    dst[static_cast<int64_t>(r) * ld_dst + c] = __float2bfloat16_rn(__ldg(src + static_cast<int64_t>(r) * ld_src + c));
  }
}

loqt_status convert_f32_bf16(const float *src, int64_t ld_src, void *dst, int64_t ld_dst, int rows, int cols,
                             cudaStream_t stream) {
  const int64_t total = static_cast<int64_t>(rows) * cols;
  if (total <= 0) return LOQT_OK;
  convert_f32_bf16_kernel<<<grid_for(convert_f32_bf16_kernel, total), kQThreads, 0, stream>>>(
      src, ld_src, static_cast<__nv_bfloat16 *>(dst), ld_dst, rows, cols);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? LOQT_OK : LOQT_ERR_CUDA;
}

// dst <- q_NF4(src); resid <- bf16(ref - deq32(dst)).  ref may equal src.
loqt_status nf4_quantize_residual(const float *src, int64_t ld_src, const float *ref, int64_t ld_ref, loqt_nf4_mat dst,
                                  void *resid, int64_t ld_resid, cudaStream_t stream) {
  const int64_t items = static_cast<int64_t>(dst.rows) * (dst.ld / kBlock);
  if (items >= (1ll << 30)) return LOQT_ERR_UNSUPPORTED;
  const bool vec = ((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(ref) | reinterpret_cast<uintptr_t>(resid)) & 15u) == 0 &&
                   (ld_src % 4) == 0 && (ld_ref % 4) == 0 && (ld_resid % 8) == 0;
  auto kernel = vec ? nf4_quantize_kernel<true, kQuantiseResidual> : nf4_quantize_kernel<false, kQuantiseResidual>;
  kernel<<<grid_for(kernel, items * 4), kQThreads, 0, stream>>>(src, ld_src, 1.0f, dst.codes, dst.absmax, dst.rows, dst.cols, dst.ld, ref,
                                                                ld_ref, static_cast<__nv_bfloat16 *>(resid), ld_resid);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? LOQT_OK : LOQT_ERR_CUDA;
}

// dst_i <- bf16(deq(src_i)) for up to kStageBatchMax matrices, one launch.
loqt_status nf4_dequantize_bf16_batch(const StageItem *items, int n, cudaStream_t stream) {
  if (n <= 0) return LOQT_OK;
  if (n > kStageBatchMax) return LOQT_ERR_INVALID_ARG;
  DequantBatch batch;
  memset(&batch, 0, sizeof(batch));
  bool vec = true;
  int64_t total = 0;
  for (int i = 0; i < n; ++i) {
    const loqt_nf4_mat &m = items[i].src;
    const int64_t words = static_cast<int64_t>(m.rows) * (m.ld / 8);
    if (words >= (1ll << 31)) return LOQT_ERR_UNSUPPORTED;
    total += words;
    vec = vec && (reinterpret_cast<uintptr_t>(items[i].dst) & 15u) == 0 && (items[i].ld_dst % 8) == 0;
  }
  auto kernel = vec ? nf4_dequantize_batch_kernel<true> : nf4_dequantize_batch_kernel<false>;
  const int cap = grid_for(kernel, (total + kDqUnroll - 1) / kDqUnroll);
  int next = 0;
  for (int i = 0; i < n; ++i) {
    const loqt_nf4_mat &m = items[i].src;
    const int64_t words = static_cast<int64_t>(m.rows) * (m.ld / 8);
    int64_t ctas = (words * cap + total - 1) / total;                     // share of the grid
    const int64_t need = (words + kQThreads * kDqUnroll - 1) / (kQThreads * kDqUnroll);  // blocks with work
    if (ctas > need) ctas = need;
    if (ctas < 1) ctas = 1;
    batch.item[i] = {m.codes, m.absmax, items[i].dst, items[i].ld_dst, m.rows, m.cols, m.ld, next, static_cast<int>(ctas)};
    next += static_cast<int>(ctas);
  }
  batch.count = n;
  kernel<<<next, kQThreads, 0, stream>>>(batch);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? LOQT_OK : LOQT_ERR_CUDA;
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
  if (items >= (1ll << 30)) return LOQT_ERR_UNSUPPORTED;  // 32-bit block indices in the kernel
  const bool vec = (reinterpret_cast<uintptr_t>(src) & 15u) == 0 && (ld_src % 4) == 0;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  auto kernel = vec ? nf4_quantize_kernel<true, kQuantise> : nf4_quantize_kernel<false, kQuantise>;
  kernel<<<grid_for(kernel, items * 4), kQThreads, 0, s>>>(src, ld_src, 1.0f, dst.codes, dst.absmax, dst.rows, dst.cols, dst.ld, nullptr, 0,
                                                           nullptr, 0);
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
  if (items >= (1ll << 31)) return LOQT_ERR_UNSUPPORTED;  // 32-bit word indices in the kernel
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const bool vec = (a & 15u) == 0 && (ld_dst % (dst_is_bf16 ? 8 : 4)) == 0;
  auto kernel = dst_is_bf16 ? (vec ? nf4_dequantize_kernel<true, true> : nf4_dequantize_kernel<true, false>)
                            : (vec ? nf4_dequantize_kernel<false, true> : nf4_dequantize_kernel<false, false>);
  kernel<<<grid_for(kernel, (items + kDqUnroll - 1) / kDqUnroll), kQThreads, 0, s>>>(src.codes, src.absmax, dst, ld_dst, src.rows,
                                                                                     src.cols, src.ld);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? LOQT_OK : LOQT_ERR_CUDA;
}

extern "C" loqt_status loqt_nf4_requantize(const float *delta, int64_t ld_delta, float s, loqt_nf4_mat Wq, void *stream) {
  loqt_status st = validate_nf4(Wq);
  if (st != LOQT_OK) return st;
  if (delta == nullptr || ld_delta < Wq.cols) return LOQT_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(delta) & 3u) != 0) return LOQT_ERR_ALIGNMENT;
  if ((st = check_arch()) != LOQT_OK) return st;
  const int64_t items = static_cast<int64_t>(Wq.rows) * (Wq.ld / kBlock);
  if (items >= (1ll << 30)) return LOQT_ERR_UNSUPPORTED;  // 32-bit block indices in the kernel
  const bool vec = (reinterpret_cast<uintptr_t>(delta) & 15u) == 0 && (ld_delta % 4) == 0;
  cudaStream_t stm = static_cast<cudaStream_t>(stream);
  auto kernel = vec ? nf4_quantize_kernel<true, kRequantise> : nf4_quantize_kernel<false, kRequantise>;
  kernel<<<grid_for(kernel, items * 4), kQThreads, 0, stm>>>(delta, ld_delta, s, Wq.codes, Wq.absmax, Wq.rows, Wq.cols, Wq.ld, nullptr, 0,
                                                             nullptr, 0);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? LOQT_OK : LOQT_ERR_CUDA;
}

extern "C" loqt_status loqt_nf4_dequantize_dq(loqt_nf4_mat src, loqt_dq_scales dq, void *dst, int64_t ld_dst, int dst_is_bf16,
                                              void *stream) {
  if (dq.codes8 == nullptr || dq.c1 == nullptr || dq.offset == nullptr) return LOQT_ERR_INVALID_ARG;
  if (src.absmax == nullptr) src.absmax = dq.c1;  // (not read: the scales come from dq)
  loqt_status st = validate_nf4(src);
  if (st != LOQT_OK) return st;
  if (dq.n != static_cast<int64_t>(src.rows) * (src.ld / kBlock)) return LOQT_ERR_INVALID_ARG;
  if (dst == nullptr || ld_dst < src.cols) return LOQT_ERR_INVALID_ARG;
  const uintptr_t a = reinterpret_cast<uintptr_t>(dst);
  if ((a & (dst_is_bf16 ? 1u : 3u)) != 0) return LOQT_ERR_ALIGNMENT;
  if ((st = check_arch()) != LOQT_OK) return st;
  const int64_t items = static_cast<int64_t>(src.rows) * (src.ld / 8);
  if (items >= (1ll << 31)) return LOQT_ERR_UNSUPPORTED;
  const bool vec = (a & 15u) == 0 && (ld_dst % (dst_is_bf16 ? 8 : 4)) == 0;
  auto kernel = dst_is_bf16 ? (vec ? nf4_dequantize_dq_kernel<true, true> : nf4_dequantize_dq_kernel<true, false>)
                            : (vec ? nf4_dequantize_dq_kernel<false, true> : nf4_dequantize_dq_kernel<false, false>);
  kernel<<<grid_for(kernel, (items + kDqUnroll - 1) / kDqUnroll), kQThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      src.codes, DqScales{dq.codes8, dq.c1, dq.offset}, dst, ld_dst, src.rows, src.cols, src.ld);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? LOQT_OK : LOQT_ERR_CUDA;
}
