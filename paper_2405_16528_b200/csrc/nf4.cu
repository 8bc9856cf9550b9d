// NF4 block quantise / requantise / dequantise streaming kernels (paper Section 5.1).
//
// All are HBM-bound: quantise moves 4 + 0.5625 bytes per element, requantise
// 4 + 2 * 0.5625, dequantise 0.5625 + 2 (bf16) or + 4 (fp32).  Loads and stores
// are 128-bit where alignment allows.  To stay memory-bound the kernels must be
// frugal with instructions (a few per element), so the work is dealt out row-wise:
// a thread keeps its position inside the row for the whole kernel and walks down
// the rows with pointer increments - no division, no 64-bit index arithmetic per
// item - and it has the loads of several rows in flight before it works on the
// first.
#include "common.cuh"

namespace loqt {

constexpr int kQThreads = 256;

// Row-wise distribution of a block's 256 threads: `per_row` threads (a power of two,
// 2^log2) side by side along a row, 256 / per_row rows per pass; blockIdx.x selects
// the chunk of the row, blockIdx.y the first rows.
struct RowDeal {
  int log2;  // log2 of the threads (or thread groups) a block puts side by side in a row
  dim3 grid;
};

// units: work units per row (one per thread or thread group); per_block: units a
// block holds (256 threads, or 64 groups of four); the grid covers the row in x and
// as many rows in y as `resident` blocks allow.
static RowDeal deal_rows(int units, int per_block, int rows, int resident) {
  RowDeal d;
  d.log2 = 0;
  while ((1 << d.log2) < units && (1 << d.log2) < per_block) ++d.log2;
  const int per_row = 1 << d.log2;
  const int gx = (units + per_row - 1) / per_row;
  const int rows_per_pass = per_block / per_row;
  int gy = (rows + rows_per_pass - 1) / rows_per_pass;
  int cap = resident / gx;
  if (cap < 1) cap = 1;
  if (gy > cap) gy = cap;
  if (gy > 65535) gy = 65535;
  d.grid = dim3(static_cast<unsigned>(gx), static_cast<unsigned>(gy > 0 ? gy : 1));
  return d;
}

template <typename Kernel>
static int resident_blocks(Kernel kernel) {
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kQThreads, 0) != cudaSuccess || per_sm < 1) per_sm = 1;
  return sm_count() * per_sm;
}

// ---------------------------------------------------------------------------
// quantise:   fp32 [rows][ld_src] -> codes [rows][ld/2], absmax [rows][ld/64]
// requantise: W_q <- q_NF4(deq32(W_q) + s * src), in place (the streaming half of
//             the two-pass merge)
// residual:   quantise `src` and also write bf16(ref - deq32(codes)) for every real
//             element (the error-compensation step: `ref` is the weight matrix
//             the quantised one should approximate, `src` what is quantised)
// Four threads share one block of 64 weights.  Where the whole block lies inside
// the matrix, thread l loads the 16-byte pieces l, l + 4, l + 8, l + 12 of its 256
// bytes, so that every load instruction of the group covers 64 contiguous bytes
// (whole 32-byte sectors); it then owns elements 16 k + 4 l .. + 3, k = 0..3, and
// the four threads exchange 16-bit pieces of their code words by shuffles so that
// each stores 8 contiguous bytes of codes.  A block cut short by the matrix edge
// is read element by element, 16 consecutive elements per thread.  The
// requantiser also loads its 16 old codes and the block's old scale.
// ---------------------------------------------------------------------------
enum : int { kQuantise = 0, kRequantise = 1, kQuantiseResidual = 2 };

struct QuantLoad {
  float v[16];
  uint2 old;
  float Mold;
};

template <bool kVec, int kMode>
__global__ void __launch_bounds__(kQThreads)
nf4_quantize_kernel(const float *__restrict__ src, int64_t ld_src, float s, uint8_t *__restrict__ codes,
                    float *__restrict__ absmax, int rows, int cols, int ld, const float *__restrict__ ref,
                    int64_t ld_ref, __nv_bfloat16 *__restrict__ resid, int64_t ld_resid, int gx_log2) {
  constexpr bool kRequant = (kMode == kRequantise);
  __shared__ Nf4Tables tab;
  nf4_tables_init(tab, threadIdx.x);
  __syncthreads();

  const int nb = ld / kBlock;
  const int l = threadIdx.x & 3;          // lane within the 4-thread group
  const int group = threadIdx.x >> 2;     // 64 groups per block
  const int gx = group & ((1 << gx_log2) - 1), gy = group >> gx_log2;
  const int b = (static_cast<int>(blockIdx.x) << gx_log2) + gx;  // NF4 block inside the row
  const int rows_per_pass = 64 >> gx_log2;
  const int row_stride = static_cast<int>(gridDim.y) * rows_per_pass;
  const int row_first = static_cast<int>(blockIdx.y) * rows_per_pass;  // of this block: the same for all its threads
  const int c0 = b * kBlock + 16 * l;  // first element of this thread's 8 bytes of codes
  const bool col_live = b < nb;
  const bool wide = kVec && (b + 1) * kBlock <= cols;  // the whole block is inside the matrix: interleaved ownership
  // element of the row that v[j] holds
  auto elem = [&](int j) { return wide ? b * kBlock + 16 * (j >> 2) + 4 * l + (j & 3) : c0 + j; };
  // Pieces of 16 bits (four codes) change hands inside the group: piece p of thread j
  // goes to position j of thread p.  Used to turn the old codes of 16 consecutive
  // elements into those of the interleaved elements and back (the map is its own
  // inverse).  All lanes of the warp take part.
  auto exchange = [&](uint2 w) {
    const unsigned long long w64 = (static_cast<unsigned long long>(w.y) << 32) | w.x;
    unsigned long long out = 0;
#pragma unroll
    for (int d = 0; d < 4; ++d) {
      const int p = l ^ d;
      uint32_t piece = static_cast<uint32_t>(w64 >> (16 * p)) & 0xFFFFu;
      if (d != 0) piece = __shfl_xor_sync(0xffffffffu, piece, d);
      out |= static_cast<unsigned long long>(piece) << (16 * p);
    }
    return make_uint2(static_cast<uint32_t>(out), static_cast<uint32_t>(out >> 32));
  };

  // Issues the loads of one item: 16 source values and, for the requantiser, the
  // 16 old codes and the old scale.  Elements past `cols` read as zero.
  auto fetch = [&](int row, QuantLoad &q) {
    const bool live = col_live && row < rows;
    q.old = make_uint2(kZeroWord, kZeroWord);
    q.Mold = 0.0f;
    if (kRequant && live) {
      q.old = *reinterpret_cast<const uint2 *>(codes + static_cast<int64_t>(row) * (ld / 2) + (c0 >> 1));
      q.Mold = absmax[static_cast<int64_t>(row) * nb + b];
    }
    const float *p = src + static_cast<int64_t>(row) * ld_src;
    if (live && wide) {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float4 a = __ldg(reinterpret_cast<const float4 *>(p + b * kBlock) + 4 * k + l);
        q.v[4 * k] = a.x; q.v[4 * k + 1] = a.y; q.v[4 * k + 2] = a.z; q.v[4 * k + 3] = a.w;
      }
    } else {
#pragma unroll
      for (int j = 0; j < 16; ++j) q.v[j] = (live && c0 + j < cols) ? __ldg(p + c0 + j) : 0.0f;
    }
  };

  // Quantises one item whose loads have arrived.  Every thread of a warp calls this
  // the same number of times (the shuffles need all lanes).
  auto work = [&](int row, QuantLoad &q) {
    const bool live = col_live && row < rows;
    if (kRequant) {
      const uint2 x = exchange(q.old);
      if (wide) q.old = x;
    }
    float m = 0.0f;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      if (kRequant) {
        const uint32_t code = ((j < 8 ? q.old.x : q.old.y) >> (4 * (j & 7))) & 15u;
        q.v[j] = fmaf(s, q.v[j], q.Mold * tab.level[code]);
      }
      m = fmaxf(m, fabsf(q.v[j]));
    }
    // (requantiser: every thread of the block has read the old scale by now - the
    // shuffles need its value - so lane 0 may replace it below)
    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
    uint2 w = make_uint2(kZeroWord, kZeroWord);  // codes of v[0..15]
    if (live && m > 0.0f) {
      const Nf4Divisor d = nf4_divisor(m);
      const float lo[8] = {q.v[0], q.v[1], q.v[2], q.v[3], q.v[4], q.v[5], q.v[6], q.v[7]};
      const float hi[8] = {q.v[8], q.v[9], q.v[10], q.v[11], q.v[12], q.v[13], q.v[14], q.v[15]};
      if (d.exact) {
        w.x = nf4_quantize8<true>(tab, lo, d);
        w.y = nf4_quantize8<true>(tab, hi, d);
      } else {
        w.x = nf4_quantize8<false>(tab, lo, d);
        w.y = nf4_quantize8<false>(tab, hi, d);
      }
    }
    const uint2 wx = exchange(w);  // (every lane: the shuffles need the whole warp)
    if (!live) return;
    *reinterpret_cast<uint2 *>(codes + static_cast<int64_t>(row) * (ld / 2) + (c0 >> 1)) = wide ? wx : w;
    if (l == 0) absmax[static_cast<int64_t>(row) * nb + b] = m;
    if (kMode == kQuantiseResidual && c0 < cols) {
      const float *rp = ref + static_cast<int64_t>(row) * ld_ref;
      __nv_bfloat16 *dp = resid + static_cast<int64_t>(row) * ld_resid;
      float e[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const uint32_t code = ((j < 8 ? w.x : w.y) >> (4 * (j & 7))) & 15u;
        const float t = (wide || c0 + j < cols) ? (ref == src ? q.v[j] : __ldg(rp + elem(j))) : 0.0f;
        e[j] = __fsub_rn(t, __fmul_rn(m, tab.level[code]));  // two roundings, as the definition has them
      }
      if (wide) {
#pragma unroll
        for (int k = 0; k < 4; ++k)  // four runs of four elements, 8 bytes each
          *reinterpret_cast<uint2 *>(dp + elem(4 * k)) = make_uint2(pack_bf16x2(e[4 * k], e[4 * k + 1]), pack_bf16x2(e[4 * k + 2], e[4 * k + 3]));
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j)
          if (c0 + j < cols) dp[c0 + j] = __float2bfloat16_rn(e[j]);
      }
    }
  };

  // Two rows per trip: both rows' loads are issued before the first is worked on.
  // (Keeping the loads of a further pair in flight costs registers and occupancy and
  // was measured slower.)
#pragma unroll 1
  for (int base = row_first; base < rows; base += 2 * row_stride) {
    QuantLoad qa, qb;
    const int ra = base + gy, rb = ra + row_stride;
    fetch(ra, qa);
    fetch(rb, qb);
    work(ra, qa);
    work(rb, qb);
  }
}

// ---------------------------------------------------------------------------
// dequantise: one thread per 8 consecutive elements (one 32-bit word of codes,
// one 16- or 32-byte store, so that a warp's stores are contiguous), the words
// of four rows in flight per trip.  Two codes are looked up at a time: a byte of
// the code word indexes a 256-entry table of level pairs, and one packed
// multiply scales the pair.
// ---------------------------------------------------------------------------
constexpr int kDqRows = 4;  // rows a thread has in flight

// Doubly quantised scales of a matrix (null codes8: plain fp32 scales are used).
struct DqScales {
  const uint8_t *codes8;
  const float *c1;
  const float *offset;
};

struct Nf4PairTable {
  float2 pair[256];  // pair[b] = {level[b & 15], level[b >> 4]}
};
__device__ __forceinline__ void nf4_pairs_init(Nf4PairTable &t, int tid) {
  if (tid < 256) t.pair[tid] = make_float2(c_nf4_level[tid & 15], c_nf4_level[tid >> 4]);
}

// Expands word h (elements 8 h .. 8 h + 7) of rows row0, row0 + row_stride, ...
template <bool kBf16, bool kVec, bool kDq>
__device__ __forceinline__ void dequantize_rows(const Nf4PairTable &tab, const uint8_t *__restrict__ codes,
                                                const float *__restrict__ absmax, DqScales dq, void *__restrict__ dst,
                                                int64_t ld_dst, int rows, int cols, int ld, int h, int row0, int row_stride) {
  const int wpr = ld / 8, nb = ld / kBlock;
  const int c0 = h * 8;
  if (h >= wpr || c0 >= cols) return;
  const bool full = kVec && (c0 + 8 <= cols);
#pragma unroll 1
  for (int base = row0; base < rows; base += kDqRows * row_stride) {
    uint32_t w[kDqRows];
    float M[kDqRows];
#pragma unroll
    for (int u = 0; u < kDqRows; ++u) {
      const int row = base + u * row_stride;
      w[u] = kZeroWord;
      M[u] = 0.0f;
      if (row < rows) {
        w[u] = __ldg(reinterpret_cast<const uint32_t *>(codes) + static_cast<int64_t>(row) * wpr + h);
        const int64_t si = static_cast<int64_t>(row) * nb + (h >> 3);
        M[u] = kDq ? dq_scale(dq.codes8, dq.c1, dq.offset, si) : __ldg(absmax + si);
      }
    }
#pragma unroll
    for (int u = 0; u < kDqRows; ++u) {
      const int row = base + u * row_stride;
      if (row >= rows) break;
      const float2 M2 = make_float2(M[u], M[u]);
      float2 p[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) p[j] = __fmul2_rn(M2, tab.pair[(w[u] >> (8 * j)) & 0xFFu]);
      if (kBf16) {
        __nv_bfloat16 *o = reinterpret_cast<__nv_bfloat16 *>(dst) + static_cast<int64_t>(row) * ld_dst + c0;
        if (full) {
          *reinterpret_cast<uint4 *>(o) = make_uint4(pack_bf16x2(p[0].x, p[0].y), pack_bf16x2(p[1].x, p[1].y),
                                                     pack_bf16x2(p[2].x, p[2].y), pack_bf16x2(p[3].x, p[3].y));
        } else {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            if (c0 + 2 * j < cols) o[2 * j] = __float2bfloat16_rn(p[j].x);
            if (c0 + 2 * j + 1 < cols) o[2 * j + 1] = __float2bfloat16_rn(p[j].y);
          }
        }
      } else {
        float *o = reinterpret_cast<float *>(dst) + static_cast<int64_t>(row) * ld_dst + c0;
        if (full) {
          reinterpret_cast<float4 *>(o)[0] = make_float4(p[0].x, p[0].y, p[1].x, p[1].y);
          reinterpret_cast<float4 *>(o)[1] = make_float4(p[2].x, p[2].y, p[3].x, p[3].y);
        } else {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            if (c0 + 2 * j < cols) o[2 * j] = p[j].x;
            if (c0 + 2 * j + 1 < cols) o[2 * j + 1] = p[j].y;
          }
        }
      }
    }
  }
}

template <bool kBf16, bool kVec, bool kDq>
__global__ void __launch_bounds__(kQThreads)
nf4_dequantize_kernel(const uint8_t *__restrict__ codes, const float *__restrict__ absmax, DqScales dq,
                      void *__restrict__ dst, int64_t ld_dst, int rows, int cols, int ld, int wx_log2) {
  __shared__ Nf4PairTable tab;
  nf4_pairs_init(tab, threadIdx.x);
  __syncthreads();
  const int tx = threadIdx.x & ((1 << wx_log2) - 1), ty = threadIdx.x >> wx_log2;
  const int rows_per_pass = kQThreads >> wx_log2;
  dequantize_rows<kBf16, kVec, kDq>(tab, codes, absmax, dq, dst, ld_dst, rows, cols, ld, (static_cast<int>(blockIdx.x) << wx_log2) + tx,
                                    static_cast<int>(blockIdx.y) * rows_per_pass + ty, static_cast<int>(gridDim.y) * rows_per_pass);
}

// Several matrices to bf16 in one launch (the staging step of a batched merge):
// the grid is dealt to the matrices in proportion to their sizes; blocks cta0 ..
// cta0 + ctas - 1 work on matrix i, `chunks` of them side by side along a row.
struct DequantBatch {
  struct Item {
    const uint8_t *codes;
    const float *absmax;
    void *dst;
    int64_t ld_dst;
    int rows, cols, ld;
    int cta0, ctas, chunks, wx_log2;
  } item[kStageBatchMax];
  int count;
};

template <bool kVec>
__global__ void __launch_bounds__(kQThreads)
nf4_dequantize_batch_kernel(const __grid_constant__ DequantBatch batch) {
  __shared__ Nf4PairTable tab;
  nf4_pairs_init(tab, threadIdx.x);
  __syncthreads();
  int i = 0;
  while (i + 1 < batch.count && static_cast<int>(blockIdx.x) >= batch.item[i + 1].cta0) ++i;
  const DequantBatch::Item &m = batch.item[i];
  const int local = static_cast<int>(blockIdx.x) - m.cta0;
  const int bx = local % m.chunks, by = local / m.chunks;
  const int tx = threadIdx.x & ((1 << m.wx_log2) - 1), ty = threadIdx.x >> m.wx_log2;
  const int rows_per_pass = kQThreads >> m.wx_log2;
  dequantize_rows<true, kVec, false>(tab, m.codes, m.absmax, DqScales{nullptr, nullptr, nullptr}, m.dst, m.ld_dst, m.rows, m.cols, m.ld,
                                     (bx << m.wx_log2) + tx, by * rows_per_pass + ty, (m.ctas / m.chunks) * rows_per_pass);
}

// fp32 -> bf16 (round to nearest even), row-major with leading dimensions: one
// thread per 8 consecutive elements of a row, rows walked as above.
template <bool kVec>
__global__ void __launch_bounds__(kQThreads)
convert_f32_bf16_kernel(const float *__restrict__ src, int64_t ld_src, __nv_bfloat16 *__restrict__ dst, int64_t ld_dst,
                        int rows, int cols, int wx_log2) {
  const int tx = threadIdx.x & ((1 << wx_log2) - 1), ty = threadIdx.x >> wx_log2;
  const int rows_per_pass = kQThreads >> wx_log2;
  const int c0 = ((static_cast<int>(blockIdx.x) << wx_log2) + tx) * 8;
  if (c0 >= cols) return;
  const bool full = kVec && c0 + 8 <= cols;
  const int row_stride = static_cast<int>(gridDim.y) * rows_per_pass;
  for (int row = static_cast<int>(blockIdx.y) * rows_per_pass + ty; row < rows; row += row_stride) {
    const float *p = src + static_cast<int64_t>(row) * ld_src + c0;
    __nv_bfloat16 *o = dst + static_cast<int64_t>(row) * ld_dst + c0;
    if (full) {
      const float4 a = __ldg(reinterpret_cast<const float4 *>(p)), b = __ldg(reinterpret_cast<const float4 *>(p) + 1);
      *reinterpret_cast<uint4 *>(o) = make_uint4(pack_bf16x2(a.x, a.y), pack_bf16x2(a.z, a.w), pack_bf16x2(b.x, b.y), pack_bf16x2(b.z, b.w));
    } else {
      for (int j = 0; j < 8 && c0 + j < cols; ++j) o[j] = __float2bfloat16_rn(__ldg(p + j));
    }
  }
}

loqt_status convert_f32_bf16(const float *src, int64_t ld_src, void *dst, int64_t ld_dst, int rows, int cols,
                             cudaStream_t stream) {
  if (rows <= 0 || cols <= 0) return LOQT_OK;
  const bool vec = ((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15u) == 0 && (ld_src % 4) == 0 && (ld_dst % 8) == 0;
  auto kernel = vec ? convert_f32_bf16_kernel<true> : convert_f32_bf16_kernel<false>;
  const RowDeal d = deal_rows((cols + 7) / 8, kQThreads, rows, resident_blocks(kernel));
  kernel<<<d.grid, kQThreads, 0, stream>>>(src, ld_src, static_cast<__nv_bfloat16 *>(dst), ld_dst, rows, cols, d.log2);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? LOQT_OK : LOQT_ERR_CUDA;
}

// Launch of the quantiser in one of its three modes.
template <int kMode>
static loqt_status launch_quantiser(const float *src, int64_t ld_src, float s, const loqt_nf4_mat &dst, const float *ref, int64_t ld_ref,
                                    void *resid, int64_t ld_resid, bool vec, cudaStream_t stream) {
  auto kernel = vec ? nf4_quantize_kernel<true, kMode> : nf4_quantize_kernel<false, kMode>;
  const RowDeal d = deal_rows(dst.ld / kBlock, kQThreads / 4, dst.rows, resident_blocks(kernel));
  kernel<<<d.grid, kQThreads, 0, stream>>>(src, ld_src, s, dst.codes, dst.absmax, dst.rows, dst.cols, dst.ld, ref, ld_ref,
                                           static_cast<__nv_bfloat16 *>(resid), ld_resid, d.log2);
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
  return launch_quantiser<kQuantiseResidual>(src, ld_src, 1.0f, dst, ref, ld_ref, resid, ld_resid, vec, stream);
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
  const int resident = resident_blocks(kernel);
  int next = 0;
  for (int i = 0; i < n; ++i) {
    const loqt_nf4_mat &m = items[i].src;
    const int64_t words = static_cast<int64_t>(m.rows) * (m.ld / 8);
    int share = static_cast<int>((words * resident + total - 1) / total);  // this matrix's part of the resident grid
    if (share < 1) share = 1;
    const RowDeal d = deal_rows(m.ld / 8, kQThreads, (m.rows + kDqRows - 1) / kDqRows, share);
    const int chunks = static_cast<int>(d.grid.x), ctas = chunks * static_cast<int>(d.grid.y);
    batch.item[i] = {m.codes, m.absmax, items[i].dst, items[i].ld_dst, m.rows, m.cols, m.ld, next, ctas, chunks, d.log2};
    next += ctas;
  }
  batch.count = n;
  kernel<<<next, kQThreads, 0, stream>>>(batch);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? LOQT_OK : LOQT_ERR_CUDA;
}

// One matrix, fp32 or doubly quantised scales, bf16 or fp32 output.
template <bool kDq>
static loqt_status launch_dequantiser(const loqt_nf4_mat &src, DqScales dq, void *dst, int64_t ld_dst, int dst_is_bf16, cudaStream_t stream) {
  const uintptr_t a = reinterpret_cast<uintptr_t>(dst);
  const bool vec = (a & 15u) == 0 && (ld_dst % (dst_is_bf16 ? 8 : 4)) == 0;
  auto kernel = dst_is_bf16 ? (vec ? nf4_dequantize_kernel<true, true, kDq> : nf4_dequantize_kernel<true, false, kDq>)
                            : (vec ? nf4_dequantize_kernel<false, true, kDq> : nf4_dequantize_kernel<false, false, kDq>);
  const RowDeal d = deal_rows(src.ld / 8, kQThreads, (src.rows + kDqRows - 1) / kDqRows, resident_blocks(kernel));
  kernel<<<d.grid, kQThreads, 0, stream>>>(src.codes, src.absmax, dq, dst, ld_dst, src.rows, src.cols, src.ld, d.log2);
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
  if (items >= (1ll << 30)) return LOQT_ERR_UNSUPPORTED;
  const bool vec = (reinterpret_cast<uintptr_t>(src) & 15u) == 0 && (ld_src % 4) == 0;
  return launch_quantiser<kQuantise>(src, ld_src, 1.0f, dst, nullptr, 0, nullptr, 0, vec, static_cast<cudaStream_t>(stream));
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
  if (items >= (1ll << 31)) return LOQT_ERR_UNSUPPORTED;
  return launch_dequantiser<false>(src, DqScales{nullptr, nullptr, nullptr}, dst, ld_dst, dst_is_bf16, static_cast<cudaStream_t>(stream));
}

extern "C" loqt_status loqt_nf4_requantize(const float *delta, int64_t ld_delta, float s, loqt_nf4_mat Wq, void *stream) {
  loqt_status st = validate_nf4(Wq);
  if (st != LOQT_OK) return st;
  if (delta == nullptr || ld_delta < Wq.cols) return LOQT_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(delta) & 3u) != 0) return LOQT_ERR_ALIGNMENT;
  if ((st = check_arch()) != LOQT_OK) return st;
  const int64_t items = static_cast<int64_t>(Wq.rows) * (Wq.ld / kBlock);
  if (items >= (1ll << 30)) return LOQT_ERR_UNSUPPORTED;
  const bool vec = (reinterpret_cast<uintptr_t>(delta) & 15u) == 0 && (ld_delta % 4) == 0;
  return launch_quantiser<kRequantise>(delta, ld_delta, s, Wq, nullptr, 0, nullptr, 0, vec, static_cast<cudaStream_t>(stream));
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
  return launch_dequantiser<true>(src, DqScales{dq.codes8, dq.c1, dq.offset}, dst, ld_dst, dst_is_bf16, static_cast<cudaStream_t>(stream));
}
