// Host side of the LoQT linear layer: argument checks, TMA descriptors, kernel
// launches for forward, backward and merge (paper Section 2, Algorithm 1).
#include <atomic>
#include <mutex>

#include "merge.cuh"

namespace loqt {

// ---------------------------------------------------------------------------
// TMA descriptor construction (driver entry point resolved at run time, so the
// library does not link against libcuda)
// ---------------------------------------------------------------------------
using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void *ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  });
  return fn;
}

// bf16 row-major matrix [outer][inner] with `ld` elements per row; box
// box_inner x box_outer, 128-byte swizzle, out-of-range elements read as zero.
static bool make_map(CUtensorMap *map, const void *base, int64_t inner, int64_t outer, int64_t ld, int box_inner,
                     int box_outer) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(inner), static_cast<cuuint64_t>(outer)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(ld) * 2};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(box_inner), static_cast<cuuint32_t>(box_outer)};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Packed NF4 codes as a byte matrix [rows][ld/2]; box in bytes x rows.
static bool make_code_map(CUtensorMap *map, const Nf4Src &m, int box_bytes, int box_rows, CUtensorMapSwizzle swz) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(m.ld / 2), static_cast<cuuint64_t>(m.rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(m.ld / 2)};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(box_bytes), static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t *>(m.codes), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// A bf16 operand of the engine.  K-major: stored [rows][K]; MN-major: stored [K][rows].
struct Bf16Operand {
  const void *ptr;
  int64_t ld;
};

static bool map_operand(CUtensorMap *map, int kind, const Bf16Operand &op, int rows, int K, int rows_tile) {
  if (kind == OP_TMA_K) return make_map(map, op.ptr, K, rows, op.ld, kBK, rows_tile);
  return make_map(map, op.ptr, rows, K, op.ld, 64, kBK);
}

static Nf4Src nf4_src(const loqt_nf4_mat &m) { return Nf4Src{m.codes, m.absmax, m.rows, m.cols, m.ld, nullptr, nullptr, nullptr}; }
// The same matrix with doubly quantised scales (m.absmax is not used).
static Nf4Src nf4_src_dq(const loqt_nf4_mat &m, const loqt_dq_scales &dq) {
  return Nf4Src{m.codes, nullptr, m.rows, m.cols, m.ld, dq.codes8, dq.c1, dq.offset};
}

static loqt_status check_bf16(const void *p, int64_t ld, int64_t cols) {
  if (p == nullptr || ld < cols) return LOQT_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(p) & 15u) != 0 || (ld & 7) != 0) return LOQT_ERR_ALIGNMENT;
  return LOQT_OK;
}

// ---------------------------------------------------------------------------
// One GEMM launch
// ---------------------------------------------------------------------------
struct GemmCall {
  GemmParams p;
  Bf16Operand a[2], b[2];
};

// Cost model of pick_tile(), in SM cycles (measured on B200): one K stage of a
// 128 x 256 MMA pass, dequantising one 64-weight block, the epilogue per 32
// output columns of a 128-row half, and the per-tile fixed cost.
constexpr double kCyclesMma256 = 700.0;
constexpr double kNarrowTilePenalty = 1.15;  // N = 128 passes move more operand bytes per flop
constexpr double kCyclesDequantRow = 3.3;
constexpr double kCyclesEpilogueRow = 400.0;
constexpr double kCyclesFixed = 3000.0;
constexpr double kPairGain = 0.85;  // stage time of a CTA pair relative to two single CTAs (measured)

// Run eligible products as tcgen05 CTA pairs (cta_group::2).
#ifndef LOQT_USE_PAIRS
#define LOQT_USE_PAIRS 1
#endif
constexpr bool kUsePairs = LOQT_USE_PAIRS != 0;

// Launches per kernel variant (instrumentation: tests ask which instantiation a
// call ran) and the tile override of loqt_set_tile_override().
static std::atomic<uint64_t> g_variant_launches[16];
static std::atomic<int> g_force_bn{0}, g_force_mh{0}, g_force_pair{0};
static int variant_index(int bn, int mh, bool two, bool nf4) {
  return (bn == 256 ? 1 : 0) | (mh == 2 ? 2 : 0) | (two ? 4 : 0) | (nf4 ? 8 : 0);
}

template <int BN, int MH, bool TWO, bool NF4>
static loqt_status launch_cfg(const GemmCall &c, cudaStream_t stream) {
  using L = SmemLayout<BN, MH, TWO, NF4>;
  constexpr int BNL = L::kBNL;  // B rows one CTA stages
  TensorMaps maps;
  memset(&maps, 0, sizeof(maps));
  for (int s = 0; s < c.p.num_segs; ++s) {
    const Segment &sg = c.p.seg[s];
    if (sg.a_kind <= OP_TMA_MN) {
      if (!map_operand(&maps.a[s], sg.a_kind, c.a[s], c.p.M, sg.K, L::kBM)) return LOQT_ERR_CUDA;
    } else if (sg.a_kind == OP_NF4_K) {
      if (!make_code_map(&maps.ca[s], sg.a_nf4, 32, L::kBM, CU_TENSOR_MAP_SWIZZLE_NONE)) return LOQT_ERR_CUDA;
    } else {
      return LOQT_ERR_UNSUPPORTED;
    }
    if (sg.b_kind <= OP_TMA_MN) {
      if (!map_operand(&maps.b[s], sg.b_kind, c.b[s], c.p.N, sg.K, BNL)) return LOQT_ERR_CUDA;
    } else if (sg.b_kind == OP_NF4_K) {
      if (!make_code_map(&maps.cb[s], sg.b_nf4, 32, BNL, CU_TENSOR_MAP_SWIZZLE_NONE)) return LOQT_ERR_CUDA;
    } else {
      if (!make_code_map(&maps.cb[s], sg.b_nf4, BNL / 2, kBK,
                         BNL == 256 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B))
        return LOQT_ERR_CUDA;
    }
  }
  auto kernel = loqt_gemm_kernel<BN, MH, TWO, NF4>;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kDynamicBytes) != cudaSuccess)
    return LOQT_ERR_CUDA;
  int mt = (c.p.M + L::kBM - 1) / L::kBM;
  if (TWO) mt = (mt + 1) & ~1;  // pairs count M tiles in twos (see Sched)
  const int nt = (c.p.N + BN - 1) / BN;
  const int units = mt * nt * c.p.splits;
  int grid = units < sm_count() ? units : sm_count();
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cudaLaunchAttribute attr[2];
  int nattr = 0;
  // programmatic dependent launch: this kernel's prologue may overlap the previous
  // kernel's tail (the kernel itself waits before it touches global memory)
  attr[nattr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[nattr].val.programmaticStreamSerializationAllowed = 1;
  ++nattr;
  if (TWO) {
    grid &= ~1;  // whole pairs (`units` is even in this mode)
    if (grid < 2) grid = 2;
    attr[nattr].id = cudaLaunchAttributeClusterDimension;
    attr[nattr].val.clusterDim.x = 2;
    attr[nattr].val.clusterDim.y = 1;
    attr[nattr].val.clusterDim.z = 1;
    ++nattr;
  }
  cfg.attrs = attr;
  cfg.numAttrs = nattr;
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kNumThreads);
  cfg.dynamicSmemBytes = L::kDynamicBytes;
  cfg.stream = stream;
  const cudaError_t err = cudaLaunchKernelEx(&cfg, kernel, maps, c.p);
  count_launch();
  g_variant_launches[variant_index(BN, MH, TWO, NF4)].fetch_add(1, std::memory_order_relaxed);
  return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? LOQT_OK : LOQT_ERR_CUDA;
}

// Tile selection.  Candidates: BN in {256, 128}, rows per CTA 128 (two TMEM
// buffers, overlapped epilogue) or 256 (one buffer, every staged B tile used by
// two MMA passes).  A stage costs the larger of its tensor / shared-memory time
// and - when the B operand is NF4 - its dequantisation time (one pass over the
// CTA's B rows per stage, whatever the tile height); the single-buffered tile
// adds an exposed epilogue.
// Estimated time = waves x (stages x stage cost + exposed epilogue); smallest wins.
struct TileCfg {
  int bn, mh;
  bool two;
};

// Two CTAs on neighbouring M tiles can run as a tcgen05 pair when tiles pair up
// exactly: 256-wide tiles, an even number of M tiles (so both CTAs of a pair
// have the same N tile) and no split-K.
static bool pair_ok(const GemmCall &c, int bn, int mh) {
  const int mt = (c.p.M + mh * kHM - 1) / (mh * kHM);
  return kUsePairs && bn == 256 && (mt % 2 == 0) && c.p.splits == 1;
}

static TileCfg pick_tile(const GemmCall &c) {
  const int sms = sm_count();
  const bool b_nf4 = c.p.seg[0].b_kind >= OP_NF4_K;
  int kb = 0;
  for (int s = 0; s < c.p.num_segs; ++s) kb += (c.p.seg[s].K + kBK - 1) / kBK;
  if (c.p.splits > 1) kb = c.p.kb_per_split;
  const TileCfg cands[4] = {{256, 1, false}, {256, 2, false}, {128, 1, false}, {128, 2, false}};
  TileCfg best = {256, 1, false};
  double best_t = 1e300;
  for (TileCfg t : cands) {
    if (t.mh == 2 && c.p.M <= kHM) continue;
    if (t.bn == 256 && c.p.N <= 128) continue;
    const int units = ((c.p.M + t.mh * kHM - 1) / (t.mh * kHM)) * ((c.p.N + t.bn - 1) / t.bn) * c.p.splits;
    const double waves = (units + sms - 1) / sms;
    const double mma = kCyclesMma256 * t.mh * (t.bn == 256 ? 1.0 : 0.5 * kNarrowTilePenalty);
    const double deq = b_nf4 ? kCyclesDequantRow * t.bn : 0.0;
    const double stage = mma > deq ? mma : deq;
    const double epi = (t.mh == 2 ? 1.0 : 0.25) * kCyclesEpilogueRow * t.mh * t.bn / 32.0;
    double cost = waves * (kb * stage + epi + kCyclesFixed);
    if (t.bn == 256 && pair_ok(c, 256, t.mh)) cost *= kPairGain;  // it will run as CTA pairs
    if (cost < best_t) {
      best_t = cost;
      best = t;
    }
  }
  // a 256-wide choice runs as pairs where it can
  best.two = pair_ok(c, best.bn, best.mh);
  // A tile forced by loqt_set_tile_override() replaces the choice wherever the
  // kernel supports it for this product: pairs need 256-wide tiles and no split-K
  // (an odd number of M tiles is rounded up by one empty tile).
  const int fbn = g_force_bn.load(std::memory_order_relaxed);
  if (fbn != 0) {
    const int fmh = g_force_mh.load(std::memory_order_relaxed);
    const bool fpair = g_force_pair.load(std::memory_order_relaxed) != 0;
    const bool ok = !(fpair && (fbn != 256 || c.p.splits != 1 || !kUsePairs));
    if (ok) best = TileCfg{fbn, fmh, fpair};
  }
  return best;
}

template <bool NF4>
static loqt_status launch_tile(const GemmCall &c, const TileCfg &t, cudaStream_t stream) {

  if (t.two) return t.mh == 2 ? launch_cfg<256, 2, true, NF4>(c, stream) : launch_cfg<256, 1, true, NF4>(c, stream);
  if (t.bn == 256) return t.mh == 2 ? launch_cfg<256, 2, false, NF4>(c, stream) : launch_cfg<256, 1, false, NF4>(c, stream);
  return t.mh == 2 ? launch_cfg<128, 2, false, NF4>(c, stream) : launch_cfg<128, 1, false, NF4>(c, stream);
}

static loqt_status launch(GemmCall &c, cudaStream_t stream) {
  c.p.has_nf4 = 0;
  for (int s = 0; s < c.p.num_segs; ++s)
    if (c.p.seg[s].a_kind >= OP_NF4_K || c.p.seg[s].b_kind >= OP_NF4_K) c.p.has_nf4 = 1;
  const TileCfg t = pick_tile(c);
  if (c.p.has_nf4) return launch_tile<true>(c, t, stream);
  return launch_tile<false>(c, t, stream);
}

// ---------------------------------------------------------------------------
// Workspace layout: [0,256) status word | region 1 | region 2
// ---------------------------------------------------------------------------
static size_t align256(size_t v) { return (v + 255) & ~static_cast<size_t>(255); }
static int64_t ld_lowrank(int r) { return (static_cast<int64_t>(r) + 63) / 64 * 64; }  // bf16 T x r scratch

// Split-K factor of the dB product (M = r, N = in, K = T): enough splits to give every SM a tile.
static void db_splits(int r, int in, int T, int &splits, int &kb_per_split) {
  const int tiles = ((r + kHM - 1) / kHM) * ((in + (in > 128 ? 255 : 127)) / (in > 128 ? 256 : 128));
  const int kb_total = (T + kBK - 1) / kBK;
  int want = sm_count() / (tiles > 0 ? tiles : 1);
  if (want < 1) want = 1;
  if (want > 16) want = 16;
  const int max_by_k = kb_total / 4 > 0 ? kb_total / 4 : 1;  // at least 4 k-blocks per split
  if (want > max_by_k) want = max_by_k;
  kb_per_split = (kb_total + want - 1) / want;
  splits = (kb_total + kb_per_split - 1) / kb_per_split;
}

// out[M x N] (fp32) = (accumulate ? out : 0) + A^T B with A stored [K][M] and B stored
// [K][N] (both bf16, K outermost), split over K when the tiles alone would not
// fill the GPU; the partial sums are then added in a fixed order.
static loqt_status gemm_tn_f32(const void *a, int64_t lda, const void *b, int64_t ldb, int M, int N, int K, float *out,
                               int64_t ld_out, int accumulate, float *partial, uint32_t *status, cudaStream_t stm) {
  GemmCall c{};
  c.p.M = M; c.p.N = N; c.p.num_segs = 1;
  c.p.seg[0].K = K; c.p.seg[0].a_kind = OP_TMA_MN; c.p.seg[0].b_kind = OP_TMA_MN;
  c.a[0] = {a, lda}; c.b[0] = {b, ldb};
  int splits = 1, kbps = 1;
  db_splits(M, N, K, splits, kbps);
  c.p.splits = splits; c.p.kb_per_split = kbps; c.p.status = status; c.p.alpha = 1.0f;
  const int64_t ldp = (static_cast<int64_t>(N) + 3) / 4 * 4;
  if (splits == 1) {
    c.p.epi = EPI_F32; c.p.out = out; c.p.ld_out = ld_out; c.p.accumulate = accumulate;
  } else {
    c.p.epi = EPI_PARTIAL; c.p.out = partial; c.p.ld_out = ldp;
  }
  loqt_status st;
  if ((st = launch(c, stm)) != LOQT_OK) return st;
  if (splits > 1) {
    const int64_t total = static_cast<int64_t>(M) * N;
    int64_t blocks = (total + 255) / 256;
    const int64_t cap = static_cast<int64_t>(sm_count()) * 8;
    if (blocks > cap) blocks = cap;
    splitk_reduce_kernel<<<static_cast<int>(blocks), 256, 0, stm>>>(partial, splits, M, N, ldp, out, ld_out, accumulate);
    count_launch();
    if (cudaGetLastError() != cudaSuccess) return LOQT_ERR_CUDA;
  }
  return LOQT_OK;
}

}  // namespace loqt

using namespace loqt;

extern "C" size_t loqt_workspace_bytes(int op, int32_t out, int32_t in, int32_t r, int32_t T) {
  size_t total = 256;
  if (op == LOQT_OP_FWD || op == LOQT_OP_BWD) total += align256(static_cast<size_t>(T > 0 ? T : 0) * ld_lowrank(r) * 2);
  if (op == LOQT_OP_BWD) {
    int splits = 1, kbps = 1;
    db_splits(r, in, T > 0 ? T : 1, splits, kbps);
    if (splits > 1) total += align256(static_cast<size_t>(splits) * r * ((static_cast<size_t>(in) + 3) / 4 * 4) * 4);
    // bf16(deq(P_q)), out x roundup(r, 64): staged once per backward for v = dy P-hat
    total += align256(static_cast<size_t>(out > 0 ? out : 0) * ld_lowrank(r) * 2);
  }
  // merge: deq(P_q) as bf16, out x roundup(r, 64)
  if (op == LOQT_OP_MERGE || op == LOQT_OP_MERGE_SPLIT)
    total += align256(static_cast<size_t>(out > 0 ? out : 0) * ld_lowrank(r) * 2);
  // two-pass merge: the fp32 product P-hat B, out x roundup(in, 64)
  if (op == LOQT_OP_MERGE_SPLIT)
    total += align256(static_cast<size_t>(out > 0 ? out : 0) * ((static_cast<size_t>(in > 0 ? in : 0) + 63) / 64 * 64) * 4);
  // error-compensated initialisation: bf16 P, bf16 residual, fp32 B (+ split-K partials)
  if (op == LOQT_OP_COMPENSATE) {
    const size_t o = static_cast<size_t>(out > 0 ? out : 0), ld64 = (static_cast<size_t>(in > 0 ? in : 0) + 63) / 64 * 64;
    const size_t ld4 = (static_cast<size_t>(in > 0 ? in : 0) + 3) / 4 * 4;
    total += align256(o * ld_lowrank(r) * 2) + align256(o * ld64 * 2) + align256(static_cast<size_t>(r) * ld4 * 4);
    int splits = 1, kbps = 1;
    db_splits(r, in, out > 0 ? out : 1, splits, kbps);
    if (splits > 1) total += align256(static_cast<size_t>(splits) * r * ld4 * 4);
  }
  // right-side variant: u (T x r) in forward; u, v (T x r) and the split-K partials of dB (out x r) in backward;
  // deq(Q_q) as bf16 (r x roundup(in, 64)) in the merge
  // (forward and backward also stage deq(Q_q) as bf16 for the product u = x Q-hat^T, which has N = r only)
  const size_t qhat_bytes = align256(static_cast<size_t>(r > 0 ? r : 0) * ((static_cast<size_t>(in > 0 ? in : 0) + 63) / 64 * 64) * 2);
  if (op == LOQT_OP_FWD_RIGHT) total += align256(static_cast<size_t>(T > 0 ? T : 0) * ld_lowrank(r) * 2) + qhat_bytes;
  if (op == LOQT_OP_BWD_RIGHT) {
    total += 2 * align256(static_cast<size_t>(T > 0 ? T : 0) * ld_lowrank(r) * 2) + qhat_bytes;
    int splits = 1, kbps = 1;
    db_splits(out, r, T > 0 ? T : 1, splits, kbps);
    if (splits > 1) total += align256(static_cast<size_t>(splits) * out * ((static_cast<size_t>(r) + 3) / 4 * 4) * 4);
  }
  // right-side compensated initialisation: bf16 Q (r x roundup(in, 64)) and the bf16 residual (out x roundup(in, 64))
  if (op == LOQT_OP_COMPENSATE_RIGHT) {
    const size_t ld64 = (static_cast<size_t>(in > 0 ? in : 0) + 63) / 64 * 64;
    total += align256(static_cast<size_t>(r > 0 ? r : 0) * ld64 * 2) + align256(static_cast<size_t>(out > 0 ? out : 0) * ld64 * 2);
  }
  if (op == LOQT_OP_MERGE_RIGHT) total += align256(static_cast<size_t>(r > 0 ? r : 0) * ((static_cast<size_t>(in > 0 ? in : 0) + 63) / 64 * 64) * 2);
  // projection: bf16 G, one fp32 iterate, its hi + lo bf16 basis, and the orthonormalisation's scratch
  if (op == LOQT_OP_PROJECTION) {
    const size_t o = static_cast<size_t>(out > 0 ? out : 0), i = static_cast<size_t>(in > 0 ? in : 0);
    const size_t big = o > i ? o : i, ldr = static_cast<size_t>(ld_lowrank(r));
    total += align256(o * ((i + 63) / 64 * 64) * 2) + align256(big * ldr * 4) + 2 * align256(big * ldr * 2) +
             orth_workspace_bytes(static_cast<int>(big), r);
  }
  // full-rank gradient: split-K partials only (K = T)
  if (op == LOQT_OP_FULL_GRADIENT) {
    int splits = 1, kbps = 1;
    db_splits(out, in, T > 0 ? T : 1, splits, kbps);
    if (splits > 1) total += align256(static_cast<size_t>(splits) * out * ((static_cast<size_t>(in) + 3) / 4 * 4) * 4);
  }
  return total;
}

static loqt_status check_layer(const loqt_nf4_mat &Wq, const loqt_nf4_mat &Pq, const void *B, int64_t ldb) {
  loqt_status st;
  if ((st = validate_nf4(Wq)) != LOQT_OK) return st;
  if ((st = validate_nf4(Pq)) != LOQT_OK) return st;
  if (Pq.rows != Wq.rows) return LOQT_ERR_INVALID_ARG;
  return check_bf16(B, ldb, Wq.cols);
}

static loqt_status check_ws(const void *ws, size_t ws_bytes, size_t need) {
  if (ws == nullptr || ws_bytes < need) return LOQT_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return LOQT_ERR_ALIGNMENT;
  return LOQT_OK;
}

// Argument checks of the forward, shared by its two entry points.
static loqt_status check_fwd_args(const loqt_nf4_mat &Wq, const loqt_nf4_mat &Pq, const void *B, int64_t ldb, const void *x,
                                  int64_t ldx, int32_t T, const void *y, int64_t ldy) {
  loqt_status st;
  if ((st = check_layer(Wq, Pq, B, ldb)) != LOQT_OK) return st;
  if (T <= 0) return LOQT_ERR_INVALID_ARG;
  if ((st = check_bf16(x, ldx, Wq.cols)) != LOQT_OK) return st;
  return check_bf16(y, ldy, Wq.rows);
}

// Forward with both NF4 operands given as engine sources (fp32 or doubly quantised scales).
static loqt_status fwd_impl(const Nf4Src &W, const Nf4Src &P, const void *B, int64_t ldb, float s, const void *x, int64_t ldx,
                            int32_t T, void *y, int64_t ldy, void *ws, size_t ws_bytes, void *stream) {
  loqt_status st;
  const int out = W.rows, in = W.cols, r = P.cols;
  if ((st = check_ws(ws, ws_bytes, loqt_workspace_bytes(LOQT_OP_FWD, out, in, r, T))) != LOQT_OK) return st;
  if ((st = check_arch()) != LOQT_OK) return st;
  cudaStream_t stm = static_cast<cudaStream_t>(stream);
  uint32_t *status = static_cast<uint32_t *>(ws);
  void *u = static_cast<uint8_t *>(ws) + 256;
  const int64_t ldu = ld_lowrank(r);

  // u = s * x B^T            (T x r; both operands K-major over `in`)
  GemmCall c1{};
  c1.p.M = T; c1.p.N = r; c1.p.num_segs = 1;
  c1.p.seg[0].K = in; c1.p.seg[0].a_kind = OP_TMA_K; c1.p.seg[0].b_kind = OP_TMA_K;
  c1.a[0] = {x, ldx}; c1.b[0] = {B, ldb};
  c1.p.splits = 1; c1.p.kb_per_split = 0;
  c1.p.epi = EPI_BF16; c1.p.out = u; c1.p.ld_out = ldu; c1.p.alpha = s; c1.p.status = status;
  if ((st = launch(c1, stm)) != LOQT_OK) return st;

  // y = x deq(W_q)^T + u deq(P_q)^T    (K = in, then K = r, one accumulator)
  GemmCall c2{};
  c2.p.M = T; c2.p.N = out; c2.p.num_segs = 2;
  c2.p.seg[0].K = in; c2.p.seg[0].a_kind = OP_TMA_K; c2.p.seg[0].b_kind = OP_NF4_K; c2.p.seg[0].b_nf4 = W;
  c2.p.seg[1].K = r; c2.p.seg[1].a_kind = OP_TMA_K; c2.p.seg[1].b_kind = OP_NF4_K; c2.p.seg[1].b_nf4 = P;
  c2.a[0] = {x, ldx}; c2.a[1] = {u, ldu};
  c2.p.splits = 1;
  c2.p.epi = EPI_BF16; c2.p.out = y; c2.p.ld_out = ldy; c2.p.alpha = 1.0f; c2.p.status = status;
  return launch(c2, stm);
}

extern "C" loqt_status loqt_linear_fwd(loqt_nf4_mat Wq, loqt_nf4_mat Pq, const void *B, int64_t ldb, float s,
                                       const void *x, int64_t ldx, int32_t T, void *y, int64_t ldy, void *ws,
                                       size_t ws_bytes, void *stream) {
  loqt_status st;
  if ((st = check_fwd_args(Wq, Pq, B, ldb, x, ldx, T, y, ldy)) != LOQT_OK) return st;
  return fwd_impl(nf4_src(Wq), nf4_src(Pq), B, ldb, s, x, ldx, T, y, ldy, ws, ws_bytes, stream);
}

// Argument checks of the backward, shared by its entry points.
static loqt_status check_bwd_args(const loqt_nf4_mat &Wq, const loqt_nf4_mat &Pq, const void *B, int64_t ldb, const void *x,
                                  int64_t ldx, const void *dy, int64_t lddy, int32_t T, const void *dx, int64_t lddx,
                                  const float *dB, int64_t lddb) {
  loqt_status st;
  if ((st = check_layer(Wq, Pq, B, ldb)) != LOQT_OK) return st;
  if (T <= 0) return LOQT_ERR_INVALID_ARG;
  if ((st = check_bf16(x, ldx, Wq.cols)) != LOQT_OK) return st;
  if ((st = check_bf16(dy, lddy, Wq.rows)) != LOQT_OK) return st;
  if (dx != nullptr && (st = check_bf16(dx, lddx, Wq.cols)) != LOQT_OK) return st;
  if (dB == nullptr || lddb < Wq.cols) return LOQT_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(dB) & 15u) != 0) return LOQT_ERR_ALIGNMENT;
  return LOQT_OK;
}

// Pq_fp32: the factor with fp32 scales when it has them (then it is staged as bf16
// for the product v), null when its scales are doubly quantised.
static loqt_status bwd_impl(const Nf4Src &W, const Nf4Src &P, const loqt_nf4_mat *Pq_fp32, const void *B, int64_t ldb, float s,
                            const void *x, int64_t ldx, const void *dy, int64_t lddy, int32_t T, void *dx, int64_t lddx, float *dB,
                            int64_t lddb, int accumulate_dB, void *ws, size_t ws_bytes, void *stream) {
  loqt_status st;
  const int out = W.rows, in = W.cols, r = P.cols;
  if ((st = check_ws(ws, ws_bytes, loqt_workspace_bytes(LOQT_OP_BWD, out, in, r, T))) != LOQT_OK) return st;
  if ((st = check_arch()) != LOQT_OK) return st;
  cudaStream_t stm = static_cast<cudaStream_t>(stream);
  uint32_t *status = static_cast<uint32_t *>(ws);
  const int64_t ldv = ld_lowrank(r);
  void *v = static_cast<uint8_t *>(ws) + 256;
  float *partial = reinterpret_cast<float *>(static_cast<uint8_t *>(v) + align256(static_cast<size_t>(T) * ldv * 2));
  int db_split = 1, db_kbps = 1;
  db_splits(r, in, T, db_split, db_kbps);
  void *phat = reinterpret_cast<uint8_t *>(partial) +
               (db_split > 1 ? align256(static_cast<size_t>(db_split) * r * ((static_cast<size_t>(in) + 3) / 4 * 4) * 4) : 0);

  // v' = s * dy deq(P_q)      (T x r; K = out).  With N = r only, dequantising P_q inside
  // the product would repeat it for every 256 token rows and bind the main loop; the
  // factor is small (out x r), so it is dequantised once into the workspace (it stays
  // in L2) and v runs as a plain bf16 product.  With doubly quantised scales P_q is
  // read in place, its blocks along N = r.
  GemmCall c1{};
  c1.p.M = T; c1.p.N = r; c1.p.num_segs = 1;
  c1.p.seg[0].K = out; c1.p.seg[0].a_kind = OP_TMA_K;
  if (Pq_fp32 != nullptr) {
    const StageItem stage{*Pq_fp32, phat, ldv};
    if ((st = nf4_dequantize_bf16_batch(&stage, 1, stm)) != LOQT_OK) return st;
    c1.p.seg[0].b_kind = OP_TMA_MN;
    c1.b[0] = {phat, ldv};
  } else {
    c1.p.seg[0].b_kind = OP_NF4_MN; c1.p.seg[0].b_nf4 = P;
  }
  c1.a[0] = {dy, lddy};
  c1.p.splits = 1;
  c1.p.epi = EPI_BF16; c1.p.out = v; c1.p.ld_out = ldv; c1.p.alpha = s; c1.p.status = status;
  if ((st = launch(c1, stm)) != LOQT_OK) return st;

  // dx = dy deq(W_q) + v' B   (T x in; K = out with W_q blocks along N = in, then K = r)
  if (dx != nullptr) {
    GemmCall c2{};
    c2.p.M = T; c2.p.N = in; c2.p.num_segs = 2;
    c2.p.seg[0].K = out; c2.p.seg[0].a_kind = OP_TMA_K; c2.p.seg[0].b_kind = OP_NF4_MN; c2.p.seg[0].b_nf4 = W;
    c2.p.seg[1].K = r; c2.p.seg[1].a_kind = OP_TMA_K; c2.p.seg[1].b_kind = OP_TMA_MN;
    c2.a[0] = {dy, lddy}; c2.a[1] = {v, ldv}; c2.b[1] = {B, ldb};
    c2.p.splits = 1;
    c2.p.epi = EPI_BF16; c2.p.out = dx; c2.p.ld_out = lddx; c2.p.alpha = 1.0f; c2.p.status = status;
    if ((st = launch(c2, stm)) != LOQT_OK) return st;
  }

  // dB = v'^T x               (r x in; K = T; both operands stored K-outermost)
  return gemm_tn_f32(v, ldv, x, ldx, r, in, T, dB, lddb, accumulate_dB, partial, status, stm);
}

extern "C" loqt_status loqt_linear_bwd(loqt_nf4_mat Wq, loqt_nf4_mat Pq, const void *B, int64_t ldb, float s,
                                       const void *x, int64_t ldx, const void *dy, int64_t lddy, int32_t T, void *dx,
                                       int64_t lddx, float *dB, int64_t lddb, int accumulate_dB, void *ws,
                                       size_t ws_bytes, void *stream) {
  loqt_status st;
  if ((st = check_bwd_args(Wq, Pq, B, ldb, x, ldx, dy, lddy, T, dx, lddx, dB, lddb)) != LOQT_OK) return st;
  return bwd_impl(nf4_src(Wq), nf4_src(Pq), &Pq, B, ldb, s, x, ldx, dy, lddy, T, dx, lddx, dB, lddb, accumulate_dB, ws, ws_bytes,
                  stream);
}

// ---------------------------------------------------------------------------
// The layer with doubly quantised block scales (Section 2.4: the quantisation state
// is itself quantised).  The operand staging decodes each block's scale from its
// 8-bit code; everything else is the forward / backward above.
// ---------------------------------------------------------------------------
static loqt_status check_dq(const loqt_nf4_mat &m, const loqt_dq_scales &dq) {
  if (dq.codes8 == nullptr || dq.c1 == nullptr || dq.offset == nullptr) return LOQT_ERR_INVALID_ARG;
  if (dq.n != static_cast<int64_t>(m.rows) * (m.ld / kBlock)) return LOQT_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(dq.c1) & 3u) != 0 || (reinterpret_cast<uintptr_t>(dq.offset) & 3u) != 0) return LOQT_ERR_ALIGNMENT;
  return LOQT_OK;
}
// validate_nf4 insists on fp32 scales; a doubly quantised view passes with any non-null stand-in
static loqt_nf4_mat with_stand_in_scales(loqt_nf4_mat m, const loqt_dq_scales &dq) {
  if (m.absmax == nullptr) m.absmax = dq.c1;
  return m;
}

extern "C" loqt_status loqt_linear_fwd_dq(loqt_nf4_mat Wq, loqt_dq_scales Wdq, loqt_nf4_mat Pq, loqt_dq_scales Pdq, const void *B,
                                          int64_t ldb, float s, const void *x, int64_t ldx, int32_t T, void *y, int64_t ldy,
                                          void *ws, size_t ws_bytes, void *stream) {
  loqt_status st;
  if ((st = check_fwd_args(with_stand_in_scales(Wq, Wdq), with_stand_in_scales(Pq, Pdq), B, ldb, x, ldx, T, y, ldy)) != LOQT_OK)
    return st;
  if ((st = check_dq(Wq, Wdq)) != LOQT_OK || (st = check_dq(Pq, Pdq)) != LOQT_OK) return st;
  return fwd_impl(nf4_src_dq(Wq, Wdq), nf4_src_dq(Pq, Pdq), B, ldb, s, x, ldx, T, y, ldy, ws, ws_bytes, stream);
}

extern "C" loqt_status loqt_linear_bwd_dq(loqt_nf4_mat Wq, loqt_dq_scales Wdq, loqt_nf4_mat Pq, loqt_dq_scales Pdq, const void *B,
                                          int64_t ldb, float s, const void *x, int64_t ldx, const void *dy, int64_t lddy,
                                          int32_t T, void *dx, int64_t lddx, float *dB, int64_t lddb, int accumulate_dB, void *ws,
                                          size_t ws_bytes, void *stream) {
  loqt_status st;
  if ((st = check_bwd_args(with_stand_in_scales(Wq, Wdq), with_stand_in_scales(Pq, Pdq), B, ldb, x, ldx, dy, lddy, T, dx, lddx, dB,
                           lddb)) != LOQT_OK)
    return st;
  if ((st = check_dq(Wq, Wdq)) != LOQT_OK || (st = check_dq(Pq, Pdq)) != LOQT_OK) return st;
  return bwd_impl(nf4_src_dq(Wq, Wdq), nf4_src_dq(Pq, Pdq), nullptr, B, ldb, s, x, ldx, dy, lddy, T, dx, lddx, dB, lddb,
                  accumulate_dB, ws, ws_bytes, stream);
}

// ---------------------------------------------------------------------------
// Merge: staging of the dequantised factor, then the batched merge kernel
// ---------------------------------------------------------------------------
static size_t merge_scratch_bytes(const loqt_nf4_mat &Pq) {
  return align256(static_cast<size_t>(Pq.rows) * ld_lowrank(Pq.cols) * 2);
}

// P-hat = bf16(deq(P_q)), once, instead of once per column tile inside the product.
static loqt_status merge_stage(const loqt_nf4_mat &Pq, void *phat, cudaStream_t stm) {
  return loqt_nf4_dequantize(Pq, phat, ld_lowrank(Pq.cols), 1, stm);
}

// One matrix of a batched merge: W_q <- q(deq32(W_q) + alpha * A Bm) with A bf16
// [M][K] (K contiguous) and Bm bf16 [K][N] (N contiguous).
struct MergeItem {
  loqt_nf4_mat Wq;
  Bf16Operand a, b;
  int K;
  float alpha;
  // compensation mode: Wq is only written; the sum starts from the fp32 matrix w32 and
  // the bf16 residual w32 - deq32(Wq) is written to resid
  const float *w32 = nullptr;
  int64_t ld_w32 = 0;
  void *resid = nullptr;
  int64_t ld_resid = 0;
};

// fp32 matrix [rows][ld] as a tensor map; box in elements x rows, 128-byte swizzle.
static bool make_f32_map(CUtensorMap *map, const float *base, int64_t cols, int64_t rows, int64_t ld, int box_cols,
                         int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(ld) * 4};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(box_cols), static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float *>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN, bool COMP = false>
static loqt_status launch_merge(const MergeItem *items, int n, uint32_t *status, cudaStream_t stream) {
  using L = MergeLayout<BN, COMP>;
  MergeBatch mb;
  memset(&mb, 0, sizeof(mb));
  if (COMP) {
    // one matrix per launch; W by TMA (16-byte aligned rows), the residual by 16-byte stores
    // that may run into the padding of its rows
    const MergeItem &it = items[0];
    if (n != 1 || (reinterpret_cast<uintptr_t>(it.w32) & 15u) != 0 || (it.ld_w32 & 3) != 0 ||
        (reinterpret_cast<uintptr_t>(it.resid) & 15u) != 0 || (it.ld_resid & 7) != 0 || it.ld_resid < it.Wq.ld)
      return LOQT_ERR_INVALID_ARG;
    if (!make_f32_map(&mb.wmap, it.w32, it.Wq.cols, it.Wq.rows, it.ld_w32, 32, 32)) return LOQT_ERR_CUDA;
  }
  int tiles = 0;
  for (int i = 0; i < n; ++i) {
    const MergeItem &it = items[i];
    const int M = it.Wq.rows, N = it.Wq.cols;
    if (!make_map(&mb.a[i], it.a.ptr, it.K, M, it.a.ld, kBK, kHM)) return LOQT_ERR_CUDA;
    if (!make_map(&mb.b[i], it.b.ptr, N, it.K, it.b.ld, 64, kBK)) return LOQT_ERR_CUDA;
    // W_q's packed codes, one box = the 128 rows x BN columns an output tile updates
    if (!make_code_map(&mb.wq[i], nf4_src(it.Wq), BN / 2, kHM, BN == 256 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B))
      return LOQT_ERR_CUDA;
    MergeProblem &pr = mb.prob[i];
    pr.wq_absmax = it.Wq.absmax;
    pr.M = M; pr.N = N; pr.K = it.K; pr.wq_ld = it.Wq.ld;
    pr.tile0 = tiles;
    pr.mt = (M + kHM - 1) / kHM;
    pr.alpha = it.alpha;
    pr.w32 = it.w32; pr.ld_w32 = it.ld_w32;
    pr.resid = static_cast<__nv_bfloat16 *>(it.resid); pr.ld_resid = it.ld_resid;
    tiles += pr.mt * ((N + BN - 1) / BN);
  }
  mb.count = n;
  mb.tiles = tiles;
  mb.status = status;
  auto kernel = loqt_merge_kernel<BN, COMP>;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kDynamicBytes) != cudaSuccess)
    return LOQT_ERR_CUDA;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // the prologue may overlap the staging kernel's tail
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cfg.gridDim = dim3(tiles < sm_count() ? tiles : sm_count());
  cfg.blockDim = dim3(kNumThreads);
  cfg.dynamicSmemBytes = L::kDynamicBytes;
  cfg.stream = stream;
  const cudaError_t err = cudaLaunchKernelEx(&cfg, kernel, mb);
  count_launch();
  g_variant_launches[variant_index(BN, 1, false, false)].fetch_add(1, std::memory_order_relaxed);
  return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? LOQT_OK : LOQT_ERR_CUDA;
}

// Up to kMergeBatchMax matrices in one persistent launch.  256-wide tiles unless
// every matrix is at most 128 columns wide or 128-wide tiles are forced.
static loqt_status merge_batch(const MergeItem *items, int n, uint32_t *status, cudaStream_t stream) {
  if (n <= 0) return LOQT_OK;
  if (n > kMergeBatchMax) return LOQT_ERR_INVALID_ARG;
  bool wide = false;
  for (int i = 0; i < n; ++i) wide = wide || items[i].Wq.cols > 128;
  const int fbn = g_force_bn.load(std::memory_order_relaxed);
  if (fbn != 0) wide = (fbn == 256);
  const bool comp = items[0].w32 != nullptr;  // a batch is all of one kind
  if (comp) return wide ? launch_merge<256, true>(items, n, status, stream) : launch_merge<128, true>(items, n, status, stream);
  return wide ? launch_merge<256>(items, n, status, stream) : launch_merge<128>(items, n, status, stream);
}

extern "C" loqt_status loqt_merge_requant_many(int32_t n, const loqt_nf4_mat *Wq, const loqt_nf4_mat *Pq,
                                               const void *const *B, const int64_t *ldb, float s, void *ws,
                                               size_t ws_bytes, void *stream) {
  if (n < 0 || (n > 0 && (Wq == nullptr || Pq == nullptr || B == nullptr || ldb == nullptr))) return LOQT_ERR_INVALID_ARG;
  loqt_status st;
  size_t slot = 0;
  for (int i = 0; i < n; ++i) {
    if ((st = check_layer(Wq[i], Pq[i], B[i], ldb[i])) != LOQT_OK) return st;
    const size_t need = merge_scratch_bytes(Pq[i]);
    if (need > slot) slot = need;
  }
  if ((st = check_ws(ws, ws_bytes, 256 + slot)) != LOQT_OK) return st;
  if ((st = check_arch()) != LOQT_OK) return st;
  if (n == 0) return LOQT_OK;
  cudaStream_t stm = static_cast<cudaStream_t>(stream);
  // Matrices are taken in batches: as many as the workspace holds dequantised
  // factors for (packed back to back) and one launch carries.  A batch's factors
  // are staged by one launch, its merges run in one persistent launch.
  uint8_t *base = static_cast<uint8_t *>(ws) + 256;
  const size_t room = ws_bytes - 256;
  for (int g0 = 0; g0 < n;) {
    StageItem stage[kMergeBatchMax];
    MergeItem items[kMergeBatchMax];
    size_t used = 0;
    int g1 = g0;
    while (g1 < n && g1 - g0 < kMergeBatchMax && used + merge_scratch_bytes(Pq[g1]) <= room) {
      void *phat = base + used;
      const int64_t ldp = ld_lowrank(Pq[g1].cols);
      stage[g1 - g0] = StageItem{Pq[g1], phat, ldp};
      items[g1 - g0] = MergeItem{Wq[g1], {phat, ldp}, {B[g1], ldb[g1]}, Pq[g1].cols, s};
      used += merge_scratch_bytes(Pq[g1]);
      ++g1;
    }
    if ((st = nf4_dequantize_bf16_batch(stage, g1 - g0, stm)) != LOQT_OK) return st;
    if ((st = merge_batch(items, g1 - g0, static_cast<uint32_t *>(ws), stm)) != LOQT_OK) return st;
    g0 = g1;
  }
  return LOQT_OK;
}

extern "C" loqt_status loqt_merge_requant(loqt_nf4_mat Wq, loqt_nf4_mat Pq, const void *B, int64_t ldb, float s,
                                          void *ws, size_t ws_bytes, void *stream) {
  const int64_t ldb1 = ldb;
  return loqt_merge_requant_many(1, &Wq, &Pq, &B, &ldb1, s, ws, ws_bytes, stream);
}

// The same merge in two passes: Delta = P-hat B written as fp32, then the
// streaming requantiser.  Same arithmetic per element as the fused epilogue.
extern "C" loqt_status loqt_merge_requant_split(loqt_nf4_mat Wq, loqt_nf4_mat Pq, const void *B, int64_t ldb, float s,
                                                void *ws, size_t ws_bytes, void *stream) {
  loqt_status st;
  if ((st = check_layer(Wq, Pq, B, ldb)) != LOQT_OK) return st;
  const size_t phat_bytes = merge_scratch_bytes(Pq);
  const size_t delta_bytes = align256(static_cast<size_t>(Wq.rows) * Wq.ld * 4);
  if ((st = check_ws(ws, ws_bytes, 256 + phat_bytes + delta_bytes)) != LOQT_OK) return st;
  if ((st = check_arch()) != LOQT_OK) return st;
  cudaStream_t stm = static_cast<cudaStream_t>(stream);
  void *phat = static_cast<uint8_t *>(ws) + 256;
  float *delta = reinterpret_cast<float *>(static_cast<uint8_t *>(phat) + phat_bytes);
  if ((st = merge_stage(Pq, phat, stm)) != LOQT_OK) return st;
  GemmCall c{};
  c.p.M = Wq.rows; c.p.N = Wq.cols; c.p.num_segs = 1;
  c.p.seg[0].K = Pq.cols; c.p.seg[0].a_kind = OP_TMA_K; c.p.seg[0].b_kind = OP_TMA_MN;
  c.a[0] = {phat, ld_lowrank(Pq.cols)}; c.b[0] = {B, ldb};
  c.p.splits = 1;
  c.p.epi = EPI_F32; c.p.out = delta; c.p.ld_out = Wq.ld; c.p.alpha = 1.0f; c.p.accumulate = 0;
  c.p.status = static_cast<uint32_t *>(ws);
  if ((st = launch(c, stm)) != LOQT_OK) return st;
  return loqt_nf4_requantize(delta, Wq.ld, s, Wq, stream);
}

// ---------------------------------------------------------------------------
// Right-side variant: W = deq(W_q) + s B deq(Q_q)   (Section 2.1: G Q for m > n)
//   Wq : out x in,  Qq : r x in (NF4, blocks along in),  B : bf16 [out][ldb] (out x r)
// Every product is a configuration of the same engine.
// ---------------------------------------------------------------------------
static loqt_status check_layer_right(const loqt_nf4_mat &Wq, const loqt_nf4_mat &Qq, const void *B, int64_t ldb) {
  loqt_status st;
  if ((st = validate_nf4(Wq)) != LOQT_OK) return st;
  if ((st = validate_nf4(Qq)) != LOQT_OK) return st;
  if (Qq.cols != Wq.cols) return LOQT_ERR_INVALID_ARG;
  return check_bf16(B, ldb, Qq.rows);
}

// u = s * x deq(Q_q)^T   (T x r; K = in).  As for v in the left-side backward: with N = r only,
// dequantising Q_q inside the product would repeat it for every 256 token rows, so the factor
// is dequantised once into `qhat` (bf16 r x Qq.ld) and the product is a plain bf16 one.
static loqt_status right_u(const loqt_nf4_mat &Qq, float s, const void *x, int64_t ldx, int T, void *u, int64_t ldu,
                           void *qhat, uint32_t *status, cudaStream_t stm) {
  const StageItem stage{Qq, qhat, Qq.ld};
  loqt_status st = nf4_dequantize_bf16_batch(&stage, 1, stm);
  if (st != LOQT_OK) return st;
  GemmCall c{};
  c.p.M = T; c.p.N = Qq.rows; c.p.num_segs = 1;
  c.p.seg[0].K = Qq.cols; c.p.seg[0].a_kind = OP_TMA_K; c.p.seg[0].b_kind = OP_TMA_K;
  c.a[0] = {x, ldx}; c.b[0] = {qhat, Qq.ld};
  c.p.splits = 1;
  c.p.epi = EPI_BF16; c.p.out = u; c.p.ld_out = ldu; c.p.alpha = s; c.p.status = status;
  return launch(c, stm);
}

extern "C" loqt_status loqt_linear_fwd_right(loqt_nf4_mat Wq, loqt_nf4_mat Qq, const void *B, int64_t ldb, float s,
                                             const void *x, int64_t ldx, int32_t T, void *y, int64_t ldy, void *ws,
                                             size_t ws_bytes, void *stream) {
  loqt_status st;
  if ((st = check_layer_right(Wq, Qq, B, ldb)) != LOQT_OK) return st;
  if (T <= 0) return LOQT_ERR_INVALID_ARG;
  const int out = Wq.rows, in = Wq.cols, r = Qq.rows;
  if ((st = check_bf16(x, ldx, in)) != LOQT_OK) return st;
  if ((st = check_bf16(y, ldy, out)) != LOQT_OK) return st;
  if ((st = check_ws(ws, ws_bytes, loqt_workspace_bytes(LOQT_OP_FWD_RIGHT, out, in, r, T))) != LOQT_OK) return st;
  if ((st = check_arch()) != LOQT_OK) return st;
  cudaStream_t stm = static_cast<cudaStream_t>(stream);
  uint32_t *status = static_cast<uint32_t *>(ws);
  void *u = static_cast<uint8_t *>(ws) + 256;
  const int64_t ldu = ld_lowrank(r);
  void *qhat = static_cast<uint8_t *>(u) + align256(static_cast<size_t>(T) * ldu * 2);
  if ((st = right_u(Qq, s, x, ldx, T, u, ldu, qhat, status, stm)) != LOQT_OK) return st;
  // y = x deq(W_q)^T + u B^T    (K = in, then K = r; B is K-major over r)
  GemmCall c{};
  c.p.M = T; c.p.N = out; c.p.num_segs = 2;
  c.p.seg[0].K = in; c.p.seg[0].a_kind = OP_TMA_K; c.p.seg[0].b_kind = OP_NF4_K; c.p.seg[0].b_nf4 = nf4_src(Wq);
  c.p.seg[1].K = r; c.p.seg[1].a_kind = OP_TMA_K; c.p.seg[1].b_kind = OP_TMA_K;
  c.a[0] = {x, ldx}; c.a[1] = {u, ldu}; c.b[1] = {B, ldb};
  c.p.splits = 1;
  c.p.epi = EPI_BF16; c.p.out = y; c.p.ld_out = ldy; c.p.alpha = 1.0f; c.p.status = status;
  return launch(c, stm);
}

extern "C" loqt_status loqt_linear_bwd_right(loqt_nf4_mat Wq, loqt_nf4_mat Qq, const void *B, int64_t ldb, float s,
                                             const void *x, int64_t ldx, const void *dy, int64_t lddy, int32_t T, void *dx,
                                             int64_t lddx, float *dB, int64_t lddb, int accumulate_dB, void *ws,
                                             size_t ws_bytes, void *stream) {
  loqt_status st;
  if ((st = check_layer_right(Wq, Qq, B, ldb)) != LOQT_OK) return st;
  if (T <= 0) return LOQT_ERR_INVALID_ARG;
  const int out = Wq.rows, in = Wq.cols, r = Qq.rows;
  if ((st = check_bf16(x, ldx, in)) != LOQT_OK) return st;
  if ((st = check_bf16(dy, lddy, out)) != LOQT_OK) return st;
  if (dx != nullptr && (st = check_bf16(dx, lddx, in)) != LOQT_OK) return st;
  if (dB == nullptr || lddb < r) return LOQT_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(dB) & 15u) != 0) return LOQT_ERR_ALIGNMENT;
  if ((st = check_ws(ws, ws_bytes, loqt_workspace_bytes(LOQT_OP_BWD_RIGHT, out, in, r, T))) != LOQT_OK) return st;
  if ((st = check_arch()) != LOQT_OK) return st;
  cudaStream_t stm = static_cast<cudaStream_t>(stream);
  uint32_t *status = static_cast<uint32_t *>(ws);
  const int64_t ldt = ld_lowrank(r);
  const size_t tr_bytes = align256(static_cast<size_t>(T) * ldt * 2);
  void *u = static_cast<uint8_t *>(ws) + 256;
  void *v = static_cast<uint8_t *>(u) + tr_bytes;
  void *qhat = static_cast<uint8_t *>(v) + tr_bytes;
  float *partial = reinterpret_cast<float *>(static_cast<uint8_t *>(qhat) + align256(static_cast<size_t>(r) * Qq.ld * 2));

  // u = s * x deq(Q_q)^T, recomputed (the forward's copy is not kept)
  if ((st = right_u(Qq, s, x, ldx, T, u, ldt, qhat, status, stm)) != LOQT_OK) return st;
  if (dx != nullptr) {
    // v = s * dy B             (T x r; K = out; B stored [K][N])
    GemmCall c1{};
    c1.p.M = T; c1.p.N = r; c1.p.num_segs = 1;
    c1.p.seg[0].K = out; c1.p.seg[0].a_kind = OP_TMA_K; c1.p.seg[0].b_kind = OP_TMA_MN;
    c1.a[0] = {dy, lddy}; c1.b[0] = {B, ldb};
    c1.p.splits = 1;
    c1.p.epi = EPI_BF16; c1.p.out = v; c1.p.ld_out = ldt; c1.p.alpha = s; c1.p.status = status;
    if ((st = launch(c1, stm)) != LOQT_OK) return st;
    // dx = dy deq(W_q) + v deq(Q_q)   (K = out with W_q blocks along N = in, then K = r with Q_q blocks along N = in)
    GemmCall c2{};
    c2.p.M = T; c2.p.N = in; c2.p.num_segs = 2;
    c2.p.seg[0].K = out; c2.p.seg[0].a_kind = OP_TMA_K; c2.p.seg[0].b_kind = OP_NF4_MN; c2.p.seg[0].b_nf4 = nf4_src(Wq);
    c2.p.seg[1].K = r; c2.p.seg[1].a_kind = OP_TMA_K; c2.p.seg[1].b_kind = OP_NF4_MN; c2.p.seg[1].b_nf4 = nf4_src(Qq);
    c2.a[0] = {dy, lddy}; c2.a[1] = {v, ldt};
    c2.p.splits = 1;
    c2.p.epi = EPI_BF16; c2.p.out = dx; c2.p.ld_out = lddx; c2.p.alpha = 1.0f; c2.p.status = status;
    if ((st = launch(c2, stm)) != LOQT_OK) return st;
  }
  // dB = dy^T u              (out x r; K = T; both operands stored K-outermost; u carries s)
  return gemm_tn_f32(dy, lddy, u, ldt, out, r, T, dB, lddb, accumulate_dB, partial, status, stm);
}

extern "C" loqt_status loqt_merge_requant_right(loqt_nf4_mat Wq, loqt_nf4_mat Qq, const void *B, int64_t ldb, float s,
                                                void *ws, size_t ws_bytes, void *stream) {
  loqt_status st;
  if ((st = check_layer_right(Wq, Qq, B, ldb)) != LOQT_OK) return st;
  const int out = Wq.rows, in = Wq.cols, r = Qq.rows;
  if ((st = check_ws(ws, ws_bytes, loqt_workspace_bytes(LOQT_OP_MERGE_RIGHT, out, in, r, 0))) != LOQT_OK) return st;
  if ((st = check_arch()) != LOQT_OK) return st;
  cudaStream_t stm = static_cast<cudaStream_t>(stream);
  // Q-hat = bf16(deq(Q_q)), once; then Delta = B Q-hat (out x in; K = r) requantised in the epilogue
  void *qhat = static_cast<uint8_t *>(ws) + 256;
  const StageItem stage{Qq, qhat, Qq.ld};
  if ((st = nf4_dequantize_bf16_batch(&stage, 1, stm)) != LOQT_OK) return st;
  const MergeItem item{Wq, {B, ldb}, {qhat, Qq.ld}, r, s};
  return merge_batch(&item, 1, static_cast<uint32_t *>(ws), stm);
}

// ---------------------------------------------------------------------------
// Full-rank gradient at merge steps (Algorithm 1: G^W before Initialize)
// ---------------------------------------------------------------------------
extern "C" loqt_status loqt_full_gradient(const void *x, int64_t ldx, const void *dy, int64_t lddy, int32_t T, int32_t out,
                                          int32_t in, float *G, int64_t ldg, int accumulate, void *ws, size_t ws_bytes,
                                          void *stream) {
  loqt_status st;
  if (T <= 0 || out <= 0 || in <= 0) return LOQT_ERR_INVALID_ARG;
  if ((st = check_bf16(x, ldx, in)) != LOQT_OK) return st;
  if ((st = check_bf16(dy, lddy, out)) != LOQT_OK) return st;
  if (G == nullptr || ldg < in) return LOQT_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(G) & 15u) != 0) return LOQT_ERR_ALIGNMENT;
  if ((st = check_ws(ws, ws_bytes, loqt_workspace_bytes(LOQT_OP_FULL_GRADIENT, out, in, 0, T))) != LOQT_OK) return st;
  if ((st = check_arch()) != LOQT_OK) return st;
  float *partial = reinterpret_cast<float *>(static_cast<uint8_t *>(ws) + 256);
  // G = dy^T x   (out x in; K = T; both operands stored K-outermost)
  return gemm_tn_f32(dy, lddy, x, ldx, out, in, T, G, ldg, accumulate, partial, static_cast<uint32_t *>(ws),
                     static_cast<cudaStream_t>(stream));
}

// ---------------------------------------------------------------------------
// Projection from the full-rank gradient (Algorithm 2, SVD lines) by randomised
// subspace iteration: products on the engine, orthonormalisation in subspace.cu
// ---------------------------------------------------------------------------
// Y (fp32, M x r) = A (hi + lo)  with the basis given as two bf16 matrices
// [K][ldq]; A is bf16 G read K-major (A = G: M = out, K = in) or MN-major
// (A = G^T: M = in, K = out).  Two K segments share the accumulator.
static loqt_status projection_product(const void *gb, int64_t ldgb, bool transposed, int M, int K, int r, const void *hi,
                                      const void *lo, int64_t ldq, float *Y, int64_t ldy, uint32_t *status, cudaStream_t stm) {
  GemmCall c{};
  c.p.M = M; c.p.N = r; c.p.num_segs = lo != nullptr ? 2 : 1;
  for (int s = 0; s < c.p.num_segs; ++s) {
    c.p.seg[s].K = K; c.p.seg[s].a_kind = transposed ? OP_TMA_MN : OP_TMA_K; c.p.seg[s].b_kind = OP_TMA_MN;
    c.a[s] = {gb, ldgb};
  }
  c.b[0] = {hi, ldq};
  c.b[1] = {lo, ldq};
  c.p.splits = 1;
  c.p.epi = EPI_F32; c.p.out = Y; c.p.ld_out = ldy; c.p.alpha = 1.0f; c.p.accumulate = 0; c.p.status = status;
  return launch(c, stm);
}

// The iteration for either side.  Left (right == false): basis of the leading left singular
// subspace, out x r, from an in x r test matrix.  Right: the same iteration on G^T - the
// roles of G and G^T in the products are exchanged - from an out x r test matrix; the basis
// (in x r) is stored transposed, r x in, the layout of the right-side variant's factor Q.
static loqt_status projection_impl(bool right, const float *G, int64_t ldg, int32_t out, int32_t in, int32_t r, const void *Omega,
                                   int64_t ldo, int32_t iters, float *basis, int64_t ld_basis, void *ws, size_t ws_bytes,
                                   void *stream) {
  loqt_status st;
  if (out <= 0 || in <= 0 || r <= 0 || r > out || r > in || r > 4096 || iters < 0 || iters > 16) return LOQT_ERR_INVALID_ARG;
  if (G == nullptr || basis == nullptr || ldg < in || ld_basis < (right ? in : r)) return LOQT_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(G) & 15u) != 0 || (reinterpret_cast<uintptr_t>(basis) & 3u) != 0) return LOQT_ERR_ALIGNMENT;
  if ((st = check_bf16(Omega, ldo, r)) != LOQT_OK) return st;
  if ((st = check_ws(ws, ws_bytes, loqt_workspace_bytes(LOQT_OP_PROJECTION, out, in, r, 0))) != LOQT_OK) return st;
  if ((st = check_arch()) != LOQT_OK) return st;
  cudaStream_t stm = static_cast<cudaStream_t>(stream);
  uint32_t *status = static_cast<uint32_t *>(ws);
  const int big = out > in ? out : in;
  const int64_t ldgb = (static_cast<int64_t>(in) + 63) / 64 * 64, ldr = ld_lowrank(r);
  uint8_t *cursor = static_cast<uint8_t *>(ws) + 256;
  void *gb = cursor;                                  cursor += align256(static_cast<size_t>(out) * ldgb * 2);
  float *Y = reinterpret_cast<float *>(cursor);       cursor += align256(static_cast<size_t>(big) * ldr * 4);
  void *hi = cursor;                                  cursor += align256(static_cast<size_t>(big) * ldr * 2);
  void *lo = cursor;                                  cursor += align256(static_cast<size_t>(big) * ldr * 2);
  void *orth_ws = cursor;

  // A = G for the left side, G^T for the right: rows m_a, columns k_a; `main` products are A (.),
  // `back` products A^T (.)
  const int m_a = right ? in : out, k_a = right ? out : in;
  auto product = [&](bool back, const void *bhi, const void *blo, int64_t ldq) {
    const bool transposed = back != right;  // whether bf16 G is read as G^T
    return projection_product(gb, ldgb, transposed, back ? k_a : m_a, back ? m_a : k_a, r, bhi, blo, ldq, Y, ldr, status, stm);
  };
  if ((st = convert_f32_bf16(G, ldg, gb, ldgb, out, in, stm)) != LOQT_OK) return st;
  // Q = orth(A Omega)
  if ((st = product(false, Omega, nullptr, ldo)) != LOQT_OK) return st;
  if ((st = orthonormalise(Y, ldr, m_a, r, iters == 0 ? basis : nullptr, ld_basis, right, hi, lo, ldr, orth_ws, status, stm)) != LOQT_OK)
    return st;
  for (int it = 1; it <= iters; ++it) {
    // Z = orth(A^T Q)
    if ((st = product(true, hi, lo, ldr)) != LOQT_OK) return st;
    if ((st = orthonormalise(Y, ldr, k_a, r, nullptr, 0, false, hi, lo, ldr, orth_ws, status, stm)) != LOQT_OK) return st;
    // Q = orth(A Z)
    if ((st = product(false, hi, lo, ldr)) != LOQT_OK) return st;
    if ((st = orthonormalise(Y, ldr, m_a, r, it == iters ? basis : nullptr, ld_basis, right, hi, lo, ldr, orth_ws, status, stm)) != LOQT_OK)
      return st;
  }
  return LOQT_OK;
}

extern "C" loqt_status loqt_projection(const float *G, int64_t ldg, int32_t out, int32_t in, int32_t r, const void *Omega,
                                       int64_t ldo, int32_t iters, float *P, int64_t ldp, void *ws, size_t ws_bytes,
                                       void *stream) {
  return projection_impl(false, G, ldg, out, in, r, Omega, ldo, iters, P, ldp, ws, ws_bytes, stream);
}

extern "C" loqt_status loqt_projection_right(const float *G, int64_t ldg, int32_t out, int32_t in, int32_t r, const void *Omega,
                                             int64_t ldo, int32_t iters, float *Q, int64_t ldq, void *ws, size_t ws_bytes,
                                             void *stream) {
  return projection_impl(true, G, ldg, out, in, r, Omega, ldo, iters, Q, ldq, ws, ws_bytes, stream);
}

// ---------------------------------------------------------------------------
// Error-compensated initialisation (Section 2.5; Algorithm 2, compensation loop)
// ---------------------------------------------------------------------------
extern "C" loqt_status loqt_compensated_init(const float *W, int64_t ldw, const float *P, int64_t ldp, int32_t steps,
                                             loqt_nf4_mat Wq, loqt_nf4_mat Pq, void *B, int64_t ldb, void *ws,
                                             size_t ws_bytes, void *stream) {
  loqt_status st;
  if ((st = validate_nf4(Wq)) != LOQT_OK) return st;
  if ((st = validate_nf4(Pq)) != LOQT_OK) return st;
  if (Pq.rows != Wq.rows || steps < 1 || steps > 16) return LOQT_ERR_INVALID_ARG;
  const int out = Wq.rows, in = Wq.cols, r = Pq.cols;
  if (W == nullptr || P == nullptr || ldw < in || ldp < r) return LOQT_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(W) & 15u) != 0 || (ldw & 3) != 0 || (reinterpret_cast<uintptr_t>(P) & 3u) != 0)
    return LOQT_ERR_ALIGNMENT;
  if ((st = check_bf16(B, ldb, in)) != LOQT_OK) return st;
  if ((st = check_ws(ws, ws_bytes, loqt_workspace_bytes(LOQT_OP_COMPENSATE, out, in, r, 0))) != LOQT_OK) return st;
  if ((st = check_arch()) != LOQT_OK) return st;
  cudaStream_t stm = static_cast<cudaStream_t>(stream);
  uint32_t *status = static_cast<uint32_t *>(ws);

  const int64_t ldr = ld_lowrank(r), ld64 = (static_cast<int64_t>(in) + 63) / 64 * 64, ld4 = (static_cast<int64_t>(in) + 3) / 4 * 4;
  uint8_t *cursor = static_cast<uint8_t *>(ws) + 256;
  void *phat = cursor;                                        cursor += align256(static_cast<size_t>(out) * ldr * 2);
  void *resid = cursor;                                       cursor += align256(static_cast<size_t>(out) * ld64 * 2);
  float *b32 = reinterpret_cast<float *>(cursor);             cursor += align256(static_cast<size_t>(r) * ld4 * 4);
  float *partial = reinterpret_cast<float *>(cursor);

  // P_q = q(P); the products below use bf16(P), the unquantised projection (Algorithm 2)
  if ((st = loqt_nf4_quantize(P, ldp, Pq, stream)) != LOQT_OK) return st;
  if ((st = convert_f32_bf16(P, ldp, phat, ldr, out, r, stm)) != LOQT_OK) return st;
  int splits = 1, kbps = 1;
  db_splits(r, in, out, splits, kbps);

  for (int c = 1; c <= steps; ++c) {
    if (c == 1) {
      // Q_1 = q(W) (B_0 = 0), residual = bf16(W - deq(Q_1)): one streaming pass
      if ((st = nf4_quantize_residual(W, ldw, W, ldw, Wq, resid, ld64, stm)) != LOQT_OK) return st;
    } else {
      // Q_c = q(W - P B_(c-1)), residual = bf16(W - deq(Q_c)): the product P B (out x in; K = r)
      // with the quantiser and the residual in its epilogue; W - P B is never written
      MergeItem item{Wq, {phat, ldr}, {B, ldb}, r, -1.0f};
      item.w32 = W; item.ld_w32 = ldw; item.resid = resid; item.ld_resid = ld64;
      if ((st = merge_batch(&item, 1, status, stm)) != LOQT_OK) return st;
    }
    // B_c = P^T residual   (r x in; K = out; both operands stored K-outermost), rounded to bf16:
    // in the product's epilogue when one pass over K does it, else after the split-K sum
    if (splits == 1) {
      GemmCall g{};
      g.p.M = r; g.p.N = in; g.p.num_segs = 1;
      g.p.seg[0].K = out; g.p.seg[0].a_kind = OP_TMA_MN; g.p.seg[0].b_kind = OP_TMA_MN;
      g.a[0] = {phat, ldr}; g.b[0] = {resid, ld64};
      g.p.splits = 1; g.p.kb_per_split = 0;
      g.p.epi = EPI_BF16; g.p.out = B; g.p.ld_out = ldb; g.p.alpha = 1.0f; g.p.status = status;
      if ((st = launch(g, stm)) != LOQT_OK) return st;
    } else {
      if ((st = gemm_tn_f32(phat, ldr, resid, ld64, r, in, out, b32, ld4, 0, partial, status, stm)) != LOQT_OK) return st;
      if ((st = convert_f32_bf16(b32, ld4, B, ldb, r, in, stm)) != LOQT_OK) return st;
    }
  }
  return LOQT_OK;
}

// The same for the right-side variant: W ~ Q_w + B Q with Q (r x in, orthonormal rows) fixed,
//   Q_c = q_NF4(W - B_(c-1) Q),   B_c = (W - deq(Q_c)) Q^T.
extern "C" loqt_status loqt_compensated_init_right(const float *W, int64_t ldw, const float *Q, int64_t ldq, int32_t steps,
                                                   loqt_nf4_mat Wq, loqt_nf4_mat Qq, void *B, int64_t ldb, void *ws,
                                                   size_t ws_bytes, void *stream) {
  loqt_status st;
  if ((st = validate_nf4(Wq)) != LOQT_OK) return st;
  if ((st = validate_nf4(Qq)) != LOQT_OK) return st;
  if (Qq.cols != Wq.cols || steps < 1 || steps > 16) return LOQT_ERR_INVALID_ARG;
  const int out = Wq.rows, in = Wq.cols, r = Qq.rows;
  if (W == nullptr || Q == nullptr || ldw < in || ldq < in) return LOQT_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(W) & 15u) != 0 || (ldw & 3) != 0 || (reinterpret_cast<uintptr_t>(Q) & 3u) != 0)
    return LOQT_ERR_ALIGNMENT;
  if ((st = check_bf16(B, ldb, r)) != LOQT_OK) return st;
  if ((st = check_ws(ws, ws_bytes, loqt_workspace_bytes(LOQT_OP_COMPENSATE_RIGHT, out, in, r, 0))) != LOQT_OK) return st;
  if ((st = check_arch()) != LOQT_OK) return st;
  cudaStream_t stm = static_cast<cudaStream_t>(stream);
  uint32_t *status = static_cast<uint32_t *>(ws);
  const int64_t ld64 = (static_cast<int64_t>(in) + 63) / 64 * 64;
  uint8_t *cursor = static_cast<uint8_t *>(ws) + 256;
  void *qhat = cursor;   cursor += align256(static_cast<size_t>(r) * ld64 * 2);
  void *resid = cursor;

  // Q_q = q(Q); the products use bf16(Q), the unquantised projection
  if ((st = loqt_nf4_quantize(Q, ldq, Qq, stream)) != LOQT_OK) return st;
  if ((st = convert_f32_bf16(Q, ldq, qhat, ld64, r, in, stm)) != LOQT_OK) return st;
  for (int c = 1; c <= steps; ++c) {
    if (c == 1) {
      if ((st = nf4_quantize_residual(W, ldw, W, ldw, Wq, resid, ld64, stm)) != LOQT_OK) return st;
    } else {
      // the product B Q (out x in; K = r) with the quantiser and the residual in its epilogue
      MergeItem item{Wq, {B, ldb}, {qhat, ld64}, r, -1.0f};
      item.w32 = W; item.ld_w32 = ldw; item.resid = resid; item.ld_resid = ld64;
      if ((st = merge_batch(&item, 1, status, stm)) != LOQT_OK) return st;
    }
    // B_c = residual Q^T   (out x r; K = in; both operands K-major), rounded to bf16 in the epilogue
    GemmCall g{};
    g.p.M = out; g.p.N = r; g.p.num_segs = 1;
    g.p.seg[0].K = in; g.p.seg[0].a_kind = OP_TMA_K; g.p.seg[0].b_kind = OP_TMA_K;
    g.a[0] = {resid, ld64}; g.b[0] = {qhat, ld64};
    g.p.splits = 1; g.p.kb_per_split = 0;
    g.p.epi = EPI_BF16; g.p.out = B; g.p.ld_out = ldb; g.p.alpha = 1.0f; g.p.status = status;
    if ((st = launch(g, stm)) != LOQT_OK) return st;
  }
  return LOQT_OK;
}

// ---------------------------------------------------------------------------
// Tile override and per-variant launch counts (testing and tuning hooks)
// ---------------------------------------------------------------------------
extern "C" loqt_status loqt_set_tile_override(int32_t bn, int32_t rows, int32_t pair) {
  if (bn == 0) {
    g_force_bn.store(0, std::memory_order_relaxed);
    return LOQT_OK;
  }
  if ((bn != 128 && bn != 256) || (rows != 128 && rows != 256) || (pair != 0 && pair != 1)) return LOQT_ERR_INVALID_ARG;
  if (pair != 0 && (bn != 256 || !kUsePairs)) return LOQT_ERR_UNSUPPORTED;
  g_force_mh.store(rows / kHM, std::memory_order_relaxed);
  g_force_pair.store(pair, std::memory_order_relaxed);
  g_force_bn.store(bn, std::memory_order_relaxed);
  return LOQT_OK;
}

extern "C" uint64_t loqt_variant_launches(int32_t bn, int32_t rows, int32_t pair, int32_t nf4) {
  if ((bn != 128 && bn != 256) || (rows != 128 && rows != 256)) return 0;
  return g_variant_launches[variant_index(bn, rows / kHM, pair != 0, nf4 != 0)].load(std::memory_order_relaxed);
}

// ---------------------------------------------------------------------------
// Forward without any caller-provided scratch (see loqt_linear_fwd_static in loqt.h)
// ---------------------------------------------------------------------------
namespace loqt {

// Status word (first 256 bytes) + the T x r intermediate of the forward.  Lives
// in every GPU context that loads this library, until the process exits.
constexpr size_t kStaticScratchBytes = 256 + LOQT_STATIC_FWD_MAX_SCRATCH;
static __device__ __align__(256) unsigned char g_static_fwd_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
static void *g_static_scratch_addr[kMaxDevices] = {nullptr};
static std::mutex g_static_scratch_mutex;

// Device address of the scratch array on the current device.  In host code the
// symbol's name is only a handle; the address a kernel can use comes from
// cudaGetSymbolAddress, asked once per device with that device current.
static loqt_status static_scratch_for_current_device(void **out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return LOQT_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return LOQT_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
  if (g_static_scratch_addr[dev] == nullptr) {
    void *ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_fwd_scratch) != cudaSuccess || ptr == nullptr) return LOQT_ERR_CUDA;
    g_static_scratch_addr[dev] = ptr;
  }
  *out = g_static_scratch_addr[dev];
  return LOQT_OK;
}

}  // namespace loqt

extern "C" loqt_status loqt_linear_fwd_static(loqt_nf4_mat Wq, loqt_nf4_mat Pq, const void *B, int64_t ldb, float s,
                                              const void *x, int64_t ldx, int32_t T, void *y, int64_t ldy,
                                              int check_device_status, void *stream) {
  // Every argument check comes before the first thing enqueued: a rejected call
  // must leave the shared status word as it was.
  loqt_status st;
  if ((st = check_fwd_args(Wq, Pq, B, ldb, x, ldx, T, y, ldy)) != LOQT_OK) return st;
  const size_t need = loqt_workspace_bytes(LOQT_OP_FWD, Wq.rows, Wq.cols, Pq.cols, T);
  if (need > kStaticScratchBytes) return LOQT_ERR_WORKSPACE;  // T * roundup(r, 64) * 2 bytes exceeds the built-in scratch
  if ((st = check_arch()) != LOQT_OK) return st;
  void *scratch = nullptr;
  if ((st = static_scratch_for_current_device(&scratch)) != LOQT_OK) return st;
  cudaStream_t stm = static_cast<cudaStream_t>(stream);
  // The array keeps whatever the previous call left; only the status word has to start at zero.
  if (cudaMemsetAsync(scratch, 0, 256, stm) != cudaSuccess) return LOQT_ERR_CUDA;
  if ((st = loqt_linear_fwd(Wq, Pq, B, ldb, s, x, ldx, T, y, ldy, scratch, kStaticScratchBytes, stream)) != LOQT_OK)
    return st;
  return check_device_status ? loqt_device_status(scratch, stream) : LOQT_OK;
}
