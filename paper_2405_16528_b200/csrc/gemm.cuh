// Warp-specialised persistent tcgen05 GEMM engine of the LoQT linear layer.
//
//   D[M x N] = sum over up to two K-segments of  A_seg[M x K_seg] * B_seg[N x K_seg]^T
//
// Each operand of each segment is either a bf16 matrix brought in by TMA (stored
// K-major or MN-major) or an NF4 matrix (paper Section 5.1).  For an NF4 operand
// TMA brings the packed 4-bit codes into shared memory and dedicated warps
// unpack and scale them straight into the 128-byte-swizzled layout the tensor
// core reads, so a dequantised weight never exists in global memory.
//
// Tile: (MH * 128) x BN outputs per CTA, K staged 64 deep.  MH = 1 keeps two
// TMEM accumulators so the epilogue of one tile overlaps the main loop of the
// next; MH = 2 computes two 128-row halves against the same B tile (each
// dequantised weight is then reused by 256 rows), filling TMEM with one tile.
//
// TWO mode (tcgen05 cta_group::2): two CTAs on neighbouring M tiles form a
// cluster and run every MMA together.  Each keeps its own A tile and its own
// accumulators but stages only half of the B tile (128 of the 256 N rows), and
// one thread of the leader CTA issues M = 256 instructions that drive both SMs'
// tensor cores.  Per SM this halves the dequantisation work, the B bytes written
// to shared memory and the B bytes the tensor core reads from it - and shared
// memory bandwidth is what bounds a single CTA here (per 256 x 256 x 64 stage the
// tensor core reads 96 KiB, TMA writes 40 KiB and the dequant warps move 40 KiB
// through a 128 B/clk port).  Barriers the MMA thread waits on live in the
// leader; the follower arrives on them through the cluster's shared-memory
// window.  "Slot free" and "accumulator ready" reach both CTAs at once: the
// commit that signals them is delivered to the same barrier in each CTA.
//
// Warp roles (480 threads): warp 0 TMA producer of the bf16 operands, warp 1
// MMA issuer + TMEM owner, warps 2-5 epilogue (one per TMEM lane quarter), warps
// 6-13 NF4 dequantisation, warp 14 TMA producer of the packed codes (their ring
// runs ahead of the operands', so it has a thread of its own).  One CTA per SM.
#pragma once
#include <type_traits>
#include "nf4_dequant.cuh"
#include "ptx.cuh"

namespace loqt {

constexpr int kHM = 128;      // rows of one MMA (M of tcgen05.mma)
constexpr int kBK = 64;       // K elements per pipeline stage (one 128-byte swizzle row of bf16)
constexpr int kUmmaK = 16;    // K of one tcgen05.mma for 16-bit inputs
constexpr int kNumThreads = 480;
constexpr int kEpiWarp0 = 2;  // warps 2..5
constexpr int kDeqWarp0 = 6;  // warps 6..13
constexpr int kDeqWarps = 8;
constexpr int kCodeWarp = 14;  // one thread: TMA producer of the packed NF4 codes

// Operand kinds
enum : int {
  OP_TMA_K = 0,   // bf16 [rows][K], K contiguous
  OP_TMA_MN = 1,  // bf16 [K][rows], rows (M or N index) contiguous
  OP_NF4_K = 2,   // NF4 [rows][K], blocks run along K
  OP_NF4_MN = 3,  // NF4 [K][rows], blocks run along the M/N index (B operand only)
};

// Epilogue kinds
enum : int {
  EPI_BF16 = 0,     // out bf16 = alpha * D
  EPI_F32 = 1,      // out fp32 = (addend, or out when accumulating, or 0) + alpha * D   (splits == 1)
  EPI_PARTIAL = 2,  // partial[split] fp32 = D                        (splits > 1)
};

// absmax: the fp32 block scales, or null when the scales are doubly quantised
// (paper Section 2.4): then scale i = fl32(fl32(E4M3(absmax8[i]) * c1[i / 256]) + *offset).
struct Nf4Src {
  const uint8_t *codes;
  const float *absmax;
  int rows, cols, ld;
  const uint8_t *absmax8;
  const float *c1;
  const float *offset;
};

struct Segment {
  int K;
  int a_kind, b_kind;
  Nf4Src a_nf4, b_nf4;
};

struct GemmParams {
  int M, N;
  int num_segs;
  Segment seg[2];
  int splits;       // split-K factor (single-segment GEMMs only)
  int kb_per_split; // k-blocks per split when splits > 1
  int epi;
  void *out;        // bf16 / fp32 output, or split-K partials
  int64_t ld_out;   // elements
  float alpha;
  int accumulate;
  const float *addend;  // EPI_F32: out = addend + alpha * D when set (16-byte aligned rows)
  int64_t ld_addend;
  uint32_t *status;  // device status word
  int has_nf4;       // any NF4 operand in any segment
};

// a/b: bf16 operands; ca/cb: packed NF4 codes viewed as a byte matrix.
struct TensorMaps {
  CUtensorMap a[2];
  CUtensorMap b[2];
  CUtensorMap ca[2];
  CUtensorMap cb[2];
};

// NF4: the kernel variant that stages NF4 operands (code ring, dequant warps); the
// variant without spends that shared memory on a deeper operand ring.
// REQ: the merge kernel (requantising epilogue): two buffers hold the packed codes
// of the output tiles' W_q blocks on their way from and to global memory.
// EXTRA: bytes of further staging after the code buffers (the compensation step's
// fp32 weights on their way to the epilogue warps, two mbarriers per warp with them).
template <int BN, int MH, bool TWO, bool NF4, bool REQ = false, int EXTRA = 0>
struct SmemLayout {
  static constexpr int kBM = MH * kHM;
  static constexpr int kBNL = TWO ? BN / 2 : BN;  // B rows staged by this CTA
  static constexpr int kABytes = kBM * kBK * 2;
  static constexpr int kBBytes = kBNL * kBK * 2;
  static constexpr int kCodeBytes = 8192;  // one code tile: up to 256 blocks x 32 bytes
  // Packed codes travel in a ring of their own with their own producer, ahead of
  // the operand ring, so that a freed operand slot can be dequantised into at once
  // instead of waiting for its codes to arrive.
  static constexpr int kStageBytes = kABytes + kBBytes;
  // The code ring is at least as deep as the operand ring (a staging group that has
  // seen operand slot `it` released may then conclude that the codes of stage
  // `it - kCodeStages` were consumed, which keeps its parity test unambiguous).
  static constexpr int kWTileBytes = REQ ? kHM * (BN / 2) : 0;  // codes of 128 rows x BN columns of W_q
  static constexpr int kWBufs = REQ ? 2 : 0;
  static constexpr int stages_for(int s) {
    return s * kStageBytes + (NF4 ? (s > 4 ? s : 4) * kCodeBytes : 0) + kWBufs * kWTileBytes + EXTRA <= 225 * 1024;
  }
  static constexpr int kStages = (!NF4 && stages_for(7)) ? 7 : stages_for(6) ? 6 : stages_for(5) ? 5 : stages_for(4) ? 4 : stages_for(3) ? 3 : 2;
  static constexpr int kCodeStages = !NF4 ? 0 : (kStages > 4 ? kStages : 4);
  static constexpr int kCodeOffset = kStages * kStageBytes;
  static constexpr int kWOffset = kCodeOffset + kCodeStages * kCodeBytes;  // (a multiple of 1024)
  static constexpr int kExtraOffset = kWOffset + kWBufs * kWTileBytes;  // (a multiple of 1024)
  static constexpr int kBarOffset = kExtraOffset + EXTRA;
  // full[S], empty[S], cfull[C], cempty[C], tfull[2], tempty[2], drain, wfull[2], wdone[2], extra[24]
  static constexpr int kNumBars = 2 * kStages + 2 * kCodeStages + 5 + 2 * kWBufs + (EXTRA > 0 ? 24 : 0);
  static constexpr int kMiscOffset = kBarOffset + kNumBars * 8;
  static constexpr int kTablesOffset = kMiscOffset + 16;
  static constexpr int kTotal = kTablesOffset + static_cast<int>(sizeof(Nf4Tables));
  static constexpr int kDynamicBytes = kTotal + 1024;  // slack for 1024-byte alignment
  static_assert(kStages >= 3, "pipeline too shallow");
  static_assert(!NF4 || kCodeStages >= kStages, "code ring too shallow");
  static_assert(kDynamicBytes <= 232448, "exceeds the 227 KiB shared memory of one CTA");
  static_assert(kBM * 32 <= kCodeBytes && kBNL * 32 <= kCodeBytes, "code tile too large");
  static_assert(!TWO || BN == 256, "pairs run 256-wide tiles");
  static_assert(!REQ || (MH == 1 && !TWO && !NF4), "the merge runs single 128-row tiles fed by TMA");
  static_assert(EXTRA % 1024 == 0, "the extra staging keeps the 1024-byte alignment of what follows");
};

// Shared-memory matrix descriptor (tcgen05), 128-byte swizzle.
//   K-major : rows of 128 bytes (64 bf16 of K), 8-row groups 1024 bytes apart.
//   MN-major: 64-element (128-byte) runs along M/N, 8 K-rows per 1024-byte group,
//             groups consecutive along K, 64-element column chunks 8192 bytes apart.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr, bool mn_major) {
  const uint64_t start = (saddr & 0x3FFFFu) >> 4;
  const uint64_t lbo = mn_major ? (8192u >> 4) : 1u;
  const uint64_t sbo = 1024u >> 4;
  return start | (lbo << 16) | (sbo << 32) | (1ull << 46) | (2ull << 61);
}

__device__ __forceinline__ uint32_t make_idesc(int m, int bn, bool a_mn, bool b_mn) {
  return (1u << 4)                                  // D format fp32
         | (1u << 7) | (1u << 10)                   // A, B format bf16
         | (a_mn ? (1u << 15) : 0u) | (b_mn ? (1u << 16) : 0u)
         | (static_cast<uint32_t>(bn >> 3) << 17)   // N
         | (static_cast<uint32_t>(m >> 4) << 24);   // M (128, or 256 for a CTA pair)
}

// Work decomposition shared by all roles.
struct Sched {
  int mt, nt, units;
  int kb_seg0, kb_total, splits, kb_per_split;
  // `pairs`: CTAs 2k and 2k+1 of the grid share every N tile, so the M tiles are
  // counted in twos; an odd count gets one tile past the matrix (its loads read
  // zeros, its rows are never stored).
  __device__ __forceinline__ Sched(const GemmParams &p, int bm, int bn, bool pairs) {
    mt = (p.M + bm - 1) / bm;
    if (pairs) mt = (mt + 1) & ~1;
    nt = (p.N + bn - 1) / bn;
    splits = p.splits;
    kb_per_split = p.kb_per_split;
    units = mt * nt * splits;
    kb_seg0 = (p.seg[0].K + kBK - 1) / kBK;
    kb_total = kb_seg0 + (p.num_segs > 1 ? (p.seg[1].K + kBK - 1) / kBK : 0);
  }
  __device__ __forceinline__ void unit(int u, int &m_blk, int &n_blk, int &split, int &kb_lo, int &kb_hi) const {
    m_blk = u % mt;
    const int t = u / mt;
    n_blk = t % nt;
    split = t / nt;
    if (splits > 1) {
      kb_lo = split * kb_per_split;
      kb_hi = min(kb_lo + kb_per_split, kb_total);
    } else {
      kb_lo = 0;
      kb_hi = kb_total;
    }
  }
};

// What one dequant thread does, fixed for as long as it stays in the same tile
// and K segment: where its 32 bytes of codes sit in a code tile, where its
// 128-byte operand row goes, and where its block scales come from.
struct DeqGeom {
  uint32_t src, src2;  // byte offsets of the two 16-byte code chunks inside the code tile
  uint32_t dst;        // byte offset of the 128-byte operand row inside the stage
  uint32_t sw;         // row index & 7 (swizzle key of the operand row)
  int active;          // 0: this thread has no row inside the matrix (outputs it would feed are discarded)
  const float *mptr;   // block scale of k-block 0 of the segment (fp32 scales)
  int64_t midx;        // its index in the matrix's sequence of scales (doubly quantised scales)
  const uint8_t *m8;   // doubly quantised scales: codes, second-level scales, offset (null otherwise)
  const float *c1;
  const float *off;
  int mstride;         // scales between consecutive k-blocks
  int kb_valid;        // k-blocks of the segment for which the row exists; later ones are the K tail (zeros)
  // A thread of a 256-row tile owns a second block, 128 tasks further on: the same
  // geometry shifted by constant offsets.
  int active2, kb_valid2;
  uint32_t d2, s2;     // byte offsets added to dst / src, src2
  int m2;              // floats added to mptr
};

// The per-stage part: the scale, fetched from global memory one stage ahead.
struct DeqTask {
  float M;
  int mode;  // 0: nothing to do, 1: dequantise, 2: write zeros
};

// BN here is the number of B rows this CTA stages (half a tile in TWO mode) and
// n_blk counts in units of it.
template <int BN, int kBM, int kABytes>
__device__ __forceinline__ DeqGeom deq_geom(const GemmParams &p, int seg_idx, int m_blk, int n_blk, int t) {
  DeqGeom g;
  g.src = g.src2 = g.dst = g.sw = 0;
  g.active = 0;
  g.mptr = nullptr;
  g.midx = 0;
  g.m8 = nullptr;
  g.c1 = nullptr;
  g.off = nullptr;
  g.mstride = 0;
  g.kb_valid = 0;
  g.active2 = g.kb_valid2 = 0;
  g.d2 = g.s2 = 0;
  g.m2 = 0;
  const Segment &sg = p.seg[seg_idx];
  const bool a_nf4 = sg.a_kind >= OP_NF4_K;
  const bool b_nf4 = sg.b_kind >= OP_NF4_K;
  if (!a_nf4 && !b_nf4) return g;
  const int kind = a_nf4 ? sg.a_kind : sg.b_kind;
  const Nf4Src &src = a_nf4 ? sg.a_nf4 : sg.b_nf4;
  const int rows_tile = a_nf4 ? kBM : BN;
  if (t >= rows_tile) return g;
  const uint32_t base = a_nf4 ? 0u : static_cast<uint32_t>(kABytes);
  const int mn0 = a_nf4 ? m_blk * kBM : n_blk * BN;
  const int nb = src.ld >> 6;
  if (kind == OP_NF4_K) {
    // tile row t <- matrix row mn0 + t, codes of one k-block; code tile is [rows][32 B]
    const int row = mn0 + t;
    g.sw = static_cast<uint32_t>(t & 7);
    g.dst = base + static_cast<uint32_t>((t >> 3) * 1024 + (t & 7) * 128);
    g.src = static_cast<uint32_t>(t * 32);
    g.src2 = g.src + 16;
    if (row >= src.rows) return g;
    g.active = 1;
    g.midx = static_cast<int64_t>(row) * nb;
    g.mstride = 1;
    g.kb_valid = 0x7fffffff;  // padded columns hold the zero level
    // second block: tile row t + 128
    g.active2 = (t + 128 < rows_tile) && (row + 128 < src.rows);
    g.kb_valid2 = g.kb_valid;
    g.d2 = 128u * 128u;
    g.s2 = 128u * 32u;
    g.m2 = 128 * nb;
  } else {
    // 64-column chunk j, K-row kk <- matrix row 64 kb + kk, codes of columns mn0 + 64 j ..
    // A warp takes 8 consecutive K-rows of every chunk, so that its operand-row
    // stores and its code-tile loads each touch 8 different swizzle positions.
    constexpr int JB = BN / 64;
    constexpr int jbits = (JB == 4) ? 2 : 1;
    const int j = (t >> 3) & (JB - 1);
    const int kk = (t & 7) | ((t >> (3 + jbits)) << 3);
    const int col0 = mn0 + 64 * j;
    g.sw = static_cast<uint32_t>(kk & 7);
    g.dst = base + static_cast<uint32_t>(j * 8192 + (kk >> 3) * 1024 + (kk & 7) * 128);
    // code tile is [64 K-rows][BN/2 bytes], TMA-swizzled (128 B rows: 128-byte
    // swizzle, 64 B rows: 64-byte swizzle): chunk ^= (offset >> 7) & mask
    constexpr uint32_t RB = BN / 2;
    constexpr uint32_t mask = (RB == 128) ? 7u : 3u;
    const uint32_t o0 = static_cast<uint32_t>(kk) * RB + static_cast<uint32_t>(j) * 32u;
    const uint32_t o1 = o0 + 16u;
    g.src = o0 ^ (((o0 >> 7) & mask) << 4);
    g.src2 = o1 ^ (((o1 >> 7) & mask) << 4);
    if (col0 >= src.ld) return g;
    g.active = 1;
    g.midx = static_cast<int64_t>(kk) * nb + (col0 >> 6);
    g.mstride = 64 * nb;
    g.kb_valid = src.rows > kk ? (src.rows - kk + 63) >> 6 : 0;  // beyond: the K tail must contribute zero
    // second block (256-row tiles only): same chunk, K-row kk + 32
    g.active2 = (BN == 256);
    g.kb_valid2 = src.rows > kk + 32 ? (src.rows - kk - 32 + 63) >> 6 : 0;
    g.d2 = 4u * 1024u;
    g.s2 = 32u * RB;
    g.m2 = 32 * nb;
  }
  if (src.absmax != nullptr) {
    g.mptr = src.absmax + g.midx;
  } else {
    g.m8 = src.absmax8;
    g.c1 = src.c1;
    g.off = src.offset;
  }
  return g;
}

template <int kSecond>
__device__ __forceinline__ DeqTask deq_fetch(const DeqGeom &g, int kb_in_seg) {
  DeqTask task;
  task.M = 0.0f;
  const int active = kSecond ? g.active2 : g.active;
  const int valid = kSecond ? g.kb_valid2 : g.kb_valid;
  task.mode = !active ? 0 : (kb_in_seg < valid ? 1 : 2);
  if (task.mode == 1) {
    const int64_t rel = static_cast<int64_t>(kb_in_seg) * g.mstride + (kSecond ? g.m2 : 0);
    if (g.m8 == nullptr) task.M = __ldg(g.mptr + rel);
    else task.M = dq_scale(g.m8, g.c1, g.off, g.midx + rel);
  }
  return task;
}

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint4 v) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
               : "memory");
}
__device__ __forceinline__ uint4 ld_shared_v4(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr)
               : "memory");
  return v;
}

template <int kSecond>
__device__ __forceinline__ void deq_store(const DeqGeom &g, const DeqTask &task, uint32_t stage_base,
                                          uint32_t code_base) {
  if (task.mode == 0) return;
  const uint32_t dst = stage_base + g.dst + (kSecond ? g.d2 : 0u);
  if (task.mode == 2) {
#pragma unroll
    for (uint32_t c = 0; c < 8; ++c) st_shared_v4(dst + ((c ^ g.sw) << 4), make_uint4(0, 0, 0, 0));
    return;
  }
  const uint4 c0 = ld_shared_v4(code_base + g.src + (kSecond ? g.s2 : 0u));
  const uint4 c1 = ld_shared_v4(code_base + g.src2 + (kSecond ? g.s2 : 0u));
  Nf4BlockTable tab;
  nf4_block_table(task.M, tab);
  const uint32_t w[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
  // the row is 128-byte aligned, so the swizzled chunk address is a pure XOR
  const uint32_t dst_x = dst ^ (g.sw << 4);
#pragma unroll
  for (uint32_t c = 0; c < 8; ++c) st_shared_v4(dst_x ^ (c << 4), nf4_dequant8(tab, w[c]));
}

// ---------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------
template <int BN, int MH, bool TWO, bool NF4>
__global__ void __launch_bounds__(kNumThreads, 1)
loqt_gemm_kernel(const __grid_constant__ TensorMaps maps, const GemmParams p) {
  using L = SmemLayout<BN, MH, TWO, NF4>;
  constexpr int kStages = L::kStages;
  constexpr int kBM = L::kBM;
  constexpr int kBNL = L::kBNL;
  constexpr int kAccBufs = (MH == 1) ? 2 : 1;  // TMEM accumulator buffers (each MH * BN columns)
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t *smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

  const uint32_t bar0 = smem_base + L::kBarOffset;
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kStages + s); };
  constexpr int kCodeStages = L::kCodeStages;
  constexpr int kCodeRing = kCodeStages > 0 ? kCodeStages : 1;  // (no code ring in kernels without NF4 operands)
  auto cfull_bar = [&](int c) { return bar0 + 8u * (2 * kStages + c); };
  auto cempty_bar = [&](int c) { return bar0 + 8u * (2 * kStages + kCodeStages + c); };
  auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * kStages + 2 * kCodeStages + a); };
  auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * kStages + 2 * kCodeStages + 2 + a); };
  const uint32_t drain_bar = bar0 + 8u * (2 * kStages + 2 * kCodeStages + 4);
  volatile uint32_t *misc = reinterpret_cast<volatile uint32_t *>(smem_gen + L::kMiscOffset);
  volatile uint32_t *tmem_slot = misc;       // written by tcgen05.alloc
  volatile uint32_t *abort_flag = misc + 1;  // raised by any role whose wait expired

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const Sched sched(p, kBM, BN, TWO);
  // TWO: rank 0 of the pair is the leader (issues the MMAs, owns the barriers the
  // MMA thread waits on).
  const uint32_t rank = TWO ? ptx::cluster_ctarank() : 0u;
  const bool leader = (rank == 0);
  // The dequant warps work as two groups of four that take the K stages of a
  // tile in turn, so that one group's barrier, fence and bookkeeping time is
  // covered by the other's table lookups (the dequantisation is bound by the
  // latency of its dependent chains, not by ALU throughput: more warps, more
  // overlap).  A group stages a whole tile: one block per thread for 128 rows,
  // two for 256.  (A third group made of the epilogue warps, idle during the main
  // loop of single-accumulator kernels, was measured 5 % slower: with three stages
  // in the ring a third group only waits for a slot.)
  constexpr int kGroupWarps = kDeqWarps / 2;
  constexpr int deq_groups = NF4 ? 2 : 0;
  const int deq_grp = (warp - kDeqWarp0) / kGroupWarps;
  constexpr uint32_t kTmemCols = 2 * BN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      // arrivals: the leader's TMA producer (which also posts the follower's bytes) and
      // the dequant warps of every CTA of the pair
      ptx::mbar_init(full_bar(s), 1 + (NF4 ? kGroupWarps * (TWO ? 2 : 1) : 0));
      ptx::mbar_init(empty_bar(s), 1);
    }
    for (int c = 0; c < kCodeStages; ++c) {
      ptx::mbar_init(cfull_bar(c), 1);             // the producer (with the tile's bytes, if any)
      ptx::mbar_init(cempty_bar(c), kGroupWarps);  // the staging group that used the tile
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(tfull_bar(a), 1);
      ptx::mbar_init(tempty_bar(a), 4 * (TWO ? 2 : 1));  // the four epilogue warps (of each CTA of a pair)
    }
    ptx::mbar_init(drain_bar, 1);
    *abort_flag = 0;
    ptx::fence_barrier_init();
  }
  if (warp == 1) {
    if (TWO) {
      ptx::tmem_alloc_pair(smem_u32(const_cast<uint32_t *>(tmem_slot)), kTmemCols);
      ptx::tmem_relinquish_pair();
    } else {
      ptx::tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_slot)), kTmemCols);
      ptx::tmem_relinquish();
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (TWO) ptx::cluster_sync_all();  // both CTAs' barriers exist before anything arrives on them
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Everything above (barriers, TMEM, tables) touched no global data, so it may
  // overlap the tail of the previous kernel of the stream; from here on global
  // memory is read and written.
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();

  // ---------------------------------------------------------- NF4 staging worker
  // State and one-stage step of a staging group.  Group g takes the stages of a
  // tile whose index within the tile is g modulo the number of groups.
  constexpr bool kTwoRows = (kBNL == 256);  // (an NF4 A tile is 128 rows: one block per thread)
  const int deq_t = (threadIdx.x - kDeqWarp0 * 32) & (kGroupWarps * 32 - 1);
  // Two cursors over this CTA's k-blocks: the one being staged and, one step
  // ahead, the one whose scale is being fetched.  A cursor recomputes its
  // geometry only when it enters a new tile or K segment.
  struct Cursor {
    int u, kb, kb_lo, kb_hi, m_blk, n_blk, seg;
    uint32_t it;  // position in the CTA's sequence of stages (all groups count alike)
    DeqGeom g;
  };
  auto cur_enter = [&](Cursor &c) {  // c.kb valid: (re)compute segment and geometry
    c.seg = c.kb < sched.kb_seg0 ? 0 : 1;
    // this CTA's B rows start at local block (TWO: 2 n_blk + rank) of kBNL rows
    c.g = deq_geom<kBNL, kBM, L::kABytes>(p, c.seg, c.m_blk, TWO ? 2 * c.n_blk + static_cast<int>(rank) : c.n_blk, deq_t);
  };
  auto cur_open = [&](Cursor &c) {
    while (c.u < sched.units) {
      int split;
      sched.unit(c.u, c.m_blk, c.n_blk, split, c.kb_lo, c.kb_hi);
      c.kb = c.kb_lo;
      if (c.kb < c.kb_hi) {
        cur_enter(c);
        return true;
      }
      c.u += gridDim.x;
    }
    return false;
  };
  auto cur_advance = [&](Cursor &c) {
    ++c.it;
    if (++c.kb < c.kb_hi) {
      if (c.kb == sched.kb_seg0) cur_enter(c);  // crossed into the second segment
      return true;
    }
    c.u += gridDim.x;
    return cur_open(c);
  };
  auto cur_mine = [&](const Cursor &c) { return (c.kb - c.kb_lo) % (NF4 ? deq_groups : 1) == deq_grp; };
  auto cur_next_mine = [&](Cursor &c) {  // to this group's next stage
    do {
      if (!cur_advance(c)) return false;
    } while (!cur_mine(c));
    return true;
  };
  auto cur_kb_in = [&](const Cursor &c) { return c.seg == 0 ? c.kb : c.kb - sched.kb_seg0; };

  Cursor cur, nxt;
  DeqTask task0, task1;
  bool deq_have = false, deq_have_next = false;
  auto deq_begin = [&]() {
    cur.u = blockIdx.x;
    cur.it = 0;
    deq_have = cur_open(cur);
    if (deq_have && !cur_mine(cur)) deq_have = cur_next_mine(cur);
    task0.mode = task1.mode = 0;
    task0.M = task1.M = 0.0f;
    if (deq_have) {
      task0 = deq_fetch<0>(cur.g, cur_kb_in(cur));
      if (kTwoRows) task1 = deq_fetch<1>(cur.g, cur_kb_in(cur));
    }
    nxt = cur;
    deq_have_next = deq_have && cur_next_mine(nxt);
  };
  // Stages the block(s) of this thread for the stage under `cur`; false when a wait expired.
  auto deq_step = [&]() -> bool {
    DeqTask next0, next1;
    next0.mode = next1.mode = 0;
    next0.M = next1.M = 0.0f;
    if (deq_have_next) {  // in flight while this stage is dequantised
      next0 = deq_fetch<0>(nxt.g, cur_kb_in(nxt));
      if (kTwoRows) next1 = deq_fetch<1>(nxt.g, cur_kb_in(nxt));
    }
    const int s = cur.it % kStages;
    const uint32_t ph = (cur.it / kStages) & 1u;
    // First the operand slot's release (the same event the producer waits for), then
    // the code tile of this stage.  The order matters: once stage `it - kStages` has
    // been consumed, every stage up to `it - kCodeStages` has been staged, so the code
    // barrier cannot still be in the phase two uses back, which a parity test would
    // read as "already complete".
    const int cs = cur.it % kCodeRing;
    const uint32_t cph = (cur.it / kCodeRing) & 1u;
    if (!ptx::mbar_wait<TWO>(empty_bar(s), ph ^ 1u, abort_flag, p.status)) return false;
    if (!ptx::mbar_wait(cfull_bar(cs), cph, abort_flag, p.status)) return false;
    const uint32_t stage_base = smem_base + s * L::kStageBytes;
    const uint32_t code_base = smem_base + L::kCodeOffset + cs * L::kCodeBytes;
    deq_store<0>(cur.g, task0, stage_base, code_base);
    if (kTwoRows) deq_store<1>(cur.g, task1, stage_base, code_base);
    ptx::fence_proxy_async_smem();  // (pairs too: the writes are to this CTA's own shared memory)
    __syncwarp();
    if (lane == 0) {
      ptx::mbar_arrive(cempty_bar(cs));  // code tile read: the producer may refill it
      if (TWO && !leader) ptx::mbar_arrive_cluster(ptx::map_to_cta(full_bar(s), 0));
      else ptx::mbar_arrive(full_bar(s));
    }
    cur = nxt;
    deq_have = deq_have_next;
    task0 = next0;
    task1 = next1;
    if (deq_have_next) deq_have_next = cur_next_mine(nxt);
    return true;
  };

  // =========================================================== TMA producer
  if (warp == 0) {
    if (lane == 0) {
      for (int s = 0; s < p.num_segs; ++s) {
        ptx::prefetch_tensormap(p.seg[s].a_kind <= OP_TMA_MN ? &maps.a[s] : &maps.ca[s]);
        ptx::prefetch_tensormap(p.seg[s].b_kind <= OP_TMA_MN ? &maps.b[s] : &maps.cb[s]);
      }
      bool ok = true;
      uint32_t it = 0;
      for (int u = blockIdx.x; ok && u < sched.units; u += gridDim.x) {
        int m_blk, n_blk, split, kb_lo, kb_hi;
        sched.unit(u, m_blk, n_blk, split, kb_lo, kb_hi);
        // first B row staged by this CTA (the follower of a pair takes the upper half of the tile)
        const int n_row0 = n_blk * BN + (TWO ? static_cast<int>(rank) * kBNL : 0);
        for (int kb = kb_lo; kb < kb_hi; ++kb, ++it) {
          const int s = it % kStages;
          const uint32_t ph = (it / kStages) & 1u;
          if (!(ok = ptx::mbar_wait<TWO>(empty_bar(s), ph ^ 1u, abort_flag, p.status))) break;
          const int sidx = kb < sched.kb_seg0 ? 0 : 1;
          const int k0 = (sidx == 0 ? kb : kb - sched.kb_seg0) * kBK;
          const Segment &sg = p.seg[sidx];
          const uint32_t a_dst = smem_base + s * L::kStageBytes;
          const uint32_t b_dst = a_dst + L::kABytes;
          uint32_t bytes = 0;
          if (sg.a_kind <= OP_TMA_MN) bytes += L::kABytes;
          if (sg.b_kind <= OP_TMA_MN) bytes += L::kBBytes;
          // the pair's full barrier lives in the leader, which expects both CTAs' bytes
          const uint32_t fbar = TWO ? ptx::map_to_cta(full_bar(s), 0) : full_bar(s);
          if (!TWO) ptx::mbar_arrive_expect_tx(fbar, bytes);
          else if (leader) ptx::mbar_arrive_expect_tx(full_bar(s), 2 * bytes);
          auto load = [&](uint32_t dst, const CUtensorMap *m, int c0, int c1) {
            if (TWO) ptx::tma_load_2d_pair(dst, m, fbar, c0, c1);
            else ptx::tma_load_2d(dst, m, fbar, c0, c1);
          };
          if (sg.a_kind == OP_TMA_K) {
            load(a_dst, &maps.a[sidx], k0, m_blk * kBM);
          } else if (sg.a_kind == OP_TMA_MN) {
#pragma unroll
            for (int j = 0; j < kBM / 64; ++j) load(a_dst + j * 8192, &maps.a[sidx], m_blk * kBM + 64 * j, k0);
          }
          if (sg.b_kind == OP_TMA_K) {
            load(b_dst, &maps.b[sidx], k0, n_row0);
          } else if (sg.b_kind == OP_TMA_MN) {
#pragma unroll
            for (int j = 0; j < kBNL / 64; ++j) load(b_dst + j * 8192, &maps.b[sidx], n_row0 + 64 * j, k0);
          }
        }
      }
      if (!ok) {
        // Give copies already in flight time to land before the CTA's shared
        // memory is released.
        const uint64_t t0 = ptx::globaltimer_ns();
        while (ptx::globaltimer_ns() - t0 < 200000ull) {
        }
      }
    }
  }
  // =========================================================== MMA issuer
  else if (warp == 1) {
    if (lane == 0 && leader) {
      uint32_t it = 0, tile = 0;
      bool ok = true;
      for (int u = blockIdx.x; ok && u < sched.units; u += gridDim.x, ++tile) {
        int m_blk, n_blk, split, kb_lo, kb_hi;
        sched.unit(u, m_blk, n_blk, split, kb_lo, kb_hi);
        const uint32_t acc = tile % kAccBufs;
        const uint32_t acc_ph = (tile / kAccBufs) & 1u;
        if (!(ok = ptx::mbar_wait<TWO>(tempty_bar(acc), acc_ph ^ 1u, abort_flag, p.status))) break;
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * (MH * BN);
        for (int kb = kb_lo; kb < kb_hi; ++kb, ++it) {
          const int s = it % kStages;
          const uint32_t ph = (it / kStages) & 1u;
          if (!(ok = ptx::mbar_wait<TWO>(full_bar(s), ph, abort_flag, p.status))) break;
          ptx::tc_fence_after();
          const Segment &sg = p.seg[kb < sched.kb_seg0 ? 0 : 1];
          const bool a_mn = (sg.a_kind == OP_TMA_MN);
          const bool b_mn = (sg.b_kind == OP_TMA_MN) || (sg.b_kind == OP_NF4_MN);
          const uint32_t idesc = make_idesc(TWO ? 2 * kHM : kHM, BN, a_mn, b_mn);
          const uint32_t a_addr = smem_base + s * L::kStageBytes;
          const uint32_t b_addr = a_addr + L::kABytes;
          const uint64_t b_desc = make_smem_desc(b_addr, b_mn);
          const uint32_t a_step = a_mn ? (2048u >> 4) : (32u >> 4);
          const uint32_t b_step = b_mn ? (2048u >> 4) : (32u >> 4);
#pragma unroll
          for (int h = 0; h < MH; ++h) {
            // half h: rows 128 h .. 128 h + 127 of the A tile (16 KiB further in either layout)
            const uint64_t a_desc = make_smem_desc(a_addr + h * (kHM * kBK * 2), a_mn);
#pragma unroll
            for (uint32_t k = 0; k < kBK / kUmmaK; ++k) {
              const uint32_t accum = (kb > kb_lo || k > 0) ? 1u : 0u;
              if (TWO) ptx::mma_bf16_ss_pair(d_tmem + h * BN, a_desc + k * a_step, b_desc + k * b_step, idesc, accum);
              else ptx::mma_bf16_ss(d_tmem + h * BN, a_desc + k * a_step, b_desc + k * b_step, idesc, accum);
            }
          }
          // stage reusable (in both CTAs) once these MMAs have read it
          if (TWO) ptx::mma_commit_pair_both(empty_bar(s));
          else ptx::mma_commit(empty_bar(s));
        }
        if (ok) {
          if (TWO) ptx::mma_commit_pair_both(tfull_bar(acc));
          else ptx::mma_commit(tfull_bar(acc));
        }
      }
      // Every MMA issued above must have finished before TMEM is freed.
      if (TWO) ptx::mma_commit_pair(drain_bar);
      else ptx::mma_commit(drain_bar);
      ptx::mbar_wait<TWO>(drain_bar, 0, abort_flag, p.status);
    }
  }
  // =========================================================== code producer
  else if (warp == kCodeWarp) {
    if (lane == 0 && NF4) {
      // A cursor over the same sequence of stages as the operand producer's; the
      // ring's depth bounds how far the codes run ahead.
      struct CodeCursor {
        int u, kb, kb_hi, m_blk, n_blk;
        uint32_t it;
        bool valid;
      };
      auto cc_open = [&](CodeCursor &c) {
        while (c.u < sched.units) {
          int split, lo;
          sched.unit(c.u, c.m_blk, c.n_blk, split, lo, c.kb_hi);
          c.kb = lo;
          if (c.kb < c.kb_hi) return true;
          c.u += gridDim.x;
        }
        return false;
      };
      bool ok = true;
      // Posts the code tile of the cursor's stage (or an empty completion when the
      // stage has no NF4 operand) and moves the cursor on.
      auto issue_codes = [&](CodeCursor &c) {
        const int cs = c.it % kCodeRing;
        const uint32_t cph = (c.it / kCodeRing) & 1u;
        if (!(ok = ptx::mbar_wait(cempty_bar(cs), cph ^ 1u, abort_flag, p.status))) return;
        const int sidx = c.kb < sched.kb_seg0 ? 0 : 1;
        const int k0 = (sidx == 0 ? c.kb : c.kb - sched.kb_seg0) * kBK;
        const Segment &sg = p.seg[sidx];
        const int n_row0 = c.n_blk * BN + (TWO ? static_cast<int>(rank) * kBNL : 0);
        const uint32_t c_dst = smem_base + L::kCodeOffset + cs * L::kCodeBytes;
        if (sg.a_kind == OP_NF4_K) {
          ptx::mbar_arrive_expect_tx(cfull_bar(cs), kBM * 32);
          ptx::tma_load_2d(c_dst, &maps.ca[sidx], cfull_bar(cs), k0 >> 1, c.m_blk * kBM);
        } else if (sg.b_kind == OP_NF4_K) {
          ptx::mbar_arrive_expect_tx(cfull_bar(cs), kBNL * 32);
          ptx::tma_load_2d(c_dst, &maps.cb[sidx], cfull_bar(cs), k0 >> 1, n_row0);
        } else if (sg.b_kind == OP_NF4_MN) {
          ptx::mbar_arrive_expect_tx(cfull_bar(cs), kBNL * 32);
          ptx::tma_load_2d(c_dst, &maps.cb[sidx], cfull_bar(cs), n_row0 >> 1, k0);
        } else {
          ptx::mbar_arrive(cfull_bar(cs));  // nothing to dequantise in this stage
        }
        ++c.it;
        if (++c.kb >= c.kb_hi) {
          c.u += gridDim.x;
          c.valid = cc_open(c);
        }
      };
      CodeCursor cc;
      cc.u = blockIdx.x;
      cc.it = 0;
      cc.valid = NF4 && cc_open(cc);
      while (ok && cc.valid) issue_codes(cc);

    }
  }
  // =========================================================== epilogue
  else if (warp < kDeqWarp0) {
    const int q = warp & 3;  // TMEM lane quarter this warp may access
    uint32_t tile = 0;
    bool ok = true;
    for (int u = blockIdx.x; ok && u < sched.units; u += gridDim.x, ++tile) {
      int m_blk, n_blk, split, kb_lo, kb_hi;
      sched.unit(u, m_blk, n_blk, split, kb_lo, kb_hi);
      const uint32_t acc = tile % kAccBufs;
      const uint32_t acc_ph = (tile / kAccBufs) & 1u;
      if (!(ok = ptx::mbar_wait<TWO>(tfull_bar(acc), acc_ph, abort_flag, p.status))) break;
      ptx::tc_fence_after();
      const int n_base = n_blk * BN;
#pragma unroll 1
      for (int h = 0; h < MH; ++h) {
        const int row = m_blk * kBM + h * kHM + q * 32 + lane;
        const bool row_ok = row < p.M;
        const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * (MH * BN) + h * BN;
        {
#pragma unroll 1
          for (int cb = 0; cb < BN / 32; ++cb) {
            uint32_t d[32];
            ptx::tmem_ld32(t_row + cb * 32, d);
            ptx::tmem_ld_wait();
            const int c0 = n_base + cb * 32;
            const bool full = (c0 + 32 <= p.N);
            if (!row_ok || c0 >= p.N) {
              // nothing to store for this thread
            } else if (p.epi == EPI_BF16) {
              __nv_bfloat16 *o = reinterpret_cast<__nv_bfloat16 *>(p.out) + static_cast<int64_t>(row) * p.ld_out + c0;
              if (full && (p.ld_out & 7) == 0) {
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                  uint4 qv;
                  qv.x = pack_bf16x2(p.alpha * __uint_as_float(d[8 * g + 0]), p.alpha * __uint_as_float(d[8 * g + 1]));
                  qv.y = pack_bf16x2(p.alpha * __uint_as_float(d[8 * g + 2]), p.alpha * __uint_as_float(d[8 * g + 3]));
                  qv.z = pack_bf16x2(p.alpha * __uint_as_float(d[8 * g + 4]), p.alpha * __uint_as_float(d[8 * g + 5]));
                  qv.w = pack_bf16x2(p.alpha * __uint_as_float(d[8 * g + 6]), p.alpha * __uint_as_float(d[8 * g + 7]));
                  reinterpret_cast<uint4 *>(o)[g] = qv;
                }
              } else {
#pragma unroll
                for (int e = 0; e < 32; ++e)
                  if (c0 + e < p.N) o[e] = __float2bfloat16_rn(p.alpha * __uint_as_float(d[e]));
              }
            } else {
              float *o;
              const int64_t ldo = p.ld_out;
              const float *base = nullptr;  // what the product is added to
              float scale = 1.0f;
              bool base_vec = true;
              if (p.epi == EPI_PARTIAL) {
                o = reinterpret_cast<float *>(p.out) + (static_cast<int64_t>(split) * p.M + row) * ldo + c0;
              } else {
                o = reinterpret_cast<float *>(p.out) + static_cast<int64_t>(row) * ldo + c0;
                scale = p.alpha;
                if (p.addend != nullptr) {
                  base = p.addend + static_cast<int64_t>(row) * p.ld_addend + c0;
                  base_vec = (p.ld_addend & 3) == 0;
                } else if (p.accumulate != 0) {
                  base = o;
                }
              }
              if (full && (ldo & 3) == 0 && base_vec) {
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                  float4 b4 = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                  if (base != nullptr) b4 = reinterpret_cast<const float4 *>(base)[g];
                  float4 f;
                  f.x = fmaf(scale, __uint_as_float(d[4 * g]), b4.x);
                  f.y = fmaf(scale, __uint_as_float(d[4 * g + 1]), b4.y);
                  f.z = fmaf(scale, __uint_as_float(d[4 * g + 2]), b4.z);
                  f.w = fmaf(scale, __uint_as_float(d[4 * g + 3]), b4.w);
                  reinterpret_cast<float4 *>(o)[g] = f;
                }
              } else {
#pragma unroll
                for (int e = 0; e < 32; ++e)
                  if (c0 + e < p.N) o[e] = fmaf(scale, __uint_as_float(d[e]), base != nullptr ? base[e] : 0.0f);
              }
            }
            __syncwarp();
          }
        }
      }
      // Accumulator fully read: hand the TMEM buffer back to the MMA warp.
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (TWO && !leader) ptx::mbar_arrive_cluster(ptx::map_to_cta(tempty_bar(acc), 0));
        else ptx::mbar_arrive(tempty_bar(acc));
      }
    }
  }
  // =========================================================== NF4 dequant
  else {
    if (NF4 && warp < kDeqWarp0 + kGroupWarps * deq_groups) {
      deq_begin();
      while (deq_have && deq_step()) {
      }
    }
  }

  // =========================================================== teardown
  ptx::tc_fence_before();
  __syncthreads();
  // neither CTA of a pair may free TMEM or leave while the other still uses the
  // pair's barriers, its shared memory (MMA operands) or its accumulators
  if (TWO) ptx::cluster_sync_all();
  if (warp == 1) {
    ptx::tc_fence_after();
    if (TWO) ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
    else ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

// Deterministic split-K reduction: out = (accumulate ? out : 0) + sum_s partial[s].
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(const float *__restrict__ partial, int splits, int M, int N, int64_t ld_partial,
                     float *__restrict__ out, int64_t ld_out, int accumulate) {
  const int64_t total = static_cast<int64_t>(M) * N;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += stride) {
    const int m = static_cast<int>(i / N);
    const int n = static_cast<int>(i - static_cast<int64_t>(m) * N);
    float acc = accumulate ? out[static_cast<int64_t>(m) * ld_out + n] : 0.0f;
    for (int s = 0; s < splits; ++s) acc += partial[(static_cast<int64_t>(s) * M + m) * ld_partial + n];
    out[static_cast<int64_t>(m) * ld_out + n] = acc;
  }
}

}  // namespace loqt
