// The periodic merge of LoQT (paper Section 2.4; Algorithm 1, merge line):
//
//   W_q <- q_NF4( deq32(W_q) + alpha * P-hat B )          in place, for a batch of matrices
//
// One persistent launch walks the output tiles of every matrix of the batch, so
// the tiles of the next matrix fill the SMs that the last wave of the previous
// one would leave idle.  P-hat (out x r, bf16, staged beforehand) and B (r x in,
// bf16) arrive by TMA; the product of a 128 x BN tile accumulates in one of two
// TMEM buffers; the epilogue reads it, one 64-column block of one row per
// thread - which is exactly one NF4 block of W_q - adds the old dequantised
// values, takes the block maximum, requantises (quantiser of Section 5.1) and
// writes codes and scale back.
//
// Warp roles (480 threads): warp 0 TMA producer, warp 1 MMA issuer and TMEM
// owner, warps 2-13 epilogue (three groups of four, one warp per TMEM lane
// quarter; the 64-column blocks are dealt to the groups round-robin, continuing
// across tiles), warp 14 mover of W_q.  The mover brings the packed codes and
// the scales of each tile's W_q blocks into shared memory ahead of the tile's
// epilogue - whole 128-byte rows by one bulk copy instead of a 32-byte access
// per thread and block - and stores the requantised tile once every epilogue
// warp is done with it.
#pragma once
#include "gemm.cuh"

namespace loqt {

constexpr int kMergeBatchMax = 32;  // matrices per launch (bounded by the kernel parameter space)

struct MergeProblem {
  float *wq_absmax;  // [M][wq_ld / 64]
  int M, N, K;       // out, in, r
  int wq_ld;
  int tile0;         // position of this matrix's first tile in the launch's sequence of tiles
  int mt;            // tiles along M (tile = tile0 + n_blk * mt + m_blk)
  float alpha;
  int pad_;
  // compensation mode only (kComp): the fp32 matrix that takes the place of deq32(W_q)
  // in the sum, and the bf16 residual W - deq32(new codes) written beside the codes
  const float *w32;       // [M][ld_w32]
  __nv_bfloat16 *resid;   // [M][ld_resid]
  int64_t ld_w32, ld_resid;
};

struct MergeBatch {
  CUtensorMap a[kMergeBatchMax];   // P-hat, bf16 [M][K]: box 64 (K) x 128 rows
  CUtensorMap b[kMergeBatchMax];   // B, bf16 [K][N]: box 64 (N) x 64 (K), an MN-major operand
  CUtensorMap wq[kMergeBatchMax];  // packed codes of W_q as bytes [M][wq_ld / 2]: box BN / 2 x 128 rows
  MergeProblem prob[kMergeBatchMax];
  CUtensorMap wmap;  // compensation mode (one matrix per launch): W, fp32 [M][ld_w32]: box 32 columns x 32 rows
  int count;
  int tiles;  // of all matrices together
  uint32_t *status;
};

// kComp = false: the merge above.  kComp = true: one step of the error-compensated
// initialisation (paper Section 2.5; Algorithm 2, compensation loop) in the same
// pipeline: the fp32 weights W take the place of deq32(W_q) in the sum,
//   Q <- q_NF4( W + alpha * A B )        (alpha = -1, A = P, B = B_(c-1)),
// the codes and scales of Q are written (nothing of W_q is read), and with them
// the bf16 residual W - deq32(Q) that the next product P^T (W - Q) consumes.  The
// corrected weights W - P B never exist in memory.
constexpr int kCompStageBytes = 32 * 128;  // per epilogue warp: 32 rows x 32 fp32 columns of W
template <int BN, bool kComp>
using MergeLayout = SmemLayout<BN, 1, false, false, true, kComp ? 12 * kCompStageBytes : 0>;

template <int BN, bool kComp = false>
__global__ void __launch_bounds__(kNumThreads, 1)
loqt_merge_kernel(const __grid_constant__ MergeBatch mb) {
  using L = MergeLayout<BN, kComp>;
  constexpr int kStages = L::kStages;
  constexpr int kEpiGroups = 3;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t *smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

  const uint32_t bar0 = smem_base + L::kBarOffset;
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kStages + s); };
  auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * kStages + a); };
  auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * kStages + 2 + a); };
  const uint32_t drain_bar = bar0 + 8u * (2 * kStages + 4);
  auto wfull_bar = [&](int b) { return bar0 + 8u * (2 * kStages + 5 + b); };
  auto wdone_bar = [&](int b) { return bar0 + 8u * (2 * kStages + 7 + b); };
  // compensation mode, per epilogue warp: staging tile filled / staging tile read by every lane
  auto stage_bar = [&](int w) { return bar0 + 8u * (2 * kStages + 9 + w); };
  auto free_bar = [&](int w) { return bar0 + 8u * (2 * kStages + 21 + w); };
  volatile uint32_t *misc = reinterpret_cast<volatile uint32_t *>(smem_gen + L::kMiscOffset);
  volatile uint32_t *tmem_slot = misc;
  volatile uint32_t *abort_flag = misc + 1;
  Nf4Tables &tables = *reinterpret_cast<Nf4Tables *>(smem_gen + L::kTablesOffset);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  constexpr uint32_t kTmemCols = 2 * BN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(tfull_bar(a), 1);
      ptx::mbar_init(tempty_bar(a), 4 * kEpiGroups);
      ptx::mbar_init(wfull_bar(a), 1);               // the mover, with the tile's bytes
      ptx::mbar_init(wdone_bar(a), 4 * kEpiGroups);  // every epilogue warp, once per tile
    }
    ptx::mbar_init(drain_bar, 1);
    if (kComp)
      for (int w = 0; w < 4 * kEpiGroups; ++w) {
        ptx::mbar_init(stage_bar(w), 1);
        ptx::mbar_init(free_bar(w), 32);
      }
    *abort_flag = 0;
    ptx::fence_barrier_init();
  }
  nf4_tables_init(tables, threadIdx.x);
  if (warp == 1) {
    ptx::tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_slot)), kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // nothing above touched global data: it may overlap the previous kernel's tail
  ptx::grid_launch_dependents();
  ptx::grid_dependency_wait();

  // Where tile g of the launch lies: matrix pi (the search resumes from the
  // caller's last position: a CTA's tiles come in ascending order) and the tile's
  // block coordinates inside it.
  auto locate = [&](int g, int &pi, int &m_blk, int &n_blk) {
    while (pi + 1 < mb.count && g >= mb.prob[pi + 1].tile0) ++pi;
    const int local = g - mb.prob[pi].tile0;
    const int mt = mb.prob[pi].mt;
    n_blk = local / mt;
    m_blk = local - n_blk * mt;
  };

  // =========================================================== TMA producer
  if (warp == 0) {
    if (lane == 0) {
      bool ok = true;
      uint32_t it = 0;
      int pi = 0, seen = -1;
      for (int g = blockIdx.x; ok && g < mb.tiles; g += gridDim.x) {
        int m_blk, n_blk;
        locate(g, pi, m_blk, n_blk);
        if (pi != seen) {
          ptx::prefetch_tensormap(&mb.a[pi]);
          ptx::prefetch_tensormap(&mb.b[pi]);
          seen = pi;
        }
        const int kbs = (mb.prob[pi].K + kBK - 1) / kBK;
        for (int kb = 0; kb < kbs; ++kb, ++it) {
          const int s = it % kStages;
          const uint32_t ph = (it / kStages) & 1u;
          if (!(ok = ptx::mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, mb.status))) break;
          const uint32_t a_dst = smem_base + s * L::kStageBytes;
          const uint32_t b_dst = a_dst + L::kABytes;
          ptx::mbar_arrive_expect_tx(full_bar(s), L::kABytes + L::kBBytes);
          ptx::tma_load_2d(a_dst, &mb.a[pi], full_bar(s), kb * kBK, m_blk * kHM);
#pragma unroll
          for (int j = 0; j < BN / 64; ++j)
            ptx::tma_load_2d(b_dst + j * 8192, &mb.b[pi], full_bar(s), n_blk * BN + 64 * j, kb * kBK);
        }
      }
      if (!ok) {
        // give copies already in flight time to land before the shared memory is released
        const uint64_t t0 = ptx::globaltimer_ns();
        while (ptx::globaltimer_ns() - t0 < 200000ull) {
        }
      }
    }
  }
  // =========================================================== MMA issuer
  else if (warp == 1) {
    if (lane == 0) {
      uint32_t it = 0, tile = 0;
      bool ok = true;
      int pi = 0;
      const uint32_t idesc = make_idesc(kHM, BN, false, true);
      for (int g = blockIdx.x; ok && g < mb.tiles; g += gridDim.x, ++tile) {
        int m_blk, n_blk;
        locate(g, pi, m_blk, n_blk);
        const int kbs = (mb.prob[pi].K + kBK - 1) / kBK;
        const uint32_t acc = tile & 1u;
        if (!(ok = ptx::mbar_wait(tempty_bar(acc), ((tile >> 1) & 1u) ^ 1u, abort_flag, mb.status))) break;
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb = 0; kb < kbs; ++kb, ++it) {
          const int s = it % kStages;
          const uint32_t ph = (it / kStages) & 1u;
          if (!(ok = ptx::mbar_wait(full_bar(s), ph, abort_flag, mb.status))) break;
          ptx::tc_fence_after();
          const uint32_t a_addr = smem_base + s * L::kStageBytes;
          const uint64_t a_desc = make_smem_desc(a_addr, false);
          const uint64_t b_desc = make_smem_desc(a_addr + L::kABytes, true);
#pragma unroll
          for (uint32_t k = 0; k < kBK / kUmmaK; ++k)
            ptx::mma_bf16_ss(d_tmem, a_desc + k * (32u >> 4), b_desc + k * (2048u >> 4), idesc, (kb > 0 || k > 0) ? 1u : 0u);
          ptx::mma_commit(empty_bar(s));
        }
        if (ok) ptx::mma_commit(tfull_bar(acc));
      }
      // every MMA issued above has finished before TMEM is freed
      ptx::mma_commit(drain_bar);
      ptx::mbar_wait(drain_bar, 0, abort_flag, mb.status);
    }
  }
  // =========================================================== mover of W_q
  else if (warp == kCodeWarp) {
    if (lane == 0) {
      // Buffer b = tile & 1.  Before a buffer is loaded again, the bulk store that
      // last read it has finished reading (stores complete in the order issued).
      bool ok = true;
      uint32_t tile = 0;
      int pi = 0, prev_pi = 0, pm = 0, pn = 0;
      auto store_prev = [&]() {
        const uint32_t pb = (tile - 1) & 1u;
        if (!(ok = ptx::mbar_wait(wdone_bar(pb), ((tile - 1) >> 1) & 1u, abort_flag, mb.status))) return;
        ptx::tma_store_2d(&mb.wq[prev_pi], smem_base + L::kWOffset + pb * L::kWTileBytes, pn * (BN / 2), pm * kHM);
        ptx::bulk_commit_group();
      };
      for (int g = blockIdx.x; ok && g < mb.tiles; g += gridDim.x, ++tile) {
        int m_blk, n_blk;
        locate(g, pi, m_blk, n_blk);
        const uint32_t b = tile & 1u;
        ptx::bulk_wait_group_read<0>();
        if (kComp) {
          // nothing to bring in: the arrival only tells the epilogue that the store which
          // last read this buffer is done with it
          ptx::mbar_arrive(wfull_bar(b));
        } else {
          ptx::mbar_arrive_expect_tx(wfull_bar(b), L::kWTileBytes);
          ptx::tma_load_2d(smem_base + L::kWOffset + b * L::kWTileBytes, &mb.wq[pi], wfull_bar(b), n_blk * (BN / 2), m_blk * kHM);
        }
        if (tile > 0) store_prev();
        prev_pi = pi;
        pm = m_blk;
        pn = n_blk;
      }
      if (ok && tile > 0) store_prev();
      // every store has left shared memory and reached global memory before the CTA ends
      ptx::bulk_wait_group<0>();
    }
  }
  // =========================================================== epilogue of the compensation step
  else if (kComp) {
    // One matrix per launch.  A thread's 64 weights W reach it through shared
    // memory: each warp owns a 32-row x 32-column fp32 staging tile that its lane 0
    // fills by TMA, half a block at a time (the second half while the first is
    // in use, the next block's first half while this block is quantised), so no
    // thread reads a 256-byte row segment of its own from global memory.  The
    // block is walked twice - once for its maximum, once for codes and residual -
    // and the accumulator is read from TMEM both times rather than kept: W, which
    // the residual needs, stays in registers instead.
    constexpr int NB = BN / 64;
    const MergeProblem &pr = mb.prob[0];
    const int q = warp & 3;
    const int ew = warp - kEpiWarp0;
    const int grp = ew >> 2;
    const uint32_t wbuf = smem_base + L::kExtraOffset + static_cast<uint32_t>(ew) * kCompStageBytes;
    const uint32_t wbar = stage_bar(ew), fbar = free_bar(ew);
    const uint32_t w_lane = wbuf + static_cast<uint32_t>(lane) * 128u;
    const uint32_t key = static_cast<uint32_t>(lane & 7);  // 128-byte swizzle: 16-byte chunk ^= row & 7
    const float alpha = pr.alpha;
    const float2 a2 = make_float2(alpha, alpha);
    uint32_t loads = 0;  // staging loads waited for so far
    bool ok = true;
    // the outcome of a wait, made the same for all lanes (the warp-wide TMEM loads and
    // barriers below need the warp whole)
    auto wait = [&](uint32_t bar, uint32_t parity) {
      return __all_sync(0xffffffffu, ptx::mbar_wait(bar, parity, abort_flag, mb.status)) != 0;
    };
    // half `half` of block `seq` of this CTA's sequence of blocks (tile seq / NB, block seq % NB)
    auto fetch = [&](uint32_t seq, int half) {
      if (lane != 0) return;
      const int g = blockIdx.x + static_cast<int>(seq / NB) * static_cast<int>(gridDim.x);
      if (g >= mb.tiles) return;
      const int n_blk = g / pr.mt, m_blk = g - n_blk * pr.mt;
      ptx::mbar_arrive_expect_tx(wbar, kCompStageBytes);
      ptx::tma_load_2d(wbuf, &mb.wmap, wbar, n_blk * BN + static_cast<int>(seq % NB) * 64 + 32 * half,
                       m_blk * kHM + q * 32);
    };
    auto take = [&](float2 *w) {  // 32 weights of this lane's row out of the staging tile
#pragma unroll
      for (uint32_t j = 0; j < 8; ++j) {
        const uint4 t = ld_shared_v4(w_lane + ((j ^ key) << 4));
        w[2 * j] = make_float2(__uint_as_float(t.x), __uint_as_float(t.y));
        w[2 * j + 1] = make_float2(__uint_as_float(t.z), __uint_as_float(t.w));
      }
    };
    {
      uint32_t first = static_cast<uint32_t>(grp);
      fetch(first, 0);
    }
    uint32_t tile = 0;
    for (int g = blockIdx.x; ok && g < mb.tiles; g += gridDim.x, ++tile) {
      const int n_blk = g / pr.mt, m_blk = g - n_blk * pr.mt;
      const uint32_t acc = tile & 1u;
      const uint32_t ph = (tile >> 1) & 1u;
      if (!(ok = wait(tfull_bar(acc), ph))) break;
      // the mover's signal that the store which last read this code buffer is done with it
      if (!(ok = wait(wfull_bar(acc), ph))) break;
      ptx::tc_fence_after();
      const int row_t = q * 32 + lane;
      const int row = m_blk * kHM + row_t;
      const bool row_ok = row < pr.M;
      const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * BN;
      const uint32_t w_row = smem_base + L::kWOffset + acc * L::kWTileBytes + static_cast<uint32_t>(row_t) * (BN / 2);
      const uint32_t w_key = (BN == 256) ? static_cast<uint32_t>(row_t & 7) : static_cast<uint32_t>((row_t >> 1) & 3);
#pragma unroll 1
      for (int jb = 0; jb < NB; ++jb) {
        const uint32_t seq = tile * NB + jb;
        if (static_cast<int>(seq % kEpiGroups) != grp) continue;
        const int c0 = n_blk * BN + jb * 64;
        const bool live = row_ok && c0 < pr.wq_ld;
        const uint32_t a0 = w_row + (((2u * jb) ^ w_key) << 4), a1 = w_row + (((2u * jb + 1u) ^ w_key) << 4);
        float2 W[32];
        uint32_t d[32];
        float mx[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        // ---- first walk: the block maximum of W + alpha * delta
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (!(ok = wait(wbar, loads & 1u))) break;
          ++loads;
          take(W + 16 * h);
          // Every lane has its copy before the staging tile is filled again: the lanes' reads
          // are ordered before their arrivals, the next copy is issued after the wait for them
          // (program order alone does not keep a shared-memory read ahead of a bulk copy).
          ptx::mbar_arrive(fbar);
          if (lane == 0) ok = ptx::mbar_wait(fbar, (loads - 1u) & 1u, abort_flag, mb.status);
          if (!(ok = __all_sync(0xffffffffu, ok) != 0)) break;
          if (h == 0) fetch(seq, 1);
          else fetch(seq + kEpiGroups, 0);
          ptx::tmem_ld32(t_row + jb * 64 + 32 * h, d);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const float2 v = __ffma2_rn(a2, make_float2(__uint_as_float(d[2 * e]), __uint_as_float(d[2 * e + 1])), W[16 * h + e]);
            mx[e & 3] = fmaxf(mx[e & 3], fmaxf(fabsf(v.x), fabsf(v.y)));
          }
        }
        if (!ok) break;
        const float Mnew = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
        const Nf4Divisor dv = nf4_divisor(Mnew);
        uint32_t o[8];
        __nv_bfloat16 *rp = pr.resid + static_cast<int64_t>(row) * pr.ld_resid + c0;
        // ---- second walk: codes, and the residual bf16( W - fl32(Mnew * q[code]) ) with the
        // two fp32 roundings of its definition (scalar intrinsics: a packed multiply and add
        // may be contracted into one fused operation)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          __syncwarp();  // the lanes' paths below differ (live rows, kind of division): whole again for the TMEM load
          ptx::tmem_ld32(t_row + jb * 64 + 32 * h, d);
          ptx::tmem_ld_wait();
          if (live) {
            auto quantise_half = [&](auto exact) {
#pragma unroll
              for (int g8 = 0; g8 < 4; ++g8) {
                auto code = [&](auto h2) {  // byte h2 of the word: columns 8 g8 + 2 h2, + 1 of this half
                  constexpr int kH2 = decltype(h2)::value;
                  const int e = 4 * g8 + kH2;
                  const float2 v = __ffma2_rn(a2, make_float2(__uint_as_float(d[2 * e]), __uint_as_float(d[2 * e + 1])), W[16 * h + e]);
                  return nf4_code2<kH2>(tables, nf4_normalise2<decltype(exact)::value>(dv, v));
                };
                using std::integral_constant;
                o[4 * h + g8] = code(integral_constant<int, 0>{}) | code(integral_constant<int, 1>{}) |
                                code(integral_constant<int, 2>{}) | code(integral_constant<int, 3>{});
              }
            };
            if (!(Mnew > 0.0f)) {
#pragma unroll
              for (int g8 = 0; g8 < 4; ++g8) o[4 * h + g8] = kZeroWord;
            } else if (dv.exact) {
              quantise_half(std::true_type{});
            } else {
              quantise_half(std::false_type{});
            }
#pragma unroll
            for (int g8 = 0; g8 < 4; ++g8) {
              uint32_t pk[4];
#pragma unroll
              for (int h2 = 0; h2 < 4; ++h2) {
                const uint32_t byte = (o[4 * h + g8] >> (8 * h2)) & 0xFFu;
                const float2 w = W[16 * h + 4 * g8 + h2];
                const float e_lo = __fsub_rn(w.x, __fmul_rn(Mnew, tables.level[byte & 15u]));
                const float e_hi = __fsub_rn(w.y, __fmul_rn(Mnew, tables.level[byte >> 4]));
                pk[h2] = pack_bf16x2(e_lo, e_hi);
              }
              reinterpret_cast<uint4 *>(rp)[4 * h + g8] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
          }
        }
        if (live) {
          st_shared_v4(a0, make_uint4(o[0], o[1], o[2], o[3]));
          st_shared_v4(a1, make_uint4(o[4], o[5], o[6], o[7]));
          pr.wq_absmax[static_cast<int64_t>(row) * (pr.wq_ld >> 6) + (c0 >> 6)] = Mnew;
        }
        __syncwarp();
      }
      if (!ok) break;
      ptx::fence_proxy_async_smem();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        ptx::mbar_arrive(wdone_bar(acc));
        ptx::mbar_arrive(tempty_bar(acc));
      }
    }
    if (!ok && lane == 0) {
      // a staging load may still be in flight: give it time to land before the shared memory is released
      const uint64_t t0 = ptx::globaltimer_ns();
      while (ptx::globaltimer_ns() - t0 < 200000ull) {
      }
    }
  }
  // =========================================================== epilogue
  else {
    const int q = warp & 3;                   // TMEM lane quarter this warp may access
    const int grp = (warp - kEpiWarp0) >> 2;  // warps 2-5, 6-9, 10-13
    uint32_t tile = 0;
    bool ok = true;
    int pi = 0;
    for (int g = blockIdx.x; ok && g < mb.tiles; g += gridDim.x, ++tile) {
      int m_blk, n_blk;
      locate(g, pi, m_blk, n_blk);
      const MergeProblem &pr = mb.prob[pi];
      const uint32_t acc = tile & 1u;
      const uint32_t ph = (tile >> 1) & 1u;
      // The old scales of this warp's blocks of the tile (one or two of the BN / 64 column
      // blocks) are asked for now, before the wait for the accumulator: a scalar load per
      // row from global memory is otherwise the longest stall of a block.  Nothing else
      // writes these scales before this thread does.
      float m_pre[BN / 64];
      {
        const int row_p = m_blk * kHM + q * 32 + lane;
#pragma unroll
        for (int jb = 0; jb < BN / 64; ++jb) {
          const int c0 = n_blk * BN + jb * 64;
          const bool mine = static_cast<int>((tile * (BN / 64) + jb) % kEpiGroups) == grp;
          m_pre[jb] = (mine && row_p < pr.M && c0 < pr.wq_ld)
                          ? pr.wq_absmax[static_cast<int64_t>(row_p) * (pr.wq_ld >> 6) + (c0 >> 6)]
                          : 0.0f;
        }
      }
      if (!(ok = ptx::mbar_wait(tfull_bar(acc), ph, abort_flag, mb.status))) break;
      // the tile's old codes (rows of BN / 2 bytes, TMA-swizzled: 16-byte chunk ^= row & 7
      // for 128-byte rows, (row >> 1) & 3 for 64-byte rows); the new ones replace them there
      if (!(ok = ptx::mbar_wait(wfull_bar(acc), ph, abort_flag, mb.status))) break;
      ptx::tc_fence_after();
      const int row_t = q * 32 + lane;  // row inside the tile
      const int row = m_blk * kHM + row_t;
      const bool row_ok = row < pr.M;
      const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * BN;
      const uint32_t w_row = smem_base + L::kWOffset + acc * L::kWTileBytes + static_cast<uint32_t>(row_t) * (BN / 2);
      const uint32_t w_key = (BN == 256) ? static_cast<uint32_t>(row_t & 7) : static_cast<uint32_t>((row_t >> 1) & 3);
      const float alpha = pr.alpha;
#pragma unroll 1
      for (int jb = 0; jb < BN / 64; ++jb) {
        const uint32_t seq = tile * (BN / 64) + jb;  // position in this CTA's sequence of blocks
        if (static_cast<int>(seq % kEpiGroups) != grp) continue;
        const int c0 = n_blk * BN + jb * 64;
        const bool live = row_ok && c0 < pr.wq_ld;
        float *mp = pr.wq_absmax + static_cast<int64_t>(row) * (pr.wq_ld >> 6) + (c0 >> 6);
        const uint32_t a0 = w_row + (((2u * jb) ^ w_key) << 4), a1 = w_row + (((2u * jb + 1u) ^ w_key) << 4);
        float Mold = 0.0f;
        uint4 ca = make_uint4(0, 0, 0, 0), cb = ca;
        float2 v[32];
#pragma unroll
        for (int k = 0; k < BN / 64; ++k)
          if (k == jb) Mold = m_pre[k];
        ca = ld_shared_v4(a0);
        cb = ld_shared_v4(a1);
        uint32_t d0[32], d1[32];
        ptx::tmem_ld32(t_row + jb * 64, d0);
        ptx::tmem_ld32(t_row + jb * 64 + 32, d1);
        ptx::tmem_ld_wait();
        if (live) {
          const uint32_t w[8] = {ca.x, ca.y, ca.z, ca.w, cb.x, cb.y, cb.z, cb.w};
          // v = deq32(old) + alpha * delta, two elements
          // per packed instruction; four running maxima keep the dependent chain of the
          // block maximum short
          float mx[4] = {0.0f, 0.0f, 0.0f, 0.0f};
          const float2 a2 = make_float2(alpha, alpha), m2 = make_float2(Mold, Mold);
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const float2 delta = make_float2(__uint_as_float(e < 16 ? d0[2 * e] : d1[2 * e - 32]),
                                             __uint_as_float(e < 16 ? d0[2 * e + 1] : d1[2 * e - 31]));
            const uint32_t word = w[e >> 2];
            const float2 lv = make_float2(tables.level[(word >> (8 * (e & 3))) & 15u],
                                          tables.level[(word >> (8 * (e & 3) + 4)) & 15u]);
            v[e] = __ffma2_rn(a2, delta, __fmul2_rn(m2, lv));
            mx[e & 3] = fmaxf(mx[e & 3], fmaxf(fabsf(v[e].x), fabsf(v[e].y)));
          }
          const float Mnew = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
          uint32_t o[8];
          const Nf4Divisor dv = nf4_divisor(Mnew);
          auto quantise_block = [&](auto exact) {
#pragma unroll
            for (int g8 = 0; g8 < 8; ++g8) {
              constexpr bool kE = decltype(exact)::value;
              o[g8] = nf4_code2<0>(tables, nf4_normalise2<kE>(dv, v[4 * g8])) |
                      nf4_code2<1>(tables, nf4_normalise2<kE>(dv, v[4 * g8 + 1])) |
                      nf4_code2<2>(tables, nf4_normalise2<kE>(dv, v[4 * g8 + 2])) |
                      nf4_code2<3>(tables, nf4_normalise2<kE>(dv, v[4 * g8 + 3]));
            }
          };
          if (!(Mnew > 0.0f)) {
#pragma unroll
            for (int g8 = 0; g8 < 8; ++g8) o[g8] = kZeroWord;
          } else if (dv.exact) {
            quantise_block(std::true_type{});
          } else {
            quantise_block(std::false_type{});
          }
          st_shared_v4(a0, make_uint4(o[0], o[1], o[2], o[3]));
          st_shared_v4(a1, make_uint4(o[4], o[5], o[6], o[7]));
          *mp = Mnew;
        }
        __syncwarp();
      }
      // This warp's blocks of the tile are in place: made visible to the bulk store,
      // then signalled; the accumulator goes back to the MMA warp.
      ptx::fence_proxy_async_smem();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        ptx::mbar_arrive(wdone_bar(acc));
        ptx::mbar_arrive(tempty_bar(acc));
      }
    }
  }

  // =========================================================== teardown
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace loqt
