// Orthonormalisation of tall thin matrices: the small dense part of finding the
// projection P from the full-rank gradient (paper Section 2.1 and Algorithm 2, the
// SVD lines: P = the r leading left singular vectors of G^W).  The library
// approximates that subspace by randomised subspace iteration (Halko, Martinsson
// and Tropp, "Finding structure with randomness", Algorithm 4.4): the large
// products G Omega, G^T Q, G Z run on the tensor-core engine (linear.cu); between
// them each m x r iterate Y is replaced by an orthonormal basis of its columns.
//
// orth(Y) here is Cholesky QR carried out in double precision on the CUDA
// cores: S = Y^T Y, S = L L^T, X = L^-1, Q = Y X^T.  Double precision because the
// Gram matrix squares the condition number of Y: with cond(Y) up to 1e6 one pass
// still gives a basis orthonormal to 1e-4, where single precision would lose
// positive definiteness beyond cond(Y) of a few thousand.
//
//   gram_kernel        S = Y^T Y        128 x 128 tiles of the lower triangle, the rows of Y
//                                       split among CTAs, partial sums added in a fixed order
//   chol_panel_kernel  S = L L^T        right-looking, 64 columns per step: the diagonal block
//   chol_update_kernel                  is factored and inverted in shared memory, the panel
//                                       below it formed, the trailing matrix updated
//   block_gemm_kernel  X = L^-1         by doubling: with the diagonal blocks A^-1, B^-1 of size h
//                                       known, the block below is -B^-1 C A^-1 (two products per
//                                       level, log2(r / 64) levels)
//   apply_kernel       Q = Y X^T        one triangular product, 128 x 128 tiles
//
// No kernel waits on another CTA (one launch per dependent step), and all sums
// run in a fixed order, so results are reproducible.
#include "common.cuh"

namespace loqt {

namespace {

constexpr int kT = 64;       // tile edge of the factorisation
constexpr int kTP = kT + 1;  // padded row of a 64-wide shared-memory tile (doubles)

// 64 x 64 tiles, 256 threads as 16 x 16: thread (ty, tx) owns rows ty + 16 i and
// columns tx + 16 j (a warp's loads of the column operand are then 16 consecutive
// doubles, free of bank conflicts, and its stores to global memory contiguous).
// acc[i][j] += sum_k a[k][ty + 16 i] * b[k][tx + 16 j], k < kc; a and b are
// shared-memory tiles stored k-outermost with padded rows of kTP doubles.
__device__ __forceinline__ void tile_fma(double (&acc)[4][4], const double *a, const double *b, int ty, int tx, int kc) {
#pragma unroll 4
  for (int k = 0; k < kc; ++k) {
    double av[4], bv[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) av[i] = a[k * kTP + ty + 16 * i];
#pragma unroll
    for (int j = 0; j < 4; ++j) bv[j] = b[k * kTP + tx + 16 * j];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = fma(av[i], bv[j], acc[i][j]);
  }
}

// The two large products work on 128 x 128 tiles: 256 threads as 16 x 16, each
// with an 8 x 8 block of the tile in registers.  Thread (ty, tx) owns rows
// 2 ty + 32 q + e and columns 2 tx + 32 q' + e' (q, q' = 0..3; e, e' = 0, 1), so that
// a warp's 16-byte loads of the column operand are contiguous and those of the row
// operand are broadcasts: 64 fused multiply-adds per 8 loads, which leaves the
// double-precision pipe, not shared memory, as the limit.
constexpr int kG = 128;      // tile edge
constexpr int kGP = kG + 2;  // padded row (doubles): rows stay 16-byte aligned
constexpr int kGK = 16;      // k-chunk staged per step
constexpr size_t kBigSmem = 2 * 2 * kGK * kGP * sizeof(double);  // two operands, two buffers

__device__ __forceinline__ int own8(int t, int i) { return 2 * t + 32 * (i >> 1) + (i & 1); }

__device__ __forceinline__ void tile_fma8(double (&acc)[8][8], const double *a, const double *b, int ty, int tx) {
#pragma unroll 2
  for (int k = 0; k < kGK; ++k) {
    double2 av[4], bv[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      av[q] = *reinterpret_cast<const double2 *>(a + k * kGP + 2 * ty + 32 * q);
      bv[q] = *reinterpret_cast<const double2 *>(b + k * kGP + 2 * tx + 32 * q);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const double ai = (i & 1) ? av[i >> 1].y : av[i >> 1].x;
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[i][j] = fma(ai, (j & 1) ? bv[j >> 1].y : bv[j >> 1].x, acc[i][j]);
    }
  }
}

// Lower-triangle tile number t -> (bi, bj), bj <= bi.
__device__ __forceinline__ void lower_tile(int t, int &bi, int &bj) {
  int i = static_cast<int>((sqrtf(8.0f * static_cast<float>(t) + 1.0f) - 1.0f) * 0.5f);
  while (i * (i + 1) / 2 > t) --i;
  while ((i + 1) * (i + 2) / 2 <= t) ++i;
  bi = i;
  bj = t - i * (i + 1) / 2;
}

// partial[split][rp][rp] (128 x 128 tiles of the lower triangle) = sum over this
// split's rows k of Y[k][i] Y[k][j].  A chunk of 16 rows of Y is staged per step
// (converted to double), the next chunk's loads are in flight meanwhile.
__global__ void __launch_bounds__(256)
gram_kernel(const float *__restrict__ Y, int64_t ldy, int m, int r, int rp, int rows_per_split, double *__restrict__ partial) {
  extern __shared__ __align__(16) double smg[];
  int bi, bj;
  lower_tile(blockIdx.x, bi, bj);
  const bool diag = bi == bj;
  const int split = blockIdx.y;
  const int k_begin = split * rows_per_split;
  const int k_end = min(m, k_begin + rows_per_split);
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  // staging: thread -> row kk of the chunk, 8 consecutive columns of the tile
  const int kk = tid >> 4, i8 = (tid & 15) * 8;
  const bool vec = (ldy & 3) == 0 && (reinterpret_cast<uintptr_t>(Y) & 15u) == 0;
  auto fetch = [&](int k0, int tile, float (&v)[8]) {
    const int row = k0 + kk, col = tile * kG + i8;
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] = 0.0f;
    if (row >= k_end) return;
    const float *p = Y + static_cast<int64_t>(row) * ldy + col;
    if (vec && col + 8 <= r) {
      const float4 a = __ldg(reinterpret_cast<const float4 *>(p)), b = __ldg(reinterpret_cast<const float4 *>(p) + 1);
      v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e)
        if (col + e < r) v[e] = __ldg(p + e);
    }
  };
  auto stash = [&](double *dst, const float (&v)[8]) {
#pragma unroll
    for (int e = 0; e < 8; e += 2)
      *reinterpret_cast<double2 *>(dst + kk * kGP + i8 + e) = make_double2(static_cast<double>(v[e]), static_cast<double>(v[e + 1]));
  };
  double acc[8][8] = {};
  float va[8], vb[8];
  fetch(k_begin, bi, va);
  if (!diag) fetch(k_begin, bj, vb);
  int buf = 0;
  stash(smg, va);
  if (!diag) stash(smg + kGK * kGP, vb);
  __syncthreads();
  for (int k0 = k_begin; k0 < k_end; k0 += kGK) {
    const bool more = k0 + kGK < k_end;
    if (more) {
      fetch(k0 + kGK, bi, va);
      if (!diag) fetch(k0 + kGK, bj, vb);
    }
    const double *a = smg + buf * 2 * kGK * kGP;
    tile_fma8(acc, a, diag ? a : a + kGK * kGP, ty, tx);
    if (more) {
      double *nxt = smg + (buf ^ 1) * 2 * kGK * kGP;
      stash(nxt, va);
      if (!diag) stash(nxt + kGK * kGP, vb);
    }
    __syncthreads();
    buf ^= 1;
  }
  double *out = partial + static_cast<int64_t>(split) * rp * rp;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int row = bi * kG + own8(ty, i);
    if (row >= rp) continue;
#pragma unroll
    for (int j = 0; j < 8; j += 2) {
      const int col = bj * kG + own8(tx, j);
      if (col < rp) *reinterpret_cast<double2 *>(out + static_cast<int64_t>(row) * rp + col) = make_double2(acc[i][j], acc[i][j + 1]);
    }
  }
}

// S = sum of the partial Gram matrices in split order, written over split 0;
// rows / columns beyond r (padding up to a multiple of 64) become those of the
// identity, so that the factorisation below runs on whole tiles.
__global__ void gram_reduce_kernel(double *__restrict__ partial, int splits, int r, int rp) {
  const int64_t total = static_cast<int64_t>(rp) * rp;
  for (int64_t e = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; e < total;
       e += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int i = static_cast<int>(e / rp), j = static_cast<int>(e % rp);
    if (j / kG > i / kG) continue;  // tiles above the diagonal were not computed and are never read
    double s = 0.0;
    for (int sp = 0; sp < splits; ++sp) s += partial[sp * total + e];
    if (i >= r || j >= r) s = (i == j) ? 1.0 : 0.0;
    partial[e] = s;
  }
}

// 1 / x without the divide sequence: the hardware estimate (20 bits) and one Newton step
// give a relative error of about 1e-12, ample for an elimination multiplier here (the
// basis it leads to is rounded to single precision), and keep the chain of dependent
// double-precision operations per elimination step short: that chain, 64 times per
// panel, is what the factorisation waits on.
__device__ __forceinline__ double fast_rcp(double x) {
  double y;
  asm("rcp.approx.ftz.f64 %0, %1;" : "=d"(y) : "d"(x));
  return fma(y, fma(-x, y, 1.0), y);
}

// Panel step p of the blocked Cholesky factorisation S = L L^T (64 columns at a
// time, right-looking).  Every CTA factors the 64 x 64 diagonal block S_pp in
// shared memory and inverts the factor; CTA 0 stores L_pp^-1 into the diagonal
// block of X (all that is ever needed of the diagonal block; S_pp itself stays as
// it is, the other CTAs of this launch are still reading it), CTA b > 0 replaces
// the block S_(p+b),p by L_(p+b),p = S_(p+b),p L_pp^-T.
// A pivot that is not positive (the iterate is rank deficient to working
// precision) is replaced by one and reported through the status word.
//
// The factorisation keeps the lower triangle in registers (its 2080 elements dealt
// over the 256 threads, nine slots each, column by column) and passes only the current column through
// shared memory: step j subtracts col[i] col[k] / pivot_j from every element (i, k)
// with k > j, and the owners of column j + 1 publish it for the next step - one
// barrier per step.  The inverse of the factor is built by doubling: 8 x 8 diagonal
// blocks by forward substitution, then three levels of X21 = -X22 (L21 X11).
__global__ void __launch_bounds__(256)
chol_panel_kernel(double *__restrict__ S, int rp, int p, double *__restrict__ X, uint32_t *status) {
  extern __shared__ __align__(16) double sm[];
  double *D = sm;                  // [64][65] the diagonal block, its factor L, finally Xt[c][i] = (L^-1)[i][c]
  double *Xs = sm + kT * kTP;      // [64][65] L^-1
  double *As = sm + 2 * kT * kTP;  // [64][65] scratch of the inversion, then As[c][a] = S_ip[a][c]
  __shared__ double col[2][kT];
  __shared__ double pivot[kT];
  const int tid = threadIdx.x;
  const int64_t d0 = static_cast<int64_t>(p) * kT;

  // ---- factorisation
  // Elements are numbered column by column (column k holds rows k .. 63), so that slot q of
  // every thread lies in a narrow band of columns: an element (i, k) is touched only while
  // j < k, and once the band of a slot is behind the current column the slot is skipped by
  // all threads at once - on average four of the nine slots are live.
  constexpr int kSlots = 9, kLower = kT * (kT + 1) / 2;
  double val[kSlots];
  int ei[kSlots], ek[kSlots], last_col[kSlots];
  {
    // idx -> (row, column) in column-major packed order; a thread's slots and the slots' last
    // elements come in ascending order, so each of the two scans passes over the columns once
    int c = 0, first = 0;    // column of the thread's current slot, number of its top element
    int lc = 0, lfirst = 0;  // the same for the last element of the slot (equal in every thread)
#pragma unroll
    for (int q = 0; q < kSlots; ++q) {
      const int idx = tid + 256 * q;
      const bool have = idx < kLower;
      while (have && first + (kT - c) <= idx) first += kT - c, ++c;
      ei[q] = have ? c + (idx - first) : 0;
      ek[q] = have ? c : -1;  // -1: empty slot
      val[q] = have ? S[(d0 + ei[q]) * rp + d0 + c] : 0.0;
      if (ek[q] == 0) col[0][ei[q]] = val[q];
      const int lidx = min(256 * q + 255, kLower - 1);
      while (lfirst + (kT - lc) <= lidx) lfirst += kT - lc, ++lc;
      last_col[q] = lc;
    }
  }
  __syncthreads();
  // Step j with slots kFirst .. 8 live.  Nothing in it branches on a thread's own elements:
  // both factors of every live slot are read, the products and the fused updates follow as
  // independent chains, and a slot outside the trailing block keeps its value by a select -
  // with a branch per slot the chains of a thread's slots ran one after the other, which
  // was most of the panel's time.
  auto step = [&](auto first_c, int j) {
    constexpr int kFirst = decltype(first_c)::value;
    const double *cur = col[j & 1];
    double *nxt = col[(j + 1) & 1];
    double piv = cur[j];
    if (!(piv > 0.0)) {  // (the same in every thread)
      if (tid == 0) atomicOr(status, kErrNumeric);
      piv = 1.0;
    }
    if (tid == 0) pivot[j] = piv;
    const double inv = fast_rcp(piv);
    double prod[kSlots];
#pragma unroll
    for (int q = kFirst; q < kSlots; ++q) prod[q] = cur[ei[q]] * cur[max(ek[q], 0)];  // does not wait for the reciprocal
#pragma unroll
    for (int q = kFirst; q < kSlots; ++q) {
      const double upd = fma(-prod[q], inv, val[q]);
      val[q] = (ek[q] > j) ? upd : val[q];
      if (ek[q] == j + 1) nxt[ei[q]] = val[q];
    }
    __syncthreads();
  };
  {
    int j = 0;
    auto run = [&](auto first_c) {  // the steps during which slot kFirst is the first live one
      constexpr int kFirst = decltype(first_c)::value;
      const int end = kFirst < kSlots ? min(last_col[kFirst < kSlots ? kFirst : 0], kT) : kT;
      for (; j < end; ++j) step(first_c, j);
    };
    run(std::integral_constant<int, 0>{});
    run(std::integral_constant<int, 1>{});
    run(std::integral_constant<int, 2>{});
    run(std::integral_constant<int, 3>{});
    run(std::integral_constant<int, 4>{});
    run(std::integral_constant<int, 5>{});
    run(std::integral_constant<int, 6>{});
    run(std::integral_constant<int, 7>{});
    run(std::integral_constant<int, 8>{});
    run(std::integral_constant<int, 9>{});  // the last columns: pivots only
  }
  // L[i][k] = value / sqrt(pivot_k), L[k][k] = sqrt(pivot_k); zero above the diagonal
#pragma unroll
  for (int e = tid; e < kT * kT; e += 256) D[(e >> 6) * kTP + (e & 63)] = 0.0, Xs[(e >> 6) * kTP + (e & 63)] = 0.0;
  __syncthreads();
#pragma unroll
  for (int q = 0; q < kSlots; ++q) {
    if (ek[q] < 0) continue;
    const double sq = sqrt(pivot[ek[q]]);
    D[ei[q] * kTP + ek[q]] = (ei[q] == ek[q]) ? sq : val[q] / sq;
  }
  __syncthreads();

  // ---- inverse of the factor
  // 8 x 8 diagonal blocks: thread (block, column) solves L x = e_c inside its block
  if (tid < kT) {
    const int b0 = tid & ~7, c = tid & 7;
    double x[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      double sum = (i == c) ? 1.0 : 0.0;
#pragma unroll
      for (int k = 0; k < 8; ++k)
        if (k < i && k >= c) sum = fma(-D[(b0 + i) * kTP + b0 + k], x[k], sum);
      x[i] = (i < c) ? 0.0 : sum / D[(b0 + i) * kTP + b0 + i];
      Xs[(b0 + i) * kTP + b0 + c] = x[i];
    }
  }
  __syncthreads();
  // doubling: for every super-block [d, d + 2h): T = L21 X11, then X21 = -X22 T.  A thread
  // has h / 8 elements of each product; their dot products advance together, each as four
  // interleaved partial sums: a dependent chain of double-precision operations is what
  // these few hundred threads wait on, so the chains run side by side, not one after another.
  auto level = [&](auto h_c) {
    constexpr int h = decltype(h_c)::value, hs = (h == 8) ? 3 : (h == 16) ? 4 : 5;
    constexpr int kE = h / 8;  // elements per thread: (kT / (2 h)) h h / 256
    auto products = [&](const double *left, int left_col, const double *right, int right_row, double *out, double sign) {
      // out[d + h + a][d + b] = sign * sum_k left[d + h + a][d + left_col + k] right[d + right_row + k][d + b]
      const double *lp[kE], *rp_[kE];
      double *op[kE];
      double s4[kE][4];
#pragma unroll
      for (int i = 0; i < kE; ++i) {
        const int e = tid + 256 * i;
        const int z = e >> (2 * hs), a = (e >> hs) & (h - 1), b = e & (h - 1), d = 2 * h * z;
        lp[i] = left + (d + h + a) * kTP + d + left_col;
        rp_[i] = right + (d + right_row) * kTP + d + b;
        op[i] = out + (d + h + a) * kTP + d + b;
#pragma unroll
        for (int u = 0; u < 4; ++u) s4[i][u] = 0.0;
      }
      for (int k = 0; k < h; k += 4) {  // (the triangular factors' stored zeros are multiplied through)
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
          for (int i = 0; i < kE; ++i) s4[i][u] = fma(lp[i][k + u], rp_[i][(k + u) * kTP], s4[i][u]);
      }
#pragma unroll
      for (int i = 0; i < kE; ++i) *op[i] = sign * ((s4[i][0] + s4[i][1]) + (s4[i][2] + s4[i][3]));
    };
    products(D, 0, Xs, 0, As, 1.0);    // T = L21 X11
    __syncthreads();
    products(Xs, h, As, h, Xs, -1.0);  // X21 = -X22 T
    __syncthreads();
  };
  level(std::integral_constant<int, 8>{});
  level(std::integral_constant<int, 16>{});
  level(std::integral_constant<int, 32>{});
  if (blockIdx.x == 0) {
  #pragma unroll
  for (int e = tid; e < kT * kT; e += 256) {
      const int i = e >> 6, j = e & 63;
      X[(d0 + i) * rp + d0 + j] = Xs[i * kTP + j];
    }
    return;
  }
  // ---- this CTA's block of the panel: L_ip = S_ip L_pp^-T
  const int64_t r0 = static_cast<int64_t>(p + blockIdx.x) * kT;
#pragma unroll
  for (int e = tid; e < kT * kT; e += 256) {
    const int a = e >> 6, c = e & 63;
    As[c * kTP + a] = S[(r0 + a) * rp + d0 + c];
    D[c * kTP + a] = Xs[a * kTP + c];  // Xt[c][i] = (L^-1)[i][c]
  }
  __syncthreads();
  const int tx = tid & 15, ty = tid >> 4;
  double acc[4][4] = {};
  tile_fma(acc, As, D, ty, tx, kT);  // sum_c S_ip[a][c] (L_pp^-1)[b][c]
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) S[(r0 + ty + 16 * i) * rp + d0 + tx + 16 * j] = acc[i][j];
}

// Trailing update after panel p: S_ij -= L_ip L_jp^T for p < j <= i.
__global__ void __launch_bounds__(256)
chol_update_kernel(double *__restrict__ S, int rp, int p) {
  __shared__ double As[32 * kTP];
  __shared__ double Bs[32 * kTP];
  int ti, tj;
  lower_tile(blockIdx.x, ti, tj);
  const int64_t i0 = static_cast<int64_t>(p + 1 + ti) * kT, j0 = static_cast<int64_t>(p + 1 + tj) * kT;
  const int64_t c0 = static_cast<int64_t>(p) * kT;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  // Everything the CTA reads from global memory is asked for at once - both halves of the two
  // panel blocks (the panel's 64 columns go through shared memory 32 at a time) and the tile
  // of S itself - so that one memory latency is waited for, not three.
  double ra[2][8], rb[2][8], cur[4][4];
#pragma unroll
  for (int half = 0; half < 2; ++half)
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int e = tid + 256 * q, a = e >> 5, c = e & 31;
      ra[half][q] = S[(i0 + a) * rp + c0 + half * 32 + c];
      rb[half][q] = S[(j0 + a) * rp + c0 + half * 32 + c];
    }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) cur[i][j] = S[(i0 + ty + 16 * i) * rp + j0 + tx + 16 * j];
  double acc[4][4] = {};
#pragma unroll
  for (int half = 0; half < 2; ++half) {
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int e = tid + 256 * q, a = e >> 5, c = e & 31;
      As[c * kTP + a] = ra[half][q];
      Bs[c * kTP + a] = rb[half][q];
    }
    __syncthreads();
    tile_fma(acc, As, Bs, ty, tx, 32);
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) S[(i0 + ty + 16 * i) * rp + j0 + tx + 16 * j] = cur[i][j] - acc[i][j];
}

// One product of the inversion by doubling, for every diagonal super-block of
// size 2 h at once (blockIdx.z): with d0 = 2 h z, the h x h blocks
//   first  (second == 0):  T(z) = C A         C = L[d0 + h .., d0 ..],  A = X[d0 .., d0 ..]
//   second (second == 1):  X[d0 + h .., d0 ..] = - B T(z)      B = X[d0 + h .., d0 + h ..]
// T(z) is kept at the position of the block it leads to.  64 x 64 output tiles, k
// over the h columns; rows and columns beyond rp count as zero.
__global__ void __launch_bounds__(256)
block_gemm_kernel(const double *__restrict__ L, double *__restrict__ X, double *__restrict__ T, int rp, int h, int second) {
  __shared__ double As[32 * kTP];
  __shared__ double Bs[32 * kTP];
  const int d0 = 2 * h * static_cast<int>(blockIdx.z);
  const int ti = static_cast<int>(blockIdx.y) * kT, tj = static_cast<int>(blockIdx.x) * kT;  // tile origin inside the h x h block
  if (d0 + h + ti >= rp) return;  // the lower block is cut off by the matrix edge (the whole CTA leaves)
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  // left operand M1 (rows d0 + h + ti .., columns m1_col0 + k) and right operand M2 (rows m2_row0 + k, columns d0 + tj ..)
  const double *M1 = second ? X : L;
  const double *M2 = second ? T : X;
  const int64_t m1_row0 = d0 + h + ti, m1_col0 = second ? d0 + h : d0;
  const int64_t m2_row0 = second ? d0 + h : d0, m2_col0 = d0 + tj;
  double acc[4][4] = {};
  // X is lower triangular: in the first product the rows of A above the column tile are zero,
  // in the second the columns of B right of the row tile are - those k are passed over (the
  // sums lose terms that are exactly zero).  The next 32 columns are on their way from global
  // memory into registers while the current ones are multiplied.
  const int k_lo = second ? 0 : tj, k_hi = second ? min(h, ti + kT) : h;
  double ra[8], rb[8];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int e = tid + 256 * q;
      {
        const int a = e >> 5, c = e & 31;  // As[c][a] = M1[row a][k0 + c]
        const int64_t row = m1_row0 + a, col = m1_col0 + k0 + c;
        ra[q] = (row < rp && col < rp) ? M1[row * rp + col] : 0.0;
      }
      {
        const int c = e >> 6, b = e & 63;  // Bs[c][b] = M2[k0 + c][column b]
        const int64_t row = m2_row0 + k0 + c, col = m2_col0 + b;
        rb[q] = (row < rp && col < rp) ? M2[row * rp + col] : 0.0;
      }
    }
  };
  fetch(k_lo);
  for (int k0 = k_lo; k0 < k_hi; k0 += 32) {
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int e = tid + 256 * q;
      As[(e & 31) * kTP + (e >> 5)] = ra[q];
      Bs[(e >> 6) * kTP + (e & 63)] = rb[q];
    }
    __syncthreads();
    if (k0 + 32 < k_hi) fetch(k0 + 32);
    tile_fma(acc, As, Bs, ty, tx, 32);
    __syncthreads();
  }
  double *dst = second ? X : T;
  const int64_t dr0 = d0 + h + ti, dc0 = d0 + tj;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int64_t row = dr0 + ty + 16 * i, col = dc0 + tx + 16 * j;
      if (row < rp && col < rp) dst[row * rp + col] = second ? -acc[i][j] : acc[i][j];
    }
}

// Q = Y X^T with X = L^-1 lower triangular: Q[a][j] = sum_(c <= j) Y[a][c] X[j][c].
// 128 x 128 tiles; the tile of column block bj sums over the columns c < 128 (bj + 1).
// Outputs (each optional): Q as fp32 (m x r, or transposed, r x m, when qf_transposed), and Q split into two bf16 matrices hi + lo
// (hi = bf16(Q), lo = bf16(Q - hi)), the form in which the next product consumes it.
__global__ void __launch_bounds__(256)
apply_kernel(const float *__restrict__ Y, int64_t ldy, int m, int r, int rp, const double *__restrict__ X,
             float *__restrict__ qf, int64_t ldqf, int qf_transposed, __nv_bfloat16 *__restrict__ qhi, __nv_bfloat16 *__restrict__ qlo,
             int64_t ldqb) {
  extern __shared__ __align__(16) double smg[];
  const int bj = static_cast<int>(gridDim.y) - 1 - static_cast<int>(blockIdx.y);  // longest sums first
  const int64_t row0 = static_cast<int64_t>(blockIdx.x) * kG;
  const int j0 = bj * kG;
  const int k_end = min(rp, j0 + kG);
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  // staging: thread -> one row of the tile (a for Y, b for X), 8 consecutive k
  const int sr = tid >> 1, sk = (tid & 1) * 8;
  auto fetch = [&](int k0, double (&va)[8], double (&vb)[8]) {
    const int64_t row = row0 + sr;
    const int c = k0 + sk;
#pragma unroll
    for (int e = 0; e < 8; ++e) va[e] = (row < m && c + e < r) ? static_cast<double>(__ldg(Y + row * ldy + c + e)) : 0.0;
    const int xr = j0 + sr;
#pragma unroll
    for (int e = 0; e < 8; ++e) vb[e] = (xr < rp && c + e < rp) ? X[static_cast<int64_t>(xr) * rp + c + e] : 0.0;
  };
  auto stash = [&](double *dst, const double (&va)[8], const double (&vb)[8]) {
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      dst[(sk + e) * kGP + sr] = va[e];
      dst[kGK * kGP + (sk + e) * kGP + sr] = vb[e];
    }
  };
  double acc[8][8] = {};
  double va[8], vb[8];
  fetch(0, va, vb);
  stash(smg, va, vb);
  __syncthreads();
  int buf = 0;
  for (int k0 = 0; k0 < k_end; k0 += kGK) {
    const bool more = k0 + kGK < k_end;
    if (more) fetch(k0 + kGK, va, vb);
    const double *a = smg + buf * 2 * kGK * kGP;
    tile_fma8(acc, a, a + kGK * kGP, ty, tx);
    if (more) stash(smg + (buf ^ 1) * 2 * kGK * kGP, va, vb);
    __syncthreads();
    buf ^= 1;
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int64_t row = row0 + own8(ty, i);
    if (row >= m) continue;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int col = j0 + own8(tx, j);
      if (col >= r) continue;
      const float f = static_cast<float>(acc[i][j]);
      if (qf != nullptr) qf[qf_transposed ? col * ldqf + row : row * ldqf + col] = f;
      if (qhi != nullptr) {
        const __nv_bfloat16 hi = __float2bfloat16_rn(f);
        qhi[row * ldqb + col] = hi;
        qlo[row * ldqb + col] = __float2bfloat16_rn(static_cast<float>(acc[i][j] - static_cast<double>(__bfloat162float(hi))));
      }
    }
  }
}

constexpr size_t kPanelSmem = 3 * kT * kTP * sizeof(double);

int gram_splits(int m, int rp) {
  const int nb = (rp + kG - 1) / kG, tiles = nb * (nb + 1) / 2;
  int splits = sm_count() / tiles;
  if (splits > 16) splits = 16;
  const int by_rows = (m + 255) / 256;
  if (splits > by_rows) splits = by_rows;
  return splits < 1 ? 1 : splits;
}

size_t up256(size_t v) { return (v + 255) & ~static_cast<size_t>(255); }

}  // namespace

size_t orth_workspace_bytes(int m, int r) {
  const size_t rp = (static_cast<size_t>(r) + kT - 1) / kT * kT;
  const size_t sq = rp * rp * sizeof(double);
  return up256(static_cast<size_t>(gram_splits(m, static_cast<int>(rp))) * sq) + 2 * up256(sq);  // Gram partials / L, X, T
}

loqt_status orthonormalise(const float *Y, int64_t ldy, int m, int r, float *qf, int64_t ldqf, bool qf_transposed, void *qhi, void *qlo,
                           int64_t ldqb, void *ws, uint32_t *status, cudaStream_t stream) {
  const int rp = (r + kT - 1) / kT * kT, nb = rp / kT;
  const int splits = gram_splits(m, rp);
  const size_t sq = static_cast<size_t>(rp) * rp * sizeof(double);
  uint8_t *cursor = static_cast<uint8_t *>(ws);
  double *S = reinterpret_cast<double *>(cursor);
  cursor += up256(static_cast<size_t>(splits) * sq);
  double *X = reinterpret_cast<double *>(cursor);
  cursor += up256(sq);
  double *T = reinterpret_cast<double *>(cursor);

  // (function attributes belong to the current device's context: set on every call, as the
  // product engine does, so that a process driving several GPUs is served on each)
  if (cudaFuncSetAttribute(chol_panel_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kPanelSmem)) != cudaSuccess ||
      cudaFuncSetAttribute(gram_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kBigSmem)) != cudaSuccess ||
      cudaFuncSetAttribute(apply_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kBigSmem)) != cudaSuccess)
    return LOQT_ERR_CUDA;
  int launches = 0;
  // S = Y^T Y
  int rows_per_split = (m + splits - 1) / splits;
  rows_per_split = (rows_per_split + kGK - 1) / kGK * kGK;
  const int gb = (rp + kG - 1) / kG;
  gram_kernel<<<dim3(gb * (gb + 1) / 2, splits), 256, kBigSmem, stream>>>(Y, ldy, m, r, rp, rows_per_split, S);
  int blocks = static_cast<int>((static_cast<int64_t>(rp) * rp + 255) / 256);
  if (blocks > sm_count() * 8) blocks = sm_count() * 8;
  gram_reduce_kernel<<<blocks, 256, 0, stream>>>(S, splits, r, rp);
  launches += 2;
  // S = L L^T (L's blocks below the diagonal replace S's), X's diagonal blocks = the inverses of L's
  if (cudaMemsetAsync(X, 0, sq, stream) != cudaSuccess) return LOQT_ERR_CUDA;
  for (int p = 0; p < nb; ++p) {
    chol_panel_kernel<<<nb - p, 256, kPanelSmem, stream>>>(S, rp, p, X, status);
    ++launches;
    const int n = nb - p - 1;
    if (n > 0) {
      chol_update_kernel<<<n * (n + 1) / 2, 256, 0, stream>>>(S, rp, p);
      ++launches;
    }
  }
  // X = L^-1 by doubling the size of the inverted diagonal blocks
  for (int h = kT; h < rp; h *= 2) {
    const int supers = (rp + 2 * h - 1) / (2 * h), ht = h / kT;
    block_gemm_kernel<<<dim3(ht, ht, supers), 256, 0, stream>>>(S, X, T, rp, h, 0);
    block_gemm_kernel<<<dim3(ht, ht, supers), 256, 0, stream>>>(S, X, T, rp, h, 1);
    launches += 2;
  }
  // Q = Y X^T
  apply_kernel<<<dim3((m + kG - 1) / kG, gb), 256, kBigSmem, stream>>>(Y, ldy, m, r, rp, X, qf, ldqf, qf_transposed ? 1 : 0, static_cast<__nv_bfloat16 *>(qhi),
                                                                       static_cast<__nv_bfloat16 *>(qlo), ldqb);
  count_launch(launches + 1);
  return cudaGetLastError() == cudaSuccess ? LOQT_OK : LOQT_ERR_CUDA;
}

}  // namespace loqt
