// Orthonormalisation of tall thin matrices: the small dense part of finding the
// projection P from the full-rank gradient (paper Section 2.1 and Algorithm 2, the
// SVD lines: P = the r leading left singular vectors of G^W).  The library
// approximates that subspace by randomised subspace iteration (Halko, Martinsson
// and Tropp, "Finding structure with randomness", Algorithm 4.4): the large
// products G Omega, G^T Q, G Z run on the tensor-core engine (linear.cu); between
// them each m x r iterate Y is replaced by an orthonormal basis of its columns.
//
// orth(Y) here is Cholesky QR carried out in double precision on the CUDA
// cores: S = Y^T Y, S = L L^T, Q = Y L^-T.  The first iterate Y = G Omega of a
// square Gaussian test block has a condition number of several thousand times
// sigma_1 / sigma_r; in double precision the Gram matrix keeps its square (up
// to about 1e14) without losing positive definiteness, so one pass gives a
// basis orthonormal to 1e-16 cond(Y)^2.  Everything is tiled 64 x 64; no kernel
// waits on another CTA (one launch per dependent step), and all sums run in a
// fixed order, so results are reproducible.
#include "common.cuh"

namespace loqt {

namespace {

constexpr int kT = 64;        // tile edge
constexpr int kTP = kT + 1;   // padded row of a shared-memory tile (doubles)

// acc[i][j] += sum_k a[k][row0 + i] * b[k][col0 + j], k < kc; a and b are
// shared-memory tiles stored k-outermost with padded rows of kTP doubles.
__device__ __forceinline__ void tile_fma(double (&acc)[4][4], const double *a, const double *b, int row0, int col0, int kc) {
#pragma unroll 4
  for (int k = 0; k < kc; ++k) {
    double av[4], bv[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) av[i] = a[k * kTP + row0 + i];
#pragma unroll
    for (int j = 0; j < 4; ++j) bv[j] = b[k * kTP + col0 + j];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = fma(av[i], bv[j], acc[i][j]);
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

// partial[split][rp][rp] (lower tiles only) = sum over this split's rows k of Y[k][i] Y[k][j].
__global__ void __launch_bounds__(256)
gram_kernel(const float *__restrict__ Y, int64_t ldy, int m, int r, int rp, int rows_per_split, double *__restrict__ partial) {
  __shared__ double As[32 * kTP];
  __shared__ double Bs[32 * kTP];
  int bi, bj;
  lower_tile(blockIdx.x, bi, bj);
  const int split = blockIdx.y;
  const int k_begin = split * rows_per_split;
  const int k_end = min(m, k_begin + rows_per_split);
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  double acc[4][4] = {};
  for (int k0 = k_begin; k0 < k_end; k0 += 32) {
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int idx = tid + e * 256, kk = idx >> 6, c = idx & 63;
      const int row = k0 + kk;
      const int ci = bi * kT + c, cj = bj * kT + c;
      const bool in_rows = row < k_end;
      As[kk * kTP + c] = (in_rows && ci < r) ? static_cast<double>(Y[static_cast<int64_t>(row) * ldy + ci]) : 0.0;
      Bs[kk * kTP + c] = (in_rows && cj < r) ? static_cast<double>(Y[static_cast<int64_t>(row) * ldy + cj]) : 0.0;
    }
    __syncthreads();
    tile_fma(acc, As, Bs, ty * 4, tx * 4, 32);
    __syncthreads();
  }
  double *out = partial + static_cast<int64_t>(split) * rp * rp;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j)
      out[static_cast<int64_t>(bi * kT + ty * 4 + i) * rp + bj * kT + tx * 4 + j] = acc[i][j];
}

// S = sum of the partial Gram matrices in split order, written over split 0;
// rows / columns beyond r (padding up to a multiple of 64) become those of the
// identity, so that the factorisation below runs on whole tiles.
__global__ void gram_reduce_kernel(double *__restrict__ partial, int splits, int r, int rp) {
  const int64_t total = static_cast<int64_t>(rp) * rp;
  for (int64_t e = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; e < total;
       e += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int i = static_cast<int>(e / rp), j = static_cast<int>(e % rp);
    if (j / kT > i / kT) continue;  // upper tiles are never read
    double s = 0.0;
    for (int sp = 0; sp < splits; ++sp) s += partial[sp * total + e];
    if (i >= r || j >= r) s = (i == j) ? 1.0 : 0.0;
    partial[e] = s;
  }
}

// Panel step p of the blocked Cholesky factorisation S = L L^T (64 columns at a
// time, right-looking).  Every CTA factors the 64 x 64 diagonal block S_pp in
// shared memory and inverts the factor; CTA 0 stores L_pp^-1 (all that is ever
// needed of the diagonal block; S_pp itself stays as it is, the other CTAs of
// this launch are still reading it), CTA b > 0 replaces the block S_(p+b),p by
// L_(p+b),p = S_(p+b),p L_pp^-T.
// A pivot that is not positive (the iterate is rank deficient to working
// precision) is replaced by one and reported through the status word.
__global__ void __launch_bounds__(256)
chol_panel_kernel(double *__restrict__ S, int rp, int p, double *__restrict__ linv, uint32_t *status) {
  extern __shared__ double sm[];
  double *D = sm;                  // [64][65] the diagonal block, then its factor
  double *Xt = sm + kT * kTP;      // [64][65] Xt[c][i] = (L_pp^-1)[i][c]
  double *As = sm + 2 * kT * kTP;  // [64][65] As[c][a] = S_ip[a][c]
  const int tid = threadIdx.x;
  const int64_t d0 = static_cast<int64_t>(p) * kT;
  for (int e = tid; e < kT * kT; e += 256) {
    const int i = e >> 6, j = e & 63;
    D[i * kTP + j] = (j <= i) ? S[(d0 + i) * rp + d0 + j] : 0.0;
  }
  __syncthreads();
  for (int j = 0; j < kT; ++j) {
    if (tid == 0) {
      double d = D[j * kTP + j];
      if (!(d > 0.0)) {
        atomicOr(status, kErrNumeric);
        d = 1.0;
      }
      D[j * kTP + j] = sqrt(d);
    }
    __syncthreads();
    const double djj = D[j * kTP + j];
    if (tid > j && tid < kT) D[tid * kTP + j] /= djj;
    __syncthreads();
    // trailing update of the block's lower triangle: D[i][k] -= D[i][j] D[k][j], j < k <= i
    for (int e = tid; e < kT * kT; e += 256) {
      const int i = e >> 6, k = e & 63;
      if (k > j && k <= i) D[i * kTP + k] -= D[i * kTP + j] * D[k * kTP + j];
    }
    __syncthreads();
  }
  // inverse of the lower-triangular factor, one column per thread (forward substitution on a unit vector)
  if (tid < kT) {
    const int c = tid;
    for (int i = 0; i < kT; ++i) {
      double x = 0.0;
      if (i >= c) {
        double sum = (i == c) ? 1.0 : 0.0;
        for (int k = c; k < i; ++k) sum -= D[i * kTP + k] * Xt[c * kTP + k];
        x = sum / D[i * kTP + i];
      }
      Xt[c * kTP + i] = x;
    }
  }
  __syncthreads();
  if (blockIdx.x == 0) {
    for (int e = tid; e < kT * kT; e += 256) {
      const int i = e >> 6, j = e & 63;
      linv[static_cast<int64_t>(p) * kT * kT + e] = Xt[j * kTP + i];
    }
    return;
  }
  const int64_t r0 = static_cast<int64_t>(p + blockIdx.x) * kT;
  for (int e = tid; e < kT * kT; e += 256) {
    const int a = e >> 6, c = e & 63;
    As[c * kTP + a] = S[(r0 + a) * rp + d0 + c];
  }
  __syncthreads();
  const int tx = tid & 15, ty = tid >> 4;
  double acc[4][4] = {};
  tile_fma(acc, As, Xt, ty * 4, tx * 4, kT);  // sum_c S_ip[a][c] (L_pp^-1)[b][c]
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) S[(r0 + ty * 4 + i) * rp + d0 + tx * 4 + j] = acc[i][j];
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
  double acc[4][4] = {};
  for (int half = 0; half < 2; ++half) {  // the panel's 64 columns, 32 at a time
    for (int e = tid; e < kT * 32; e += 256) {
      const int a = e >> 5, c = e & 31;
      As[c * kTP + a] = S[(i0 + a) * rp + c0 + half * 32 + c];
      Bs[c * kTP + a] = S[(j0 + a) * rp + c0 + half * 32 + c];
    }
    __syncthreads();
    tile_fma(acc, As, Bs, ty * 4, tx * 4, 32);
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) S[(i0 + ty * 4 + i) * rp + j0 + tx * 4 + j] -= acc[i][j];
}

// Q = Y L^-T by blocks of 64 columns: Q_j = (Y_j - sum_(k<j) Q_k L_jk^T) L_jj^-T.
// A CTA owns 32 rows of Y and walks the column blocks in order; its rows of Q
// stay in double precision in `qd` for the later blocks.  Outputs (each
// optional): Q as fp32, and Q split into two bf16 matrices hi + lo (hi =
// bf16(Q), lo = bf16(Q - hi)), the form in which the next product consumes it.
__global__ void __launch_bounds__(128)
solve_kernel(const float *__restrict__ Y, int64_t ldy, int m, int r, int rp, const double *__restrict__ L,
             const double *__restrict__ linv, double *__restrict__ qd, float *__restrict__ qf, int64_t ldqf,
             __nv_bfloat16 *__restrict__ qhi, __nv_bfloat16 *__restrict__ qlo, int64_t ldqb) {
  extern __shared__ double sm[];
  double *As = sm;             // [64][65] As[c][a], a < 32
  double *Bs = sm + kT * kTP;  // [64][65]
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;  // 16 x 8 threads, 4 x 4 outputs each
  const int64_t row0 = static_cast<int64_t>(blockIdx.x) * 32;
  const int nb = rp / kT;
  for (int j = 0; j < nb; ++j) {
    double acc[4][4] = {};
    for (int k = 0; k < j; ++k) {
      for (int e = tid; e < 32 * kT; e += 128) {
        const int a = e >> 6, c = e & 63;
        As[c * kTP + a] = (row0 + a < m) ? qd[(row0 + a) * rp + k * kT + c] : 0.0;
      }
      for (int e = tid; e < kT * kT; e += 128) {
        const int b = e >> 6, c = e & 63;
        Bs[c * kTP + b] = L[static_cast<int64_t>(j * kT + b) * rp + k * kT + c];
      }
      __syncthreads();
      tile_fma(acc, As, Bs, ty * 4, tx * 4, kT);
      __syncthreads();
    }
    // T = Y_j - acc, stored k-outermost for the product with L_jj^-T
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
        const int64_t row = row0 + ty * 4 + i;
        const int col = j * kT + tx * 4 + jj;
        const double y = (row < m && col < r) ? static_cast<double>(Y[row * ldy + col]) : 0.0;
        As[(tx * 4 + jj) * kTP + ty * 4 + i] = y - acc[i][jj];
      }
    for (int e = tid; e < kT * kT; e += 128) {
      const int b = e >> 6, c = e & 63;
      Bs[c * kTP + b] = linv[static_cast<int64_t>(j) * kT * kT + e];  // Bs[c][b] = (L_jj^-1)[b][c]
    }
    __syncthreads();
    double q[4][4] = {};
    tile_fma(q, As, Bs, ty * 4, tx * 4, kT);
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
        const int64_t row = row0 + ty * 4 + i;
        const int col = j * kT + tx * 4 + jj;
        if (row >= m) continue;
        qd[row * rp + col] = q[i][jj];
        if (col >= r) continue;
        const float f = static_cast<float>(q[i][jj]);
        if (qf != nullptr) qf[row * ldqf + col] = f;
        if (qhi != nullptr) {
          const __nv_bfloat16 hi = __float2bfloat16_rn(f);
          qhi[row * ldqb + col] = hi;
          qlo[row * ldqb + col] = __float2bfloat16_rn(static_cast<float>(q[i][jj] - static_cast<double>(__bfloat162float(hi))));
        }
      }
    __syncthreads();
  }
}

constexpr size_t kPanelSmem = 3 * kT * kTP * sizeof(double);
constexpr size_t kSolveSmem = 2 * kT * kTP * sizeof(double);

int gram_splits(int m, int rp) {
  const int nb = rp / kT, tiles = nb * (nb + 1) / 2;
  int splits = sm_count() / tiles;
  if (splits > 16) splits = 16;
  const int by_rows = (m + 255) / 256;
  if (splits > by_rows) splits = by_rows;
  return splits < 1 ? 1 : splits;
}

}  // namespace

size_t orth_workspace_bytes(int m, int r) {
  const size_t rp = (static_cast<size_t>(r) + kT - 1) / kT * kT;
  const size_t gram = static_cast<size_t>(gram_splits(m, static_cast<int>(rp))) * rp * rp * sizeof(double);
  const size_t inv = rp * kT * sizeof(double);
  const size_t qd = static_cast<size_t>(m) * rp * sizeof(double);
  auto up = [](size_t v) { return (v + 255) & ~static_cast<size_t>(255); };
  return up(gram) + up(inv) + up(qd);
}

loqt_status orthonormalise(const float *Y, int64_t ldy, int m, int r, float *qf, int64_t ldqf, void *qhi, void *qlo,
                           int64_t ldqb, void *ws, uint32_t *status, cudaStream_t stream) {
  const int rp = (r + kT - 1) / kT * kT, nb = rp / kT;
  const int splits = gram_splits(m, rp);
  auto up = [](size_t v) { return (v + 255) & ~static_cast<size_t>(255); };
  uint8_t *cursor = static_cast<uint8_t *>(ws);
  double *S = reinterpret_cast<double *>(cursor);
  cursor += up(static_cast<size_t>(splits) * rp * rp * sizeof(double));
  double *linv = reinterpret_cast<double *>(cursor);
  cursor += up(static_cast<size_t>(rp) * kT * sizeof(double));
  double *qd = reinterpret_cast<double *>(cursor);

  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(chol_panel_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kPanelSmem)) != cudaSuccess ||
        cudaFuncSetAttribute(solve_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kSolveSmem)) != cudaSuccess)
      return LOQT_ERR_CUDA;
    attr_set = true;
  }
  int rows_per_split = (m + splits - 1) / splits;
  rows_per_split = (rows_per_split + 31) / 32 * 32;
  const int tiles = nb * (nb + 1) / 2;
  gram_kernel<<<dim3(tiles, splits), 256, 0, stream>>>(Y, ldy, m, r, rp, rows_per_split, S);
  int blocks = static_cast<int>((static_cast<int64_t>(rp) * rp + 255) / 256);
  if (blocks > sm_count() * 8) blocks = sm_count() * 8;
  gram_reduce_kernel<<<blocks, 256, 0, stream>>>(S, splits, r, rp);
  int launches = 2;
  for (int p = 0; p < nb; ++p) {
    chol_panel_kernel<<<nb - p, 256, kPanelSmem, stream>>>(S, rp, p, linv, status);
    ++launches;
    const int n = nb - p - 1;
    if (n > 0) {
      chol_update_kernel<<<n * (n + 1) / 2, 256, 0, stream>>>(S, rp, p);
      ++launches;
    }
  }
  solve_kernel<<<(m + 31) / 32, 128, kSolveSmem, stream>>>(Y, ldy, m, r, rp, S, linv, qd, qf, ldqf,
                                                           static_cast<__nv_bfloat16 *>(qhi), static_cast<__nv_bfloat16 *>(qlo), ldqb);
  count_launch(launches + 1);
  return cudaGetLastError() == cudaSuccess ? LOQT_OK : LOQT_ERR_CUDA;
}

}  // namespace loqt
