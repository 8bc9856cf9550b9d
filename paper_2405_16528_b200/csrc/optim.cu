// Optimiser step on the trainable factor B (paper Algorithm 1, the update line
// B <- B - rho(G^B) with rho = Adam; optimiser states in bf16).  One streaming
// pass: 4 bytes of gradient and 2 + 2 + 2 bytes of B and the two moments in,
// 2 + 2 + 2 bytes out per element.
#include <mutex>

#include "common.cuh"

namespace loqt {

constexpr int kOptThreads = 256;

struct AdamConsts {
  float lr, beta1, beta2, one_minus_beta1, one_minus_beta2, eps, weight_decay;
  float inv_bc1, inv_bc2;  // 1 / (1 - beta^t)
};

__device__ __forceinline__ float bf16_bits_to_float(uint32_t bits16) { return __uint_as_float(bits16 << 16); }

// Adam (Kingma & Ba, Algorithm 1) with decoupled weight decay, fp32 arithmetic.
__device__ __forceinline__ void adam_element(const AdamConsts &h, float g, float &b, float &m, float &v) {
  m = fmaf(h.beta1, m, h.one_minus_beta1 * g);
  v = fmaf(h.beta2, v, (h.one_minus_beta2 * g) * g);
  const float mhat = m * h.inv_bc1;
  const float vhat = v * h.inv_bc2;
  const float upd = __fdiv_rn(mhat, __fsqrt_rn(vhat) + h.eps) + h.weight_decay * b;
  b = fmaf(-h.lr, upd, b);
}

template <bool kVec>
__global__ void __launch_bounds__(kOptThreads)
adam_step_kernel(__nv_bfloat16 *__restrict__ B, int64_t ldb, const float *__restrict__ g, int64_t ldg,
                 __nv_bfloat16 *__restrict__ m, __nv_bfloat16 *__restrict__ v, int64_t lds, int rows, int cols,
                 AdamConsts h) {
  const uint32_t gpr = static_cast<uint32_t>((cols + 7) / 8);  // groups of 8 elements per row
  const uint32_t n_items = static_cast<uint32_t>(rows) * gpr;  // (host checks < 2^31)
  const uint32_t stride = gridDim.x * kOptThreads;
  for (uint32_t item = blockIdx.x * kOptThreads + threadIdx.x; item < n_items; item += stride) {
    const uint32_t row = item / gpr;
    const int c0 = static_cast<int>(item - row * gpr) * 8;
    __nv_bfloat16 *bp = B + static_cast<int64_t>(row) * ldb + c0;
    __nv_bfloat16 *mp = m + static_cast<int64_t>(row) * lds + c0;
    __nv_bfloat16 *vp = v + static_cast<int64_t>(row) * lds + c0;
    const float *gp = g + static_cast<int64_t>(row) * ldg + c0;
    if (kVec && c0 + 8 <= cols) {
      const uint4 bw = *reinterpret_cast<const uint4 *>(bp);
      const uint4 mw = *reinterpret_cast<const uint4 *>(mp);
      const uint4 vw = *reinterpret_cast<const uint4 *>(vp);
      const float4 g0 = __ldg(reinterpret_cast<const float4 *>(gp));
      const float4 g1 = __ldg(reinterpret_cast<const float4 *>(gp) + 1);
      const uint32_t bb[4] = {bw.x, bw.y, bw.z, bw.w}, mm[4] = {mw.x, mw.y, mw.z, mw.w}, vv[4] = {vw.x, vw.y, vw.z, vw.w};
      const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
      uint32_t ob[4], om[4], ov[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        float b0 = bf16_bits_to_float(bb[k] & 0xFFFFu), b1 = bf16_bits_to_float(bb[k] >> 16);
        float m0 = bf16_bits_to_float(mm[k] & 0xFFFFu), m1 = bf16_bits_to_float(mm[k] >> 16);
        float v0 = bf16_bits_to_float(vv[k] & 0xFFFFu), v1 = bf16_bits_to_float(vv[k] >> 16);
        adam_element(h, gg[2 * k], b0, m0, v0);
        adam_element(h, gg[2 * k + 1], b1, m1, v1);
        ob[k] = pack_bf16x2(b0, b1);
        om[k] = pack_bf16x2(m0, m1);
        ov[k] = pack_bf16x2(v0, v1);
      }
      *reinterpret_cast<uint4 *>(bp) = make_uint4(ob[0], ob[1], ob[2], ob[3]);
      *reinterpret_cast<uint4 *>(mp) = make_uint4(om[0], om[1], om[2], om[3]);
      *reinterpret_cast<uint4 *>(vp) = make_uint4(ov[0], ov[1], ov[2], ov[3]);
    } else {
      for (int j = 0; j < 8 && c0 + j < cols; ++j) {
        float b = __bfloat162float(bp[j]), mj = __bfloat162float(mp[j]), vj = __bfloat162float(vp[j]);
        adam_element(h, __ldg(gp + j), b, mj, vj);
        bp[j] = __float2bfloat16_rn(b);
        mp[j] = __float2bfloat16_rn(mj);
        vp[j] = __float2bfloat16_rn(vj);
      }
    }
  }
}

}  // namespace loqt

using namespace loqt;

extern "C" loqt_status loqt_adam_step(void *B, int64_t ldb, const float *dB, int64_t lddb, void *m, void *v, int64_t ld_state,
                                      int32_t r, int32_t in, loqt_adam_params hp, void *stream) {
  if (B == nullptr || dB == nullptr || m == nullptr || v == nullptr) return LOQT_ERR_INVALID_ARG;
  if (r <= 0 || in <= 0 || ldb < in || lddb < in || ld_state < in || hp.step < 1) return LOQT_ERR_INVALID_ARG;
  if (!(hp.beta1 >= 0.0f && hp.beta1 < 1.0f && hp.beta2 >= 0.0f && hp.beta2 < 1.0f)) return LOQT_ERR_INVALID_ARG;
  const uintptr_t all = reinterpret_cast<uintptr_t>(B) | reinterpret_cast<uintptr_t>(m) | reinterpret_cast<uintptr_t>(v);
  if ((all & 1u) != 0 || (reinterpret_cast<uintptr_t>(dB) & 3u) != 0) return LOQT_ERR_ALIGNMENT;
  loqt_status st;
  if ((st = check_arch()) != LOQT_OK) return st;
  const int64_t items = static_cast<int64_t>(r) * ((in + 7) / 8);
  if (items >= (1ll << 31)) return LOQT_ERR_UNSUPPORTED;
  AdamConsts h;
  h.lr = hp.lr; h.beta1 = hp.beta1; h.beta2 = hp.beta2; h.eps = hp.eps; h.weight_decay = hp.weight_decay;
  h.one_minus_beta1 = static_cast<float>(1.0 - static_cast<double>(hp.beta1));
  h.one_minus_beta2 = static_cast<float>(1.0 - static_cast<double>(hp.beta2));
  h.inv_bc1 = static_cast<float>(1.0 / (1.0 - pow(static_cast<double>(hp.beta1), hp.step)));
  h.inv_bc2 = static_cast<float>(1.0 / (1.0 - pow(static_cast<double>(hp.beta2), hp.step)));
  const bool vec = ((all | reinterpret_cast<uintptr_t>(dB)) & 15u) == 0 && (ldb % 8) == 0 && (ld_state % 8) == 0 && (lddb % 4) == 0;
  auto kernel = vec ? adam_step_kernel<true> : adam_step_kernel<false>;
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kOptThreads, 0) != cudaSuccess || per_sm < 1) per_sm = 1;
  int64_t blocks = (items + kOptThreads - 1) / kOptThreads;
  const int64_t cap = static_cast<int64_t>(sm_count()) * per_sm;
  if (blocks > cap) blocks = cap;
  kernel<<<static_cast<int>(blocks), kOptThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<__nv_bfloat16 *>(B), ldb, dB, lddb, static_cast<__nv_bfloat16 *>(m), static_cast<__nv_bfloat16 *>(v), ld_state,
      r, in, h);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? LOQT_OK : LOQT_ERR_CUDA;
}

// ---------------------------------------------------------------------------
// The same step with the two moments held in 8 bits (the paper's "8-bit Adam",
// after Dettmers et al., "8-bit Optimizers via Block-wise Quantization"): blocks
// of 2048 consecutive elements of the row-major flattened r x in moments, one
// fp32 scale (the block's largest magnitude) per block, codes in the dynamic tree
// data type - a sign bit, a run of E zero bits (base-10 exponent), an indicator
// bit and f fraction bits; magnitude = 10^-E (0.1 + 0.9 (j + 1) / 2^f), which makes
// the magnitude bits, read as an integer 2^f + j, ascend with the magnitude.  The
// second moment is non-negative and uses the sign bit as one more fraction bit.
// One CTA per block: dequantise, update in fp32, take the new block maxima,
// quantise (nearest magnitude by binary search over the exact midpoints).
// 12 bytes per element: 4 (gradient) + 2 + 2 (B) + 1 + 1 (m) + 1 + 1 (v).
// ---------------------------------------------------------------------------
namespace loqt {

constexpr int kOpt8Block = 2048;
constexpr int kOpt8Threads = 256;  // 8 elements per thread

// magnitudes and decision thresholds of both data types (thr[k]: largest fp32 not
// above the midpoint of magnitudes k and k + 1, so that  a > thr[k]  <=>  a > midpoint)
struct Dyn8Tables {
  float mag_m[128], thr_m[128];
  float mag_v[256], thr_v[256];
};

static void build_dyn8(int bits, float *mag, float *thr) {
  const int n = 1 << bits;
  static const double kPow10[8] = {1.0, 1e-1, 1e-2, 1e-3, 1e-4, 1e-5, 1e-6, 1e-7};
  mag[0] = 0.0f;
  for (int f = 0; f < bits; ++f) {
    const int E = bits - 1 - f;
    for (int j = 0; j < (1 << f); ++j)
      mag[(1 << f) + j] = static_cast<float>((0.1 + 0.9 * (j + 1) / static_cast<double>(1 << f)) * kPow10[E]);
  }
  for (int k = 0; k + 1 < n; ++k) {
    const double mid = (static_cast<double>(mag[k]) + static_cast<double>(mag[k + 1])) / 2.0;
    float t = static_cast<float>(mid);
    if (static_cast<double>(t) > mid) t = nextafterf(t, -1.0f);
    thr[k] = t;
  }
  thr[n - 1] = 3.0e38f;  // sentinel: no normalised magnitude exceeds it
}

static const Dyn8Tables &dyn8_tables() {
  static Dyn8Tables t;
  static bool ready = false;
  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);
  if (!ready) {
    build_dyn8(7, t.mag_m, t.thr_m);
    build_dyn8(8, t.mag_v, t.thr_v);
    ready = true;
  }
  return t;
}

// number of thresholds below a (a >= 0): index of the nearest magnitude, the smaller on a tie
template <int kBits>
__device__ __forceinline__ uint32_t dyn8_index(const float *thr, float a) {
  uint32_t lo = 0;
#pragma unroll
  for (int step = 1 << (kBits - 1); step > 0; step >>= 1)
    if (a > thr[lo + step - 1]) lo += step;
  return lo;
}

template <bool kVec>
__global__ void __launch_bounds__(kOpt8Threads)
adam8_step_kernel(__nv_bfloat16 *__restrict__ B, int64_t ldb, const float *__restrict__ g, int64_t ldg, uint8_t *__restrict__ m8,
                  float *__restrict__ m_absmax, uint8_t *__restrict__ v8, float *__restrict__ v_absmax, int rows, int cols,
                  AdamConsts h, const __grid_constant__ Dyn8Tables tabs) {
  __shared__ Dyn8Tables t;
  __shared__ float red_m[kOpt8Threads / 32], red_v[kOpt8Threads / 32];
  {
    const float *src = reinterpret_cast<const float *>(&tabs);
    float *dst = reinterpret_cast<float *>(&t);
    for (int i = threadIdx.x; i < static_cast<int>(sizeof(Dyn8Tables) / 4); i += kOpt8Threads) dst[i] = src[i];
  }
  __syncthreads();
  const int64_t total = static_cast<int64_t>(rows) * cols;
  const int64_t e0 = static_cast<int64_t>(blockIdx.x) * kOpt8Block + threadIdx.x * 8;
  const float Mm = m_absmax[blockIdx.x], Mv = v_absmax[blockIdx.x];
  float b[8], m[8], v[8];
  bool live[8];
  const bool full = kVec && (e0 + 8 <= total);
  int64_t row0 = 0;
  int col0 = 0;
  if (e0 < total) {
    row0 = e0 / cols;
    col0 = static_cast<int>(e0 - row0 * cols);
  }
  if (full) {
    // (kVec: cols % 8 == 0, so the eight elements share a row and every access is 16-byte aligned)
    const uint2 mc = *reinterpret_cast<const uint2 *>(m8 + e0), vc = *reinterpret_cast<const uint2 *>(v8 + e0);
    const uint4 bw = *reinterpret_cast<const uint4 *>(B + row0 * ldb + col0);
    const float4 g0 = __ldg(reinterpret_cast<const float4 *>(g + row0 * ldg + col0));
    const float4 g1 = __ldg(reinterpret_cast<const float4 *>(g + row0 * ldg + col0) + 1);
    const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
    const uint32_t bb[4] = {bw.x, bw.y, bw.z, bw.w};
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const uint32_t cm = ((k < 4 ? mc.x : mc.y) >> (8 * (k & 3))) & 0xFFu, cv = ((k < 4 ? vc.x : vc.y) >> (8 * (k & 3))) & 0xFFu;
      const float am = __fmul_rn(t.mag_m[cm & 0x7Fu], Mm);
      m[k] = (cm & 0x80u) ? -am : am;
      v[k] = __fmul_rn(t.mag_v[cv], Mv);
      b[k] = bf16_bits_to_float((k & 1) ? (bb[k >> 1] >> 16) : (bb[k >> 1] & 0xFFFFu));
      live[k] = true;
      adam_element(h, gg[k], b[k], m[k], v[k]);
    }
  } else {
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int64_t e = e0 + k;
      live[k] = e < total;
      b[k] = m[k] = v[k] = 0.0f;
      if (live[k]) {
        const int64_t row = e / cols;
        const int col = static_cast<int>(e - row * cols);
        const uint32_t cm = m8[e], cv = v8[e];
        const float am = __fmul_rn(t.mag_m[cm & 0x7Fu], Mm);
        m[k] = (cm & 0x80u) ? -am : am;
        v[k] = __fmul_rn(t.mag_v[cv], Mv);
        b[k] = __bfloat162float(B[row * ldb + col]);
        adam_element(h, __ldg(g + row * ldg + col), b[k], m[k], v[k]);
      }
    }
  }
  // the block's new scales
  float mm = 0.0f, mv = 0.0f;
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    mm = fmaxf(mm, fabsf(m[k]));
    mv = fmaxf(mv, v[k]);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    mm = fmaxf(mm, __shfl_xor_sync(0xffffffffu, mm, o));
    mv = fmaxf(mv, __shfl_xor_sync(0xffffffffu, mv, o));
  }
  if ((threadIdx.x & 31) == 0) {
    red_m[threadIdx.x >> 5] = mm;
    red_v[threadIdx.x >> 5] = mv;
  }
  __syncthreads();
  mm = red_m[0];
  mv = red_v[0];
#pragma unroll
  for (int w = 1; w < kOpt8Threads / 32; ++w) {
    mm = fmaxf(mm, red_m[w]);
    mv = fmaxf(mv, red_v[w]);
  }
  if (threadIdx.x == 0) {
    m_absmax[blockIdx.x] = mm;
    v_absmax[blockIdx.x] = mv;
  }
  uint32_t om[8], ov[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    om[k] = ov[k] = 0;
    if (mm > 0.0f) {
      const float n = __fdiv_rn(m[k], mm);
      const uint32_t idx = dyn8_index<7>(t.thr_m, fabsf(n));
      om[k] = (n < 0.0f && idx > 0) ? (idx | 0x80u) : idx;
    }
    if (mv > 0.0f) ov[k] = dyn8_index<8>(t.thr_v, __fdiv_rn(v[k], mv));
  }
  if (full) {
    uint2 mc, vc;
    mc.x = om[0] | (om[1] << 8) | (om[2] << 16) | (om[3] << 24);
    mc.y = om[4] | (om[5] << 8) | (om[6] << 16) | (om[7] << 24);
    vc.x = ov[0] | (ov[1] << 8) | (ov[2] << 16) | (ov[3] << 24);
    vc.y = ov[4] | (ov[5] << 8) | (ov[6] << 16) | (ov[7] << 24);
    *reinterpret_cast<uint2 *>(m8 + e0) = mc;
    *reinterpret_cast<uint2 *>(v8 + e0) = vc;
    *reinterpret_cast<uint4 *>(B + row0 * ldb + col0) =
        make_uint4(pack_bf16x2(b[0], b[1]), pack_bf16x2(b[2], b[3]), pack_bf16x2(b[4], b[5]), pack_bf16x2(b[6], b[7]));
  } else {
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      if (!live[k]) continue;
      const int64_t e = e0 + k;
      const int64_t row = e / cols;
      const int col = static_cast<int>(e - row * cols);
      m8[e] = static_cast<uint8_t>(om[k]);
      v8[e] = static_cast<uint8_t>(ov[k]);
      B[row * ldb + col] = __float2bfloat16_rn(b[k]);
    }
  }
}

}  // namespace loqt

extern "C" loqt_status loqt_adam8_step(void *B, int64_t ldb, const float *dB, int64_t lddb, loqt_adam8_state st, int32_t r,
                                       int32_t in, loqt_adam_params hp, void *stream) {
  if (B == nullptr || dB == nullptr || st.m8 == nullptr || st.v8 == nullptr || st.m_absmax == nullptr || st.v_absmax == nullptr)
    return LOQT_ERR_INVALID_ARG;
  if (r <= 0 || in <= 0 || ldb < in || lddb < in || hp.step < 1) return LOQT_ERR_INVALID_ARG;
  if (!(hp.beta1 >= 0.0f && hp.beta1 < 1.0f && hp.beta2 >= 0.0f && hp.beta2 < 1.0f)) return LOQT_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(B) & 1u) != 0 || (reinterpret_cast<uintptr_t>(dB) & 3u) != 0 ||
      ((reinterpret_cast<uintptr_t>(st.m_absmax) | reinterpret_cast<uintptr_t>(st.v_absmax)) & 3u) != 0)
    return LOQT_ERR_ALIGNMENT;
  loqt_status s;
  if ((s = check_arch()) != LOQT_OK) return s;
  const int64_t total = static_cast<int64_t>(r) * in;
  const int64_t blocks = (total + kOpt8Block - 1) / kOpt8Block;
  if (blocks >= (1ll << 31)) return LOQT_ERR_UNSUPPORTED;
  AdamConsts h;
  h.lr = hp.lr; h.beta1 = hp.beta1; h.beta2 = hp.beta2; h.eps = hp.eps; h.weight_decay = hp.weight_decay;
  h.one_minus_beta1 = static_cast<float>(1.0 - static_cast<double>(hp.beta1));
  h.one_minus_beta2 = static_cast<float>(1.0 - static_cast<double>(hp.beta2));
  h.inv_bc1 = static_cast<float>(1.0 / (1.0 - pow(static_cast<double>(hp.beta1), hp.step)));
  h.inv_bc2 = static_cast<float>(1.0 / (1.0 - pow(static_cast<double>(hp.beta2), hp.step)));
  const uintptr_t all = reinterpret_cast<uintptr_t>(B) | reinterpret_cast<uintptr_t>(dB);
  const bool vec = (all & 15u) == 0 && ((reinterpret_cast<uintptr_t>(st.m8) | reinterpret_cast<uintptr_t>(st.v8)) & 7u) == 0 &&
                   (in % 8) == 0 && (ldb % 8) == 0 && (lddb % 4) == 0;
  auto kernel = vec ? adam8_step_kernel<true> : adam8_step_kernel<false>;
  kernel<<<static_cast<int>(blocks), kOpt8Threads, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<__nv_bfloat16 *>(B), ldb, dB, lddb, st.m8, st.m_absmax, st.v8, st.v_absmax, r, in, h, dyn8_tables());
  count_launch();
  return cudaGetLastError() == cudaSuccess ? LOQT_OK : LOQT_ERR_CUDA;
}
