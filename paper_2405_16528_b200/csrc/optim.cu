// Optimiser step on the trainable factor B (paper Algorithm 1, the update line
// B <- B - rho(G^B) with rho = Adam; optimiser states in bf16).  One streaming
// pass: 4 bytes of gradient and 2 + 2 + 2 bytes of B and the two moments in,
// 2 + 2 + 2 bytes out per element.
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
