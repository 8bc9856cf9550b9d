// Register-only NF4 -> bf16 dequantisation of one block of 64 weights
// (paper Section 5.1: w = M * q[code]), for staging GEMM operands.
//
// A block shares one scale M, so the 16 possible outputs bf16(M * q_i) are
// formed once per block (16 multiplies, 8 packed conversions) and each code is
// then a lookup.  The table lives in registers as two byte planes (low bytes
// and high bytes of the 16 bf16 values, 4 registers each); a byte-permute picks
// 4 entries at a time from the lower or upper 8 entries, and bit 3 of each code
// selects between the two.  Every output equals bf16_rne(fl32(M * q_i)) exactly.
#pragma once
#include "common.cuh"

namespace loqt {

#ifdef __CUDA_ARCH__
#define LOQT_HD __host__ __device__ __forceinline__
#else
#define LOQT_HD inline
#endif

LOQT_HD uint32_t hd_prmt(uint32_t a, uint32_t b, uint32_t s) {
#ifdef __CUDA_ARCH__
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(s));
  return d;
#else
  const uint64_t src = (static_cast<uint64_t>(b) << 32) | a;
  uint32_t d = 0;
  for (int i = 0; i < 4; ++i) {
    const uint32_t n = (s >> (4 * i)) & 0xFu;
    uint32_t byte = static_cast<uint32_t>(src >> (8 * (n & 7u))) & 0xFFu;
    if (n & 8u) byte = (byte & 0x80u) ? 0xFFu : 0x00u;
    d |= byte << (8 * i);
  }
  return d;
#endif
}

LOQT_HD uint32_t hd_pack_bf16x2(float lo, float hi) {
#ifdef __CUDA_ARCH__
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
#else
  auto rne = [](float f) -> uint32_t {
    uint32_t u;
    __builtin_memcpy(&u, &f, 4);
    return (u + 0x7FFFu + ((u >> 16) & 1u)) >> 16;
  };
  return rne(lo) | (rne(hi) << 16);
#endif
}

// Byte planes of the scaled table of one block.
struct Nf4BlockTable {
  uint32_t lo[4];  // lo[j] = low bytes of entries 4j .. 4j+3
  uint32_t hi[4];  // hi[j] = high bytes of entries 4j .. 4j+3
};

LOQT_HD void nf4_block_table(float M, Nf4BlockTable &t) {
  constexpr float lv[16] = LOQT_NF4_LEVELS;
  uint32_t p[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) p[j] = hd_pack_bf16x2(M * lv[2 * j], M * lv[2 * j + 1]);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    t.lo[j] = hd_prmt(p[2 * j], p[2 * j + 1], 0x6420u);
    t.hi[j] = hd_prmt(p[2 * j], p[2 * j + 1], 0x7531u);
  }
}

// One code word (8 codes, element j in nibble j) -> 8 bf16 (16 bytes).
// Codes 0..3 use the selector's low half directly; codes 4..7 the same word
// shifted down.  Bit 3 of every code is turned into a byte mask by a permute in
// sign-replication mode: the sign bits of bytes 0..3 of w hold bit 3 of the odd
// codes, those of w << 4 bit 3 of the even codes.
LOQT_HD uint4 nf4_dequant8(const Nf4BlockTable &t, uint32_t w) {
  const uint32_t w4 = w << 4;
  const uint32_t idx = w & 0x77777777u;  // 3-bit table indices; a permute reads the low 16 bits of its selector
  const uint32_t idxh = idx >> 16;
  const uint32_t up_l = hd_prmt(w4, w, 0xD9C8u);  // byte e = 0xFF iff code e >= 8       (e = 0..3)
  const uint32_t up_h = hd_prmt(w4, w, 0xFBEAu);  // byte e = 0xFF iff code 4 + e >= 8
  uint4 o;
  {
    const uint32_t lo = (hd_prmt(t.lo[0], t.lo[1], idx) & ~up_l) | (hd_prmt(t.lo[2], t.lo[3], idx) & up_l);
    const uint32_t hi = (hd_prmt(t.hi[0], t.hi[1], idx) & ~up_l) | (hd_prmt(t.hi[2], t.hi[3], idx) & up_l);
    o.x = hd_prmt(lo, hi, 0x5140u);
    o.y = hd_prmt(lo, hi, 0x7362u);
  }
  {
    const uint32_t lo = (hd_prmt(t.lo[0], t.lo[1], idxh) & ~up_h) | (hd_prmt(t.lo[2], t.lo[3], idxh) & up_h);
    const uint32_t hi = (hd_prmt(t.hi[0], t.hi[1], idxh) & ~up_h) | (hd_prmt(t.hi[2], t.hi[3], idxh) & up_h);
    o.z = hd_prmt(lo, hi, 0x5140u);
    o.w = hd_prmt(lo, hi, 0x7362u);
  }
  return o;
}

}  // namespace loqt
