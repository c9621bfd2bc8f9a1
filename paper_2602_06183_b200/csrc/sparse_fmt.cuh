// Device helpers for the two packed activation formats of the step: the V:N:M form with groups of
// eight columns (Section 2.3) and its re-expression as a plain 2:4 operand over all columns.
// Shared by the stand-alone sparsify kernel, the fused epilogue of the y1 product, the dy1 epilogue
// and the operand expanders of the weight-gradient products.
#pragma once

#include "sf_common.cuh"

namespace sf {

// max(x, 0) and x * x on a packed pair of bf16 (the multiply is correctly rounded, which equals
// rounding the exact float32 square)
__device__ __forceinline__ uint32_t bf2_relu(uint32_t w) {
  __nv_bfloat162 x = *reinterpret_cast<__nv_bfloat162*>(&w);
  __nv_bfloat162 z = __hmax2(x, __float2bfloat162_rn(0.f));
  return *reinterpret_cast<uint32_t*>(&z);
}
__device__ __forceinline__ uint32_t bf2_sq(uint32_t r) {
  __nv_bfloat162 x = *reinterpret_cast<__nv_bfloat162*>(&r);
  __nv_bfloat162 z = __hmul2(x, x);
  return *reinterpret_cast<uint32_t*>(&z);
}

// Byte-permute selectors for one group of eight columns whose row keeps the pair of columns
// ca < cb (each 0..7). With `pair` = the two kept values (first in the low half):
//   sel.x, sel.y   four 16-bit selectors: dense word j (columns 2j, 2j+1) = byte_perm(pair, 0, s_j)
//   sel.z          low half: picks the two values at columns (ca & 3), (cb & 3) out of a pair of words;
//                  high half: then chooses between the words of columns 0..3 and 4..7
//   sel.w          the same pair laid out as a 2:4 operand: low half = stored pair of columns 0..3,
//                  high half = stored pair of columns 4..7 (zeros where a half keeps fewer than two)
//   nib24          the two position nibbles of that 2:4 layout (low = columns 0..3). A half that
//                  keeps one value at position p pairs it with a zero at position 1 (p = 0) or 0
//                  (p > 0); a half that keeps none records positions (0, 1).
__device__ __forceinline__ void vnm8_pair_selectors(uint32_t ca, uint32_t cb, uint4& sel, uint32_t& nib24) {
  uint32_t sd[4];
#pragma unroll
  for (uint32_t j = 0; j < 4; ++j) {
    const uint32_t lo = ca == 2 * j ? 0x10u : (cb == 2 * j ? 0x32u : 0x44u);
    const uint32_t hi = ca == 2 * j + 1 ? 0x10u : (cb == 2 * j + 1 ? 0x32u : 0x44u);
    sd[j] = lo | (hi << 8);
  }
  const uint32_t pa = ca & 3u, pb = cb & 3u;
  const uint32_t s1 = (2u * pa) | ((2u * pa + 1u) << 4) | ((2u * pb) << 8) | ((2u * pb + 1u) << 12);
  const uint32_t s2 = (ca < 4u ? 0x10u : 0x54u) | ((cb < 4u ? 0x32u : 0x76u) << 8);
  const bool both_lo = cb < 4u, both_hi = ca >= 4u;
  const uint32_t s_wlo = both_lo ? 0x3210u : (both_hi ? 0x4444u : (pa == 0u ? 0x4410u : 0x1044u));
  const uint32_t s_whi = both_hi ? 0x3210u : (both_lo ? 0x4444u : (pb == 0u ? 0x4432u : 0x3244u));
  const uint32_t pair_nib = pa | (pb << 2);
  const uint32_t nlo = both_lo ? pair_nib : (both_hi ? 4u : (pa == 0u ? 4u : (pa << 2)));
  const uint32_t nhi = both_hi ? pair_nib : (both_lo ? 4u : (pb == 0u ? 4u : (pb << 2)));
  sel = make_uint4(sd[0] | (sd[1] << 16), sd[2] | (sd[3] << 16), s1 | (s2 << 16), s_wlo | (s_whi << 16));
  nib24 = nlo | (nhi << 4);
}

// The six legal position pairs of a 2:4 nibble are distinct modulo 7: table slot of a nibble.
__device__ __forceinline__ uint32_t nib_slot(uint32_t nib) { return nib - 7u * ((nib * 37u) >> 8); }

// One 2:4 group back to its four dense columns: `pair` holds the two stored values (first in the
// low half), `nib` = pos0 | pos1 << 2. w0 = columns 0, 1; w1 = columns 2, 3; dropped columns are +0.
__device__ __forceinline__ void expand24(uint32_t pair, uint32_t nib, uint32_t& w0, uint32_t& w1) {
  const uint32_t s0 = (nib & 3u) * 8u, s1 = (nib >> 2) * 8u;      // selector field of each kept column
  uint32_t s = 0x44444444u;                                      // every byte from the zero operand
  s = (s & ~(0xFFu << s0)) | (0x10u << s0);
  s = (s & ~(0xFFu << s1)) | (0x32u << s1);
  w0 = __byte_perm(pair, 0u, s & 0xFFFFu);
  w1 = __byte_perm(pair, 0u, s >> 16);
}

// Eight dense columns (16 bytes) from the 2:4 layout: `v` = the four stored values of the two
// groups, `mb` = their two nibbles (low nibble = first group).
__device__ __forceinline__ uint4 expand24_x8(uint2 v, uint32_t mb) {
  uint4 d;
  expand24(v.x, mb & 0xFu, d.x, d.y);
  expand24(v.y, (mb >> 4) & 0xFu, d.z, d.w);
  return d;
}

}  // namespace sf
