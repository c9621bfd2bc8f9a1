// E4M3 conversion helpers shared by the quantising passes.
#pragma once

#include <cuda_fp8.h>

#include "sf_common.cuh"

namespace sf {

// two floats -> two E4M3 codes (low byte = first): round to nearest even, magnitudes above 448 clamp
__device__ __forceinline__ uint32_t e4m3x2(float a, float b) {
  return (uint32_t)__nv_cvt_float2_to_fp8x2(make_float2(a, b), __NV_SATFINITE, __NV_E4M3);
}
// a word of two bf16 patterns -> two codes of float(x) * scale, in the low 16 bits
__device__ __forceinline__ uint32_t quant2(uint32_t w, float scale) {
  return e4m3x2(__fmul_rn(bf16_bits_to_float(w & 0xFFFFu), scale), __fmul_rn(bf16_bits_to_float(w >> 16), scale));
}

}  // namespace sf
