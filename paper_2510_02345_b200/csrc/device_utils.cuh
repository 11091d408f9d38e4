// Small device helpers shared by the kernels: INT4 decoding, warp reductions, erf-GELU.
#pragma once

#include <cuda_fp16.h>
#include <stdint.h>

namespace cmoe {

// Sign-extend a 4-bit two's-complement code held in the low nibble.
__device__ __forceinline__ int sext4(int nib) { return ((nib & 0xF) ^ 8) - 8; }

// Element `flat` of a packed INT4 factor times the fp16 scale of its group of 32 (Sec. 3.4).
__device__ __forceinline__ float deq4(const uint8_t* __restrict__ q, const __half* __restrict__ s,
                                      long long flat) {
  int b = q[flat >> 1];
  int code = sext4((flat & 1) ? (b >> 4) : b);
  return (float)code * __half2float(s[flat >> 5]);
}

// The eight codes of a 32-bit word of a packed INT4 factor as floats, without integer-to-float
// conversions: (nibble ^ 8) = code + 8 is placed in the mantissa of 2^23, then 2^23 + 8 is subtracted.
__device__ __forceinline__ void int4x8_to_float(uint32_t word, float* out) {
#pragma unroll
  for (int n = 0; n < 8; ++n) {
    const uint32_t bits = ((word >> (4 * n)) & 0xFu) ^ 0x4B000008u;
    out[n] = __uint_as_float(bits) - 8388616.0f;
  }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// GELU(u) = u/2 (1 + erf(u / sqrt 2))
__device__ __forceinline__ float gelu_erf(float u) {
  return 0.5f * u * (1.0f + erff(u * 0.70710678118654752f));
}

}  // namespace cmoe
