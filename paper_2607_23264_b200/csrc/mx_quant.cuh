// Block-scaled FP8 (MXFP8) helpers shared by the quantisation kernel and the Linear-1 epilogue: 32 consecutive
// elements along K share a scale 2^e stored as the byte e + 127 (E8M0), elements are E4M3.
#pragma once
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace mx {

// Scale byte of a block whose largest magnitude is amax (fp32, finite, >= 0): the smallest e with
// amax * 2^-e <= 448, not below -127.  448 = 1.75 * 2^8, so on the bits of amax this is
// e = (unbiased exponent) - 8 + [mantissa field > 0x600000].  Integer work only: reproducible bit for bit.
__device__ __forceinline__ uint32_t scale_byte(float amax) {
  const uint32_t bits = __float_as_uint(amax);
  int e = static_cast<int>((bits >> 23) & 0xFFu) - 127 - 8 + ((bits & 0x7FFFFFu) > 0x600000u ? 1 : 0);
  e = e < -127 ? -127 : e;          // zero and subnormal blocks; the upper end (120) is never exceeded
  return static_cast<uint32_t>(e + 127);
}
// 2^-e as an fp32 (exponent field 254 - byte, always a normal number); multiplying by it is exact.
__device__ __forceinline__ float inverse_scale(uint32_t byte) { return __uint_as_float((254u - byte) << 23); }

// Four values -> four E4M3 codes in one word (lowest byte first), nearest-even, saturating.
__device__ __forceinline__ uint32_t pack4(float a, float b, float c, float d) {
  const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(a, b), __NV_SATFINITE, __NV_E4M3);
  const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(c, d), __NV_SATFINITE, __NV_E4M3);
  return lo | (hi << 16);
}

// Quantise one block of 32 fp32 values: returns the scale byte, writes the 32 codes as 8 words.
__device__ __forceinline__ uint32_t quantize_block(const float (&v)[32], uint32_t (&codes)[8]) {
  float amax = 0.f;
#pragma unroll
  for (int i = 0; i < 32; ++i) amax = fmaxf(amax, fabsf(v[i]));
  const uint32_t byte = scale_byte(amax);
  const float inv = inverse_scale(byte);
#pragma unroll
  for (int i = 0; i < 8; ++i) codes[i] = pack4(v[4 * i] * inv, v[4 * i + 1] * inv, v[4 * i + 2] * inv, v[4 * i + 3] * inv);
  return byte;
}

// Scale bytes live in words of four (one word = the four 32-blocks of a 128-element K stage), words stored
// [K/128][rows]: byte address of block b of row r.
__device__ __forceinline__ size_t scale_byte_index(long long rows, long long r, int b) {
  return (static_cast<size_t>(b >> 2) * rows + r) * 4 + (b & 3);
}

}  // namespace mx
