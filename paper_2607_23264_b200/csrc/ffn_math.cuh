// Small device helpers shared by the grouped-GEMM epilogues.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

// SwiGLU merge of the two Linear-1 halves: silu(g) * u with the fast exponential and division (both sides of a
// parity test see the result through a 5e-3 relative bound).
__device__ __forceinline__ float silu_mul(float g, float u) { return __fdividef(g, 1.f + __expf(-g)) * u; }

// Two fp32 values -> one word of two bf16 (nearest-even), lower address first.
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&v);
}
