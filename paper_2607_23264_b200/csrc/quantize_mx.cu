// Block-scaled FP8 (MXFP8) support kernels: quantisation of bf16 matrices in 32-element blocks along K, and the
// dispatch of quantised rows with their scale words.
//
// quantize_rows_mx : one thread per block: 64 bytes of bf16 in (four 16-byte loads), the block maximum, the scale
//   byte, 32 codes out (two 16-byte stores).  Scale bytes are stored four to a word, words as [K/128][rows], so that
//   the GEMM's scale loader reads one word per row per 128-element K stage, consecutive rows side by side.
// dispatch_rows_mx : the token-centric row mover on 1-byte elements, plus the K/128 scale words of each row.
#include <cuda_bf16.h>

#include "moe_internal.h"
#include "mx_quant.cuh"

namespace {

constexpr int kQThreads = 256;

__global__ void __launch_bounds__(kQThreads)
quantize_rows_mx(const uint4* __restrict__ in, long long rows, int blocks_per_row, uint4* __restrict__ codes,
                 unsigned char* __restrict__ sf_bytes) {
  const long long total = rows * blocks_per_row;
  for (long long g = static_cast<long long>(blockIdx.x) * kQThreads + threadIdx.x; g < total;
       g += static_cast<long long>(gridDim.x) * kQThreads) {
    const long long row = g / blocks_per_row;
    const int b = static_cast<int>(g - row * blocks_per_row);
    float v[32];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint4 q = __ldg(in + g * 4 + u);
      const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&q);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 f = __bfloat1622float2(p[i]);
        v[8 * u + 2 * i] = f.x;
        v[8 * u + 2 * i + 1] = f.y;
      }
    }
    uint32_t c[8];
    const uint32_t byte = mx::quantize_block(v, c);
    codes[g * 2] = make_uint4(c[0], c[1], c[2], c[3]);
    codes[g * 2 + 1] = make_uint4(c[4], c[5], c[6], c[7]);
    sf_bytes[mx::scale_byte_index(rows, row, b)] = static_cast<unsigned char>(byte);
  }
}

constexpr int kVecPerLane = 4;
constexpr int kVecPerPass = 32 * kVecPerLane;

__global__ void __launch_bounds__(kQThreads)
dispatch_rows_mx(const uint4* __restrict__ xq, const uint32_t* __restrict__ sfx, const int32_t* __restrict__ inv_perm,
                 uint4* __restrict__ xq_perm, uint32_t* __restrict__ sfx_perm, int T, int k, int vec_per_row,
                 int words_per_row) {
  const int lane = threadIdx.x & 31;
  const int warps_total = gridDim.x * (kQThreads / 32);
  const int gwarp = blockIdx.x * (kQThreads / 32) + (threadIdx.x >> 5);
  const size_t R = static_cast<size_t>(T) * k;
  for (int t = gwarp; t < T; t += warps_total) {
    const int my_row = (lane < k) ? inv_perm[static_cast<size_t>(t) * k + lane] : 0;
    for (int wd0 = 0; wd0 < words_per_row; wd0 += 32) {          // uniform trip count: the shuffles need every lane
      const int wd = wd0 + lane;
      const bool valid = wd < words_per_row;
      const uint32_t word = valid ? sfx[static_cast<size_t>(wd) * T + t] : 0u;
      for (int j = 0; j < k; ++j) {
        const int row = __shfl_sync(0xFFFFFFFFu, my_row, j);
        if (valid) sfx_perm[static_cast<size_t>(wd) * R + row] = word;
      }
    }
    const uint4* src = xq + static_cast<size_t>(t) * vec_per_row;
    for (int v0 = 0; v0 < vec_per_row; v0 += kVecPerPass) {
      uint4 buf[kVecPerLane];
#pragma unroll
      for (int u = 0; u < kVecPerLane; ++u) {
        const int v = v0 + u * 32 + lane;
        if (v < vec_per_row) buf[u] = __ldg(src + v);
      }
      for (int j = 0; j < k; ++j) {
        const int row = __shfl_sync(0xFFFFFFFFu, my_row, j);
        uint4* dst = xq_perm + static_cast<size_t>(row) * vec_per_row;
#pragma unroll
        for (int u = 0; u < kVecPerLane; ++u) {
          const int v = v0 + u * 32 + lane;
          if (v < vec_per_row) dst[v] = buf[u];
        }
      }
    }
  }
}

}  // namespace

namespace moe {

cudaError_t launch_quantize_rows_mx(moe_ctx* ctx, const void* in_bf16, long long rows, int cols, void* codes,
                                    uint32_t* sf_words, cudaStream_t stream) {
  if (rows == 0) return cudaSuccess;
  const long long total = rows * (cols / 32);
  long long blocks = (total + kQThreads - 1) / kQThreads;
  const long long cap = static_cast<long long>(ctx->num_sms) * 32;
  if (blocks > cap) blocks = cap;
  quantize_rows_mx<<<static_cast<int>(blocks), kQThreads, 0, stream>>>(
      static_cast<const uint4*>(in_bf16), rows, cols / 32, static_cast<uint4*>(codes),
      reinterpret_cast<unsigned char*>(sf_words));
  ctx->last_launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_dispatch_mx(moe_ctx* ctx, const void* xq, const uint32_t* sfx, const int32_t* inv_perm,
                               void* xq_perm, uint32_t* sfx_perm, cudaStream_t stream) {
  const moe_shape& s = ctx->shape;
  const int warps_per_block = kQThreads / 32;
  int blocks = (s.T + warps_per_block - 1) / warps_per_block;
  const int cap = ctx->num_sms * 8;
  if (blocks > cap) blocks = cap;
  dispatch_rows_mx<<<blocks, kQThreads, 0, stream>>>(static_cast<const uint4*>(xq), sfx, inv_perm,
                                                    static_cast<uint4*>(xq_perm), sfx_perm, s.T, s.k, s.H / 16,
                                                    s.H / 128);
  moe_mark(ctx, 4, stream);
  ctx->last_launches += 1;
  return cudaGetLastError();
}

}  // namespace moe
