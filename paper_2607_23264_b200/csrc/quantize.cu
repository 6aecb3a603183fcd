// FP8 (E4M3) support kernels: row-wise quantisation of bf16 matrices and the dispatch of quantised rows.
//
// quantize_rows: one CTA per row.  Pass 1 reads the row with 16-byte loads and reduces max|v| (exact in fp32);
//   scale = amax / 448 (1 for an all-zero row); pass 2 re-reads the row (from L1/L2), divides in fp32 and converts
//   with round-to-nearest-even, saturating at +-448.  8 codes leave as one 8-byte store.
// dispatch_rows_fp8: the token-centric row mover of the bf16 path on 1-byte elements, plus the scale of each row.
#include <cuda_bf16.h>
#include <cuda_fp8.h>

#include "moe_internal.h"

namespace {

constexpr int kQThreads = 256;

__global__ void __launch_bounds__(kQThreads)
quantize_rows(const uint4* __restrict__ in, long long rows, int vec_per_row, uint2* __restrict__ codes,
              float* __restrict__ scales) {
  __shared__ float s_part[kQThreads / 32];
  __shared__ float s_scale;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (long long row = blockIdx.x; row < rows; row += gridDim.x) {
    const uint4* src = in + row * vec_per_row;
    float amax = 0.f;
    for (int v = tid; v < vec_per_row; v += kQThreads) {
      const uint4 q = __ldg(src + v);
      const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&q);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 f = __bfloat1622float2(p[i]);
        amax = fmaxf(amax, fmaxf(fabsf(f.x), fabsf(f.y)));
      }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, off));
    if (lane == 0) s_part[warp] = amax;
    __syncthreads();
    if (tid == 0) {
      float m = s_part[0];
      for (int w = 1; w < kQThreads / 32; ++w) m = fmaxf(m, s_part[w]);
      const float sc = m > 0.f ? __fdiv_rn(m, 448.f) : 1.f;
      s_scale = sc;
      scales[row] = sc;
    }
    __syncthreads();
    const float sc = s_scale;
    uint2* dst = codes + row * vec_per_row;
    for (int v = tid; v < vec_per_row; v += kQThreads) {
      const uint4 q = __ldg(src + v);
      const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&q);
      unsigned char c[8];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 f = __bfloat1622float2(p[i]);
        c[2 * i] = static_cast<unsigned char>(__nv_cvt_float_to_fp8(__fdiv_rn(f.x, sc), __NV_SATFINITE, __NV_E4M3));
        c[2 * i + 1] = static_cast<unsigned char>(__nv_cvt_float_to_fp8(__fdiv_rn(f.y, sc), __NV_SATFINITE, __NV_E4M3));
      }
      uint2 o;
      o.x = c[0] | (c[1] << 8) | (c[2] << 16) | (static_cast<uint32_t>(c[3]) << 24);
      o.y = c[4] | (c[5] << 8) | (c[6] << 16) | (static_cast<uint32_t>(c[7]) << 24);
      dst[v] = o;
    }
    __syncthreads();   // s_part / s_scale are reused by the next row
  }
}

constexpr int kVecPerLane = 4;
constexpr int kVecPerPass = 32 * kVecPerLane;

__global__ void __launch_bounds__(kQThreads)
dispatch_rows_fp8(const uint4* __restrict__ xq, const float* __restrict__ sx, const int32_t* __restrict__ inv_perm,
                  uint4* __restrict__ xq_perm, float* __restrict__ sx_perm, int T, int k, int vec_per_row) {
  const int lane = threadIdx.x & 31;
  const int warps_total = gridDim.x * (kQThreads / 32);
  const int gwarp = blockIdx.x * (kQThreads / 32) + (threadIdx.x >> 5);
  for (int t = gwarp; t < T; t += warps_total) {
    const int my_row = (lane < k) ? inv_perm[static_cast<size_t>(t) * k + lane] : 0;
    if (lane < k) sx_perm[my_row] = sx[t];
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

cudaError_t launch_quantize_rows(moe_ctx* ctx, const void* in_bf16, long long rows, int cols, void* codes,
                                 float* scales, cudaStream_t stream) {
  if (rows == 0) return cudaSuccess;
  long long blocks = rows;
  const long long cap = static_cast<long long>(ctx->num_sms) * 16;
  if (blocks > cap) blocks = cap;
  quantize_rows<<<static_cast<int>(blocks), kQThreads, 0, stream>>>(static_cast<const uint4*>(in_bf16), rows, cols / 8,
                                                                  static_cast<uint2*>(codes), scales);
  ctx->last_launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_dispatch_fp8(moe_ctx* ctx, const void* xq, const float* sx, const int32_t* inv_perm,
                                void* xq_perm, float* sx_perm, cudaStream_t stream) {
  const moe_shape& s = ctx->shape;
  const int warps_per_block = kQThreads / 32;
  int blocks = (s.T + warps_per_block - 1) / warps_per_block;
  const int cap = ctx->num_sms * 8;
  if (blocks > cap) blocks = cap;
  dispatch_rows_fp8<<<blocks, kQThreads, 0, stream>>>(static_cast<const uint4*>(xq), sx, inv_perm,
                                                     static_cast<uint4*>(xq_perm), sx_perm, s.T, s.k, s.H / 16);
  moe_mark(ctx, 4, stream);
  ctx->last_launches += 1;
  return cudaGetLastError();
}

}  // namespace moe
