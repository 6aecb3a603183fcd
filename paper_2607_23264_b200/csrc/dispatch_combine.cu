// Dispatch and combine: the two HBM-bound row movers of the layer.
//
// dispatch: token-centric.  A warp owns one token at a time, reads its row once with 16-byte loads and
//           writes it to the k rows of the expert-contiguous buffer named by inv_perm.  Algorithmic
//           traffic: 2H(T + R) bytes.
// combine : a warp owns a (token, column block) item, gathers the k expert rows named by inv_perm,
//           accumulates w[t,j] * y in fp32 in ascending j and writes bf16.  No atomics, fixed order.
//           Algorithmic traffic: 2H(R + T) + 8R bytes.
#include <cuda_bf16.h>

#include "moe_internal.h"

namespace {

constexpr int kThreads = 256;
constexpr int kVecPerLane = 4;                       // 16-byte vectors a lane keeps in flight
constexpr int kVecPerPass = 32 * kVecPerLane;        // vectors a warp moves per pass (2 KiB)

__global__ void __launch_bounds__(kThreads)
dispatch_rows(const uint4* __restrict__ x, const int32_t* __restrict__ inv_perm, uint4* __restrict__ x_perm,
              int T, int k, int vec_per_row) {
  const int lane = threadIdx.x & 31;
  const int warps_total = gridDim.x * (kThreads / 32);
  const int gwarp = blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
  for (int t = gwarp; t < T; t += warps_total) {
    const int my_row = (lane < k) ? inv_perm[static_cast<size_t>(t) * k + lane] : 0;
    const uint4* src = x + static_cast<size_t>(t) * vec_per_row;
    for (int v0 = 0; v0 < vec_per_row; v0 += kVecPerPass) {
      uint4 buf[kVecPerLane];
#pragma unroll
      for (int u = 0; u < kVecPerLane; ++u) {
        const int v = v0 + u * 32 + lane;
        if (v < vec_per_row) buf[u] = __ldg(src + v);
      }
      for (int j = 0; j < k; ++j) {
        const int row = __shfl_sync(0xFFFFFFFFu, my_row, j);
        uint4* dst = x_perm + static_cast<size_t>(row) * vec_per_row;
#pragma unroll
        for (int u = 0; u < kVecPerLane; ++u) {
          const int v = v0 + u * 32 + lane;
          if (v < vec_per_row) dst[v] = buf[u];
        }
      }
    }
  }
}

__device__ __forceinline__ void fma8(float (&acc)[8], float w, const uint4& v) {
  const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = __bfloat1622float2(p[i]);
    acc[2 * i] = fmaf(w, f.x, acc[2 * i]);
    acc[2 * i + 1] = fmaf(w, f.y, acc[2 * i + 1]);
  }
}

constexpr int kCombVec = 2;                      // vectors per lane per item
constexpr int kCombPass = 32 * kCombVec;         // vectors per item (1 KiB of bf16 per row)

__global__ void __launch_bounds__(kThreads)
combine_rows(const uint4* __restrict__ y_perm, const int32_t* __restrict__ inv_perm,
             const float* __restrict__ topk_w, uint4* __restrict__ out, int T, int k, int vec_per_row,
             int blocks_per_row) {
  const int lane = threadIdx.x & 31;
  const long long warps_total = static_cast<long long>(gridDim.x) * (kThreads / 32);
  const long long gwarp = static_cast<long long>(blockIdx.x) * (kThreads / 32) + (threadIdx.x >> 5);
  const long long items = static_cast<long long>(T) * blocks_per_row;
  for (long long item = gwarp; item < items; item += warps_total) {
    const int t = static_cast<int>(item / blocks_per_row);
    const int v0 = static_cast<int>(item % blocks_per_row) * kCombPass;
    int my_row = 0;
    float my_w = 0.f;
    if (lane < k) {
      my_row = inv_perm[static_cast<size_t>(t) * k + lane];
      my_w = topk_w[static_cast<size_t>(t) * k + lane];
    }
    float acc[kCombVec][8];
#pragma unroll
    for (int u = 0; u < kCombVec; ++u)
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[u][i] = 0.f;
#pragma unroll 4
    for (int j = 0; j < k; ++j) {                 // ascending j: the summation order is part of the contract
      const int row = __shfl_sync(0xFFFFFFFFu, my_row, j);
      const float w = __shfl_sync(0xFFFFFFFFu, my_w, j);
      const uint4* src = y_perm + static_cast<size_t>(row) * vec_per_row;
#pragma unroll
      for (int u = 0; u < kCombVec; ++u) {
        const int v = v0 + u * 32 + lane;
        if (v < vec_per_row) fma8(acc[u], w, __ldg(src + v));
      }
    }
#pragma unroll
    for (int u = 0; u < kCombVec; ++u) {
      const int v = v0 + u * 32 + lane;
      if (v < vec_per_row) {
        uint4 o;
        __nv_bfloat162* p = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
        for (int i = 0; i < 4; ++i) p[i] = __floats2bfloat162_rn(acc[u][2 * i], acc[u][2 * i + 1]);
        out[static_cast<size_t>(t) * vec_per_row + v] = o;
      }
    }
  }
}

}  // namespace

namespace moe {

cudaError_t launch_dispatch(moe_ctx* ctx, const void* x, const int32_t* inv_perm, void* x_perm,
                            cudaStream_t stream) {
  const moe_shape& s = ctx->shape;
  const int vec_per_row = s.H / 8;
  const int warps_per_block = kThreads / 32;
  int blocks = (s.T + warps_per_block - 1) / warps_per_block;
  const int cap = ctx->num_sms * 8;
  if (blocks > cap) blocks = cap;
  dispatch_rows<<<blocks, kThreads, 0, stream>>>(static_cast<const uint4*>(x), inv_perm,
                                                 static_cast<uint4*>(x_perm), s.T, s.k, vec_per_row);
  moe_mark(ctx, 4, stream);
  ctx->last_launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_combine(moe_ctx* ctx, const void* y_perm, const int32_t* inv_perm, const float* topk_w,
                           void* out, cudaStream_t stream) {
  const moe_shape& s = ctx->shape;
  const int vec_per_row = s.H / 8;
  const int blocks_per_row = (vec_per_row + kCombPass - 1) / kCombPass;
  const long long items = static_cast<long long>(s.T) * blocks_per_row;
  const int warps_per_block = kThreads / 32;
  long long blocks = (items + warps_per_block - 1) / warps_per_block;
  const long long cap = static_cast<long long>(ctx->num_sms) * 8;
  if (blocks > cap) blocks = cap;
  combine_rows<<<static_cast<int>(blocks), kThreads, 0, stream>>>(
      static_cast<const uint4*>(y_perm), inv_perm, topk_w, static_cast<uint4*>(out), s.T, s.k, vec_per_row,
      blocks_per_row);
  moe_mark(ctx, 7, stream);
  ctx->last_launches += 1;
  return cudaGetLastError();
}

}  // namespace moe
