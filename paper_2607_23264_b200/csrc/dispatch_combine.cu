// Dispatch and combine: the two HBM-bound row movers of the layer.
//
// dispatch: token-centric.  A warp owns a (token, column block) item, reads that part of the token's row once
//           with 16-byte loads and writes it to the k rows of the expert-contiguous buffer named by
//           inv_perm.  Algorithmic traffic: 2H(T + R) bytes.
// combine : a warp owns a (token, column block) item, gathers the k expert rows named by inv_perm,
//           accumulates w[t,j] * y in fp32 in ascending j and writes bf16.  No atomics, fixed order.
//           Algorithmic traffic: 2H(R + T) + 8R bytes.
#include <cuda_bf16.h>

#include "moe_internal.h"

namespace {

constexpr int kThreads = 256;

// 16-byte load of data read once: through the read-only path, not kept in L1
__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// One item = one token x (32 * V) 16-byte vectors of its row: read once, written to the k rows inv_perm names.
// Items rather than whole tokens per warp keep enough independent loads in flight for rows of several KiB.
template <int V>
__global__ void __launch_bounds__(kThreads)
dispatch_rows(const uint4* __restrict__ x, const int32_t* __restrict__ inv_perm, uint4* __restrict__ x_perm,
              int T, int k, int vec_per_row, int blocks_per_row) {
  const int lane = threadIdx.x & 31;
  const long long warps_total = static_cast<long long>(gridDim.x) * (kThreads / 32);
  const long long gwarp = static_cast<long long>(blockIdx.x) * (kThreads / 32) + (threadIdx.x >> 5);
  const long long items = static_cast<long long>(T) * blocks_per_row;
  for (long long item = gwarp; item < items; item += warps_total) {
    const int t = static_cast<int>(item / blocks_per_row);
    const int v0 = static_cast<int>(item % blocks_per_row) * (32 * V);
    const int my_row = (lane < k) ? __ldg(inv_perm + static_cast<size_t>(t) * k + lane) : 0;
    const uint4* src = x + static_cast<size_t>(t) * vec_per_row;
    uint4 buf[V];
#pragma unroll
    for (int u = 0; u < V; ++u) {
      const int v = v0 + u * 32 + lane;
      if (v < vec_per_row) buf[u] = ld_stream(src + v);
    }
    for (int j = 0; j < k; ++j) {
      const int row = __shfl_sync(0xFFFFFFFFu, my_row, j);
      uint4* dst = x_perm + static_cast<size_t>(row) * vec_per_row;
#pragma unroll
      for (int u = 0; u < V; ++u) {
        const int v = v0 + u * 32 + lane;
        if (v < vec_per_row) dst[v] = buf[u];
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

// One item = one token x (32 * V) 16-byte vectors of its row.  The k expert rows are fetched in batches of kCombBatch
// rows: all loads of a batch (kCombBatch * V per lane) are issued before the first of its FMAs, which then run in
// ascending j, so the memory system sees the whole batch at once while the summation order stays the contract's.
// What bounds the kernel is the bytes an SM keeps in flight (resident warps x loads per lane x 16 bytes); V and the
// batch are template parameters because registers decide how many warps are resident (the launcher picks them).
template <int V, int kCombBatch>
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
    const int v0 = static_cast<int>(item % blocks_per_row) * (32 * V);
    int my_row = 0;
    float my_w = 0.f;
    if (lane < k) {
      my_row = __ldg(inv_perm + static_cast<size_t>(t) * k + lane);
      my_w = __ldg(topk_w + static_cast<size_t>(t) * k + lane);
    }
    float acc[V][8];
#pragma unroll
    for (int u = 0; u < V; ++u)
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[u][i] = 0.f;
    for (int j0 = 0; j0 < k; j0 += kCombBatch) {
      uint4 buf[kCombBatch][V];
      float w[kCombBatch];
#pragma unroll
      for (int b = 0; b < kCombBatch; ++b) {
        const int j = j0 + b;                       // j >= k reads lane j's zeros: row 0, weight 0, skipped below
        const int row = __shfl_sync(0xFFFFFFFFu, my_row, j & 31);
        w[b] = __shfl_sync(0xFFFFFFFFu, my_w, j & 31);
        const uint4* src = y_perm + static_cast<size_t>(row) * vec_per_row;
#pragma unroll
        for (int u = 0; u < V; ++u) {
          const int v = v0 + u * 32 + lane;
          if (j < k && v < vec_per_row) buf[b][u] = ld_stream(src + v);
        }
      }
#pragma unroll
      for (int b = 0; b < kCombBatch; ++b) {       // ascending j: the summation order is part of the contract
        if (j0 + b < k) {
#pragma unroll
          for (int u = 0; u < V; ++u)
            if (v0 + u * 32 + lane < vec_per_row) fma8(acc[u], w[b], buf[b][u]);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < V; ++u) {
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
  int V = moe_knob_value(ctx, "dispatch_vec", 0);
  if (V != 1 && V != 2 && V != 4) V = 4;
  while (V > 1 && vec_per_row < 32 * V) V >>= 1;
  const int blocks_per_row = (vec_per_row + 32 * V - 1) / (32 * V);
  const long long items = static_cast<long long>(s.T) * blocks_per_row;
  const int warps_per_block = kThreads / 32;
  long long blocks = (items + warps_per_block - 1) / warps_per_block;
  const long long cap = static_cast<long long>(ctx->num_sms) * moe_knob_value(ctx, "dispatch_ctas_per_sm", 16);
  if (blocks > cap && cap > 0) blocks = cap;
  auto kernel = V == 4 ? dispatch_rows<4> : V == 2 ? dispatch_rows<2> : dispatch_rows<1>;
  kernel<<<static_cast<int>(blocks), kThreads, 0, stream>>>(static_cast<const uint4*>(x), inv_perm,
                                                            static_cast<uint4*>(x_perm), s.T, s.k, vec_per_row,
                                                            blocks_per_row);
  moe_mark(ctx, 4, stream);
  ctx->last_launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_combine(moe_ctx* ctx, const void* y_perm, const int32_t* inv_perm, const float* topk_w,
                           void* out, cudaStream_t stream) {
  const moe_shape& s = ctx->shape;
  const int vec_per_row = s.H / 8;
  // Measured on the Mixtral-like (k = 2) and DeepSeek-V3-like (k = 8) movers: four vectors per lane, rows taken one at
  // a time (72 registers, three resident CTAs per SM), beats every variant that batches rows or narrows the item; only
  // batches of a few dozen tokens prefer one vector per lane with the rows batched (more warps, fewer bytes each).
  int batch = 1, V = 4;
  if (s.T < 2 * ctx->num_sms) { V = 1; batch = s.k >= 4 ? 4 : s.k >= 2 ? 2 : 1; }
  while (V > 1 && vec_per_row < 32 * V) V >>= 1;
  const int kv = moe_knob_value(ctx, "combine_vec", 0), kb = moe_knob_value(ctx, "combine_batch", 0);
  if (kv == 1 || kv == 2 || kv == 4) V = kv;
  if (kb == 1 || kb == 2 || kb == 4 || kb == 8) batch = kb;
  const int blocks_per_row = (vec_per_row + 32 * V - 1) / (32 * V);
  const long long items = static_cast<long long>(s.T) * blocks_per_row;
  const int warps_per_block = kThreads / 32;
  long long blocks = (items + warps_per_block - 1) / warps_per_block;
  const long long cap = static_cast<long long>(ctx->num_sms) * moe_knob_value(ctx, "combine_ctas_per_sm", 3);
  if (blocks > cap && cap > 0) blocks = cap;
  using kernel_t = void (*)(const uint4*, const int32_t*, const float*, uint4*, int, int, int, int);
  static const kernel_t table[3][4] = {
      {combine_rows<1, 1>, combine_rows<1, 2>, combine_rows<1, 4>, combine_rows<1, 8>},
      {combine_rows<2, 1>, combine_rows<2, 2>, combine_rows<2, 4>, combine_rows<2, 8>},
      {combine_rows<4, 1>, combine_rows<4, 2>, combine_rows<4, 4>, combine_rows<4, 8>}};
  const kernel_t kernel = table[V == 4 ? 2 : V == 2 ? 1 : 0][batch == 8 ? 3 : batch == 4 ? 2 : batch == 2 ? 1 : 0];
  kernel<<<static_cast<int>(blocks), kThreads, 0, stream>>>(static_cast<const uint4*>(y_perm), inv_perm, topk_w,
                                                            static_cast<uint4*>(out), s.T, s.k, vec_per_row,
                                                            blocks_per_row);
  moe_mark(ctx, 7, stream);
  ctx->last_launches += 1;
  return cudaGetLastError();
}

}  // namespace moe
