// Top-k selection of one token by one warp, shared by the routing plan (logits given) and the router
// front end (logits computed in the same kernel), so that both take the same decisions on the same fp32 values.
#pragma once
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

namespace moe {

// Order-preserving map fp32 -> uint32 (a > b as floats <=> key(a) > key(b) as unsigned, for non-NaN values;
// -0 is first turned into +0 so that the two zeros tie as they do in a float comparison).  Every key is > 0.
__device__ __forceinline__ uint32_t order_key(float v) {
  const uint32_t u = __float_as_uint(v + 0.0f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_value(uint32_t key) {
  return __uint_as_float((key & 0x80000000u) ? (key ^ 0x80000000u) : ~key);
}

// NT tokens at once (their chains of reductions are independent, so the warp overlaps them).  A token's E logits
// are read once from rows[n] (lane l keeps entries l, l+32, ... as keys in registers; EL = entries per lane,
// E <= 32*EL).  k passes of warp arg-max, ties to the lower expert index: a scan of the lane's own keys and two
// warp-wide integer reductions (the largest key, then the lowest index holding it); the picked entry is cleared in
// its owner's register.  Slot j receives the j-th largest logit.  Weights = softmax over the k selected logits
// (fp32).  Lane j < k returns its slot's expert id and weight for token n in id[n], w[n].
template <int EL, int NT>
__device__ __forceinline__ void warp_select_topk_regs(const float* const (&rows)[NT], int E, int k, int lane,
                                                      int (&id)[NT], float (&w)[NT]) {
  constexpr unsigned kFull = 0xFFFFFFFFu;
  uint32_t key[NT][EL];
#pragma unroll
  for (int n = 0; n < NT; ++n)
#pragma unroll
    for (int i = 0; i < EL; ++i) {
      const int e = lane + 32 * i;
      key[n][i] = e < E ? order_key(rows[n][e]) : 0u;   // 0 is below every key: never picked while an entry is left
    }
  uint32_t sel_key[NT];    // lane j keeps the key picked in pass j
#pragma unroll
  for (int n = 0; n < NT; ++n) { sel_key[n] = 0; id[n] = 0; }
  for (int j = 0; j < k; ++j) {
    // stage by stage over the NT tokens, so that their reductions are issued back to back
    uint32_t best[NT], top[NT];
    int best_e[NT], pick[NT];
#pragma unroll
    for (int n = 0; n < NT; ++n) {
      best[n] = 0;
      best_e[n] = 0x7FFFFFFF;
#pragma unroll
      for (int i = 0; i < EL; ++i)                  // ascending index with strict '>' keeps the lowest index
        if (key[n][i] > best[n]) { best[n] = key[n][i]; best_e[n] = lane + 32 * i; }
    }
#pragma unroll
    for (int n = 0; n < NT; ++n) top[n] = __reduce_max_sync(kFull, best[n]);
#pragma unroll
    for (int n = 0; n < NT; ++n) pick[n] = __reduce_min_sync(kFull, best[n] == top[n] ? best_e[n] : 0x7FFFFFFF);
#pragma unroll
    for (int n = 0; n < NT; ++n) {
      if (pick[n] >= E) pick[n] = E - 1;            // nothing left to pick (cannot happen for k <= E): stay in range
#pragma unroll
      for (int i = 0; i < EL; ++i)
        if (pick[n] == lane + 32 * i) key[n][i] = 0u;   // taken
      if (lane == j) { sel_key[n] = top[n]; id[n] = pick[n]; }
    }
  }
  // softmax over the k selected logits; pass 0 picked the maximum.  Lanes >= k hold 0, so a butterfly over the
  // smallest power of two >= k lanes sums everything.
  int width = 1;
  while (width < k) width <<= 1;
#pragma unroll
  for (int n = 0; n < NT; ++n) {
    const float sel_logit = key_value(sel_key[n]);
    const float m = __shfl_sync(kFull, sel_logit, 0);
    const float p = (lane < k) ? expf(sel_logit - m) : 0.f;
    float sum = p;
    for (int off = width >> 1; off > 0; off >>= 1) sum += __shfl_xor_sync(kFull, sum, off);
    w[n] = p / sum;
  }
}

// E <= 1024.  The rows may be shared or global memory; they are only read.
template <int NT>
__device__ __forceinline__ void warp_select_topk_n(const float* const (&rows)[NT], int E, int k, int lane,
                                                   int (&id)[NT], float (&w)[NT]) {
  if (E <= 32) warp_select_topk_regs<1, NT>(rows, E, k, lane, id, w);
  else if (E <= 64) warp_select_topk_regs<2, NT>(rows, E, k, lane, id, w);
  else if (E <= 128) warp_select_topk_regs<4, NT>(rows, E, k, lane, id, w);
  else if (E <= 256) warp_select_topk_regs<8, NT>(rows, E, k, lane, id, w);
  else if (E <= 512) warp_select_topk_regs<16, NT>(rows, E, k, lane, id, w);
  else warp_select_topk_regs<32, NT>(rows, E, k, lane, id, w);
}

__device__ __forceinline__ void warp_select_topk(const float* row, int E, int k, int lane, int* id, float* w) {
  const float* const rows[1] = {row};
  int ids[1];
  float ws[1];
  warp_select_topk_n<1>(rows, E, k, lane, ids, ws);
  *id = ids[0];
  *w = ws[0];
}

}  // namespace moe
