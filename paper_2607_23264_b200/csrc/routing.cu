// Routing plan: top-k + softmax weights, per-expert histogram, exclusive scan, stable permutation.
//
// The token range is cut into chunks of `tokens_per_chunk` tokens (at most 256 slots).  Three launches:
//   1. route_topk_hist : one CTA per chunk; a warp per token selects the k largest logits by k passes of
//                        warp arg-max (integer warp reductions on order-preserving keys, ties to the lower
//                        index) and computes the softmax weights; the CTA then histograms its slots per expert.
//   2. route_scan      : one CTA; exclusive prefix of the chunk histograms over chunks (per expert) and
//                        the exclusive scan of the totals over experts (offsets).
//   3. route_scatter   : one CTA per chunk, one thread per slot; the stable rank of a slot among the
//                        slots of its expert is (slots of earlier chunks) + (slots of earlier warps in
//                        the chunk) + (earlier lanes in the warp, from a match-any ballot).
// Everything is integer work on identical fp32 inputs, so ids, counts, offsets and both permutations are
// reproducible bit for bit.
#include <atomic>

#include "moe_internal.h"
#include "route_select.cuh"

namespace {

constexpr unsigned kFull = 0xFFFFFFFFu;

__global__ void __launch_bounds__(kRouteThreads)
route_topk_hist(const float* __restrict__ logits, int T, int E, int k, int tokens_per_chunk,
                int32_t* __restrict__ topk_ids, float* __restrict__ topk_w, int32_t* __restrict__ chunk_hist) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int warps = kRouteThreads / 32;
  int32_t* s_hist = reinterpret_cast<int32_t*>(smem_raw);                 // [E]
  int32_t* s_ids = s_hist + E;                                            // [256]

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int chunk = blockIdx.x;
  const int t_begin = chunk * tokens_per_chunk;
  const int t_end = min(T, t_begin + tokens_per_chunk);

  for (int e = tid; e < E; e += kRouteThreads) s_hist[e] = 0;

  for (int t = t_begin + warp; t < t_end; t += warps) {
    int sel_id;
    float sel_w;
    moe::warp_select_topk(logits + static_cast<size_t>(t) * E, E, k, lane, &sel_id, &sel_w);
    if (lane < k) {
      const size_t s = static_cast<size_t>(t) * k + lane;
      topk_ids[s] = sel_id;
      topk_w[s] = sel_w;
      s_ids[(t - t_begin) * k + lane] = sel_id;
    }
  }
  __syncthreads();
  const int n_slots = (t_end - t_begin) * k;
  if (tid < n_slots) atomicAdd(&s_hist[s_ids[tid]], 1);   // integer counts: order does not matter
  __syncthreads();
  for (int e = tid; e < E; e += kRouteThreads) chunk_hist[static_cast<size_t>(chunk) * E + e] = s_hist[e];
}

// Histogram of externally supplied expert ids (same chunking as route_topk_hist).  An id outside [0, E) violates
// the contract: it is reported through the status word and counted as expert 0 so that nothing is written out of
// bounds; the plan is then meaningless.
__global__ void __launch_bounds__(kRouteThreads)
route_hist_ids(const int32_t* __restrict__ topk_ids, int T, int E, int k, int tokens_per_chunk,
               int32_t* __restrict__ ids_checked, int32_t* __restrict__ chunk_hist, int32_t* __restrict__ status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  int32_t* s_hist = reinterpret_cast<int32_t*>(smem_raw);   // [E]
  const int tid = threadIdx.x, chunk = blockIdx.x;
  const int t_begin = chunk * tokens_per_chunk;
  const int t_end = min(T, t_begin + tokens_per_chunk);
  const int n_slots = (t_end - t_begin) * k;
  for (int e = tid; e < E; e += kRouteThreads) s_hist[e] = 0;
  __syncthreads();
  if (tid < n_slots) {
    const size_t s = static_cast<size_t>(t_begin) * k + tid;
    int e = topk_ids[s];
    if (e < 0 || e >= E) {
      atomicCAS(&status[0], 0, MOE_ERR_BAD_ROUTING);
      atomicCAS(&status[1], 0, static_cast<int>(s));
      e = 0;
    }
    ids_checked[s] = e;
    atomicAdd(&s_hist[e], 1);
  }
  __syncthreads();
  for (int e = tid; e < E; e += kRouteThreads) chunk_hist[static_cast<size_t>(chunk) * E + e] = s_hist[e];
}

// One CTA of 1024 threads, E <= 1024.  With few experts (at least 8 threads per expert) and at least 64 chunks the
// chunks are cut into
// S = min(1024 / E, num_chunks) segments; thread (expert e, segment s) = e + s * E sums its segment (independent
// loads, consecutive e side by side), the segment sums are scanned over s in shared memory, then the thread writes
// the exclusive prefixes of its chunks.  With many experts one thread per expert walks all chunks once.  A block scan
// over the experts' totals gives the offsets.
__global__ void __launch_bounds__(1024)
route_scan(const int32_t* __restrict__ chunk_hist, int32_t* __restrict__ chunk_base, int num_chunks, int E,
           int32_t* __restrict__ counts, int32_t* __restrict__ offsets) {
  __shared__ int32_t s_warp[32];
  __shared__ int32_t s_seg[2][1024];      // [buffer][s * E + e]: inclusive scan over s, ping-pong
  __shared__ int32_t s_total[1024];       // per expert
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  int S = 1024 / E;
  if (S > num_chunks) S = num_chunks;
  if (S < 1) S = 1;
  // many experts or few chunks: one thread per expert walks all chunks once (no second pass, no segment scan)
  if (S < 8 || num_chunks < 64) S = 1;
  const int seg_len = (num_chunks + S - 1) / S;
  const int e_of = tid % E, seg = tid / E;
  const bool active = seg < S;
  const int c_begin = seg * seg_len;
  const int c_end = min(num_chunks, c_begin + seg_len);
  int32_t sum = 0;
  if (S == 1) {
    // single pass: the prefix is written while summing
    if (active) {
      int c = 0;
      for (; c + 8 <= num_chunks; c += 8) {
        int32_t v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = chunk_hist[static_cast<size_t>(c + u) * E + e_of];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          chunk_base[static_cast<size_t>(c + u) * E + e_of] = sum;
          sum += v[u];
        }
      }
      for (; c < num_chunks; ++c) {
        const size_t i = static_cast<size_t>(c) * E + e_of;
        const int32_t v = chunk_hist[i];
        chunk_base[i] = sum;
        sum += v;
      }
      s_total[e_of] = sum;
    }
  } else if (active) {
    int c = c_begin;
    for (; c + 8 <= c_end; c += 8) {        // eight independent loads per step
      int32_t v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = chunk_hist[static_cast<size_t>(c + u) * E + e_of];
#pragma unroll
      for (int u = 0; u < 8; ++u) sum += v[u];
    }
    for (; c < c_end; ++c) sum += chunk_hist[static_cast<size_t>(c) * E + e_of];
    s_seg[0][tid] = sum;
  }
  __syncthreads();
  // inclusive scan over the segments of each expert (entries e + s * E, stride E); nothing to do for one segment
  int cur = 0;
  for (int off = 1; off < S; off <<= 1) {
    if (active) {
      int32_t v = s_seg[cur][tid];
      if (seg >= off) v += s_seg[cur][tid - off * E];
      s_seg[cur ^ 1][tid] = v;
    }
    cur ^= 1;
    __syncthreads();
  }
  if (active && S > 1) {
    int32_t running = s_seg[cur][tid] - sum;                 // slots of this expert in earlier segments
    int c = c_begin;
    for (; c + 8 <= c_end; c += 8) {        // eight loads in flight, then the eight prefixes
      int32_t v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = chunk_hist[static_cast<size_t>(c + u) * E + e_of];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        chunk_base[static_cast<size_t>(c + u) * E + e_of] = running;
        running += v[u];
      }
    }
    for (; c < c_end; ++c) {
      const size_t i = static_cast<size_t>(c) * E + e_of;
      const int32_t v = chunk_hist[i];
      chunk_base[i] = running;
      running += v;
    }
    if (seg == S - 1) s_total[e_of] = s_seg[cur][tid];       // inclusive over all segments = the expert's count
  }
  __syncthreads();
  const int e = tid;
  int32_t total = 0;
  if (e < E) {
    total = s_total[e];
    counts[e] = total;
  }
  int32_t incl = total;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int32_t o = __shfl_up_sync(kFull, incl, off);
    if (lane >= off) incl += o;
  }
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int32_t w = s_warp[lane];
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int32_t o = __shfl_up_sync(kFull, w, off);
      if (lane >= off) w += o;
    }
    s_warp[lane] = w;   // inclusive over warps
  }
  __syncthreads();
  const int32_t before = (warp ? s_warp[warp - 1] : 0) + incl - total;   // exclusive prefix of counts
  if (e < E) offsets[e] = before;
  if (e == E - 1) offsets[E] = before + total;
}

__global__ void __launch_bounds__(kRouteThreads)
route_scatter(const int32_t* __restrict__ topk_ids, const int32_t* __restrict__ offsets,
              const int32_t* __restrict__ chunk_base, int T, int E, int k, int tokens_per_chunk,
              int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int warps = kRouteThreads / 32;
  int32_t* s_warp_cnt = reinterpret_cast<int32_t*>(smem_raw);   // [warps][E]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int chunk = blockIdx.x;
  const int t_begin = chunk * tokens_per_chunk;
  const int t_end = min(T, t_begin + tokens_per_chunk);
  const int n_slots = (t_end - t_begin) * k;
  const int s = t_begin * k + tid;

  for (int i = tid; i < warps * E; i += kRouteThreads) s_warp_cnt[i] = 0;
  __syncthreads();

  const bool active = tid < n_slots;
  const int e = active ? topk_ids[s] : (E + lane);   // idle lanes get distinct keys outside [0,E)
  const unsigned same = __match_any_sync(kFull, e);
  const int rank_in_warp = __popc(same & ((1u << lane) - 1u));
  if (active && rank_in_warp == 0) s_warp_cnt[warp * E + e] = __popc(same);
  __syncthreads();
  if (active) {
    int before = 0;
    for (int w = 0; w < warp; ++w) before += s_warp_cnt[w * E + e];
    const int row = offsets[e] + chunk_base[static_cast<size_t>(chunk) * E + e] + before + rank_in_warp;
    perm[row] = s;
    inv_perm[s] = row;
  }
}

}  // namespace

namespace moe {

cudaError_t launch_plan_routing(moe_ctx* ctx, const float* logits, int32_t* topk_ids, float* topk_w,
                                int32_t* counts, int32_t* offsets, int32_t* perm, int32_t* inv_perm,
                                cudaStream_t stream) {
  const moe_shape& s = ctx->shape;
  const int warps = kRouteThreads / 32;
  const size_t smem1 = (static_cast<size_t>(s.E) + 256) * 4;
  const size_t smem3 = static_cast<size_t>(warps) * s.E * 4;
  route_topk_hist<<<ctx->num_chunks, kRouteThreads, smem1, stream>>>(logits, s.T, s.E, s.k, ctx->tokens_per_chunk,
                                                                     topk_ids, topk_w, ctx->d_chunk_hist);
  moe_mark(ctx, 1, stream);
  route_scan<<<1, 1024, 0, stream>>>(ctx->d_chunk_hist, ctx->d_chunk_base, ctx->num_chunks, s.E, counts, offsets);
  moe_mark(ctx, 2, stream);
  route_scatter<<<ctx->num_chunks, kRouteThreads, smem3, stream>>>(topk_ids, offsets, ctx->d_chunk_base, s.T, s.E,
                                                                   s.k, ctx->tokens_per_chunk, perm, inv_perm);
  moe_mark(ctx, 3, stream);
  ctx->last_launches += 3;
  return cudaGetLastError();
}

cudaError_t launch_plan_from_topk(moe_ctx* ctx, const int32_t* topk_ids, int32_t* ids_checked, int32_t* counts,
                                  int32_t* offsets, int32_t* perm, int32_t* inv_perm, cudaStream_t stream) {
  const moe_shape& s = ctx->shape;
  const int warps = kRouteThreads / 32;
  route_hist_ids<<<ctx->num_chunks, kRouteThreads, static_cast<size_t>(s.E) * 4, stream>>>(
      topk_ids, s.T, s.E, s.k, ctx->tokens_per_chunk, ids_checked, ctx->d_chunk_hist, ctx->d_status);
  moe_mark(ctx, 1, stream);
  route_scan<<<1, 1024, 0, stream>>>(ctx->d_chunk_hist, ctx->d_chunk_base, ctx->num_chunks, s.E, counts, offsets);
  moe_mark(ctx, 2, stream);
  route_scatter<<<ctx->num_chunks, kRouteThreads, static_cast<size_t>(warps) * s.E * 4, stream>>>(
      ids_checked, offsets, ctx->d_chunk_base, s.T, s.E, s.k, ctx->tokens_per_chunk, perm, inv_perm);
  moe_mark(ctx, 3, stream);
  ctx->last_launches += 3;
  return cudaGetLastError();
}

}  // namespace moe


// ------------------------------------------------------------------------------------------------
// Routing plan without any allocation: same three kernels, scratch in a file-scope device array.
// ------------------------------------------------------------------------------------------------
namespace {

// Largest num_chunks * E the static scratch holds (two arrays of this many int32: 512 KiB in total,
// resident on every GPU that loads the library until the process exits).
constexpr int kStaticScratchInts = 65536;
static __device__ __align__(256) int32_t g_route_static_scratch[2 * kStaticScratchInts];

constexpr int kMaxDevices = 64;
// device address of the array, per device, once resolved (host threads may race to resolve it: they store the
// same value)
std::atomic<int32_t*> g_route_static_addr[kMaxDevices];

// Set-up, once per device, with that device current: in host code the array's name is only a stand-in, the address
// a kernel may use comes from cudaGetSymbolAddress.  Returns nullptr on failure.
int32_t* static_scratch_address() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  int32_t* scratch = g_route_static_addr[dev].load(std::memory_order_acquire);
  if (!scratch) {
    void* addr = nullptr;
    if (cudaGetSymbolAddress(&addr, g_route_static_scratch) != cudaSuccess || !addr) return nullptr;
    scratch = static_cast<int32_t*>(addr);
    g_route_static_addr[dev].store(scratch, std::memory_order_release);
  }
  return scratch;
}

}  // namespace

extern "C" moe_status moe_plan_routing_static(const moe_shape* shape, const float* logits, int32_t* topk_ids,
                                              float* topk_w, int32_t* counts, int32_t* offsets, int32_t* perm,
                                              int32_t* inv_perm, void* stream) {
  if (!shape) return MOE_ERR_INVALID_ARG;
  if (shape->ep_size != 1 || shape->ep_rank != 0) return MOE_ERR_UNSUPPORTED;
  if (shape->T < 0 || shape->E <= 0 || shape->k <= 0 || shape->E > 1024 || shape->k > 32 || shape->k > shape->E)
    return MOE_ERR_UNSUPPORTED_SHAPE;
  if (!counts || !offsets) return MOE_ERR_INVALID_ARG;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const int T = shape->T, E = shape->E, k = shape->k;
  // resolved before anything else that can succeed, so that any first call (an empty batch included) is the set-up
  int32_t* scratch = static_scratch_address();
  if (!scratch) return MOE_ERR_CUDA;
  if (T == 0) {
    if (cudaMemsetAsync(counts, 0, static_cast<size_t>(E) * 4, cs) != cudaSuccess) return MOE_ERR_CUDA;
    if (cudaMemsetAsync(offsets, 0, static_cast<size_t>(E + 1) * 4, cs) != cudaSuccess) return MOE_ERR_CUDA;
    return MOE_OK;
  }
  if (!logits || !topk_ids || !topk_w || !perm || !inv_perm) return MOE_ERR_INVALID_ARG;
  const void* ptrs[] = {logits, topk_ids, topk_w, counts, offsets, perm, inv_perm};
  for (const void* q : ptrs)
    if (reinterpret_cast<uintptr_t>(q) & 15u) return MOE_ERR_INVALID_ARG;

  const int tokens_per_chunk = kRouteThreads / k;
  const long long num_chunks = (static_cast<long long>(T) + tokens_per_chunk - 1) / tokens_per_chunk;
  if (num_chunks * E > kStaticScratchInts) return MOE_ERR_STATIC_SCRATCH_TOO_SMALL;

  int32_t* chunk_hist = scratch;                        // [num_chunks, E], every entry rewritten by kernel 1
  int32_t* chunk_base = scratch + kStaticScratchInts;   // [num_chunks, E], every entry rewritten by kernel 2

  const int warps = kRouteThreads / 32;
  const size_t smem1 = (static_cast<size_t>(E) + 256) * 4;
  const size_t smem3 = static_cast<size_t>(warps) * E * 4;
  const int nc = static_cast<int>(num_chunks);
  route_topk_hist<<<nc, kRouteThreads, smem1, cs>>>(logits, T, E, k, tokens_per_chunk, topk_ids, topk_w, chunk_hist);
  route_scan<<<1, 1024, 0, cs>>>(chunk_hist, chunk_base, nc, E, counts, offsets);
  route_scatter<<<nc, kRouteThreads, smem3, cs>>>(topk_ids, offsets, chunk_base, T, E, k, tokens_per_chunk, perm,
                                                  inv_perm);
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}
