// Router front end: logits = x . W_r (+ bias) and the top-k selection in one kernel.
//
// The paper leaves the router as it is (Sec. 7: routing, placement and dependencies unchanged); this is the
// step in front of the Dispatch bookkeeping of Sec. 4.3, for callers that hold the router matrix rather than logits.
//
// Arithmetic.  x is bf16, W_r is fp32.  W_r is split once into two bf16 terms W1 + W2 (W2 the bf16 rounding of what
// W1 left over: 16 significant bits together, relative error below 2^-17), so the product runs on the bf16 tensor
// path with every partial product exact in fp32.  A third term would restore all 24 bits but buys nothing: the
// tensor pipe's fp32 accumulation (addends aligned and truncated, about 2^-24 of the running sum per instruction)
// already leaves 3e-5 to 6e-5 at H = 4096 to 7168, above what the dropped bits contribute (about 5e-6).  The
// top-k is then taken on those fp32 values by the same warp selection the routing plan uses.
//
// Work.  Persistent CTAs (at most one per SM) draw items from one counter.  GEMM items come first: (128-token row
// tile, column tile of at most 128 experts, K split): TMA brings a stage of x[128 x 64] and the two weight terms
// [BN x 64] each, one thread issues 8 tcgen05.mma per stage into one TMEM accumulator, four warps write the fp32
// partial tile to the caller's scratch and the row tile's count moves.  Selection items follow: 32 tokens each; the
// CTA waits (bounded) until the row tile's partials are all there, adds them in split order, adds the bias, and
// its 16 warps select the top k per token and write ids, weights and, if asked, the logits.  The K split only
// spreads small batches over the SMs.
#include <cuda_bf16.h>

#include "moe_internal.h"
#include "ptx_sm100.cuh"
#include "route_select.cuh"

namespace {

constexpr int kThreads = 512;          // warp 0 TMA, warp 1 MMA, warps 2-5 epilogue; all sixteen reduce and select
constexpr int BM = 128;                // tokens per row tile
constexpr int BK = 64;                 // K elements per stage: one 128-byte swizzle row of bf16
constexpr int UMMA_K = 16;
constexpr int kTerms = 2;              // bf16 terms of the fp32 router matrix
constexpr int kABytes = BM * BK * 2;
constexpr int kMaxStages = 8;
constexpr int kRingBudget = 200 * 1024;
constexpr int kTmemCols = 128;         // one accumulator of at most 128 fp32 columns
constexpr int kMaxSplits = 8;
constexpr int kSelectTokens = 32;      // tokens of a selection item: two per warp; divides BM
constexpr int kSumBatch = 2;           // entries (16 bytes each where E % 4 == 0) a thread sums per batch, all splits in flight

struct RouterGeom {
  int BN;          // experts per column tile (multiple of 16, at most 128)
  int EpT;         // padded expert count = col_tiles * BN: row pitch of the partials, rows per weight term
  int col_tiles;
  int row_tiles;
  int S;           // K splits
  int k_blocks;    // H / 64
  int stages;
  int stage_bytes;
};

RouterGeom geometry(int T, int H, int E, int num_sms) {
  RouterGeom g{};
  const int e16 = (E + 15) / 16 * 16;
  g.col_tiles = (e16 + 127) / 128;
  g.BN = g.col_tiles > 1 ? 128 : e16;
  g.EpT = g.col_tiles * g.BN;
  g.row_tiles = (T + BM - 1) / BM;
  g.k_blocks = H / BK;
  const int tiles = g.row_tiles * g.col_tiles;
  int S = tiles > 0 ? num_sms / tiles : 1;
  if (S > kMaxSplits) S = kMaxSplits;
  if (S > g.k_blocks) S = g.k_blocks;
  if (S < 1) S = 1;
  g.S = S;
  g.stage_bytes = kABytes + kTerms * g.BN * BK * 2;
  g.stages = kRingBudget / g.stage_bytes;
  if (g.stages > kMaxStages) g.stages = kMaxStages;
  return g;
}

struct RouterParams {
  int T, E, k;
  RouterGeom g;
  const float* bias;       // [E] or null
  float* partials;         // [S][T][EpT] fp32
  float* logits_out;       // [T][E] or null
  int32_t* topk_ids;       // [T][k]
  float* topk_w;           // [T][k]
  int32_t* done;           // [row_tiles] partial tiles written so far, per row tile; zero at launch
  int32_t* ticket;         // work counter; zero at launch
  int32_t* status;         // device status word
};

struct RouterTail {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t tmem_full;
  uint32_t tmem_base;
  int abort_flag;
  int ticket;
};

__device__ __forceinline__ void router_timeout(const RouterParams& p, int where) {
  atomicCAS(&p.status[0], 0, MOE_ERR_TIMEOUT);
  atomicCAS(&p.status[1], 0, 100 + where);
}

// Bounded wait until *counter reaches `need` (an acquire load per poll); false when the budget ran out.
__device__ __forceinline__ bool wait_count(const int32_t* counter, int need, long long budget) {
  const long long t0 = clock64();
  for (;;) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
    if (v >= need) return true;
    if (clock64() - t0 > budget) return false;
    __nanosleep(200);
  }
}

__global__ void __launch_bounds__(kThreads, 1)
router_logits_topk(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
                   const RouterParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
  unsigned char* stage_base = smem_raw + pad;                 // 1024-byte aligned: required by the swizzle
  const uint32_t stage_u32 = raw + pad;
  const RouterGeom& g = p.g;
  RouterTail* st = reinterpret_cast<RouterTail*>(stage_base + static_cast<size_t>(g.stages) * g.stage_bytes);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b_bytes = g.BN * BK * 2;                           // one weight term of a stage
  const int gemm_items = g.row_tiles * g.col_tiles * g.S;
  const int select_items = (p.T + kSelectTokens - 1) / kSelectTokens;

  if (tid == 0) {
    for (int s = 0; s < g.stages; ++s) {
      ptx::mbar_init(ptx::smem_u32(&st->full[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&st->empty[s]), 1);
    }
    ptx::mbar_init(ptx::smem_u32(&st->tmem_full), 1);
    st->abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::fence_proxy_async_smem();
  }
  if (warp == 0 && lane == 0) {
    ptx::prefetch_tensormap(&tm_x);
    ptx::prefetch_tensormap(&tm_w);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(&st->tmem_base), kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = st->tmem_base;
  volatile int* abort_flag = &st->abort_flag;

  // Ring and accumulator state of the roles; it runs on from one GEMM item of this CTA to the next.
  int stage = 0;
  uint32_t phase = 0;
  uint32_t acc_phase = 0;

  // Work is drawn from one ticket counter: first every GEMM item, then every selection item.  A selection item
  // waits for the partial tiles of its row tile; whoever holds those GEMM tickets is running and waits for nothing,
  // so the wait ends whatever the order in which CTAs reach the SMs.
  for (;;) {
    if (tid == 0) st->ticket = atomicAdd(p.ticket, 1);
    __syncthreads();
    const int ticket = st->ticket;
    if (ticket >= gemm_items + select_items || st->abort_flag) break;

    if (ticket < gemm_items) {
      const int split = ticket % g.S;
      const int col_tile = (ticket / g.S) % g.col_tiles;
      const int row_tile = ticket / (g.S * g.col_tiles);
      const int row0 = row_tile * BM;
      const int kb0 = static_cast<int>(static_cast<long long>(split) * g.k_blocks / g.S);
      const int kb1 = static_cast<int>(static_cast<long long>(split + 1) * g.k_blocks / g.S);
      if (warp == 0) {
        // -------------------------------------------------------------- TMA producer
        if (lane == 0) {
          for (int kb = kb0; kb < kb1; ++kb) {
            if (!ptx::mbar_wait(ptx::smem_u32(&st->empty[stage]), phase ^ 1u, abort_flag)) {
              router_timeout(p, 1);
              break;
            }
            const uint32_t full = ptx::smem_u32(&st->full[stage]);
            const uint32_t sa = stage_u32 + stage * g.stage_bytes;
            ptx::mbar_expect_tx(full, g.stage_bytes);
            ptx::tma_load_2d(sa, &tm_x, full, kb * BK, row0);
#pragma unroll
            for (int term = 0; term < kTerms; ++term)
              ptx::tma_load_2d(sa + kABytes + term * b_bytes, &tm_w, full, kb * BK, term * g.EpT + col_tile * g.BN);
            if (++stage == g.stages) { stage = 0; phase ^= 1u; }
          }
        }
        __syncwarp();
      } else if (warp == 1) {
        // -------------------------------------------------------------- MMA issuer
        if (lane == 0) {
          const uint32_t idesc = ptx::idesc_bf16_f32(BM, g.BN);
          bool ok = true;
          ptx::tc_fence_after_sync();
          for (int kb = kb0; kb < kb1; ++kb) {
            if (!ptx::mbar_wait(ptx::smem_u32(&st->full[stage]), phase, abort_flag)) {
              router_timeout(p, 2);
              ok = false;
              break;
            }
            ptx::tc_fence_after_sync();
            const uint32_t sa = stage_u32 + stage * g.stage_bytes;
            const uint64_t a_desc = ptx::smem_desc_sw128(sa);
#pragma unroll
            for (int term = 0; term < kTerms; ++term) {
              const uint64_t b_desc = ptx::smem_desc_sw128(sa + kABytes + term * b_bytes);
#pragma unroll
              for (int k4 = 0; k4 < BK / UMMA_K; ++k4) {
                const uint64_t adv = static_cast<uint64_t>(2 * k4);   // +32 bytes along K inside the swizzle row
                ptx::tc_mma_bf16(tmem_base, a_desc + adv, b_desc + adv, idesc,
                                 (kb > kb0 || term > 0 || k4 > 0) ? 1u : 0u);
              }
            }
            ptx::tc_commit(ptx::smem_u32(&st->empty[stage]));
            if (++stage == g.stages) { stage = 0; phase ^= 1u; }
          }
          if (ok) ptx::tc_commit(ptx::smem_u32(&st->tmem_full));
        }
        __syncwarp();
      } else if (warp < 6) {
        // -------------------------------------------------------------- epilogue: partial tile to scratch
        const int quarter = warp & 3;                 // TMEM lane quarter this warp may read
        const int row = row0 + quarter * 32 + lane;
        if (!ptx::mbar_wait(ptx::smem_u32(&st->tmem_full), acc_phase, abort_flag)) {
          if (lane == 0) router_timeout(p, 3);
        } else {
          ptx::tc_fence_after_sync();
          const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
          float* dst = p.partials + (static_cast<size_t>(split) * p.T + row) * g.EpT + col_tile * g.BN;
          for (int c0 = 0; c0 < g.BN; c0 += 16) {
            uint32_t v[16];
            ptx::tmem_ld_32x16(t_addr + c0, v);
            ptx::tmem_ld_wait();
            if (row < p.T) {
#pragma unroll
              for (int i = 0; i < 16; i += 4)
                *reinterpret_cast<uint4*>(dst + c0 + i) = make_uint4(v[i], v[i + 1], v[i + 2], v[i + 3]);
            }
          }
          ptx::tc_fence_before_sync();
        }
      }
      acc_phase ^= 1u;
      // publish: the partial tile is visible before the row tile's count moves
      __threadfence();
      __syncthreads();
      if (tid == 0 && !st->abort_flag) atomicAdd(&p.done[row_tile], 1);
    } else {
      // ---------------------------------------------------------------- selection item: kSelectTokens tokens
      const int t0 = (ticket - gemm_items) * kSelectTokens;
      const int n_rows = min(kSelectTokens, p.T - t0);
      if (tid == 0 && !wait_count(&p.done[t0 / BM], g.col_tiles * g.S, ptx::kWaitClockBudget)) {
        router_timeout(p, 4);
        st->abort_flag = 1;
      }
      __syncthreads();
      if (st->abort_flag) break;
      __threadfence();
      // The ring is idle (every stage this CTA loaded has been consumed): it holds the summed logits of the item.
      float* rows = reinterpret_cast<float*>(stage_base);
      const size_t split_pitch = static_cast<size_t>(p.T) * g.EpT;
      const float* part = p.partials + static_cast<size_t>(t0) * g.EpT;
      // all warps: partials summed in split order, then the bias; coalesced along e.  Every load of a batch (all
      // splits of kSumBatch entries) is issued before anything is added or stored, so that they are in flight
      // together; splits beyond S contribute an exact +0.
      if ((p.E & 3) == 0) {
        const int e4 = p.E >> 2;
        const int n4 = n_rows * e4;
        for (int base = 0; base < n4; base += kThreads * kSumBatch) {
          float4 a[kSumBatch][kMaxSplits];
#pragma unroll
          for (int u = 0; u < kSumBatch; ++u) {
            const int i = base + u * kThreads + tid;
            const int r = i / e4;
            const float* src = part + r * g.EpT + 4 * (i - r * e4);
#pragma unroll
            for (int s = 0; s < kMaxSplits; ++s)
              a[u][s] = (i < n4 && s < g.S) ? __ldcg(reinterpret_cast<const float4*>(src + s * split_pitch))
                                            : make_float4(0.f, 0.f, 0.f, 0.f);
          }
#pragma unroll
          for (int u = 0; u < kSumBatch; ++u) {
            const int i = base + u * kThreads + tid;
            if (i >= n4) continue;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int s = 0; s < kMaxSplits; ++s) { v.x += a[u][s].x; v.y += a[u][s].y; v.z += a[u][s].z; v.w += a[u][s].w; }
            if (p.bias != nullptr) {
              const float4 bb = *reinterpret_cast<const float4*>(p.bias + 4 * (i % e4));
              v.x += bb.x; v.y += bb.y; v.z += bb.z; v.w += bb.w;
            }
            reinterpret_cast<float4*>(rows)[i] = v;
            if (p.logits_out != nullptr)
              reinterpret_cast<float4*>(p.logits_out + static_cast<size_t>(t0) * p.E)[i] = v;
          }
        }
      } else {
        const int n = n_rows * p.E;
        for (int base = 0; base < n; base += kThreads * kSumBatch) {
          float a[kSumBatch][kMaxSplits];
#pragma unroll
          for (int u = 0; u < kSumBatch; ++u) {
            const int i = base + u * kThreads + tid;
            const int r = i / p.E;
            const float* src = part + r * g.EpT + (i - r * p.E);
#pragma unroll
            for (int s = 0; s < kMaxSplits; ++s) a[u][s] = (i < n && s < g.S) ? __ldcg(src + s * split_pitch) : 0.f;
          }
#pragma unroll
          for (int u = 0; u < kSumBatch; ++u) {
            const int i = base + u * kThreads + tid;
            if (i >= n) continue;
            float v = 0.f;
#pragma unroll
            for (int s = 0; s < kMaxSplits; ++s) v += a[u][s];
            if (p.bias != nullptr) v += p.bias[i % p.E];
            rows[i] = v;
            if (p.logits_out != nullptr) p.logits_out[static_cast<size_t>(t0) * p.E + i] = v;
          }
        }
      }
      __syncthreads();
      // two tokens per warp, selected together: rows warp and warp + 16 of the item
      {
        static_assert(kSelectTokens == 2 * (kThreads / 32), "a selection item is two tokens per warp");
        const int r0 = warp, r1 = warp + kThreads / 32;
        if (r1 < n_rows) {
          const float* const two[2] = {rows + r0 * p.E, rows + r1 * p.E};
          int ids[2];
          float ws[2];
          moe::warp_select_topk_n<2>(two, p.E, p.k, lane, ids, ws);
          if (lane < p.k) {
            const size_t s0 = static_cast<size_t>(t0 + r0) * p.k + lane, s1 = static_cast<size_t>(t0 + r1) * p.k + lane;
            p.topk_ids[s0] = ids[0];
            p.topk_w[s0] = ws[0];
            p.topk_ids[s1] = ids[1];
            p.topk_w[s1] = ws[1];
          }
        } else if (r0 < n_rows) {
          int sel_id;
          float sel_w;
          moe::warp_select_topk(rows + r0 * p.E, p.E, p.k, lane, &sel_id, &sel_w);
          if (lane < p.k) {
            const size_t s0 = static_cast<size_t>(t0 + r0) * p.k + lane;
            p.topk_ids[s0] = sel_id;
            p.topk_w[s0] = sel_w;
          }
        }
      }
    }
    __syncthreads();   // the ticket slot and the ring are reused by the next item
  }

  __syncthreads();
  if (st->abort_flag) {
    // a wait gave up: give copies still in flight time to land before the shared memory is released
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

// W_r [H,E] fp32 -> kTerms bf16 terms, each [EpT, H] with H contiguous (rows e >= E are zero).
__global__ void __launch_bounds__(256)
router_split_weights(const float* __restrict__ w_router, int H, int E, int EpT, __nv_bfloat16* __restrict__ out) {
  const long long idx = static_cast<long long>(blockIdx.x) * 256 + threadIdx.x;
  const long long n = static_cast<long long>(EpT) * H;
  if (idx >= n) return;
  const int h = static_cast<int>(idx % H);
  const int e = static_cast<int>(idx / H);
  const float w = e < E ? w_router[static_cast<size_t>(h) * E + e] : 0.f;
  const __nv_bfloat16 b1 = __float2bfloat16_rn(w);
  const float r1 = w - __bfloat162float(b1);           // exact: the difference fits an fp32
  const __nv_bfloat16 b2 = __float2bfloat16_rn(r1);
  static_assert(kTerms == 2, "the split below writes two terms");
  out[idx] = b1;
  out[n + idx] = b2;
}

CUresult encode_rows(moe_ctx* ctx, CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(BK), box_rows};
  const cuuint32_t elem[2] = {1u, 1u};
  return ctx->encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

}  // namespace

namespace moe {

size_t router_weight_bytes(const moe_shape& s) {
  const RouterGeom g = geometry(s.T, s.H, s.E, 1);
  return static_cast<size_t>(kTerms) * g.EpT * s.H * 2;
}

size_t router_scratch_bytes(const moe_shape& s) {
  const RouterGeom g = geometry(s.T, s.H, s.E, 1);
  return static_cast<size_t>(kMaxSplits) * s.T * g.EpT * 4;
}

cudaError_t launch_router_prepare(moe_ctx* ctx, const float* w_router, void* w_split, cudaStream_t stream) {
  const moe_shape& s = ctx->shape;
  const RouterGeom g = geometry(s.T, s.H, s.E, ctx->num_sms);
  const long long n = static_cast<long long>(g.EpT) * s.H;
  router_split_weights<<<static_cast<unsigned>((n + 255) / 256), 256, 0, stream>>>(
      w_router, s.H, s.E, g.EpT, static_cast<__nv_bfloat16*>(w_split));
  ctx->last_launches += 1;
  return cudaGetLastError();
}

moe_status launch_router(moe_ctx* ctx, const void* x, const void* w_split, const float* bias, void* scratch,
                         float* logits_out, int32_t* topk_ids, float* topk_w, cudaStream_t stream) {
  const moe_shape& s = ctx->shape;
  const RouterGeom g = geometry(s.T, s.H, s.E, ctx->num_sms);
  CUtensorMap tm_x, tm_w;
  if (encode_rows(ctx, &tm_x, x, s.T, s.H, BM) != CUDA_SUCCESS) return MOE_ERR_CUDA;
  if (encode_rows(ctx, &tm_w, w_split, static_cast<uint64_t>(kTerms) * g.EpT, s.H, g.BN) != CUDA_SUCCESS)
    return MOE_ERR_CUDA;
  RouterParams p{};
  p.T = s.T;
  p.E = s.E;
  p.k = s.k;
  p.g = g;
  p.bias = bias;
  p.partials = static_cast<float*>(scratch);
  p.logits_out = logits_out;
  p.topk_ids = topk_ids;
  p.topk_w = topk_w;
  p.ticket = ctx->d_router_done;           // word 0: the ticket counter, then one count per row tile
  p.done = ctx->d_router_done + 1;
  p.status = ctx->d_status;
  if (cudaMemsetAsync(ctx->d_router_done, 0, static_cast<size_t>(g.row_tiles + 1) * 4, stream) != cudaSuccess)
    return MOE_ERR_CUDA;
  const size_t smem = 1024 + static_cast<size_t>(g.stages) * g.stage_bytes + sizeof(RouterTail);
  const int items = g.row_tiles * g.col_tiles * g.S + (s.T + kSelectTokens - 1) / kSelectTokens;
  const int grid = items < ctx->num_sms ? items : ctx->num_sms;   // persistent: at most one CTA per SM
  router_logits_topk<<<grid, kThreads, smem, stream>>>(tm_x, tm_w, p);
  ctx->last_launches += 1;
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

cudaError_t prepare_router(moe_ctx* ctx) {
  (void)ctx;
  return cudaFuncSetAttribute(router_logits_topk, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              1024 + kRingBudget + static_cast<int>(sizeof(RouterTail)));
}

}  // namespace moe
