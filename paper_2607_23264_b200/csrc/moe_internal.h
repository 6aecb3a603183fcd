// Internal declarations shared by the translation units of the library (not part of the C ABI).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/moe.h"

// Rows per M tile of the grouped GEMM and slots per routing chunk.
constexpr int kRouteThreads = 256;
// Kernels of one forward, in launch order: top-k+histogram, scan, scatter, dispatch, Linear-1, Linear-2, combine.
constexpr int kMoeKernels = 7;
constexpr int kMoeTimingSlots = 32;   // calls whose per-kernel events are kept (a ring: one slot per timed call)
// Wait counters one CTA of a grouped GEMM records when tracing is on (SM clocks unless noted):
// 0 producer loop span, 1 producer waited for a free stage, 2 MMA waited for data, 3 MMA waited for a free
// accumulator (the epilogue's back-pressure), 4 epilogue waited for an accumulator, 5 epilogue drain+store span,
// 6 tiles processed (count), 7 epilogue held by the pacing gap; and, by the MMA warp, per tile class: 8 tiles computed
// with swapped operands (count), 9 their time from the first operand wait to the last MMA issued, 10 the part of it
// spent waiting for operands, 11 the time of the other (full 128-row) tiles.
constexpr int kMoeTraceFields = 12;
// Tile codes (phase << 30 | index in the phase's tile list, -1 = end) a CTA logs when tracing a one-launch run.
constexpr int kMoeOrderLogCap = 512;

typedef CUresult (*moe_encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                        const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                        CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                        CUtensorMapFloatOOBfill);

// Development knobs given as "x.<name>=<int>" entries of the MOE_TUNING environment variable (see moe_create).
constexpr int kMoeMaxKnobs = 16;
struct moe_knob {
  char name[24];
  int32_t value;
};

// Tensor maps the grouped GEMMs built for recent calls (see tensor_map_2d).
constexpr int kMoeMapCache = 24;
struct moe_map_entry {
  const void* base;
  uint64_t rows, cols;
  int elem_bytes, box_rows;
  CUtensorMap map;
};

struct moe_ctx {
  moe_shape shape;
  int has_env_tuning;    // MOE_TUNING named at least one moe_tuning field: env_tuning replaces the defaults of a
  moe_tuning env_tuning; // call that passes tuning = NULL
  int num_knobs;
  moe_knob knobs[kMoeMaxKnobs];
  int device;
  int num_sms;
  int max_pairs;         // CTA pairs (clusters of two) of the pair kernel that can be resident at once
  int max_tokens;        // T given at creation: the size of the routing scratch; shape.T is the active batch
  int tokens_per_chunk;  // routing: tokens handled by one CTA, so that a chunk has at most 256 slots
  int num_chunks;
  int32_t* d_chunk_hist;  // [num_chunks, E] slots of each chunk per expert
  int32_t* d_chunk_base;  // [num_chunks, E] exclusive prefix of d_chunk_hist over chunks
  int32_t* d_status;      // [2] device status word: code, detail
  int32_t* d_sched;       // [4] tile scheduler of the two grouped GEMMs: {next tile, CTAs done} each; zero when idle
  int32_t* d_ready;       // [T*k/128 + E + 1] per 128-row block: Linear-1 warps that published its h rows; zero when idle
  int32_t* d_router_done; // [1 + T/128 + 1] router front end: work ticket, then partial tiles written per row tile
  int32_t* d_order;       // [num_sms][kMoeOrderLogCap] tile codes drawn by each CTA in the last traced one-launch run
  unsigned long long* d_trace;   // [2][num_sms][kMoeTraceFields] wait counters of Linear-1 and Linear-2
  moe_encode_tiled_fn encode_tiled;
  int num_maps;
  unsigned next_map_victim;
  moe_map_entry maps[kMoeMapCache];
  int32_t last_launches;
  // Two-deep pipeline of moe_fused_forward_host_pipelined: copy streams, per-slot events, next slot.
  cudaStream_t s_h2d, s_d2h;
  cudaEvent_t ev_h2d[2], ev_compute[2], ev_d2h[2];
  int pipe_slot;
  // Optional per-kernel timing: event i is recorded after kernel i (event 0 before the first kernel).
  int timing;
  int ev_slot;                                  // slot of the last timed call
  uint32_t ev_recorded[kMoeTimingSlots];        // bit i set when ev[slot][i] was recorded by that slot's call
  cudaEvent_t ev[kMoeTimingSlots][kMoeKernels + 1];
};

// Value of the development knob "x.<name>" from MOE_TUNING, or dflt.
inline int moe_knob_value(const moe_ctx* ctx, const char* name, int dflt) {
  for (int i = 0; i < ctx->num_knobs; ++i) {
    const char *a = ctx->knobs[i].name, *b = name;
    while (*a && *a == *b) { ++a; ++b; }
    if (*a == 0 && *b == 0) return ctx->knobs[i].value;
  }
  return dflt;
}

// The tuning a call runs with: the caller's, else the one MOE_TUNING gave at moe_create, else the built-in default.
inline moe_tuning moe_effective_tuning(const moe_ctx* ctx, const moe_tuning* given) {
  if (given) return *given;
  if (ctx->has_env_tuning) return ctx->env_tuning;
  return moe_tuning{1, 0, 1, 0, 0, 0};
}

// Record timing mark i on the stream when per-kernel timing is enabled.
inline void moe_mark(moe_ctx* ctx, int i, cudaStream_t stream) {
  if (ctx->timing && cudaEventRecord(ctx->ev[ctx->ev_slot][i], stream) == cudaSuccess)
    ctx->ev_recorded[ctx->ev_slot] |= 1u << i;
}

// Launchers (each returns the cudaError_t of its launches).  `stream` is the caller's stream.
namespace moe {

cudaError_t launch_plan_routing(moe_ctx* ctx, const float* logits, int32_t* topk_ids, float* topk_w,
                                int32_t* counts, int32_t* offsets, int32_t* perm, int32_t* inv_perm,
                                cudaStream_t stream);

// Plan from expert ids chosen by the caller; ids_checked receives the ids with out-of-range ones replaced by 0.
cudaError_t launch_plan_from_topk(moe_ctx* ctx, const int32_t* topk_ids, int32_t* ids_checked, int32_t* counts,
                                  int32_t* offsets, int32_t* perm, int32_t* inv_perm, cudaStream_t stream);

cudaError_t launch_dispatch(moe_ctx* ctx, const void* x, const int32_t* inv_perm, void* x_perm,
                            cudaStream_t stream);

cudaError_t launch_combine(moe_ctx* ctx, const void* y_perm, const int32_t* inv_perm, const float* topk_w,
                           void* out, cudaStream_t stream);

// Returns MOE_OK, MOE_ERR_CUDA (driver/runtime failure) or MOE_ERR_INVALID_ARG.
moe_status launch_expert_ffn(moe_ctx* ctx, const void* x_perm, const int32_t* offsets, const void* w_gate,
                             const void* w_up, const void* w_down, void* h_ws, void* y_perm,
                             float* h_fp32_debug, const moe_tuning* tuning, cudaStream_t stream);

moe_status launch_expert_ffn_fp8(moe_ctx* ctx, const moe_fp8_ffn_args* args, const moe_tuning* tuning,
                                 cudaStream_t stream);

// bf16 [rows, cols] -> E4M3 codes [rows, cols] + one fp32 scale per row (amax / 448).
cudaError_t launch_quantize_rows(moe_ctx* ctx, const void* in_bf16, long long rows, int cols, void* codes,
                                 float* scales, cudaStream_t stream);

// Row mover for E4M3 rows with their scales: xq_perm[inv_perm[t*k+j]] = xq[t], sx_perm[..] = sx[t].
cudaError_t launch_dispatch_fp8(moe_ctx* ctx, const void* xq, const float* sx, const int32_t* inv_perm,
                                void* xq_perm, float* sx_perm, cudaStream_t stream);

// Router front end.  Sizes of the prepared weights (two bf16 terms of W_r, expert rows padded) and of the scratch
// for the K-split partial logits; the split of W_r; logits + top-k in one kernel (ids and weights only: the plan's
// histogram, scan and scatter follow through launch_plan_from_topk).
size_t router_weight_bytes(const moe_shape& s);
size_t router_scratch_bytes(const moe_shape& s);
cudaError_t launch_router_prepare(moe_ctx* ctx, const float* w_router, void* w_split, cudaStream_t stream);
moe_status launch_router(moe_ctx* ctx, const void* x, const void* w_split, const float* bias, void* scratch,
                         float* logits_out, int32_t* topk_ids, float* topk_w, cudaStream_t stream);
cudaError_t prepare_router(moe_ctx* ctx);      // one-time kernel attributes

// Block-scaled FP8 (MXFP8): row quantisation in 32-element blocks, dispatch of quantised rows, the two GEMMs.
cudaError_t launch_quantize_rows_mx(moe_ctx* ctx, const void* in_bf16, long long rows, int cols, void* codes,
                                    uint32_t* sf_words, cudaStream_t stream);
cudaError_t launch_dispatch_mx(moe_ctx* ctx, const void* xq, const uint32_t* sfx, const int32_t* inv_perm,
                               void* xq_perm, uint32_t* sfx_perm, cudaStream_t stream);
moe_status launch_expert_ffn_mx(moe_ctx* ctx, const moe_mx_ffn_args* args, cudaStream_t stream);
cudaError_t prepare_expert_ffn_mx(moe_ctx* ctx);

cudaError_t prepare_expert_ffn(moe_ctx* ctx);  // one-time kernel attributes (dynamic shared memory size)

}  // namespace moe
