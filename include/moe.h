/*
 * moe.h -- C ABI of the B200 (sm_100a) MoE forward library, EP=1 on one GPU.
 *
 * The calls restate the expert-parallel problem the paper analyses (Sec. 2.2: token hidden vectors are
 * sent to their experts, expert outputs are returned to the rank that owns the token; Sec. 4.3: the fused
 * kernel is Dispatch, Linear-1, Linear-2 and a Combine buffer written by the Linear-2 epilogue), run with
 * a single rank.  The per-expert receive buffer (x_perm) and the combine buffer (y_perm) that the paper's
 * kernels reach with remote stores are ordinary allocations in this GPU's HBM, separate from x and out.
 *
 * Conventions for every call
 *   - All tensor pointers are DEVICE pointers unless the parameter name ends in _host.  The caller owns
 *     every buffer; the library keeps no reference after the call's work has finished on the stream.
 *   - bf16 tensors are passed as void* (2 bytes per element, row-major, innermost dimension contiguous).
 *   - Pointers must be 16-byte aligned.  H and F must be multiples of 64; 1 <= k <= min(E, 32); E <= 1024.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls are asynchronous:
 *     they enqueue work and return.  Argument and shape errors are returned synchronously, before any
 *     launch.  Errors detected on the device (a bounded wait that expired) are written to a status word
 *     read by moe_last_device_status; kernels never trap.
 *   - The context's device must be the calling thread's current device.
 *   - Notation: T tokens, H hidden, F per-expert ffn width, E experts, k experts per token, R = T*k rows.
 */
#ifndef MOE_B200_H_
#define MOE_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  MOE_OK = 0,
  MOE_ERR_INVALID_ARG = 1,         /* null pointer, misaligned pointer, wrong device, bad tuning value */
  MOE_ERR_UNSUPPORTED_SHAPE = 2,   /* H or F not a multiple of 64, k or E out of range, T < 0 */
  MOE_ERR_WORKSPACE_TOO_SMALL = 3,
  MOE_ERR_BAD_ROUTING = 4,         /* device status: an expert id given to moe_plan_routing_from_topk is outside
                                      [0, E); returned by a call only from the debug check of the logits
                                      (MOE_TUNING entry x.check_logits=1: non-finite logits, tested on the host) */
  MOE_ERR_CUDA = 5,                /* a CUDA runtime or driver call failed */
  MOE_ERR_TIMEOUT = 6,             /* device status only: a bounded on-device wait expired */
  MOE_ERR_UNSUPPORTED = 7,         /* ep_size != 1, unknown schedule */
  MOE_ERR_STATIC_SCRATCH_TOO_SMALL = 8  /* moe_plan_routing_static: the shape exceeds the built-in scratch */
} moe_status;

typedef struct {
  int32_t T, H, F, E, k;
  int32_t ep_size, ep_rank;        /* must be 1 and 0: nothing is sharded across GPUs */
} moe_shape;

/*
 * Store pacing of the grouped-GEMM epilogue: the one part of the paper's burst/gap idea (Sec. 3.1: a
 * producer emits a burst, then an interval with no stores; Eq. 1) that has a meaning on local HBM.
 * A "store tile" is 128 rows x 32 output columns of bf16 (8 KiB), the unit one pass of the four epilogue
 * warps drains from tensor memory.  A burst is `store_burst_tiles` store tiles issued back to back by a
 * CTA.  interleave_mode 0 ("after-mainloop"): bursts follow one another with no enforced gap.
 * interleave_mode 1 ("every-k-iterations"): after each burst the epilogue holds its next store until the
 * MMA warp has issued `interleave_k` more 64-deep K-blocks (of the following tiles' mainloops) than when
 * the burst ended, or has nothing left to issue.  In the CTA-pair kernel both CTAs of a pair pace on the
 * leader's MMA warp, so every CTA that stores is a paced producer in the sense of Eq. 1.  Tiles computed
 * with swapped operands (a few rows) are not paced.  Pacing never changes values: outputs are bitwise
 * identical for every setting.
 */
typedef struct {
  int32_t store_burst_tiles;       /* 1, 2, 4, 8 or 16; a CTA counts its store tiles across output tiles, so a burst
                                      may span accumulators (an output tile is 4 store tiles in Linear-1, 8 in Linear-2) */
  int32_t interleave_mode;         /* 0 or 1 */
  int32_t interleave_k;            /* 1, 2 or 4; used when interleave_mode == 1 */
  int32_t schedule;                /* 0 = Expert-Wave order (Sec. 4.3): all Linear-1 tiles, then all Linear-2 tiles;
                                      1 = interleaved order (Algorithm 1): both tile lists row-major (a row is one
                                      128-row block), CTA g of G owns tiles g, g+G, ... of each and places its
                                      Linear-2 tiles between its Linear-1 tiles as early as a lead of dep_lead_D
                                      rows allows; one launch, Linear-2 tiles wait for their row's h.
                                      Values are bitwise identical for both schedules. */
  int32_t dep_lead_D;              /* schedule 1: minimum row lead D >= 1 of Linear-1 over Linear-2; 0 = the
                                      anti-starvation knee ceil(128 * SMs / (2 F)) (App. A.2).  Must be 0 for
                                      schedule 0. */
  int32_t debug_flags;             /* bit 0: record per-CTA wait counters (moe_get_ffn_trace); bit 1: run
                                      schedule 0 as one launch with ready counters instead of two (layers whose
                                      tiles fit in about one wave of CTAs always do); bit 2: failure drill, requested
                                      by the host: runs as one launch in which Linear-1 never publishes its rows, so
                                      every Linear-2 wait expires (after about 0.1 s), the kernel unwinds and the
                                      status word reads MOE_ERR_TIMEOUT; outputs are then undefined; bit 3: use the
                                      CTA-pair kernel (clusters of two CTAs on 256-row tiles) for two-launch runs; by
                                      default every layer runs the single-CTA kernel, which cuts many-row experts
                                      into 256-row tiles on its two accumulators, except Linear-1 of the FP8 (per-row
                                      scales) path on layers averaging 1024 rows per expert or more, which runs as
                                      CTA pairs; bit 4: the single-CTA kernel there as well; other bits 0 */
} moe_tuning;

/*
 * Environment override for sweeps (no counterpart in the paper).  moe_create reads the variable MOE_TUNING once:
 * a comma-separated list of key=value entries with the keys burst, mode, k, schedule, lead, flags (the six fields
 * above, in that order; fields not named keep their defaults 1, 0, 1, 0, 0, 0).  The result replaces the built-in
 * default that a call uses when it is given tuning = NULL; a call that passes a moe_tuning is not affected.
 * Entries "x.<name>=<int>" are development knobs of individual kernels (unstable, undocumented on purpose: they
 * select between variants under measurement and never change results).  An unknown key, a malformed number or a
 * combination moe_tuning does not allow makes moe_create return MOE_ERR_INVALID_ARG.
 * moe_parse_tuning applies the same parser to `text` (NULL = empty) without touching the environment or a device:
 * *out_tuning receives the fields, *out_named_field (may be NULL) 1 when at least one of the six keys was named.
 */
moe_status moe_parse_tuning(const char* text, moe_tuning* out_tuning, int32_t* out_named_field);

/* Byte offsets of the slices of the workspace used by moe_fused_forward (each 256-byte aligned). */
typedef struct {
  size_t topk_ids;   /* int32 [T,k]  */
  size_t topk_w;     /* fp32  [T,k]  */
  size_t counts;     /* int32 [E]    */
  size_t offsets;    /* int32 [E+1]  */
  size_t perm;       /* int32 [R]    */
  size_t inv_perm;   /* int32 [R]    */
  size_t x_perm;     /* bf16  [R,H]  expert-contiguous receive buffer (Dispatch) */
  size_t h;          /* bf16  [R,F]  Linear-1 output after SiLU*mul */
  size_t y_perm;     /* bf16  [R,H]  combine buffer written by the Linear-2 epilogue */
  size_t x_stage;    /* bf16  [T,H]  device staging for moe_fused_forward_host */
  size_t logits_stage; /* fp32 [T,E] device staging for moe_fused_forward_host */
  size_t out_stage;  /* bf16  [T,H]  device staging for moe_fused_forward_host */
  size_t x_stage_b;  /* second staging slot of moe_fused_forward_host_pipelined: bf16 [T,H] */
  size_t logits_stage_b; /* fp32 [T,E] */
  size_t out_stage_b;    /* bf16 [T,H] */
  size_t total;      /* = moe_workspace_bytes */
} moe_workspace_layout;

typedef struct moe_ctx moe_ctx;    /* opaque: shape, device, SM count, small device scratch */

/* Human-readable name of a status code.  Never NULL. */
const char* moe_status_string(moe_status s);

/*
 * Create a context for one layer shape on `device` (must be the current device).  Allocates the small
 * device scratch the routing kernels need (per-chunk histograms, a status word); no later call allocates.
 * Errors: INVALID_ARG, UNSUPPORTED_SHAPE, UNSUPPORTED (ep_size != 1), CUDA.
 */
moe_status moe_create(moe_ctx** out_ctx, const moe_shape* shape, int device);
void moe_destroy(moe_ctx* ctx);

/*
 * Serving batches vary in size: a context created for T tokens also runs any smaller batch.  This sets the
 * number of tokens the following calls process (0 <= tokens <= the T given to moe_create); every tensor
 * argument then has `tokens` rows ([tokens,H], [tokens*k], ...), and the workspace slices are those of
 * moe_get_workspace_layout for a shape with T = tokens (a workspace sized for the creation shape always suffices).
 * No device work, no allocation.  Errors: INVALID_ARG.
 */
moe_status moe_set_active_tokens(moe_ctx* ctx, int32_t tokens);

/* Size and slicing of the caller-provided workspace of moe_fused_forward.  Returns 0 / fills zeros for a
 * shape moe_create would reject. */
size_t moe_workspace_bytes(const moe_shape* shape);
moe_status moe_get_workspace_layout(const moe_shape* shape, moe_workspace_layout* out_layout);

/*
 * Routing plan (the Dispatch bookkeeping of Sec. 4.3; the paper leaves routing unchanged, Sec. 7).
 * For each token: the k largest logits (ties to the lower expert index), slots in descending-logit
 * order, weights = softmax over the k selected logits (fp32).  Then per-expert counts, exclusive
 * offsets, and the stable permutation: flat slot s = t*k+j is placed at row offsets[e] + (number of
 * slots s' < s with the same expert).  perm[row] = s, inv_perm[s] = row.
 *   logits [T,E] fp32 (finite)  ->  topk_ids [T,k] int32, topk_w [T,k] fp32, counts [E] int32,
 *   offsets [E+1] int32, perm [R] int32, inv_perm [R] int32.
 * T == 0 writes zero counts/offsets and launches nothing else.  Infinite or NaN logits violate the contract and are
 * not tested on the device; a context created with the MOE_TUNING entry x.check_logits=1 (a debug aid: it copies the
 * logits to the host and synchronises the stream in every call that takes logits) returns MOE_ERR_BAD_ROUTING for them
 * before anything is launched.
 */
moe_status moe_plan_routing(moe_ctx* ctx, const float* logits, int32_t* topk_ids, float* topk_w,
                            int32_t* counts, int32_t* offsets, int32_t* perm, int32_t* inv_perm,
                            void* stream);

/*
 * The same plan for routers the library does not know (sigmoid scores, bias-corrected or group-limited top-k, ...):
 * the caller supplies the expert ids it chose, topk_ids [T,k] int32, and keeps its own combine weights for
 * moe_combine.  Counts, offsets and the stable permutation are built exactly as in moe_plan_routing.  Every id
 * must lie in [0, E); an id outside is reported through the status word (MOE_ERR_BAD_ROUTING, detail = the flat
 * slot t*k+j) and treated as expert 0 so that no write goes out of bounds; the plan is then meaningless.
 * topk_ids_checked [T,k] int32 receives the ids actually used (it may be the same buffer as topk_ids).
 */
moe_status moe_plan_routing_from_topk(moe_ctx* ctx, const int32_t* topk_ids, int32_t* topk_ids_checked,
                                      int32_t* counts, int32_t* offsets, int32_t* perm, int32_t* inv_perm,
                                      void* stream);

/*
 * The routing plan for callers that must not allocate.  (The paper has no counterpart: this entry point
 * exists for the library's users, not for the method.)
 *
 * moe_create obtains its scratch with cudaMalloc.  Some callers cannot do that: code that runs after a
 * framework has handed the whole device to its own memory pool, plugins whose execute hook is forbidden
 * to allocate, or a serving loop that cannot afford the device-wide synchronisation an allocation may
 * imply.  This call needs no context and calls no cudaMalloc, cudaFree or allocating library routine.
 * Its scratch (the per-chunk histograms and their prefix) is a fixed array of 512 KiB that is part of
 * the library image: every GPU on which the library is loaded holds it until the process exits.
 *
 * Same inputs, outputs and results as moe_plan_routing (shape->T, E, k are used; H and F are ignored).
 *   - Limit: ceil(T / floor(256/k)) * E <= 65536, e.g. T <= 8192 at E = 256, k = 8.  Beyond it the call
 *     returns MOE_ERR_STATIC_SCRATCH_TOO_SMALL and launches nothing.
 *   - The first call on each device that passes the argument checks (a call with T = 0 counts) looks up
 *     the array's device address, with that device current.  Make that first call outside any stream
 *     capture.  Host threads may make it concurrently: the lookup is idempotent and its result is
 *     published atomically.
 *   - All calls on a device share the one array.  Nothing in it has to start at zero (each call
 *     rewrites every entry it later reads), so calls may follow one another on a stream freely; two
 *     calls that overlap on the GPU (different streams, no ordering) race on it and give wrong plans.
 *   - Works on the calling thread's current device.  Errors: INVALID_ARG (null or misaligned pointer),
 *     UNSUPPORTED_SHAPE, UNSUPPORTED (ep_size != 1), STATIC_SCRATCH_TOO_SMALL, CUDA.
 */
moe_status moe_plan_routing_static(const moe_shape* shape, const float* logits, int32_t* topk_ids,
                                   float* topk_w, int32_t* counts, int32_t* offsets, int32_t* perm,
                                   int32_t* inv_perm, void* stream);

/*
 * Router front end: the step before the Dispatch bookkeeping of Sec. 4.3, for callers that hold the router matrix
 * instead of logits.  The paper does not change the router (Sec. 7) and gives no kernel for it; the operation is
 *     logits[t,e] = sum_c x[t,c] * w_router[c,e] (+ bias[e]),
 * followed by the plan of moe_plan_routing on those logits.
 *
 * moe_router_prepare splits w_router [H,E] fp32 (device) once into two bf16 terms (the bf16 rounding of the value
 * and the bf16 rounding of the remainder: 16 significant bits, relative error below 2^-17), stored as [2][Epad][H]
 * with H contiguous and the expert rows padded to Epad (a multiple of 16, of 128 above 128 experts; padding rows are
 * zero); w_split (device, caller-owned) holds moe_router_weight_bytes bytes.  With bf16 x every partial product is
 * exact in fp32; what separates the logits from an fp64 product is the tensor path's fp32 accumulation (about 2^-24
 * of the running sum per instruction) and the bits the split drops: |delta| <= 1e-4 * (1 + |logit|) for H <= 8192
 * on N(0,1) data (about 6e-5 at H = 7168).
 *
 * moe_route_tokens computes the logits on the bf16 tensor path and selects the top k per token in the same kernel,
 * on the fp32 logits it computed, with the rules of moe_plan_routing (ties to the lower expert index, softmax over
 * the k selected logits); counts, offsets, perm and inv_perm follow as in moe_plan_routing_from_topk.  The result
 * is bit-identical to moe_plan_routing applied to the returned logits, and run-to-run deterministic.
 *   x [T,H] bf16, w_split from moe_router_prepare, bias [E] fp32 or NULL,
 *   scratch: device, at least moe_router_scratch_bytes bytes (partial sums of the K split; contents undefined after),
 *   logits_out: NULL, or fp32 [T,E] that receives the logits the selection used,
 *   -> topk_ids, topk_w, counts, offsets, perm, inv_perm as moe_plan_routing.
 * Errors: INVALID_ARG, WORKSPACE_TOO_SMALL (scratch), CUDA; TIMEOUT through the status word (detail 101-103).
 */
size_t moe_router_weight_bytes(const moe_shape* shape);
size_t moe_router_scratch_bytes(const moe_shape* shape);
moe_status moe_router_prepare(moe_ctx* ctx, const float* w_router, void* w_split, void* stream);
moe_status moe_route_tokens(moe_ctx* ctx, const void* x, const void* w_split, const float* bias, void* scratch,
                            size_t scratch_bytes, float* logits_out, int32_t* topk_ids, float* topk_w,
                            int32_t* counts, int32_t* offsets, int32_t* perm, int32_t* inv_perm, void* stream);

/*
 * Dispatch (Sec. 2.2 / Sec. 4.3 "Dispatch input"): x_perm[inv_perm[t*k+j], :] = x[t, :] for every slot,
 * i.e. x_perm[row, :] = x[perm[row] div k, :].  Each token row is read once and written k times with
 * 16-byte accesses.   x [T,H] bf16, inv_perm [R] int32 -> x_perm [R,H] bf16 (bit-exact copies).
 */
moe_status moe_dispatch(moe_ctx* ctx, const void* x, const int32_t* inv_perm, void* x_perm, void* stream);

/*
 * Expert feed-forward over the expert-contiguous buffer (Sec. 4.3 "Linear-1", "Linear-2"; Linear-1 is
 * twice the intermediate width, App. A.2, i.e. a gate half and an up half).  For expert e and its rows
 * offsets[e] <= r < offsets[e+1]:
 *     h[r,f] = silu(sum_c x_perm[r,c] w_gate[e,f,c]) * (sum_c x_perm[r,c] w_up[e,f,c])      (bf16 out)
 *     y_perm[r,c] = sum_f h[r,f] w_down[e,c,f]                                               (bf16 out)
 * bf16 operands, fp32 accumulation in tensor memory, outputs rounded to nearest even.
 *   x_perm [R,H] bf16, offsets [E+1] int32, w_gate/w_up [E,F,H] bf16, w_down [E,H,F] bf16
 *   -> h_ws [R,F] bf16 (also the Linear-2 input), y_perm [R,H] bf16.
 *   h_fp32_debug: NULL, or fp32 [R,F] that receives h before its rounding to bf16.
 *   tuning: NULL for defaults {1,0,1,0,0,0}.
 * Rows of empty experts do not exist; rows outside every expert are never written.
 */
moe_status moe_expert_ffn(moe_ctx* ctx, const void* x_perm, const int32_t* offsets, const void* w_gate,
                          const void* w_up, const void* w_down, void* h_ws, void* y_perm,
                          float* h_fp32_debug, const moe_tuning* tuning, void* stream);

/*
 * Combine (Sec. 2.2: expert outputs return to the token's owner; Sec. 4.3 "Combine buffer"):
 *     out[t,:] = bf16( sum_{j=0..k-1} topk_w[t,j] * float(y_perm[inv_perm[t*k+j], :]) )
 * summed in ascending j with fp32 accumulation: deterministic, no atomics.
 *   y_perm [R,H] bf16, inv_perm [R] int32, topk_w [T,k] fp32 -> out [T,H] bf16.
 */
moe_status moe_combine(moe_ctx* ctx, const void* y_perm, const int32_t* inv_perm, const float* topk_w,
                       void* out, void* stream);

/*
 * The whole layer on one stream: plan_routing, dispatch, expert_ffn, combine (Sec. 4.3, the fused
 * Dispatch + Linear-1 + Linear-2 + Combine path).  Intermediates live in `workspace` at the offsets
 * moe_get_workspace_layout reports.  Errors: as the four calls, plus WORKSPACE_TOO_SMALL.
 */
moe_status moe_fused_forward(moe_ctx* ctx, const void* x, const float* logits, const void* w_gate,
                             const void* w_up, const void* w_down, void* out, void* workspace,
                             size_t workspace_bytes, const moe_tuning* tuning, void* stream);

/*
 * The whole layer starting from the router matrix: moe_route_tokens (logits not kept), dispatch, expert_ffn,
 * combine on one stream.  w_split from moe_router_prepare; bias [E] fp32 or NULL; router_scratch as the scratch of
 * moe_route_tokens (at least moe_router_scratch_bytes bytes); everything else as moe_fused_forward.
 */
moe_status moe_fused_forward_routed(moe_ctx* ctx, const void* x, const void* w_split, const float* bias,
                                    const void* w_gate, const void* w_up, const void* w_down, void* out,
                                    void* workspace, size_t workspace_bytes, void* router_scratch,
                                    size_t router_scratch_bytes, const moe_tuning* tuning, void* stream);

/*
 * moe_fused_forward with the per-step tensors in HOST memory (pinned memory makes the copies asynchronous):
 * x_host [T,H] bf16 and logits_host [T,E] fp32 are copied to the workspace's staging slices, the layer
 * runs, and out [T,H] bf16 is copied back to out_host, all on `stream`.  Expert weights stay on the
 * device.  The caller synchronises the stream before reading out_host.
 */
moe_status moe_fused_forward_host(moe_ctx* ctx, const void* x_host, const float* logits_host,
                                  const void* w_gate, const void* w_up, const void* w_down,
                                  void* out_host, void* workspace, size_t workspace_bytes,
                                  const moe_tuning* tuning, void* stream);

/* ------------------------------------------------------------------------------------------------------------
 * FP8 (W8A8) variant of the expert FFN.  The paper's kernels run W8A8 / W4A8 (Sec. 5.3) without saying how values
 * are scaled; the scheme here needs no scaling inside the MMA loop: E4M3 storage (round to nearest even, saturating
 * at 448), one fp32 scale per row of every quantised matrix (per token row for x and h, per output channel for the
 * weights), scale = amax(|row|) / 448 (1 for an all-zero row), code = convert(fp32(v) / scale); a GEMM multiplies
 * codes with fp32 accumulation and its epilogue applies row scale x column scale.  h is produced in bf16, then
 * quantised row by row for Linear-2; y_perm and out stay bf16.  Routing, combine and all plan arrays are those of
 * the bf16 layer.  H and F must be multiples of 128.
 * ------------------------------------------------------------------------------------------------------------ */

/* in_bf16 [rows, cols] bf16 (cols a multiple of 8) -> codes [rows, cols] E4M3 bytes, scales [rows] fp32. */
moe_status moe_quantize_rows(moe_ctx* ctx, const void* in_bf16, int64_t rows, int32_t cols, void* codes,
                             float* scales, void* stream);

/* xq_perm[inv_perm[t*k+j], :] = xq[t, :] (E4M3 bytes, [T,H] -> [R,H]) and sx_perm[inv_perm[t*k+j]] = sx[t]. */
moe_status moe_dispatch_fp8(moe_ctx* ctx, const void* xq, const float* sx, const int32_t* inv_perm, void* xq_perm,
                            float* sx_perm, void* stream);

typedef struct {
  const void* xq_perm;      /* E4M3 [R,H] expert-contiguous rows */
  const float* sx_perm;     /* fp32 [R]   their scales */
  const int32_t* offsets;   /* int32 [E+1] */
  const void* wq_gate;      /* E4M3 [E,F,H] */
  const float* s_gate;      /* fp32 [E,F] */
  const void* wq_up;        /* E4M3 [E,F,H] */
  const float* s_up;        /* fp32 [E,F] */
  const void* wq_down;      /* E4M3 [E,H,F] */
  const float* s_down;      /* fp32 [E,H] */
  void* h_ws;               /* out: bf16 [R,F]  silu(g)*u */
  void* hq_ws;              /* out: E4M3 [R,F]  its quantised copy (Linear-2 input) */
  float* sh_ws;             /* out: fp32 [R]    row scales of hq */
  void* y_perm;             /* out: bf16 [R,H] */
} moe_fp8_ffn_args;

/* Linear-1 (E4M3 x E4M3 -> fp32, scales, SiLU*mul) -> h bf16 -> row quantisation -> Linear-2 -> y_perm bf16.
 * Three launches; Expert-Wave order only (tuning->schedule must be 0). */
moe_status moe_expert_ffn_fp8(moe_ctx* ctx, const moe_fp8_ffn_args* args, const moe_tuning* tuning, void* stream);

/* Byte offsets of the workspace slices of moe_fused_forward_fp8 (256-byte aligned). */
typedef struct {
  size_t topk_ids, topk_w, counts, offsets, perm, inv_perm;   /* as in moe_workspace_layout */
  size_t xq;         /* E4M3 [T,H] */
  size_t sx;         /* fp32 [T]   */
  size_t xq_perm;    /* E4M3 [R,H] */
  size_t sx_perm;    /* fp32 [R]   */
  size_t h;          /* bf16 [R,F] */
  size_t hq;         /* E4M3 [R,F] */
  size_t sh;         /* fp32 [R]   */
  size_t y_perm;     /* bf16 [R,H] */
  size_t total;
} moe_workspace_layout_fp8;
moe_status moe_get_workspace_layout_fp8(const moe_shape* shape, moe_workspace_layout_fp8* out_layout);

/* The whole layer with FP8 experts on one stream: plan_routing, quantize x, dispatch_fp8, expert_ffn_fp8, combine.
 * x [T,H] bf16 and logits as in moe_fused_forward; weights pre-quantised (moe_quantize_rows over their rows). */
moe_status moe_fused_forward_fp8(moe_ctx* ctx, const void* x, const float* logits, const void* wq_gate,
                                 const float* s_gate, const void* wq_up, const float* s_up, const void* wq_down,
                                 const float* s_down, void* out, void* workspace, size_t workspace_bytes,
                                 const moe_tuning* tuning, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Block-scaled FP8 experts (MXFP8).  The paper's kernels are W8A8 / W4A8 (Sec. 5.3) and do not say how values are
 * scaled; this is the block-scaled reading in the form the sm_100a tensor pipe applies inside the MMA: E4M3
 * elements, 32 consecutive elements along K share a scale 2^e kept as the byte e + 127 (E8M0), e = the smallest
 * integer with amax * 2^-e <= 448 (not below -127), code = convert(value * 2^-e) to nearest-even, never clipped.
 * Scale bytes are stored four to a 32-bit word (the four blocks of a 128-element K stage, lowest block in the lowest
 * byte), words as [K/128][rows].  H and F must be multiples of 128 (MOE_ERR_UNSUPPORTED_SHAPE otherwise).
 * ------------------------------------------------------------------------------------------------ */

/* in_bf16 [rows, cols] bf16 -> codes [rows, cols] E4M3 + sf_words [cols/128][rows] uint32.  cols % 128 == 0. */
moe_status moe_quantize_rows_mx(moe_ctx* ctx, const void* in_bf16, int64_t rows, int32_t cols, void* codes,
                                uint32_t* sf_words, void* stream);

/* Dispatch of quantised token rows: xq_perm[inv_perm[t*k+j], :] = xq[t, :], sfx_perm[w][inv_perm[t*k+j]] = sfx[w][t].
 *   xq [T,H] E4M3, sfx [H/128][T] -> xq_perm [R,H], sfx_perm [H/128][R]. */
moe_status moe_dispatch_mx(moe_ctx* ctx, const void* xq, const uint32_t* sfx, const int32_t* inv_perm, void* xq_perm,
                           uint32_t* sfx_perm, void* stream);

typedef struct {
  const void* xq_perm;      /* E4M3 [R,H] */
  const uint32_t* sfx_perm; /* [H/128][R] */
  const int32_t* offsets;   /* [E+1] */
  const void* wq_gate;      /* E4M3 [E*F, H] */
  const uint32_t* sf_gate;  /* [H/128][E*F] */
  const void* wq_up;        /* E4M3 [E*F, H] */
  const uint32_t* sf_up;    /* [H/128][E*F] */
  const void* wq_down;      /* E4M3 [E*H, F] */
  const uint32_t* sf_down;  /* [F/128][E*H] */
  void* hq_ws;              /* out: E4M3 [R,F]: h = silu(gate) * up, quantised from its fp32 value (Linear-2 input) */
  uint32_t* sfh_ws;         /* out: [F/128][R] */
  void* y_perm;             /* out: bf16 [R,H] */
  float* h_fp32_debug;      /* NULL, or fp32 [R,F] that receives h before its quantisation */
} moe_mx_ffn_args;

/* Linear-1 (block-scaled MMA, SiLU*mul, h quantised in the epilogue) and Linear-2 (-> y_perm bf16): two launches,
 * 128 x 256 tiles, Expert-Wave order.  For expert e and its rows r, with deq() the dequantised operands:
 *   h[r,f] = silu(sum_c deq(x)[r,c] deq(w_gate)[e,f,c]) * (sum_c deq(x)[r,c] deq(w_up)[e,f,c]),
 *   y_perm[r,c] = sum_f deq(hq)[r,f] deq(w_down)[e,c,f]   (fp32 accumulation, bf16 out). */
moe_status moe_expert_ffn_mx(moe_ctx* ctx, const moe_mx_ffn_args* args, void* stream);

/* Byte offsets of the workspace slices of moe_fused_forward_mx (256-byte aligned). */
typedef struct {
  size_t topk_ids, topk_w, counts, offsets, perm, inv_perm;   /* as in moe_workspace_layout */
  size_t xq;         /* E4M3 [T,H] */
  size_t sfx;        /* uint32 [H/128][T] */
  size_t xq_perm;    /* E4M3 [R,H] */
  size_t sfx_perm;   /* uint32 [H/128][R] */
  size_t hq;         /* E4M3 [R,F] */
  size_t sfh;        /* uint32 [F/128][R] */
  size_t y_perm;     /* bf16 [R,H] */
  size_t total;
} moe_workspace_layout_mx;
moe_status moe_get_workspace_layout_mx(const moe_shape* shape, moe_workspace_layout_mx* out_layout);

/* The whole layer with block-scaled FP8 experts on one stream: plan_routing, quantize x, dispatch_mx, expert_ffn_mx,
 * combine.  x [T,H] bf16 and logits as in moe_fused_forward; weights pre-quantised (moe_quantize_rows_mx over the
 * rows of each matrix: [E*F, H] for gate and up, [E*H, F] for down). */
moe_status moe_fused_forward_mx(moe_ctx* ctx, const void* x, const float* logits, const void* wq_gate,
                                const uint32_t* sf_gate, const void* wq_up, const uint32_t* sf_up, const void* wq_down,
                                const uint32_t* sf_down, void* out, void* workspace, size_t workspace_bytes,
                                void* stream);

/*
 * The host-buffer call as a two-deep pipeline, for callers that run step after step (serving): consecutive calls
 * alternate between two staging slots, the input copy of call i+1 runs on an internal copy stream while call i
 * computes on `stream`, and the output copy of call i runs on a second internal stream while call i+1 computes.
 * The intermediates are single-buffered, so the layers themselves still run one after another on `stream`.
 * Same arguments as moe_fused_forward_host; x_host, logits_host and out_host should be pinned and must stay
 * valid until the pipeline is flushed.  out_host of call i is complete only after a later
 * moe_host_pipeline_flush(ctx, stream) followed by a synchronisation of `stream` (the flush makes `stream` wait
 * for every copy issued so far).  Use one `stream` per context, and flush before mixing in calls of
 * moe_fused_forward_host, which shares the first staging slot.
 */
moe_status moe_fused_forward_host_pipelined(moe_ctx* ctx, const void* x_host, const float* logits_host,
                                            const void* w_gate, const void* w_up, const void* w_down,
                                            void* out_host, void* workspace, size_t workspace_bytes,
                                            const moe_tuning* tuning, void* stream);
moe_status moe_host_pipeline_flush(moe_ctx* ctx, void* stream);

/*
 * Synchronise `stream`, then read and clear the device status word.  *code is MOE_OK or MOE_ERR_TIMEOUT;
 * *detail identifies the wait that gave up (kernel id * 65536 + role).  Blocking.
 */
moe_status moe_last_device_status(moe_ctx* ctx, int32_t* code, int32_t* detail, void* stream);

/* Number of kernels the last call on this context launched (host-side count, for benchmarking). */
int32_t moe_last_launch_count(const moe_ctx* ctx);

/*
 * Wait counters of the two grouped GEMMs (the instrumentation of Sec. 5.1 / App. A.2: per-tile store spans and
 * the MMA-side wait for a free accumulator, there read with clock64()).  When a call ran with
 * tuning->debug_flags bit 0 set, every CTA of Linear-1 and of Linear-2 recorded twelve 64-bit counters, in SM
 * clocks: 0 producer loop span, 1 producer waited for a free shared-memory stage, 2 MMA warp waited for
 * operands, 3 MMA warp waited for a free accumulator (the epilogue's back-pressure, the paper's tmem_empty
 * wait), 4 epilogue waited for a finished accumulator, 5 epilogue drain-and-store span, 6 tiles processed
 * (a count), 7 epilogue held by the pacing gap, 8 tiles computed with swapped operands (a count), 9 the MMA
 * warp's time in those tiles, 10 the part of it spent waiting for operands, 11 its time in the other tiles
 * (8-11: the single-CTA bf16/E4M3 kernel; the block-scaled FP8 kernel, whose counters moe_expert_ffn_mx records
 * while per-kernel timing is enabled, writes 8, 9 and 11; zero in the CTA-pair kernel).  This call synchronises `stream` and copies
 * counters_host[2][*num_ctas][12] (Linear-1 first) to HOST memory; capacity is in 64-bit elements and must be
 * at least 24 * (number of SMs).
 */
moe_status moe_get_ffn_trace(moe_ctx* ctx, uint64_t* counters_host, int32_t capacity, int32_t* num_ctas,
                             void* stream);

/*
 * Tile order of the last one-launch expert FFN that ran with tuning->debug_flags bit 0 set (schedule 1, or
 * schedule 0 with debug bit 1): the codes each CTA drew, in its own order, so that the emitted schedule can be
 * checked against Algorithm 1.  A code is (phase << 30) | index, phase 0 = Linear-1, 1 = Linear-2; for
 * schedule 1 the index is the row-major tile number k (row k / n_blocks, column k % n_blocks, with n_blocks =
 * ceil(F/128) for Linear-1 and ceil(H/256) for Linear-2); -1 ends a CTA's list.  Synchronises `stream` and copies
 * codes_host[*num_ctas][*codes_per_cta] (int32, HOST); capacity is in elements and must cover that.
 */
moe_status moe_get_ffn_order(moe_ctx* ctx, int32_t* codes_host, int32_t capacity, int32_t* num_ctas,
                             int32_t* codes_per_cta, void* stream);

/*
 * Calibration probe of the tensor pipe (in the spirit of the paper's independent calibration, Sec. 3.3: measure
 * the platform parameter alone before using it in a kernel model).  One CTA issues `iters` tcgen05.mma of shape
 * M x N x 16 (bf16 in, fp32 accumulate; M in {64,128}, N a multiple of 16 up to 256) back to back on operands
 * resident in shared memory; *cycles_per_mma (HOST) receives the SM clocks per instruction.  Blocking.
 */
moe_status moe_probe_mma_cycles(moe_ctx* ctx, int32_t M, int32_t N, int32_t iters, double* cycles_per_mma,
                                void* stream);
/* The same probe for the other operand kinds: kind 0 = bf16 (K = 16 per instruction), 1 = E4M3 (kind::f8f6f4,
 * K = 32), 2 = block-scaled E4M3 (kind::mxf8f6f4.block_scale, K = 32, M = 128 only; scales resident in tensor memory),
 * 3 = the same with three tcgen05.cp scale copies (512 bytes each) in front of every four instructions, as one K stage
 * of the block-scaled GEMM issues them. */
moe_status moe_probe_mma_cycles_kind(moe_ctx* ctx, int32_t kind, int32_t M, int32_t N, int32_t iters,
                                     double* cycles_per_mma, void* stream);

/*
 * Per-kernel timing (measurement aid; the paper times its kernel with CUDA events, Sec. 5.1).  When
 * enabled, each call records a CUDA event on the stream before its first kernel and after every kernel.
 * moe_get_kernel_times waits for the last call's events and writes the seven device durations in
 * milliseconds, in launch order {top-k + histogram, scan, scatter, dispatch, Linear-1, Linear-2, combine},
 * to the HOST array ms_host[n], n == 7; kernels the last call did not launch read -1.
 * The events of the last 32 timed calls are kept (a ring, one slot per call), so a run of back-to-back calls can be
 * timed per kernel without a host synchronisation between them: moe_get_kernel_times_back reads the call that
 * was `calls_back` timed calls before the last one (0 = the last; 0 <= calls_back < 32, else MOE_ERR_INVALID_ARG;
 * a slot no call has used since timing was enabled reads -1 throughout).  Enabling or disabling clears the ring.
 */
moe_status moe_set_kernel_timing(moe_ctx* ctx, int32_t enable);
moe_status moe_get_kernel_times(moe_ctx* ctx, float* ms_host, int32_t n);
moe_status moe_get_kernel_times_back(moe_ctx* ctx, int32_t calls_back, float* ms_host, int32_t n);

#ifdef __cplusplus
}
#endif
#endif /* MOE_B200_H_ */
