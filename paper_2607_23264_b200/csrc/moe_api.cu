// Host side of the C ABI (include/moe.h): argument validation, context, workspace carving, call order.
#include <climits>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "moe_internal.h"

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

moe_status check_shape(const moe_shape* s) {
  if (!s) return MOE_ERR_INVALID_ARG;
  if (s->ep_size != 1 || s->ep_rank != 0) return MOE_ERR_UNSUPPORTED;
  if (s->T < 0 || s->H <= 0 || s->F <= 0 || s->E <= 0 || s->k <= 0) return MOE_ERR_UNSUPPORTED_SHAPE;
  if (s->H % 64 != 0 || s->F % 64 != 0) return MOE_ERR_UNSUPPORTED_SHAPE;
  if (s->E > 1024 || s->k > 32 || s->k > s->E) return MOE_ERR_UNSUPPORTED_SHAPE;
  if (static_cast<long long>(s->T) * s->k > 0x7FFFFFFFLL / 2) return MOE_ERR_UNSUPPORTED_SHAPE;
  return MOE_OK;
}

moe_status check_tuning(const moe_tuning* t) {
  if (!t) return MOE_OK;
  const int b = t->store_burst_tiles;
  if (!(b == 1 || b == 2 || b == 4 || b == 8 || b == 16)) return MOE_ERR_INVALID_ARG;
  if (t->interleave_mode != 0 && t->interleave_mode != 1) return MOE_ERR_INVALID_ARG;
  if (!(t->interleave_k == 1 || t->interleave_k == 2 || t->interleave_k == 4)) return MOE_ERR_INVALID_ARG;
  if (t->schedule != 0 && t->schedule != 1) return MOE_ERR_UNSUPPORTED;
  if (t->dep_lead_D < 0 || (t->schedule == 0 && t->dep_lead_D != 0) || (t->debug_flags & ~31) != 0)
    return MOE_ERR_INVALID_ARG;
  return MOE_OK;
}

// One "key=value" entry of MOE_TUNING.  Returns false on an unknown key or a malformed number.
bool apply_tuning_entry(const char* key, size_t key_len, const char* val, moe_tuning* t, int* named_field,
                        moe_knob* knobs, int* num_knobs) {
  char* end = nullptr;
  const long v = std::strtol(val, &end, 0);
  if (end == val || (*end != 0 && *end != ',') || v < INT32_MIN || v > INT32_MAX) return false;
  auto is = [&](const char* name) { return std::strlen(name) == key_len && std::strncmp(key, name, key_len) == 0; };
  int32_t* field = is("burst") ? &t->store_burst_tiles : is("mode") ? &t->interleave_mode : is("k") ? &t->interleave_k
                 : is("schedule") ? &t->schedule : is("lead") ? &t->dep_lead_D : is("flags") ? &t->debug_flags : nullptr;
  if (field) {
    *field = static_cast<int32_t>(v);
    *named_field = 1;
    return true;
  }
  if (key_len > 2 && key[0] == 'x' && key[1] == '.' && key_len - 2 < sizeof(knobs[0].name)) {
    if (!knobs || !num_knobs) return true;
    if (*num_knobs >= kMoeMaxKnobs) return false;
    moe_knob& k = knobs[(*num_knobs)++];
    std::memcpy(k.name, key + 2, key_len - 2);
    k.name[key_len - 2] = 0;
    k.value = static_cast<int32_t>(v);
    return true;
  }
  return false;
}

moe_status parse_tuning_text(const char* text, moe_tuning* t, int* named_field, moe_knob* knobs, int* num_knobs) {
  *t = moe_tuning{1, 0, 1, 0, 0, 0};
  *named_field = 0;
  if (num_knobs) *num_knobs = 0;
  if (!text) return MOE_OK;
  const char* p = text;
  while (*p) {
    while (*p == ',' || *p == ' ') ++p;
    if (!*p) break;
    const char* eq = p;
    while (*eq && *eq != '=' && *eq != ',') ++eq;
    if (*eq != '=' || eq == p) return MOE_ERR_INVALID_ARG;
    if (!apply_tuning_entry(p, static_cast<size_t>(eq - p), eq + 1, t, named_field, knobs, num_knobs))
      return MOE_ERR_INVALID_ARG;
    p = eq + 1;
    while (*p && *p != ',') ++p;
  }
  return *named_field ? check_tuning(t) : MOE_OK;
}

// Debug aid (development knob x.check_logits=1): copy the logits to the host, wait, and refuse non-finite values,
// which the top-k contract excludes and the kernels do not test.  Synchronises the stream; not for timed runs.
moe_status check_logits_on_host(const moe_ctx* ctx, const float* logits, cudaStream_t cs) {
  if (moe_knob_value(ctx, "check_logits", 0) == 0) return MOE_OK;
  const size_t n = static_cast<size_t>(ctx->shape.T) * ctx->shape.E;
  float* host = static_cast<float*>(std::malloc(n * sizeof(float)));
  if (!host) return MOE_ERR_CUDA;
  moe_status st = MOE_OK;
  if (cudaMemcpyAsync(host, logits, n * sizeof(float), cudaMemcpyDeviceToHost, cs) != cudaSuccess ||
      cudaStreamSynchronize(cs) != cudaSuccess) {
    st = MOE_ERR_CUDA;
  } else {
    for (size_t i = 0; i < n; ++i) {
      uint32_t bits;
      std::memcpy(&bits, host + i, 4);
      if ((bits & 0x7F800000u) == 0x7F800000u) {   // exponent all ones: infinity or NaN
        st = MOE_ERR_BAD_ROUTING;
        break;
      }
    }
  }
  std::free(host);
  return st;
}

moe_status check_ctx(const moe_ctx* ctx) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return MOE_ERR_CUDA;
  return dev == ctx->device ? MOE_OK : MOE_ERR_INVALID_ARG;
}

// Start of a public call: reset the launch counter and the timing marks, record the mark that
// precedes the call's first kernel.
inline void begin_call(moe_ctx* ctx, int first_mark, void* stream) {
  ctx->last_launches = 0;
  if (ctx->timing) {                      // a timed call takes the next slot of the event ring
    ctx->ev_slot = (ctx->ev_slot + 1) % kMoeTimingSlots;
    ctx->ev_recorded[ctx->ev_slot] = 0;
  }
  moe_mark(ctx, first_mark, static_cast<cudaStream_t>(stream));
}

// A routing chunk holds at most 256 slots (k <= 32, so at least 8 tokens).  Small batches use smaller chunks,
// down to one token per warp, so that the top-k work spreads over about two CTAs per SM.
void set_chunking(moe_ctx* ctx, int tokens) {
  ctx->tokens_per_chunk = kRouteThreads / ctx->shape.k;
  const int spread = (tokens + 2 * ctx->num_sms - 1) / (2 * ctx->num_sms);
  if (spread < ctx->tokens_per_chunk) ctx->tokens_per_chunk = spread < 8 ? 8 : spread;
  ctx->num_chunks = tokens ? (tokens + ctx->tokens_per_chunk - 1) / ctx->tokens_per_chunk : 0;
}

inline size_t up256(size_t v) { return (v + 255) & ~static_cast<size_t>(255); }

void fill_layout(const moe_shape& s, moe_workspace_layout* L) {
  const size_t T = s.T, H = s.H, F = s.F, E = s.E, k = s.k, R = T * k;
  size_t off = 0;
  auto take = [&](size_t bytes) { const size_t at = off; off += up256(bytes); return at; };
  L->topk_ids = take(R * 4);
  L->topk_w = take(R * 4);
  L->counts = take(E * 4);
  L->offsets = take((E + 1) * 4);
  L->perm = take(R * 4);
  L->inv_perm = take(R * 4);
  L->x_perm = take(R * H * 2);
  L->h = take(R * F * 2);
  L->y_perm = take(R * H * 2);
  L->x_stage = take(T * H * 2);
  L->logits_stage = take(T * E * 4);
  L->out_stage = take(T * H * 2);
  L->x_stage_b = take(T * H * 2);
  L->logits_stage_b = take(T * E * 4);
  L->out_stage_b = take(T * H * 2);
  L->total = off;
}

}  // namespace

extern "C" {

const char* moe_status_string(moe_status s) {
  switch (s) {
    case MOE_OK: return "MOE_OK";
    case MOE_ERR_INVALID_ARG: return "MOE_ERR_INVALID_ARG";
    case MOE_ERR_UNSUPPORTED_SHAPE: return "MOE_ERR_UNSUPPORTED_SHAPE";
    case MOE_ERR_WORKSPACE_TOO_SMALL: return "MOE_ERR_WORKSPACE_TOO_SMALL";
    case MOE_ERR_BAD_ROUTING: return "MOE_ERR_BAD_ROUTING";
    case MOE_ERR_CUDA: return "MOE_ERR_CUDA";
    case MOE_ERR_TIMEOUT: return "MOE_ERR_TIMEOUT";
    case MOE_ERR_UNSUPPORTED: return "MOE_ERR_UNSUPPORTED";
    case MOE_ERR_STATIC_SCRATCH_TOO_SMALL: return "MOE_ERR_STATIC_SCRATCH_TOO_SMALL";
  }
  return "MOE_ERR_UNKNOWN";
}

size_t moe_workspace_bytes(const moe_shape* shape) {
  if (check_shape(shape) != MOE_OK) return 0;
  moe_workspace_layout L;
  fill_layout(*shape, &L);
  return L.total;
}

moe_status moe_get_workspace_layout(const moe_shape* shape, moe_workspace_layout* out_layout) {
  if (!out_layout) return MOE_ERR_INVALID_ARG;
  std::memset(out_layout, 0, sizeof(*out_layout));
  const moe_status st = check_shape(shape);
  if (st != MOE_OK) return st;
  fill_layout(*shape, out_layout);
  return MOE_OK;
}

moe_status moe_parse_tuning(const char* text, moe_tuning* out_tuning, int32_t* out_named_field) {
  if (!out_tuning) return MOE_ERR_INVALID_ARG;
  int named = 0;
  const moe_status st = parse_tuning_text(text, out_tuning, &named, nullptr, nullptr);
  if (out_named_field) *out_named_field = named;
  return st;
}

moe_status moe_create(moe_ctx** out_ctx, const moe_shape* shape, int device) {
  if (!out_ctx) return MOE_ERR_INVALID_ARG;
  *out_ctx = nullptr;
  const moe_status st = check_shape(shape);
  if (st != MOE_OK) return st;
  moe_tuning env_tuning;
  moe_knob env_knobs[kMoeMaxKnobs];
  int env_named = 0, env_knob_count = 0;
  if (parse_tuning_text(std::getenv("MOE_TUNING"), &env_tuning, &env_named, env_knobs, &env_knob_count) != MOE_OK)
    return MOE_ERR_INVALID_ARG;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return MOE_ERR_CUDA;
  if (dev != device) return MOE_ERR_INVALID_ARG;

  moe_ctx* ctx = new (std::nothrow) moe_ctx();
  if (!ctx) return MOE_ERR_CUDA;
  ctx->shape = *shape;
  ctx->device = device;
  ctx->last_launches = 0;
  ctx->has_env_tuning = env_named;
  ctx->env_tuning = env_tuning;
  ctx->num_knobs = env_knob_count;
  std::memcpy(ctx->knobs, env_knobs, sizeof(env_knobs));
  if (cudaDeviceGetAttribute(&ctx->num_sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
    delete ctx;
    return MOE_ERR_CUDA;
  }
  ctx->max_tokens = shape->T;
  set_chunking(ctx, shape->T);
  // scratch for the finest chunking any batch up to T can use (8 tokens per chunk)
  const size_t hist_elems = static_cast<size_t>(shape->T / 8 + 1) * shape->E;

  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !fn) {
    delete ctx;
    return MOE_ERR_CUDA;
  }
  ctx->encode_tiled = reinterpret_cast<moe_encode_tiled_fn>(fn);

  bool ok = cudaMalloc(&ctx->d_chunk_hist, hist_elems * 4) == cudaSuccess;
  ok = ok && cudaMalloc(&ctx->d_chunk_base, hist_elems * 4) == cudaSuccess;
  ok = ok && cudaMalloc(&ctx->d_status, 2 * 4) == cudaSuccess;
  ok = ok && cudaMemset(ctx->d_status, 0, 2 * 4) == cudaSuccess;
  const size_t trace_bytes = static_cast<size_t>(2) * ctx->num_sms * kMoeTraceFields * 8;
  ok = ok && cudaMalloc(&ctx->d_trace, trace_bytes) == cudaSuccess;
  ok = ok && cudaMemset(ctx->d_trace, 0, trace_bytes) == cudaSuccess;
  const size_t order_bytes = static_cast<size_t>(ctx->num_sms) * kMoeOrderLogCap * 4;
  ok = ok && cudaMalloc(&ctx->d_order, order_bytes) == cudaSuccess;
  ok = ok && cudaMemset(ctx->d_order, 0xFF, order_bytes) == cudaSuccess;
  const size_t ready_bytes = (static_cast<size_t>(shape->T) * shape->k / 128 + shape->E + 1) * 4;
  ok = ok && cudaMalloc(&ctx->d_ready, ready_bytes) == cudaSuccess;
  ok = ok && cudaMemset(ctx->d_ready, 0, ready_bytes) == cudaSuccess;
  ok = ok && cudaMalloc(&ctx->d_sched, 4 * 4) == cudaSuccess;
  ok = ok && cudaMemset(ctx->d_sched, 0, 4 * 4) == cudaSuccess;
  const size_t done_bytes = static_cast<size_t>(shape->T / 128 + 2) * 4;
  ok = ok && cudaMalloc(&ctx->d_router_done, done_bytes) == cudaSuccess;
  ok = ok && cudaMemset(ctx->d_router_done, 0, done_bytes) == cudaSuccess;
  ok = ok && moe::prepare_expert_ffn(ctx) == cudaSuccess;
  ok = ok && moe::prepare_router(ctx) == cudaSuccess;
  ok = ok && moe::prepare_expert_ffn_mx(ctx) == cudaSuccess;
  for (int sl = 0; ok && sl < kMoeTimingSlots; ++sl)
    for (int i = 0; ok && i <= kMoeKernels; ++i) ok = cudaEventCreate(&ctx->ev[sl][i]) == cudaSuccess;
  ok = ok && cudaStreamCreateWithFlags(&ctx->s_h2d, cudaStreamNonBlocking) == cudaSuccess;
  ok = ok && cudaStreamCreateWithFlags(&ctx->s_d2h, cudaStreamNonBlocking) == cudaSuccess;
  for (int i = 0; ok && i < 2; ++i) {
    ok = cudaEventCreateWithFlags(&ctx->ev_h2d[i], cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&ctx->ev_compute[i], cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&ctx->ev_d2h[i], cudaEventDisableTiming) == cudaSuccess;
  }
  if (!ok) {
    moe_destroy(ctx);
    return MOE_ERR_CUDA;
  }
  *out_ctx = ctx;
  return MOE_OK;
}

moe_status moe_set_active_tokens(moe_ctx* ctx, int32_t tokens) {
  if (!ctx || tokens < 0 || tokens > ctx->max_tokens) return MOE_ERR_INVALID_ARG;
  ctx->shape.T = tokens;
  set_chunking(ctx, tokens);
  return MOE_OK;
}

void moe_destroy(moe_ctx* ctx) {
  if (!ctx) return;
  if (ctx->d_chunk_hist) cudaFree(ctx->d_chunk_hist);
  if (ctx->d_chunk_base) cudaFree(ctx->d_chunk_base);
  if (ctx->d_status) cudaFree(ctx->d_status);
  if (ctx->d_sched) cudaFree(ctx->d_sched);
  if (ctx->d_trace) cudaFree(ctx->d_trace);
  if (ctx->d_ready) cudaFree(ctx->d_ready);
  if (ctx->d_order) cudaFree(ctx->d_order);
  if (ctx->d_router_done) cudaFree(ctx->d_router_done);
  for (int sl = 0; sl < kMoeTimingSlots; ++sl)
    for (int i = 0; i <= kMoeKernels; ++i)
      if (ctx->ev[sl][i]) cudaEventDestroy(ctx->ev[sl][i]);
  for (int i = 0; i < 2; ++i) {
    if (ctx->ev_h2d[i]) cudaEventDestroy(ctx->ev_h2d[i]);
    if (ctx->ev_compute[i]) cudaEventDestroy(ctx->ev_compute[i]);
    if (ctx->ev_d2h[i]) cudaEventDestroy(ctx->ev_d2h[i]);
  }
  if (ctx->s_h2d) cudaStreamDestroy(ctx->s_h2d);
  if (ctx->s_d2h) cudaStreamDestroy(ctx->s_d2h);
  delete ctx;
}

moe_status moe_plan_routing(moe_ctx* ctx, const float* logits, int32_t* topk_ids, float* topk_w,
                            int32_t* counts, int32_t* offsets, int32_t* perm, int32_t* inv_perm,
                            void* stream) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  begin_call(ctx, 0, stream);
  const moe_shape& s = ctx->shape;
  if (!counts || !offsets) return MOE_ERR_INVALID_ARG;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  if (s.T == 0) {
    if (cudaMemsetAsync(counts, 0, static_cast<size_t>(s.E) * 4, cs) != cudaSuccess) return MOE_ERR_CUDA;
    if (cudaMemsetAsync(offsets, 0, static_cast<size_t>(s.E + 1) * 4, cs) != cudaSuccess) return MOE_ERR_CUDA;
    return MOE_OK;
  }
  if (!logits || !topk_ids || !topk_w || !perm || !inv_perm) return MOE_ERR_INVALID_ARG;
  if (!aligned16(logits) || !aligned16(topk_ids) || !aligned16(topk_w) || !aligned16(counts) ||
      !aligned16(offsets) || !aligned16(perm) || !aligned16(inv_perm))
    return MOE_ERR_INVALID_ARG;
  st = check_logits_on_host(ctx, logits, cs);
  if (st != MOE_OK) return st;
  return moe::launch_plan_routing(ctx, logits, topk_ids, topk_w, counts, offsets, perm, inv_perm, cs) == cudaSuccess
             ? MOE_OK
             : MOE_ERR_CUDA;
}

moe_status moe_plan_routing_from_topk(moe_ctx* ctx, const int32_t* topk_ids, int32_t* topk_ids_checked,
                                      int32_t* counts, int32_t* offsets, int32_t* perm, int32_t* inv_perm,
                                      void* stream) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  begin_call(ctx, 0, stream);
  const moe_shape& s = ctx->shape;
  if (!counts || !offsets) return MOE_ERR_INVALID_ARG;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  if (s.T == 0) {
    if (cudaMemsetAsync(counts, 0, static_cast<size_t>(s.E) * 4, cs) != cudaSuccess) return MOE_ERR_CUDA;
    if (cudaMemsetAsync(offsets, 0, static_cast<size_t>(s.E + 1) * 4, cs) != cudaSuccess) return MOE_ERR_CUDA;
    return MOE_OK;
  }
  if (!topk_ids || !topk_ids_checked || !perm || !inv_perm) return MOE_ERR_INVALID_ARG;
  if (!aligned16(topk_ids) || !aligned16(topk_ids_checked) || !aligned16(counts) || !aligned16(offsets) ||
      !aligned16(perm) || !aligned16(inv_perm))
    return MOE_ERR_INVALID_ARG;
  return moe::launch_plan_from_topk(ctx, topk_ids, topk_ids_checked, counts, offsets, perm, inv_perm, cs) == cudaSuccess
             ? MOE_OK
             : MOE_ERR_CUDA;
}

moe_status moe_dispatch(moe_ctx* ctx, const void* x, const int32_t* inv_perm, void* x_perm, void* stream) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  begin_call(ctx, 3, stream);
  if (ctx->shape.T == 0) return MOE_OK;
  if (!x || !inv_perm || !x_perm) return MOE_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(inv_perm) || !aligned16(x_perm)) return MOE_ERR_INVALID_ARG;
  return moe::launch_dispatch(ctx, x, inv_perm, x_perm, static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? MOE_OK
             : MOE_ERR_CUDA;
}

moe_status moe_expert_ffn(moe_ctx* ctx, const void* x_perm, const int32_t* offsets, const void* w_gate,
                          const void* w_up, const void* w_down, void* h_ws, void* y_perm,
                          float* h_fp32_debug, const moe_tuning* tuning, void* stream) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  begin_call(ctx, 4, stream);
  st = check_tuning(tuning);
  if (st != MOE_OK) return st;
  if (ctx->shape.T == 0) return MOE_OK;
  if (!x_perm || !offsets || !w_gate || !w_up || !w_down || !h_ws || !y_perm) return MOE_ERR_INVALID_ARG;
  if (!aligned16(x_perm) || !aligned16(offsets) || !aligned16(w_gate) || !aligned16(w_up) || !aligned16(w_down) ||
      !aligned16(h_ws) || !aligned16(y_perm) || !aligned16(h_fp32_debug))
    return MOE_ERR_INVALID_ARG;
  return moe::launch_expert_ffn(ctx, x_perm, offsets, w_gate, w_up, w_down, h_ws, y_perm, h_fp32_debug, tuning,
                                static_cast<cudaStream_t>(stream));
}

moe_status moe_combine(moe_ctx* ctx, const void* y_perm, const int32_t* inv_perm, const float* topk_w,
                       void* out, void* stream) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  begin_call(ctx, 6, stream);
  if (ctx->shape.T == 0) return MOE_OK;
  if (!y_perm || !inv_perm || !topk_w || !out) return MOE_ERR_INVALID_ARG;
  if (!aligned16(y_perm) || !aligned16(inv_perm) || !aligned16(topk_w) || !aligned16(out)) return MOE_ERR_INVALID_ARG;
  return moe::launch_combine(ctx, y_perm, inv_perm, topk_w, out, static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? MOE_OK
             : MOE_ERR_CUDA;
}

moe_status moe_fused_forward(moe_ctx* ctx, const void* x, const float* logits, const void* w_gate,
                             const void* w_up, const void* w_down, void* out, void* workspace,
                             size_t workspace_bytes, const moe_tuning* tuning, void* stream) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  st = check_tuning(tuning);
  if (st != MOE_OK) return st;
  const moe_shape& s = ctx->shape;
  if (s.T == 0) { ctx->last_launches = 0; return MOE_OK; }
  if (!x || !logits || !w_gate || !w_up || !w_down || !out || !workspace) return MOE_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(logits) || !aligned16(w_gate) || !aligned16(w_up) || !aligned16(w_down) ||
      !aligned16(out) || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
    return MOE_ERR_INVALID_ARG;
  moe_workspace_layout L;
  fill_layout(s, &L);
  if (workspace_bytes < L.total) return MOE_ERR_WORKSPACE_TOO_SMALL;

  unsigned char* ws = static_cast<unsigned char*>(workspace);
  int32_t* topk_ids = reinterpret_cast<int32_t*>(ws + L.topk_ids);
  float* topk_w = reinterpret_cast<float*>(ws + L.topk_w);
  int32_t* counts = reinterpret_cast<int32_t*>(ws + L.counts);
  int32_t* offsets = reinterpret_cast<int32_t*>(ws + L.offsets);
  int32_t* perm = reinterpret_cast<int32_t*>(ws + L.perm);
  int32_t* inv_perm = reinterpret_cast<int32_t*>(ws + L.inv_perm);
  void* x_perm = ws + L.x_perm;
  void* h = ws + L.h;
  void* y_perm = ws + L.y_perm;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);

  begin_call(ctx, 0, stream);
  st = check_logits_on_host(ctx, logits, cs);
  if (st != MOE_OK) return st;
  if (moe::launch_plan_routing(ctx, logits, topk_ids, topk_w, counts, offsets, perm, inv_perm, cs) != cudaSuccess)
    return MOE_ERR_CUDA;
  if (moe::launch_dispatch(ctx, x, inv_perm, x_perm, cs) != cudaSuccess) return MOE_ERR_CUDA;
  st = moe::launch_expert_ffn(ctx, x_perm, offsets, w_gate, w_up, w_down, h, y_perm, nullptr, tuning, cs);
  if (st != MOE_OK) return st;
  if (moe::launch_combine(ctx, y_perm, inv_perm, topk_w, out, cs) != cudaSuccess) return MOE_ERR_CUDA;
  return MOE_OK;
}

// ------------------------------------------------------------------------------------------------ router front end

size_t moe_router_weight_bytes(const moe_shape* shape) {
  return check_shape(shape) == MOE_OK ? moe::router_weight_bytes(*shape) : 0;
}

size_t moe_router_scratch_bytes(const moe_shape* shape) {
  return check_shape(shape) == MOE_OK ? moe::router_scratch_bytes(*shape) : 0;
}

moe_status moe_router_prepare(moe_ctx* ctx, const float* w_router, void* w_split, void* stream) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  ctx->last_launches = 0;
  if (!w_router || !w_split || !aligned16(w_router) || !aligned16(w_split)) return MOE_ERR_INVALID_ARG;
  return moe::launch_router_prepare(ctx, w_router, w_split, static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? MOE_OK
             : MOE_ERR_CUDA;
}

moe_status moe_route_tokens(moe_ctx* ctx, const void* x, const void* w_split, const float* bias, void* scratch,
                            size_t scratch_bytes, float* logits_out, int32_t* topk_ids, float* topk_w,
                            int32_t* counts, int32_t* offsets, int32_t* perm, int32_t* inv_perm, void* stream) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  begin_call(ctx, 0, stream);
  const moe_shape& s = ctx->shape;
  if (!counts || !offsets) return MOE_ERR_INVALID_ARG;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  if (s.T == 0) {
    if (cudaMemsetAsync(counts, 0, static_cast<size_t>(s.E) * 4, cs) != cudaSuccess) return MOE_ERR_CUDA;
    if (cudaMemsetAsync(offsets, 0, static_cast<size_t>(s.E + 1) * 4, cs) != cudaSuccess) return MOE_ERR_CUDA;
    return MOE_OK;
  }
  if (!x || !w_split || !scratch || !topk_ids || !topk_w || !perm || !inv_perm) return MOE_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(w_split) || !aligned16(bias) || !aligned16(scratch) || !aligned16(logits_out) ||
      !aligned16(topk_ids) || !aligned16(topk_w) || !aligned16(counts) || !aligned16(offsets) || !aligned16(perm) ||
      !aligned16(inv_perm))
    return MOE_ERR_INVALID_ARG;
  if (scratch_bytes < moe::router_scratch_bytes(s)) return MOE_ERR_WORKSPACE_TOO_SMALL;
  st = moe::launch_router(ctx, x, w_split, bias, scratch, logits_out, topk_ids, topk_w, cs);
  if (st != MOE_OK) return st;
  return moe::launch_plan_from_topk(ctx, topk_ids, topk_ids, counts, offsets, perm, inv_perm, cs) == cudaSuccess
             ? MOE_OK
             : MOE_ERR_CUDA;
}

moe_status moe_fused_forward_routed(moe_ctx* ctx, const void* x, const void* w_split, const float* bias,
                                    const void* w_gate, const void* w_up, const void* w_down, void* out,
                                    void* workspace, size_t workspace_bytes, void* router_scratch,
                                    size_t router_scratch_bytes, const moe_tuning* tuning, void* stream) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  st = check_tuning(tuning);
  if (st != MOE_OK) return st;
  const moe_shape& s = ctx->shape;
  if (s.T == 0) { ctx->last_launches = 0; return MOE_OK; }
  if (!x || !w_split || !w_gate || !w_up || !w_down || !out || !workspace || !router_scratch)
    return MOE_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(w_split) || !aligned16(bias) || !aligned16(w_gate) || !aligned16(w_up) ||
      !aligned16(w_down) || !aligned16(out) || !aligned16(router_scratch) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
    return MOE_ERR_INVALID_ARG;
  moe_workspace_layout L;
  fill_layout(s, &L);
  if (workspace_bytes < L.total || router_scratch_bytes < moe::router_scratch_bytes(s))
    return MOE_ERR_WORKSPACE_TOO_SMALL;

  unsigned char* ws = static_cast<unsigned char*>(workspace);
  int32_t* topk_ids = reinterpret_cast<int32_t*>(ws + L.topk_ids);
  float* topk_w = reinterpret_cast<float*>(ws + L.topk_w);
  int32_t* counts = reinterpret_cast<int32_t*>(ws + L.counts);
  int32_t* offsets = reinterpret_cast<int32_t*>(ws + L.offsets);
  int32_t* perm = reinterpret_cast<int32_t*>(ws + L.perm);
  int32_t* inv_perm = reinterpret_cast<int32_t*>(ws + L.inv_perm);
  void* x_perm = ws + L.x_perm;
  void* h = ws + L.h;
  void* y_perm = ws + L.y_perm;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);

  begin_call(ctx, 0, stream);
  st = moe::launch_router(ctx, x, w_split, bias, router_scratch, nullptr, topk_ids, topk_w, cs);
  if (st != MOE_OK) return st;
  if (moe::launch_plan_from_topk(ctx, topk_ids, topk_ids, counts, offsets, perm, inv_perm, cs) != cudaSuccess)
    return MOE_ERR_CUDA;
  if (moe::launch_dispatch(ctx, x, inv_perm, x_perm, cs) != cudaSuccess) return MOE_ERR_CUDA;
  st = moe::launch_expert_ffn(ctx, x_perm, offsets, w_gate, w_up, w_down, h, y_perm, nullptr, tuning, cs);
  if (st != MOE_OK) return st;
  if (moe::launch_combine(ctx, y_perm, inv_perm, topk_w, out, cs) != cudaSuccess) return MOE_ERR_CUDA;
  return MOE_OK;
}

// ------------------------------------------------------------------------------------------------ FP8 variant
namespace {
void fill_layout_fp8(const moe_shape& s, moe_workspace_layout_fp8* L) {
  const size_t T = s.T, H = s.H, F = s.F, E = s.E, k = s.k, R = T * k;
  size_t off = 0;
  auto take = [&](size_t bytes) { const size_t at = off; off += up256(bytes); return at; };
  L->topk_ids = take(R * 4);
  L->topk_w = take(R * 4);
  L->counts = take(E * 4);
  L->offsets = take((E + 1) * 4);
  L->perm = take(R * 4);
  L->inv_perm = take(R * 4);
  L->xq = take(T * H);
  L->sx = take(T * 4);
  L->xq_perm = take(R * H);
  L->sx_perm = take(R * 4);
  L->h = take(R * F * 2);
  L->hq = take(R * F);
  L->sh = take(R * 4);
  L->y_perm = take(R * H * 2);
  L->total = off;
}
moe_status check_fp8_shape(const moe_ctx* ctx) {
  return (ctx->shape.H % 128 == 0 && ctx->shape.F % 128 == 0) ? MOE_OK : MOE_ERR_UNSUPPORTED_SHAPE;
}
}  // namespace

moe_status moe_get_workspace_layout_fp8(const moe_shape* shape, moe_workspace_layout_fp8* out_layout) {
  if (!out_layout) return MOE_ERR_INVALID_ARG;
  std::memset(out_layout, 0, sizeof(*out_layout));
  moe_status st = check_shape(shape);
  if (st != MOE_OK) return st;
  if (shape->H % 128 != 0 || shape->F % 128 != 0) return MOE_ERR_UNSUPPORTED_SHAPE;
  fill_layout_fp8(*shape, out_layout);
  return MOE_OK;
}

moe_status moe_quantize_rows(moe_ctx* ctx, const void* in_bf16, int64_t rows, int32_t cols, void* codes,
                             float* scales, void* stream) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  ctx->last_launches = 0;
  if (rows < 0 || cols <= 0 || cols % 8 != 0) return MOE_ERR_INVALID_ARG;
  if (rows == 0) return MOE_OK;
  if (!in_bf16 || !codes || !scales || !aligned16(in_bf16) || (reinterpret_cast<uintptr_t>(codes) & 7u) != 0)
    return MOE_ERR_INVALID_ARG;
  return moe::launch_quantize_rows(ctx, in_bf16, rows, cols, codes, scales, static_cast<cudaStream_t>(stream)) ==
                 cudaSuccess
             ? MOE_OK
             : MOE_ERR_CUDA;
}

moe_status moe_dispatch_fp8(moe_ctx* ctx, const void* xq, const float* sx, const int32_t* inv_perm, void* xq_perm,
                            float* sx_perm, void* stream) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  st = check_fp8_shape(ctx);
  if (st != MOE_OK) return st;
  begin_call(ctx, 3, stream);
  if (ctx->shape.T == 0) return MOE_OK;
  if (!xq || !sx || !inv_perm || !xq_perm || !sx_perm) return MOE_ERR_INVALID_ARG;
  if (!aligned16(xq) || !aligned16(inv_perm) || !aligned16(xq_perm)) return MOE_ERR_INVALID_ARG;
  return moe::launch_dispatch_fp8(ctx, xq, sx, inv_perm, xq_perm, sx_perm, static_cast<cudaStream_t>(stream)) ==
                 cudaSuccess
             ? MOE_OK
             : MOE_ERR_CUDA;
}

moe_status moe_expert_ffn_fp8(moe_ctx* ctx, const moe_fp8_ffn_args* a, const moe_tuning* tuning, void* stream) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  st = check_fp8_shape(ctx);
  if (st != MOE_OK) return st;
  begin_call(ctx, 4, stream);
  st = check_tuning(tuning);
  if (st != MOE_OK) return st;
  if (tuning && (tuning->schedule != 0 || (tuning->debug_flags & 6) != 0)) return MOE_ERR_UNSUPPORTED;
  if (ctx->shape.T == 0) return MOE_OK;
  if (!a) return MOE_ERR_INVALID_ARG;
  const void* ptrs[] = {a->xq_perm, a->sx_perm, a->offsets, a->wq_gate, a->s_gate, a->wq_up, a->s_up,
                        a->wq_down, a->s_down, a->h_ws, a->hq_ws, a->sh_ws, a->y_perm};
  for (const void* q : ptrs)
    if (!q || (reinterpret_cast<uintptr_t>(q) & 15u) != 0) return MOE_ERR_INVALID_ARG;
  return moe::launch_expert_ffn_fp8(ctx, a, tuning, static_cast<cudaStream_t>(stream));
}

moe_status moe_fused_forward_fp8(moe_ctx* ctx, const void* x, const float* logits, const void* wq_gate,
                                 const float* s_gate, const void* wq_up, const float* s_up, const void* wq_down,
                                 const float* s_down, void* out, void* workspace, size_t workspace_bytes,
                                 const moe_tuning* tuning, void* stream) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  st = check_fp8_shape(ctx);
  if (st != MOE_OK) return st;
  st = check_tuning(tuning);
  if (st != MOE_OK) return st;
  if (tuning && (tuning->schedule != 0 || (tuning->debug_flags & 6) != 0)) return MOE_ERR_UNSUPPORTED;
  const moe_shape& s = ctx->shape;
  if (s.T == 0) { ctx->last_launches = 0; return MOE_OK; }
  const void* ptrs[] = {x, logits, wq_gate, s_gate, wq_up, s_up, wq_down, s_down, out};
  for (const void* q : ptrs)
    if (!q || (reinterpret_cast<uintptr_t>(q) & 15u) != 0) return MOE_ERR_INVALID_ARG;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MOE_ERR_INVALID_ARG;
  moe_workspace_layout_fp8 L;
  fill_layout_fp8(s, &L);
  if (workspace_bytes < L.total) return MOE_ERR_WORKSPACE_TOO_SMALL;
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  int32_t* topk_ids = reinterpret_cast<int32_t*>(ws + L.topk_ids);
  float* topk_w = reinterpret_cast<float*>(ws + L.topk_w);
  int32_t* counts = reinterpret_cast<int32_t*>(ws + L.counts);
  int32_t* offsets = reinterpret_cast<int32_t*>(ws + L.offsets);
  int32_t* perm = reinterpret_cast<int32_t*>(ws + L.perm);
  int32_t* inv_perm = reinterpret_cast<int32_t*>(ws + L.inv_perm);
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  begin_call(ctx, 0, stream);
  st = check_logits_on_host(ctx, logits, cs);
  if (st != MOE_OK) return st;
  if (moe::launch_plan_routing(ctx, logits, topk_ids, topk_w, counts, offsets, perm, inv_perm, cs) != cudaSuccess)
    return MOE_ERR_CUDA;
  if (moe::launch_quantize_rows(ctx, x, s.T, s.H, ws + L.xq, reinterpret_cast<float*>(ws + L.sx), cs) != cudaSuccess)
    return MOE_ERR_CUDA;
  if (moe::launch_dispatch_fp8(ctx, ws + L.xq, reinterpret_cast<const float*>(ws + L.sx), inv_perm, ws + L.xq_perm,
                               reinterpret_cast<float*>(ws + L.sx_perm), cs) != cudaSuccess)
    return MOE_ERR_CUDA;
  moe_fp8_ffn_args a;
  a.xq_perm = ws + L.xq_perm;
  a.sx_perm = reinterpret_cast<const float*>(ws + L.sx_perm);
  a.offsets = offsets;
  a.wq_gate = wq_gate;
  a.s_gate = s_gate;
  a.wq_up = wq_up;
  a.s_up = s_up;
  a.wq_down = wq_down;
  a.s_down = s_down;
  a.h_ws = ws + L.h;
  a.hq_ws = ws + L.hq;
  a.sh_ws = reinterpret_cast<float*>(ws + L.sh);
  a.y_perm = ws + L.y_perm;
  st = moe::launch_expert_ffn_fp8(ctx, &a, tuning, cs);
  if (st != MOE_OK) return st;
  if (moe::launch_combine(ctx, ws + L.y_perm, inv_perm, topk_w, out, cs) != cudaSuccess) return MOE_ERR_CUDA;
  return MOE_OK;
}

// ------------------------------------------------------------------------------------------------ MXFP8 variant
}  // extern "C"
namespace {
void fill_layout_mx(const moe_shape& s, moe_workspace_layout_mx* L) {
  const size_t T = s.T, H = s.H, F = s.F, E = s.E, k = s.k, R = T * k;
  size_t off = 0;
  auto take = [&](size_t bytes) { const size_t at = off; off += up256(bytes); return at; };
  L->topk_ids = take(R * 4);
  L->topk_w = take(R * 4);
  L->counts = take(E * 4);
  L->offsets = take((E + 1) * 4);
  L->perm = take(R * 4);
  L->inv_perm = take(R * 4);
  L->xq = take(T * H);
  L->sfx = take(H / 128 * T * 4);
  L->xq_perm = take(R * H);
  L->sfx_perm = take(H / 128 * R * 4);
  L->hq = take(R * F);
  L->sfh = take(F / 128 * R * 4);
  L->y_perm = take(R * H * 2);
  L->total = off;
}
moe_status check_mx_shape(const moe_ctx* ctx) {
  return (ctx->shape.H % 128 == 0 && ctx->shape.F % 128 == 0) ? MOE_OK : MOE_ERR_UNSUPPORTED_SHAPE;
}
}  // namespace
extern "C" {

moe_status moe_quantize_rows_mx(moe_ctx* ctx, const void* in_bf16, int64_t rows, int32_t cols, void* codes,
                                uint32_t* sf_words, void* stream) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  ctx->last_launches = 0;
  if (rows < 0 || cols <= 0 || cols % 128 != 0) return MOE_ERR_INVALID_ARG;
  if (rows == 0) return MOE_OK;
  if (!in_bf16 || !codes || !sf_words || !aligned16(in_bf16) || !aligned16(codes) || !aligned16(sf_words))
    return MOE_ERR_INVALID_ARG;
  return moe::launch_quantize_rows_mx(ctx, in_bf16, rows, cols, codes, sf_words, static_cast<cudaStream_t>(stream)) ==
                 cudaSuccess
             ? MOE_OK
             : MOE_ERR_CUDA;
}

moe_status moe_dispatch_mx(moe_ctx* ctx, const void* xq, const uint32_t* sfx, const int32_t* inv_perm, void* xq_perm,
                           uint32_t* sfx_perm, void* stream) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  st = check_mx_shape(ctx);
  if (st != MOE_OK) return st;
  begin_call(ctx, 3, stream);
  if (ctx->shape.T == 0) return MOE_OK;
  const void* ptrs[] = {xq, sfx, inv_perm, xq_perm, sfx_perm};
  for (const void* q : ptrs)
    if (!q || !aligned16(q)) return MOE_ERR_INVALID_ARG;
  return moe::launch_dispatch_mx(ctx, xq, sfx, inv_perm, xq_perm, sfx_perm, static_cast<cudaStream_t>(stream)) ==
                 cudaSuccess
             ? MOE_OK
             : MOE_ERR_CUDA;
}

moe_status moe_expert_ffn_mx(moe_ctx* ctx, const moe_mx_ffn_args* a, void* stream) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  st = check_mx_shape(ctx);
  if (st != MOE_OK) return st;
  begin_call(ctx, 4, stream);
  if (!a) return MOE_ERR_INVALID_ARG;
  if (ctx->shape.T == 0) return MOE_OK;
  const void* ptrs[] = {a->xq_perm, a->sfx_perm, a->offsets, a->wq_gate, a->sf_gate, a->wq_up, a->sf_up,
                        a->wq_down, a->sf_down, a->hq_ws, a->sfh_ws, a->y_perm};
  for (const void* q : ptrs)
    if (!q || !aligned16(q)) return MOE_ERR_INVALID_ARG;
  if (!aligned16(a->h_fp32_debug)) return MOE_ERR_INVALID_ARG;
  return moe::launch_expert_ffn_mx(ctx, a, static_cast<cudaStream_t>(stream));
}

moe_status moe_get_workspace_layout_mx(const moe_shape* shape, moe_workspace_layout_mx* out_layout) {
  if (!out_layout) return MOE_ERR_INVALID_ARG;
  std::memset(out_layout, 0, sizeof(*out_layout));
  const moe_status st = check_shape(shape);
  if (st != MOE_OK) return st;
  if (shape->H % 128 != 0 || shape->F % 128 != 0) return MOE_ERR_UNSUPPORTED_SHAPE;
  fill_layout_mx(*shape, out_layout);
  return MOE_OK;
}

moe_status moe_fused_forward_mx(moe_ctx* ctx, const void* x, const float* logits, const void* wq_gate,
                                const uint32_t* sf_gate, const void* wq_up, const uint32_t* sf_up, const void* wq_down,
                                const uint32_t* sf_down, void* out, void* workspace, size_t workspace_bytes,
                                void* stream) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  st = check_mx_shape(ctx);
  if (st != MOE_OK) return st;
  const moe_shape& s = ctx->shape;
  if (s.T == 0) { ctx->last_launches = 0; return MOE_OK; }
  const void* ptrs[] = {x, logits, wq_gate, sf_gate, wq_up, sf_up, wq_down, sf_down, out};
  for (const void* q : ptrs)
    if (!q || !aligned16(q)) return MOE_ERR_INVALID_ARG;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MOE_ERR_INVALID_ARG;
  moe_workspace_layout_mx L;
  fill_layout_mx(s, &L);
  if (workspace_bytes < L.total) return MOE_ERR_WORKSPACE_TOO_SMALL;
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  int32_t* topk_ids = reinterpret_cast<int32_t*>(ws + L.topk_ids);
  float* topk_w = reinterpret_cast<float*>(ws + L.topk_w);
  int32_t* counts = reinterpret_cast<int32_t*>(ws + L.counts);
  int32_t* offsets = reinterpret_cast<int32_t*>(ws + L.offsets);
  int32_t* perm = reinterpret_cast<int32_t*>(ws + L.perm);
  int32_t* inv_perm = reinterpret_cast<int32_t*>(ws + L.inv_perm);
  uint32_t* sfx = reinterpret_cast<uint32_t*>(ws + L.sfx);
  uint32_t* sfx_perm = reinterpret_cast<uint32_t*>(ws + L.sfx_perm);
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  begin_call(ctx, 0, stream);
  st = check_logits_on_host(ctx, logits, cs);
  if (st != MOE_OK) return st;
  if (moe::launch_plan_routing(ctx, logits, topk_ids, topk_w, counts, offsets, perm, inv_perm, cs) != cudaSuccess)
    return MOE_ERR_CUDA;
  if (moe::launch_quantize_rows_mx(ctx, x, s.T, s.H, ws + L.xq, sfx, cs) != cudaSuccess) return MOE_ERR_CUDA;
  if (moe::launch_dispatch_mx(ctx, ws + L.xq, sfx, inv_perm, ws + L.xq_perm, sfx_perm, cs) != cudaSuccess)
    return MOE_ERR_CUDA;
  moe_mx_ffn_args a{};
  a.xq_perm = ws + L.xq_perm;
  a.sfx_perm = sfx_perm;
  a.offsets = offsets;
  a.wq_gate = wq_gate;
  a.sf_gate = sf_gate;
  a.wq_up = wq_up;
  a.sf_up = sf_up;
  a.wq_down = wq_down;
  a.sf_down = sf_down;
  a.hq_ws = ws + L.hq;
  a.sfh_ws = reinterpret_cast<uint32_t*>(ws + L.sfh);
  a.y_perm = ws + L.y_perm;
  a.h_fp32_debug = nullptr;
  st = moe::launch_expert_ffn_mx(ctx, &a, cs);
  if (st != MOE_OK) return st;
  if (moe::launch_combine(ctx, ws + L.y_perm, inv_perm, topk_w, out, cs) != cudaSuccess) return MOE_ERR_CUDA;
  return MOE_OK;
}

moe_status moe_fused_forward_host(moe_ctx* ctx, const void* x_host, const float* logits_host,
                                  const void* w_gate, const void* w_up, const void* w_down,
                                  void* out_host, void* workspace, size_t workspace_bytes,
                                  const moe_tuning* tuning, void* stream) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  const moe_shape& s = ctx->shape;
  if (s.T == 0) { ctx->last_launches = 0; return MOE_OK; }
  if (!x_host || !logits_host || !out_host || !workspace) return MOE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MOE_ERR_INVALID_ARG;
  moe_workspace_layout L;
  fill_layout(s, &L);
  if (workspace_bytes < L.total) return MOE_ERR_WORKSPACE_TOO_SMALL;
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const size_t act_bytes = static_cast<size_t>(s.T) * s.H * 2;
  const size_t logit_bytes = static_cast<size_t>(s.T) * s.E * 4;
  if (cudaMemcpyAsync(ws + L.x_stage, x_host, act_bytes, cudaMemcpyHostToDevice, cs) != cudaSuccess) return MOE_ERR_CUDA;
  if (cudaMemcpyAsync(ws + L.logits_stage, logits_host, logit_bytes, cudaMemcpyHostToDevice, cs) != cudaSuccess)
    return MOE_ERR_CUDA;
  st = moe_fused_forward(ctx, ws + L.x_stage, reinterpret_cast<const float*>(ws + L.logits_stage), w_gate, w_up,
                         w_down, ws + L.out_stage, workspace, workspace_bytes, tuning, stream);
  if (st != MOE_OK) return st;
  if (cudaMemcpyAsync(out_host, ws + L.out_stage, act_bytes, cudaMemcpyDeviceToHost, cs) != cudaSuccess)
    return MOE_ERR_CUDA;
  return MOE_OK;
}

moe_status moe_fused_forward_host_pipelined(moe_ctx* ctx, const void* x_host, const float* logits_host,
                                            const void* w_gate, const void* w_up, const void* w_down,
                                            void* out_host, void* workspace, size_t workspace_bytes,
                                            const moe_tuning* tuning, void* stream) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  const moe_shape& s = ctx->shape;
  if (s.T == 0) { ctx->last_launches = 0; return MOE_OK; }
  if (!x_host || !logits_host || !out_host || !workspace) return MOE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MOE_ERR_INVALID_ARG;
  moe_workspace_layout L;
  fill_layout(s, &L);
  if (workspace_bytes < L.total) return MOE_ERR_WORKSPACE_TOO_SMALL;
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const int slot = ctx->pipe_slot;
  unsigned char* x_dev = ws + (slot ? L.x_stage_b : L.x_stage);
  unsigned char* lg_dev = ws + (slot ? L.logits_stage_b : L.logits_stage);
  unsigned char* out_dev = ws + (slot ? L.out_stage_b : L.out_stage);
  const size_t act_bytes = static_cast<size_t>(s.T) * s.H * 2;
  const size_t logit_bytes = static_cast<size_t>(s.T) * s.E * 4;
  // input copy: once the layer that last read this slot (two calls ago) has finished
  bool ok = cudaStreamWaitEvent(ctx->s_h2d, ctx->ev_compute[slot], 0) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(x_dev, x_host, act_bytes, cudaMemcpyHostToDevice, ctx->s_h2d) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(lg_dev, logits_host, logit_bytes, cudaMemcpyHostToDevice, ctx->s_h2d) == cudaSuccess;
  ok = ok && cudaEventRecord(ctx->ev_h2d[slot], ctx->s_h2d) == cudaSuccess;
  // the layer: after its inputs have landed and the slot's previous output has left
  ok = ok && cudaStreamWaitEvent(cs, ctx->ev_h2d[slot], 0) == cudaSuccess;
  ok = ok && cudaStreamWaitEvent(cs, ctx->ev_d2h[slot], 0) == cudaSuccess;
  if (!ok) return MOE_ERR_CUDA;
  st = moe_fused_forward(ctx, x_dev, reinterpret_cast<const float*>(lg_dev), w_gate, w_up, w_down, out_dev, workspace,
                         workspace_bytes, tuning, stream);
  if (st != MOE_OK) return st;
  ok = cudaEventRecord(ctx->ev_compute[slot], cs) == cudaSuccess;
  // output copy: overlaps the next call's layer
  ok = ok && cudaStreamWaitEvent(ctx->s_d2h, ctx->ev_compute[slot], 0) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(out_host, out_dev, act_bytes, cudaMemcpyDeviceToHost, ctx->s_d2h) == cudaSuccess;
  ok = ok && cudaEventRecord(ctx->ev_d2h[slot], ctx->s_d2h) == cudaSuccess;
  if (!ok) return MOE_ERR_CUDA;
  ctx->pipe_slot = slot ^ 1;
  return MOE_OK;
}

moe_status moe_host_pipeline_flush(moe_ctx* ctx, void* stream) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  for (int i = 0; i < 2; ++i) {
    if (cudaStreamWaitEvent(cs, ctx->ev_d2h[i], 0) != cudaSuccess) return MOE_ERR_CUDA;
    if (cudaStreamWaitEvent(cs, ctx->ev_h2d[i], 0) != cudaSuccess) return MOE_ERR_CUDA;
  }
  return MOE_OK;
}

moe_status moe_last_device_status(moe_ctx* ctx, int32_t* code, int32_t* detail, void* stream) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  if (!code || !detail) return MOE_ERR_INVALID_ARG;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  int32_t host[2] = {0, 0};
  if (cudaMemcpyAsync(host, ctx->d_status, sizeof(host), cudaMemcpyDeviceToHost, cs) != cudaSuccess) return MOE_ERR_CUDA;
  if (cudaMemsetAsync(ctx->d_status, 0, sizeof(host), cs) != cudaSuccess) return MOE_ERR_CUDA;
  if (cudaStreamSynchronize(cs) != cudaSuccess) return MOE_ERR_CUDA;
  *code = host[0];
  *detail = host[1];
  return MOE_OK;
}

int32_t moe_last_launch_count(const moe_ctx* ctx) { return ctx ? ctx->last_launches : 0; }

moe_status moe_get_ffn_trace(moe_ctx* ctx, uint64_t* counters_host, int32_t capacity, int32_t* num_ctas, void* stream) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  if (!counters_host || !num_ctas) return MOE_ERR_INVALID_ARG;
  const int32_t need = 2 * ctx->num_sms * kMoeTraceFields;
  *num_ctas = ctx->num_sms;
  if (capacity < need) return MOE_ERR_INVALID_ARG;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(counters_host, ctx->d_trace, static_cast<size_t>(need) * 8, cudaMemcpyDeviceToHost, cs) !=
      cudaSuccess)
    return MOE_ERR_CUDA;
  return cudaStreamSynchronize(cs) == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

moe_status moe_get_ffn_order(moe_ctx* ctx, int32_t* codes_host, int32_t capacity, int32_t* num_ctas,
                             int32_t* codes_per_cta, void* stream) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  if (!codes_host || !num_ctas || !codes_per_cta) return MOE_ERR_INVALID_ARG;
  const int32_t need = ctx->num_sms * kMoeOrderLogCap;
  *num_ctas = ctx->num_sms;
  *codes_per_cta = kMoeOrderLogCap;
  if (capacity < need) return MOE_ERR_INVALID_ARG;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(codes_host, ctx->d_order, static_cast<size_t>(need) * 4, cudaMemcpyDeviceToHost, cs) != cudaSuccess)
    return MOE_ERR_CUDA;
  return cudaStreamSynchronize(cs) == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

moe_status moe_set_kernel_timing(moe_ctx* ctx, int32_t enable) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  ctx->timing = enable ? 1 : 0;
  for (int sl = 0; sl < kMoeTimingSlots; ++sl) ctx->ev_recorded[sl] = 0;
  return MOE_OK;
}

moe_status moe_get_kernel_times_back(moe_ctx* ctx, int32_t calls_back, float* ms_host, int32_t n) {
  moe_status st = check_ctx(ctx);
  if (st != MOE_OK) return st;
  if (!ms_host || n != kMoeKernels || calls_back < 0 || calls_back >= kMoeTimingSlots) return MOE_ERR_INVALID_ARG;
  const int sl = ((ctx->ev_slot - calls_back) % kMoeTimingSlots + kMoeTimingSlots) % kMoeTimingSlots;
  for (int i = 0; i < kMoeKernels; ++i) {
    ms_host[i] = -1.f;
    const uint32_t need = (1u << i) | (1u << (i + 1));
    if ((ctx->ev_recorded[sl] & need) != need) continue;
    if (cudaEventSynchronize(ctx->ev[sl][i + 1]) != cudaSuccess) return MOE_ERR_CUDA;
    if (cudaEventElapsedTime(&ms_host[i], ctx->ev[sl][i], ctx->ev[sl][i + 1]) != cudaSuccess) return MOE_ERR_CUDA;
  }
  return MOE_OK;
}

moe_status moe_get_kernel_times(moe_ctx* ctx, float* ms_host, int32_t n) {
  return moe_get_kernel_times_back(ctx, 0, ms_host, n);
}

}  // extern "C"
