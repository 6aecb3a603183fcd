"""ctypes binding of libmoe_b200.so: the same names as include/moe.h, argument marshalling only.

Tensors are torch CUDA tensors (torch is used for device memory and streams); bf16 buffers are
``torch.bfloat16`` (or int16/uint16 views of the same bytes).  Every step of the path runs inside the
library's kernels.  Loading fails loudly when the library has not been built: there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libmoe_b200.so")

MOE_OK = 0
STATUS_NAMES = {
    0: "MOE_OK", 1: "MOE_ERR_INVALID_ARG", 2: "MOE_ERR_UNSUPPORTED_SHAPE", 3: "MOE_ERR_WORKSPACE_TOO_SMALL",
    4: "MOE_ERR_BAD_ROUTING", 5: "MOE_ERR_CUDA", 6: "MOE_ERR_TIMEOUT", 7: "MOE_ERR_UNSUPPORTED",
    8: "MOE_ERR_STATIC_SCRATCH_TOO_SMALL",
}

EXPORTS = (
    "moe_status_string", "moe_create", "moe_destroy", "moe_workspace_bytes", "moe_get_workspace_layout",
    "moe_plan_routing", "moe_dispatch", "moe_expert_ffn", "moe_combine", "moe_fused_forward",
    "moe_fused_forward_host", "moe_last_device_status", "moe_last_launch_count", "moe_set_kernel_timing",
    "moe_get_kernel_times", "moe_plan_routing_static", "moe_get_ffn_trace", "moe_probe_mma_cycles",
    "moe_get_ffn_order", "moe_fused_forward_host_pipelined", "moe_host_pipeline_flush", "moe_quantize_rows",
    "moe_dispatch_fp8", "moe_expert_ffn_fp8", "moe_get_workspace_layout_fp8", "moe_fused_forward_fp8",
    "moe_set_active_tokens", "moe_plan_routing_from_topk", "moe_router_weight_bytes", "moe_router_scratch_bytes",
    "moe_router_prepare", "moe_route_tokens", "moe_fused_forward_routed", "moe_quantize_rows_mx", "moe_dispatch_mx",
    "moe_expert_ffn_mx", "moe_get_workspace_layout_mx", "moe_fused_forward_mx", "moe_probe_mma_cycles_kind",
    "moe_parse_tuning", "moe_get_kernel_times_back",
)

TIMING_SLOTS = 32     # timed calls whose per-kernel events the library keeps (moe_get_kernel_times_back)

TRACE_FIELDS = ("producer_span", "producer_wait_stage", "mma_wait_operands", "mma_wait_accumulator",
                "epilogue_wait_accumulator", "epilogue_store_span", "tiles", "epilogue_pacing_gap",
                "swapped_tiles", "swapped_tile_clocks", "swapped_wait_operands", "full_tile_clocks")

KERNEL_NAMES = ("route_topk_hist", "route_scan", "route_scatter", "dispatch_rows", "expert_ffn_linear1",
                "expert_ffn_linear2", "combine_rows")


class MoeError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {STATUS_NAMES.get(code, code)}")


class moe_shape(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("T", "H", "F", "E", "k", "ep_size", "ep_rank")]


class moe_tuning(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("store_burst_tiles", "interleave_mode", "interleave_k", "schedule",
                                         "dep_lead_D", "debug_flags")]


class moe_workspace_layout(C.Structure):
    _fields_ = [(n, C.c_size_t) for n in ("topk_ids", "topk_w", "counts", "offsets", "perm", "inv_perm", "x_perm",
                                          "h", "y_perm", "x_stage", "logits_stage", "out_stage", "x_stage_b",
                                          "logits_stage_b", "out_stage_b", "total")]


class moe_fp8_ffn_args(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("xq_perm", "sx_perm", "offsets", "wq_gate", "s_gate", "wq_up", "s_up",
                                          "wq_down", "s_down", "h_ws", "hq_ws", "sh_ws", "y_perm")]


class moe_workspace_layout_fp8(C.Structure):
    _fields_ = [(n, C.c_size_t) for n in ("topk_ids", "topk_w", "counts", "offsets", "perm", "inv_perm", "xq", "sx",
                                          "xq_perm", "sx_perm", "h", "hq", "sh", "y_perm", "total")]


class moe_mx_ffn_args(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("xq_perm", "sfx_perm", "offsets", "wq_gate", "sf_gate", "wq_up", "sf_up",
                                          "wq_down", "sf_down", "hq_ws", "sfh_ws", "y_perm", "h_fp32_debug")]


class moe_workspace_layout_mx(C.Structure):
    _fields_ = [(n, C.c_size_t) for n in ("topk_ids", "topk_w", "counts", "offsets", "perm", "inv_perm", "xq", "sfx",
                                          "xq_perm", "sfx_perm", "hq", "sfh", "y_perm", "total")]


_lib = None


def load_library() -> C.CDLL:
    """dlopen the library (once) and declare the prototypes.  Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2607_23264_b200.build` "
            "(the MoE path has no CPU or PyTorch fallback)")
    lib = C.CDLL(_LIB_PATH)
    vp, i32p, f32p = C.c_void_p, C.c_void_p, C.c_void_p
    lib.moe_status_string.restype = C.c_char_p
    lib.moe_status_string.argtypes = [C.c_int]
    lib.moe_create.argtypes = [C.POINTER(C.c_void_p), C.POINTER(moe_shape), C.c_int]
    lib.moe_destroy.argtypes = [C.c_void_p]
    lib.moe_destroy.restype = None
    lib.moe_workspace_bytes.argtypes = [C.POINTER(moe_shape)]
    lib.moe_workspace_bytes.restype = C.c_size_t
    lib.moe_get_workspace_layout.argtypes = [C.POINTER(moe_shape), C.POINTER(moe_workspace_layout)]
    lib.moe_plan_routing.argtypes = [vp, f32p, i32p, f32p, i32p, i32p, i32p, i32p, vp]
    lib.moe_plan_routing_static.argtypes = [C.POINTER(moe_shape), f32p, i32p, f32p, i32p, i32p, i32p, i32p, vp]
    lib.moe_dispatch.argtypes = [vp, vp, i32p, vp, vp]
    lib.moe_expert_ffn.argtypes = [vp, vp, i32p, vp, vp, vp, vp, vp, f32p, C.POINTER(moe_tuning), vp]
    lib.moe_combine.argtypes = [vp, vp, i32p, f32p, vp, vp]
    lib.moe_fused_forward.argtypes = [vp, vp, f32p, vp, vp, vp, vp, vp, C.c_size_t, C.POINTER(moe_tuning), vp]
    lib.moe_fused_forward_host.argtypes = [vp, vp, f32p, vp, vp, vp, vp, vp, C.c_size_t, C.POINTER(moe_tuning), vp]
    lib.moe_fused_forward_host_pipelined.argtypes = lib.moe_fused_forward_host.argtypes
    lib.moe_host_pipeline_flush.argtypes = [vp, vp]
    lib.moe_quantize_rows.argtypes = [vp, vp, C.c_int64, C.c_int32, vp, f32p, vp]
    lib.moe_dispatch_fp8.argtypes = [vp, vp, f32p, i32p, vp, f32p, vp]
    lib.moe_expert_ffn_fp8.argtypes = [vp, C.POINTER(moe_fp8_ffn_args), C.POINTER(moe_tuning), vp]
    lib.moe_get_workspace_layout_fp8.argtypes = [C.POINTER(moe_shape), C.POINTER(moe_workspace_layout_fp8)]
    lib.moe_fused_forward_fp8.argtypes = [vp, vp, f32p, vp, f32p, vp, f32p, vp, f32p, vp, vp, C.c_size_t,
                                          C.POINTER(moe_tuning), vp]
    lib.moe_set_active_tokens.argtypes = [vp, C.c_int32]
    lib.moe_plan_routing_from_topk.argtypes = [vp, i32p, i32p, i32p, i32p, i32p, i32p, vp]
    lib.moe_router_weight_bytes.argtypes = [C.POINTER(moe_shape)]
    lib.moe_router_weight_bytes.restype = C.c_size_t
    lib.moe_router_scratch_bytes.argtypes = [C.POINTER(moe_shape)]
    lib.moe_router_scratch_bytes.restype = C.c_size_t
    lib.moe_router_prepare.argtypes = [vp, f32p, vp, vp]
    lib.moe_route_tokens.argtypes = [vp, vp, vp, f32p, vp, C.c_size_t, f32p, i32p, f32p, i32p, i32p, i32p, i32p, vp]
    lib.moe_fused_forward_routed.argtypes = [vp, vp, vp, f32p, vp, vp, vp, vp, vp, C.c_size_t, vp, C.c_size_t,
                                             C.POINTER(moe_tuning), vp]
    lib.moe_quantize_rows_mx.argtypes = [vp, vp, C.c_int64, C.c_int32, vp, vp, vp]
    lib.moe_dispatch_mx.argtypes = [vp, vp, vp, i32p, vp, vp, vp]
    lib.moe_expert_ffn_mx.argtypes = [vp, C.POINTER(moe_mx_ffn_args), vp]
    lib.moe_get_workspace_layout_mx.argtypes = [C.POINTER(moe_shape), C.POINTER(moe_workspace_layout_mx)]
    lib.moe_fused_forward_mx.argtypes = [vp, vp, f32p, vp, vp, vp, vp, vp, vp, vp, vp, C.c_size_t, vp]
    lib.moe_last_device_status.argtypes = [vp, C.POINTER(C.c_int32), C.POINTER(C.c_int32), vp]
    lib.moe_last_launch_count.argtypes = [vp]
    lib.moe_last_launch_count.restype = C.c_int32
    lib.moe_set_kernel_timing.argtypes = [vp, C.c_int32]
    lib.moe_get_kernel_times.argtypes = [vp, C.POINTER(C.c_float), C.c_int32]
    lib.moe_get_kernel_times_back.argtypes = [vp, C.c_int32, C.POINTER(C.c_float), C.c_int32]
    lib.moe_probe_mma_cycles.argtypes = [vp, C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_double), vp]
    lib.moe_probe_mma_cycles_kind.argtypes = [vp, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_double), vp]
    lib.moe_get_ffn_order.argtypes = [vp, C.POINTER(C.c_int32), C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_int32), vp]
    lib.moe_get_ffn_trace.argtypes = [vp, C.POINTER(C.c_uint64), C.c_int32, C.POINTER(C.c_int32), vp]
    for name in EXPORTS:
        if name not in ("moe_status_string", "moe_destroy", "moe_workspace_bytes", "moe_last_launch_count",
                        "moe_router_weight_bytes", "moe_router_scratch_bytes"):
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def _ptr(t):
    """Device (or host) address of a tensor, None -> NULL."""
    if t is None:
        return None
    if isinstance(t, int):
        return C.c_void_p(t)
    if not t.is_contiguous():
        raise ValueError("tensors passed to the MoE library must be contiguous")
    return C.c_void_p(t.data_ptr())


def _stream(stream):
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _check(code: int, where: str):
    if code != MOE_OK:
        raise MoeError(code, where)


def make_tuning(store_burst_tiles=1, interleave_mode=0, interleave_k=1, schedule=0, dep_lead_D=0, debug_flags=0):
    return moe_tuning(store_burst_tiles, interleave_mode, interleave_k, schedule, dep_lead_D, debug_flags)


def moe_parse_tuning(text):
    """Parse a MOE_TUNING string.  Returns (moe_tuning, named_field: bool); raises MoeError on a bad string."""
    t = moe_tuning()
    named = C.c_int32(0)
    _check(load_library().moe_parse_tuning(None if text is None else text.encode(), C.byref(t), C.byref(named)),
           "moe_parse_tuning")
    return t, bool(named.value)


def _tuning_ref(tuning):
    return None if tuning is None else C.byref(tuning)


def moe_status_string(code: int) -> str:
    return load_library().moe_status_string(code).decode()


def moe_workspace_bytes(T, H, F, E, k) -> int:
    return load_library().moe_workspace_bytes(C.byref(moe_shape(T, H, F, E, k, 1, 0)))


def moe_get_workspace_layout(T, H, F, E, k) -> dict:
    L = moe_workspace_layout()
    _check(load_library().moe_get_workspace_layout(C.byref(moe_shape(T, H, F, E, k, 1, 0)), C.byref(L)),
           "moe_get_workspace_layout")
    return {n: getattr(L, n) for n, _ in moe_workspace_layout._fields_}


def moe_plan_routing_static(T, E, k, logits, topk_ids, topk_w, counts, offsets, perm, inv_perm, stream=None):
    """Routing plan through the entry point that allocates nothing and needs no context: its scratch is a
    fixed array inside the library (see include/moe.h for the size limit and the sharing rules)."""
    shape = moe_shape(T, 0, 0, E, k, 1, 0)
    _check(load_library().moe_plan_routing_static(C.byref(shape), _ptr(logits), _ptr(topk_ids), _ptr(topk_w),
                                                  _ptr(counts), _ptr(offsets), _ptr(perm), _ptr(inv_perm),
                                                  _stream(stream)), "moe_plan_routing_static")


@dataclass
class Context:
    """Owner of a moe_ctx*; methods carry the C function names."""
    T: int
    H: int
    F: int
    E: int
    k: int
    device: int = 0
    ep_size: int = 1
    ep_rank: int = 0

    def __post_init__(self):
        import torch
        self._lib = load_library()
        self._handle = C.c_void_p()
        torch.cuda.set_device(self.device)
        torch.cuda.init()
        torch.zeros(1, device=f"cuda:{self.device}")  # make sure the primary context exists and is current
        shape = moe_shape(self.T, self.H, self.F, self.E, self.k, self.ep_size, self.ep_rank)
        _check(self._lib.moe_create(C.byref(self._handle), C.byref(shape), self.device), "moe_create")

    @property
    def R(self):
        return self.T * self.k

    def close(self):
        if getattr(self, "_handle", None) and self._handle.value:
            self._lib.moe_destroy(self._handle)
            self._handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def moe_set_active_tokens(self, tokens: int):
        """Process `tokens` <= the creation T in the following calls (tensor arguments shrink accordingly)."""
        _check(self._lib.moe_set_active_tokens(self._handle, tokens), "moe_set_active_tokens")
        self.T = tokens

    def workspace_bytes(self) -> int:
        return moe_workspace_bytes(self.T, self.H, self.F, self.E, self.k)

    def workspace_layout(self) -> dict:
        return moe_get_workspace_layout(self.T, self.H, self.F, self.E, self.k)

    def moe_plan_routing(self, logits, topk_ids, topk_w, counts, offsets, perm, inv_perm, stream=None):
        _check(self._lib.moe_plan_routing(self._handle, _ptr(logits), _ptr(topk_ids), _ptr(topk_w), _ptr(counts),
                                          _ptr(offsets), _ptr(perm), _ptr(inv_perm), _stream(stream)),
               "moe_plan_routing")

    def moe_plan_routing_from_topk(self, topk_ids, topk_ids_checked, counts, offsets, perm, inv_perm, stream=None):
        _check(self._lib.moe_plan_routing_from_topk(self._handle, _ptr(topk_ids), _ptr(topk_ids_checked), _ptr(counts),
                                                    _ptr(offsets), _ptr(perm), _ptr(inv_perm), _stream(stream)),
               "moe_plan_routing_from_topk")

    def _shape(self):
        return moe_shape(self.T, self.H, self.F, self.E, self.k, self.ep_size, self.ep_rank)

    def router_weight_bytes(self) -> int:
        """Bytes of the prepared router weights (two bf16 terms of W_r, expert rows padded)."""
        return int(self._lib.moe_router_weight_bytes(C.byref(self._shape())))

    def router_scratch_bytes(self) -> int:
        """Bytes of the scratch moe_route_tokens needs for the K-split partial logits."""
        return int(self._lib.moe_router_scratch_bytes(C.byref(self._shape())))

    def moe_router_prepare(self, w_router, w_split, stream=None):
        _check(self._lib.moe_router_prepare(self._handle, _ptr(w_router), _ptr(w_split), _stream(stream)),
               "moe_router_prepare")

    def moe_route_tokens(self, x, w_split, bias, scratch, logits_out, topk_ids, topk_w, counts, offsets, perm,
                         inv_perm, stream=None):
        _check(self._lib.moe_route_tokens(self._handle, _ptr(x), _ptr(w_split), _ptr(bias), _ptr(scratch),
                                          scratch.numel() * scratch.element_size(), _ptr(logits_out), _ptr(topk_ids),
                                          _ptr(topk_w), _ptr(counts), _ptr(offsets), _ptr(perm), _ptr(inv_perm),
                                          _stream(stream)), "moe_route_tokens")

    def moe_fused_forward_routed(self, x, w_split, bias, w_gate, w_up, w_down, out, workspace, router_scratch,
                                 tuning=None, stream=None):
        _check(self._lib.moe_fused_forward_routed(self._handle, _ptr(x), _ptr(w_split), _ptr(bias), _ptr(w_gate),
                                                  _ptr(w_up), _ptr(w_down), _ptr(out), _ptr(workspace),
                                                  workspace.numel() * workspace.element_size(), _ptr(router_scratch),
                                                  router_scratch.numel() * router_scratch.element_size(),
                                                  _tuning_ref(tuning), _stream(stream)), "moe_fused_forward_routed")

    def moe_dispatch(self, x, inv_perm, x_perm, stream=None):
        _check(self._lib.moe_dispatch(self._handle, _ptr(x), _ptr(inv_perm), _ptr(x_perm), _stream(stream)),
               "moe_dispatch")

    def moe_expert_ffn(self, x_perm, offsets, w_gate, w_up, w_down, h_ws, y_perm, h_fp32_debug=None, tuning=None,
                       stream=None):
        _check(self._lib.moe_expert_ffn(self._handle, _ptr(x_perm), _ptr(offsets), _ptr(w_gate), _ptr(w_up),
                                        _ptr(w_down), _ptr(h_ws), _ptr(y_perm), _ptr(h_fp32_debug),
                                        _tuning_ref(tuning), _stream(stream)), "moe_expert_ffn")

    def moe_combine(self, y_perm, inv_perm, topk_w, out, stream=None):
        _check(self._lib.moe_combine(self._handle, _ptr(y_perm), _ptr(inv_perm), _ptr(topk_w), _ptr(out),
                                     _stream(stream)), "moe_combine")

    def moe_fused_forward(self, x, logits, w_gate, w_up, w_down, out, workspace, tuning=None, stream=None):
        _check(self._lib.moe_fused_forward(self._handle, _ptr(x), _ptr(logits), _ptr(w_gate), _ptr(w_up),
                                           _ptr(w_down), _ptr(out), _ptr(workspace),
                                           workspace.numel() * workspace.element_size(), _tuning_ref(tuning),
                                           _stream(stream)), "moe_fused_forward")

    def moe_fused_forward_host(self, x_host, logits_host, w_gate, w_up, w_down, out_host, workspace, tuning=None,
                               stream=None):
        _check(self._lib.moe_fused_forward_host(self._handle, _ptr(x_host), _ptr(logits_host), _ptr(w_gate),
                                                _ptr(w_up), _ptr(w_down), _ptr(out_host), _ptr(workspace),
                                                workspace.numel() * workspace.element_size(), _tuning_ref(tuning),
                                                _stream(stream)), "moe_fused_forward_host")

    def moe_fused_forward_host_pipelined(self, x_host, logits_host, w_gate, w_up, w_down, out_host, workspace,
                                         tuning=None, stream=None):
        _check(self._lib.moe_fused_forward_host_pipelined(self._handle, _ptr(x_host), _ptr(logits_host), _ptr(w_gate),
                                                          _ptr(w_up), _ptr(w_down), _ptr(out_host), _ptr(workspace),
                                                          workspace.numel() * workspace.element_size(),
                                                          _tuning_ref(tuning), _stream(stream)),
               "moe_fused_forward_host_pipelined")

    def moe_host_pipeline_flush(self, stream=None):
        _check(self._lib.moe_host_pipeline_flush(self._handle, _stream(stream)), "moe_host_pipeline_flush")

    # ---- FP8 (E4M3, W8A8) variant
    def workspace_layout_fp8(self) -> dict:
        L = moe_workspace_layout_fp8()
        shape = moe_shape(self.T, self.H, self.F, self.E, self.k, 1, 0)
        _check(self._lib.moe_get_workspace_layout_fp8(C.byref(shape), C.byref(L)), "moe_get_workspace_layout_fp8")
        return {n: getattr(L, n) for n, _ in moe_workspace_layout_fp8._fields_}

    def moe_quantize_rows(self, in_bf16, rows, cols, codes, scales, stream=None):
        _check(self._lib.moe_quantize_rows(self._handle, _ptr(in_bf16), rows, cols, _ptr(codes), _ptr(scales),
                                           _stream(stream)), "moe_quantize_rows")

    def moe_dispatch_fp8(self, xq, sx, inv_perm, xq_perm, sx_perm, stream=None):
        _check(self._lib.moe_dispatch_fp8(self._handle, _ptr(xq), _ptr(sx), _ptr(inv_perm), _ptr(xq_perm),
                                          _ptr(sx_perm), _stream(stream)), "moe_dispatch_fp8")

    def moe_expert_ffn_fp8(self, xq_perm, sx_perm, offsets, wq_gate, s_gate, wq_up, s_up, wq_down, s_down, h_ws, hq_ws,
                           sh_ws, y_perm, tuning=None, stream=None):
        tensors = (xq_perm, sx_perm, offsets, wq_gate, s_gate, wq_up, s_up, wq_down, s_down, h_ws, hq_ws, sh_ws, y_perm)
        args = moe_fp8_ffn_args(*[None if t is None else t.data_ptr() for t in tensors])
        _check(self._lib.moe_expert_ffn_fp8(self._handle, C.byref(args), _tuning_ref(tuning), _stream(stream)),
               "moe_expert_ffn_fp8")

    def moe_fused_forward_fp8(self, x, logits, wq_gate, s_gate, wq_up, s_up, wq_down, s_down, out, workspace,
                              tuning=None, stream=None):
        _check(self._lib.moe_fused_forward_fp8(self._handle, _ptr(x), _ptr(logits), _ptr(wq_gate), _ptr(s_gate),
                                               _ptr(wq_up), _ptr(s_up), _ptr(wq_down), _ptr(s_down), _ptr(out),
                                               _ptr(workspace), workspace.numel() * workspace.element_size(),
                                               _tuning_ref(tuning), _stream(stream)), "moe_fused_forward_fp8")

    def workspace_layout_mx(self) -> dict:
        L = moe_workspace_layout_mx()
        _check(self._lib.moe_get_workspace_layout_mx(C.byref(self._shape()), C.byref(L)), "moe_get_workspace_layout_mx")
        return {n: getattr(L, n) for n, _ in moe_workspace_layout_mx._fields_}

    def moe_quantize_rows_mx(self, in_bf16, rows, cols, codes, sf_words, stream=None):
        _check(self._lib.moe_quantize_rows_mx(self._handle, _ptr(in_bf16), rows, cols, _ptr(codes), _ptr(sf_words),
                                              _stream(stream)), "moe_quantize_rows_mx")

    def moe_dispatch_mx(self, xq, sfx, inv_perm, xq_perm, sfx_perm, stream=None):
        _check(self._lib.moe_dispatch_mx(self._handle, _ptr(xq), _ptr(sfx), _ptr(inv_perm), _ptr(xq_perm),
                                         _ptr(sfx_perm), _stream(stream)), "moe_dispatch_mx")

    def moe_expert_ffn_mx(self, xq_perm, sfx_perm, offsets, wq_gate, sf_gate, wq_up, sf_up, wq_down, sf_down, hq_ws,
                          sfh_ws, y_perm, h_fp32_debug=None, stream=None):
        vals = [xq_perm, sfx_perm, offsets, wq_gate, sf_gate, wq_up, sf_up, wq_down, sf_down, hq_ws, sfh_ws, y_perm,
                h_fp32_debug]
        args = moe_mx_ffn_args(*[None if v is None else v.data_ptr() for v in vals])
        _check(self._lib.moe_expert_ffn_mx(self._handle, C.byref(args), _stream(stream)), "moe_expert_ffn_mx")

    def moe_fused_forward_mx(self, x, logits, wq_gate, sf_gate, wq_up, sf_up, wq_down, sf_down, out, workspace,
                             stream=None):
        _check(self._lib.moe_fused_forward_mx(self._handle, _ptr(x), _ptr(logits), _ptr(wq_gate), _ptr(sf_gate),
                                              _ptr(wq_up), _ptr(sf_up), _ptr(wq_down), _ptr(sf_down), _ptr(out),
                                              _ptr(workspace), workspace.numel() * workspace.element_size(),
                                              _stream(stream)), "moe_fused_forward_mx")

    def moe_last_device_status(self, stream=None):
        code, detail = C.c_int32(0), C.c_int32(0)
        _check(self._lib.moe_last_device_status(self._handle, C.byref(code), C.byref(detail), _stream(stream)),
               "moe_last_device_status")
        return code.value, detail.value

    def moe_last_launch_count(self) -> int:
        return self._lib.moe_last_launch_count(self._handle)

    def moe_get_ffn_trace(self, stream=None):
        """Wait counters of the last traced call as a numpy array [2 (Linear-1, Linear-2), CTAs, 8]."""
        import numpy as np
        cap = 2 * 1024 * len(TRACE_FIELDS)
        buf = (C.c_uint64 * cap)()
        n = C.c_int32(0)
        _check(self._lib.moe_get_ffn_trace(self._handle, buf, cap, C.byref(n), _stream(stream)), "moe_get_ffn_trace")
        a = np.frombuffer(buf, dtype=np.uint64)[: 2 * n.value * len(TRACE_FIELDS)]
        return a.reshape(2, n.value, len(TRACE_FIELDS)).copy()

    def moe_get_ffn_order(self, stream=None):
        """Tile codes each CTA drew in the last traced one-launch run: list (per CTA) of lists of
        (phase, index), the terminating -1 dropped."""
        cap = 1024 * 512
        buf = (C.c_int32 * cap)()
        n, per = C.c_int32(0), C.c_int32(0)
        _check(self._lib.moe_get_ffn_order(self._handle, buf, cap, C.byref(n), C.byref(per), _stream(stream)),
               "moe_get_ffn_order")
        out = []
        for g in range(n.value):
            seq = []
            for i in range(per.value):
                code = buf[g * per.value + i]
                if code < 0:
                    break
                seq.append((code >> 30, code & ((1 << 30) - 1)))
            out.append(seq)
        return out

    def moe_probe_mma_cycles(self, M: int, N: int, iters: int = 4096, stream=None) -> float:
        out = C.c_double(0.0)
        _check(self._lib.moe_probe_mma_cycles(self._handle, M, N, iters, C.byref(out), _stream(stream)),
               "moe_probe_mma_cycles")
        return out.value

    def moe_probe_mma_cycles_kind(self, kind: int, M: int, N: int, iters: int = 4096, stream=None) -> float:
        """kind 0 bf16, 1 E4M3, 2 block-scaled E4M3."""
        out = C.c_double(0.0)
        _check(self._lib.moe_probe_mma_cycles_kind(self._handle, kind, M, N, iters, C.byref(out), _stream(stream)),
               "moe_probe_mma_cycles_kind")
        return out.value

    def moe_set_kernel_timing(self, enable: bool):
        _check(self._lib.moe_set_kernel_timing(self._handle, 1 if enable else 0), "moe_set_kernel_timing")

    def moe_get_kernel_times(self) -> list:
        ms = (C.c_float * len(KERNEL_NAMES))()
        _check(self._lib.moe_get_kernel_times(self._handle, ms, len(KERNEL_NAMES)), "moe_get_kernel_times")
        return list(ms)

    def moe_get_kernel_times_back(self, calls_back: int) -> list:
        ms = (C.c_float * len(KERNEL_NAMES))()
        _check(self._lib.moe_get_kernel_times_back(self._handle, calls_back, ms, len(KERNEL_NAMES)),
               "moe_get_kernel_times_back")
        return list(ms)
