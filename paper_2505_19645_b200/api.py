"""Thin Python binding over the C ABI of ``libmoe_verify.so`` (argument marshalling only).

Every step of the layer runs in the library's CUDA kernels; torch is used for device memory
and streams.  There is no CPU fallback: if the library is missing or a call fails, an
exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libmoe_verify.so")

MOE_OK = 0
STATUS_NAMES = {0: "MOE_OK", 1: "MOE_ERR_INVALID_ARG", 2: "MOE_ERR_UNSUPPORTED",
                3: "MOE_ERR_WORKSPACE", 4: "MOE_ERR_CUDA", 5: "MOE_ERR_TIMEOUT"}

EXPORTS = ["moe_workspace_bytes", "moe_router_logits", "moe_route_topk", "moe_permute",
           "moe_grouped_swiglu", "moe_combine", "moe_verify_layer", "moe_check",
           "moe_last_launch_count", "moe_status_string", "moe_profile_stage",
           "moe_selftest_wait_limit", "moe_workspace_region", "moe_grouped_swiglu_static",
           "moe_check_static", "moe_selftest_wait_limit_static"]

STAGES = {"router_logits": 0, "route_topk": 1, "permute": 2, "plan": 3, "gate_up": 4, "down": 5,
          "combine": 6, "gather": 7}


class MoeError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %s (%s)" % (where, STATUS_NAMES.get(status, status),
                                                 status_string(status)))


class CConfig(ctypes.Structure):
    _fields_ = [("hidden", ctypes.c_int32), ("n_experts", ctypes.c_int32),
                ("top_k", ctypes.c_int32), ("inter", ctypes.c_int32),
                ("shared_inter", ctypes.c_int32), ("score_fn", ctypes.c_int32),
                ("renormalize", ctypes.c_int32), ("shared_gate", ctypes.c_int32),
                ("routed_scale", ctypes.c_float)]


class CWeights(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("w_router", "router_bias", "w_gate", "w_up", "w_down", "ws_gate", "ws_up",
                 "ws_down", "w_shared_gate")]


class CDebugOut(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("logits", "topk_idx", "topk_w", "counts", "offsets", "perm", "inv_perm",
                 "active", "n_active")]


_lib = None


def load_library():
    """Load libmoe_verify.so (built in-tree by ``paper_2505_19645_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            "CUDA library %s is missing: run `python -m paper_2505_19645_b200.build` "
            "(there is no CPU fallback)" % LIB_PATH)
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
    cfgp, wp = ctypes.POINTER(CConfig), ctypes.POINTER(CWeights)
    lib.moe_workspace_bytes.restype = sz
    lib.moe_workspace_bytes.argtypes = [cfgp, i32]
    lib.moe_router_logits.restype = i32
    lib.moe_router_logits.argtypes = [cfgp, wp, vp, i32, vp, vp, vp]
    lib.moe_route_topk.restype = i32
    lib.moe_route_topk.argtypes = [cfgp, vp, i32, vp, vp, vp]
    lib.moe_permute.restype = i32
    lib.moe_permute.argtypes = [cfgp, vp, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.moe_grouped_swiglu.restype = i32
    lib.moe_grouped_swiglu.argtypes = [cfgp, wp, vp, i32, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.moe_combine.restype = i32
    lib.moe_combine.argtypes = [cfgp, vp, vp, vp, vp, vp, i32, vp, vp]
    lib.moe_verify_layer.restype = i32
    lib.moe_verify_layer.argtypes = [cfgp, wp, vp, i32, i32, vp, ctypes.POINTER(CDebugOut), vp,
                                     sz, vp]
    lib.moe_check.restype = i32
    lib.moe_check.argtypes = [vp, vp]
    lib.moe_profile_stage.restype = i32
    lib.moe_profile_stage.argtypes = [i32, vp, vp]
    lib.moe_selftest_wait_limit.restype = i32
    lib.moe_selftest_wait_limit.argtypes = [vp, i32, vp]
    lib.moe_workspace_region.restype = i32
    lib.moe_workspace_region.argtypes = [cfgp, i32, i32, ctypes.POINTER(sz), ctypes.POINTER(sz)]
    lib.moe_grouped_swiglu_static.restype = i32
    lib.moe_grouped_swiglu_static.argtypes = [cfgp, wp, vp, i32] + [vp] * 7
    lib.moe_check_static.restype = i32
    lib.moe_check_static.argtypes = [vp]
    lib.moe_selftest_wait_limit_static.restype = i32
    lib.moe_selftest_wait_limit_static.argtypes = [i32, vp]
    lib.moe_last_launch_count.restype = i32
    lib.moe_last_launch_count.argtypes = []
    lib.moe_status_string.restype = ctypes.c_char_p
    lib.moe_status_string.argtypes = [i32]
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().moe_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != MOE_OK:
        raise MoeError(status, where)


def make_config(shape) -> CConfig:
    """``shape``: a workloads.LayerShape (or anything with the same attributes)."""
    return CConfig(shape.hidden, shape.n_experts, shape.top_k, shape.inter, shape.shared_inter,
                   shape.score_fn, shape.renormalize, shape.shared_gate, shape.routed_scale)


def _ptr(t, dtype=None):
    """Device address of a tensor as an int (ctypes converts it for a c_void_p argument)."""
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor (the library takes device pointers)")
    if not t.is_contiguous():
        raise ValueError("expected a contiguous tensor")
    if dtype is not None and t.dtype is not dtype:
        raise ValueError("expected dtype %s, got %s" % (dtype, t.dtype))
    return t.data_ptr()


def make_weights(w: dict) -> CWeights:
    """``w``: dict of CUDA tensors as produced by workloads.make_weights(device='cuda')."""
    bf, f32 = torch.bfloat16, torch.float32
    return CWeights(_ptr(w["w_router"], f32), _ptr(w.get("router_bias"), f32),
                    _ptr(w["w_gate"], bf), _ptr(w["w_up"], bf), _ptr(w["w_down"], bf),
                    _ptr(w.get("ws_gate"), bf), _ptr(w.get("ws_up"), bf), _ptr(w.get("ws_down"), bf),
                    _ptr(w.get("w_shared_gate"), bf))


try:  # the raw handle of torch's current stream without building a Stream object (about 1 us less)
    _raw_stream = torch._C._cuda_getCurrentRawStream
except AttributeError:  # pragma: no cover - older torch
    _raw_stream = None


def _stream_ptr(stream=None, device_index=None):
    if stream is not None:
        return stream.cuda_stream
    if _raw_stream is not None:
        return _raw_stream(torch.cuda.current_device() if device_index is None else device_index)
    return torch.cuda.current_stream().cuda_stream


def moe_workspace_bytes(cfg: CConfig, max_tokens: int) -> int:
    return int(load_library().moe_workspace_bytes(ctypes.byref(cfg), int(max_tokens)))


def alloc_workspace(cfg: CConfig, max_tokens: int, device="cuda") -> torch.Tensor:
    n = moe_workspace_bytes(cfg, max_tokens)
    if n == 0:
        raise MoeError(1, "moe_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=device)


def moe_router_logits(cfg, weights, x, logits, shared_scale=None, stream=None):
    T = x.shape[0]
    _check(load_library().moe_router_logits(
        ctypes.byref(cfg), ctypes.byref(weights), _ptr(x, torch.bfloat16), T,
        _ptr(logits, torch.float32), _ptr(shared_scale, torch.float32), _stream_ptr(stream)),
        "moe_router_logits")


def moe_route_topk(cfg, logits, topk_idx, topk_w, stream=None):
    T = logits.shape[0]
    _check(load_library().moe_route_topk(
        ctypes.byref(cfg), _ptr(logits, torch.float32), T, _ptr(topk_idx, torch.int32),
        _ptr(topk_w, torch.float32), _stream_ptr(stream)), "moe_route_topk")


@dataclass
class Grouping:
    counts: torch.Tensor
    offsets: torch.Tensor
    perm: torch.Tensor
    inv_perm: torch.Tensor
    active: torch.Tensor
    n_active: torch.Tensor


def alloc_grouping(cfg: CConfig, T: int, device="cuda") -> Grouping:
    E, A = cfg.n_experts, T * cfg.top_k
    mk = lambda n: torch.empty(n, dtype=torch.int32, device=device)  # noqa: E731
    return Grouping(mk(E), mk(E + 1), mk(A), mk(A), mk(E), mk(1))


def moe_permute(cfg, topk_idx, grouping: Grouping, stream=None):
    T = topk_idx.shape[0]
    g = grouping
    i32 = torch.int32
    _check(load_library().moe_permute(
        ctypes.byref(cfg), _ptr(topk_idx, i32), T, _ptr(g.counts, i32), _ptr(g.offsets, i32),
        _ptr(g.perm, i32), _ptr(g.inv_perm, i32), _ptr(g.active, i32), _ptr(g.n_active, i32),
        _stream_ptr(stream)), "moe_permute")


def moe_grouped_swiglu(cfg, weights, x, grouping: Grouping, y, shared_y, ws, stream=None):
    T = x.shape[0]
    g = grouping
    i32 = torch.int32
    _check(load_library().moe_grouped_swiglu(
        ctypes.byref(cfg), ctypes.byref(weights), _ptr(x, torch.bfloat16), T, _ptr(g.offsets, i32),
        _ptr(g.perm, i32), _ptr(g.active, i32), _ptr(g.n_active, i32), _ptr(y, torch.bfloat16),
        _ptr(shared_y, torch.bfloat16), _ptr(ws), ws.numel() * ws.element_size(),
        _stream_ptr(stream)), "moe_grouped_swiglu")


STATIC_SCRATCH_BYTES = 8 << 20


def moe_grouped_swiglu_static(cfg, weights, x, grouping: Grouping, y, shared_y, stream=None):
    """moe_grouped_swiglu for callers that cannot hand over a workspace (no allocation may
    happen where they run, e.g. a server with a frozen memory plan): scratch is a fixed
    array of STATIC_SCRATCH_BYTES inside the library, shared by all calls on the device.
    Raises MoeError(MOE_ERR_WORKSPACE) if the request does not fit.  Make the first call on
    a device outside stream capture; do not let two calls overlap on the GPU."""
    T = x.shape[0]
    g = grouping
    i32 = torch.int32
    lib = load_library()
    _check(lib.moe_grouped_swiglu_static(
        ctypes.byref(cfg), ctypes.byref(weights), _ptr(x, torch.bfloat16), T, _ptr(g.offsets, i32),
        _ptr(g.perm, i32), _ptr(g.active, i32), _ptr(g.n_active, i32), _ptr(y, torch.bfloat16),
        _ptr(shared_y, torch.bfloat16), _stream_ptr(stream)), "moe_grouped_swiglu_static")


def moe_check_static(stream=None):
    """moe_check for the static entry point: synchronises the stream and raises MoeError
    (MOE_ERR_TIMEOUT) if a bounded wait gave up in a static call since the last report."""
    _check(load_library().moe_check_static(_stream_ptr(stream)), "moe_check_static")


def moe_selftest_wait_limit_static(limit_us: int, stream=None):
    _check(load_library().moe_selftest_wait_limit_static(int(limit_us), _stream_ptr(stream)),
           "moe_selftest_wait_limit_static")


def workspace_regions(cfg: CConfig, T: int):
    """[(offset, bytes)] of every region a call with T tokens uses inside its workspace."""
    lib = load_library()
    out = []
    off, n = ctypes.c_size_t(), ctypes.c_size_t()
    i = 0
    while lib.moe_workspace_region(ctypes.byref(cfg), int(T), i, ctypes.byref(off),
                                   ctypes.byref(n)) == MOE_OK:
        out.append((int(off.value), int(n.value)))
        i += 1
    return out


def moe_combine(cfg, y, inv_perm, topk_w, shared_y, shared_scale, out, stream=None):
    T = out.shape[0]
    _check(load_library().moe_combine(
        ctypes.byref(cfg), _ptr(y, torch.bfloat16), _ptr(inv_perm, torch.int32),
        _ptr(topk_w, torch.float32), _ptr(shared_y, torch.bfloat16),
        _ptr(shared_scale, torch.float32), T, _ptr(out, torch.bfloat16), _stream_ptr(stream)),
        "moe_combine")


def alloc_debug(cfg: CConfig, T: int, device="cuda") -> dict:
    E, k = cfg.n_experts, cfg.top_k
    A = T * k
    i32, f32 = torch.int32, torch.float32
    mk = lambda shp, dt: torch.empty(shp, dtype=dt, device=device)  # noqa: E731
    return {"logits": mk((T, E), f32), "topk_idx": mk((T, k), i32), "topk_w": mk((T, k), f32),
            "counts": mk((E,), i32), "offsets": mk((E + 1,), i32), "perm": mk((A,), i32),
            "inv_perm": mk((A,), i32), "active": mk((E,), i32), "n_active": mk((1,), i32)}


def moe_verify_layer(cfg, weights, x, B: int, gamma: int, out, ws, dbg: dict | None = None,
                     stream=None):
    """One MoE FFN layer pass for B sequences x (gamma+1) tokens; x, out are [B*(gamma+1), H]."""
    cdbg = None
    if dbg is not None:
        cdbg = ctypes.byref(CDebugOut(*[_ptr(dbg.get(n)) for n, _ in CDebugOut._fields_]))
    status = _lib.moe_verify_layer(
        ctypes.byref(cfg), ctypes.byref(weights), _ptr(x, torch.bfloat16), int(B), int(gamma),
        _ptr(out, torch.bfloat16), cdbg, _ptr(ws), ws.nbytes,
        _stream_ptr(stream, x.device.index)) if _lib is not None else load_library() and None
    if status is None:   # first call: the library was not loaded yet
        return moe_verify_layer(cfg, weights, x, B, gamma, out, ws, dbg, stream)
    if status != MOE_OK:
        raise MoeError(status, "moe_verify_layer")


def moe_check(ws, stream=None):
    _check(load_library().moe_check(_ptr(ws), _stream_ptr(stream)), "moe_check")


def moe_selftest_wait_limit(ws, limit_us: int, stream=None):
    """Enqueue the bounded-wait self-test; moe_check(ws) then raises MOE_ERR_TIMEOUT."""
    _check(load_library().moe_selftest_wait_limit(_ptr(ws), int(limit_us), _stream_ptr(stream)),
           "moe_selftest_wait_limit")


def moe_profile_stage(stage, start_event=None, stop_event=None):
    """Record the two (already created) torch.cuda.Event objects around one kernel of every
    following moe_verify_layer call of this thread; stage None / -1 switches it off."""
    if stage is None or (isinstance(stage, int) and stage < 0):
        _check(load_library().moe_profile_stage(-1, None, None), "moe_profile_stage")
        return
    sid = STAGES[stage] if isinstance(stage, str) else int(stage)
    _check(load_library().moe_profile_stage(sid, ctypes.c_void_p(start_event.cuda_event),
                                            ctypes.c_void_p(stop_event.cuda_event)),
           "moe_profile_stage")


def moe_last_launch_count() -> int:
    return int(load_library().moe_last_launch_count())
