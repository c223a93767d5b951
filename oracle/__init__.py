"""ctypes shim over the plain-C CPU oracle (``moe_oracle.c``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the CPU-baseline leg of the
benchmark may import this package; the CUDA product path never does.  The oracle is a
token-major fp64 restatement of the sparse-MoE FFN layer (router -> top-k -> per-token
expert SwiGLU FFNs -> gate-weighted sum, plus an optional shared expert) and of the
closed forms of Sec. 3.2 (Eq. N(t), Eq. T_exp, Eq. T_thres).  It shares no code with
the CUDA path.

Arrays are numpy arrays (bf16 data as ``uint16`` bit patterns); torch CPU tensors are
accepted and viewed without copying.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "moe_oracle.c")
_LIB = os.path.join(_HERE, "libmoe_oracle.so")

SCORE_SOFTMAX = 0
SCORE_SIGMOID = 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP over tokens) if it is out of date."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    c_int, c_dbl, c_vp = ctypes.c_int, ctypes.c_double, ctypes.c_void_p
    lib.oracle_num_threads.restype = c_int
    lib.oracle_expected_active.restype = c_dbl
    lib.oracle_expected_active.argtypes = [c_int, c_int, c_dbl]
    lib.oracle_mean_tokens_per_expert.restype = c_dbl
    lib.oracle_mean_tokens_per_expert.argtypes = [c_dbl, c_dbl]
    lib.oracle_token_threshold.restype = c_int
    lib.oracle_token_threshold.argtypes = [c_dbl, c_dbl]
    lib.oracle_router_logits.restype = None
    lib.oracle_router_logits.argtypes = [c_vp, c_vp, c_vp, c_int, c_int, c_int, c_vp]
    lib.oracle_shared_gate.restype = None
    lib.oracle_shared_gate.argtypes = [c_vp, c_vp, c_int, c_int, c_vp]
    lib.oracle_route_topk.restype = None
    lib.oracle_route_topk.argtypes = [c_vp, c_int, c_int, c_int, c_int, c_int, c_dbl, c_vp, c_vp]
    lib.oracle_permute.restype = None
    lib.oracle_permute.argtypes = [c_vp, c_int, c_int, c_int] + [c_vp] * 6
    lib.oracle_expert_ffn.restype = None
    lib.oracle_expert_ffn.argtypes = [c_vp] * 4 + [c_int] * 3 + [c_vp]
    layer_args = [c_vp] + [c_int] * 6 + [c_vp] * 9
    lib.oracle_layer.restype = None
    lib.oracle_layer.argtypes = layer_args + [c_vp, c_int, c_vp]
    lib.oracle_layer_dense_masked.restype = None
    lib.oracle_layer_dense_masked.argtypes = layer_args + [c_vp]
    _lib = lib
    return lib


def _np(a, dtype):
    """Return a C-contiguous numpy view of ``a`` with ``dtype`` (bf16 tensors -> uint16)."""
    if a is None:
        return None
    if not isinstance(a, np.ndarray):  # torch CPU tensor
        import torch

        t = a.detach().contiguous()
        if t.dtype == torch.bfloat16:
            t = t.view(torch.uint16)
        a = t.numpy()
    a = np.ascontiguousarray(a)
    if a.dtype != dtype:
        if dtype == np.uint16:
            raise TypeError("bf16 data must be given as uint16 bit patterns or a bf16 tensor")
        a = a.astype(dtype)
    return a


def _p(a):
    return None if a is None else ctypes.c_void_p(a.ctypes.data)


def num_threads() -> int:
    return _load().oracle_num_threads()


# ---- closed forms (Sec. 3.2) ---------------------------------------------------------

def expected_active(E: int, K: int, t: float) -> float:
    """Eq. N(t): expected activated experts after ``t`` tokens."""
    return _load().oracle_expected_active(int(E), int(K), float(t))


def mean_tokens_per_expert(rho: float, t: float) -> float:
    """Eq. T_exp: mean tokens per activated expert."""
    return _load().oracle_mean_tokens_per_expert(float(rho), float(t))


def token_threshold(rho: float, tau: float = 0.95) -> int:
    """Eq. T_thres: tokens needed for N(t) >= tau*E."""
    return _load().oracle_token_threshold(float(rho), float(tau))


# ---- layer steps ---------------------------------------------------------------------

def router_logits(x, w_router, bias=None):
    """z[t,e] = x[t,:] . w_router[e,:] (+ bias[e]); fp64 accumulation, one rounding to fp32."""
    x = _np(x, np.uint16)
    w = _np(w_router, np.float32)
    b = _np(bias, np.float32)
    T, H = x.shape
    E = w.shape[0]
    assert w.shape == (E, H)
    z = np.empty((T, E), np.float32)
    _load().oracle_router_logits(_p(x), _p(w), _p(b), T, H, E, _p(z))
    return z


def shared_gate(x, w_sg):
    """s[t] = sigmoid(x[t,:] . w_sg) in fp64."""
    x = _np(x, np.uint16)
    w = _np(w_sg, np.uint16).reshape(-1)
    T, H = x.shape
    s = np.empty((T,), np.float64)
    _load().oracle_shared_gate(_p(x), _p(w), T, H, _p(s))
    return s


def route_topk(z, k: int, score_fn: int, renormalize: bool, routed_scale: float = 1.0):
    """Select on the fp32 logits (ties -> lower index), then score; returns (idx i32, w f64)."""
    z = _np(z, np.float32)
    T, E = z.shape
    idx = np.empty((T, k), np.int32)
    w = np.empty((T, k), np.float64)
    _load().oracle_route_topk(_p(z), T, E, int(k), int(score_fn), int(bool(renormalize)),
                              float(routed_scale), _p(idx), _p(w))
    return idx, w


@dataclass
class Grouping:
    counts: np.ndarray
    offsets: np.ndarray
    perm: np.ndarray
    inv_perm: np.ndarray
    active: np.ndarray
    n_active: int


def permute(topk_idx, E: int) -> Grouping:
    """Stable grouping of the assignments a = t*k+j by expert."""
    idx = _np(topk_idx, np.int32)
    T, k = idx.shape
    A = T * k
    counts = np.empty((E,), np.int32)
    offsets = np.empty((E + 1,), np.int32)
    perm = np.empty((A,), np.int32)
    inv_perm = np.empty((A,), np.int32)
    active = np.empty((E,), np.int32)
    n_active = np.zeros((1,), np.int32)
    _load().oracle_permute(_p(idx), T, k, E, _p(counts), _p(offsets), _p(perm), _p(inv_perm),
                           _p(active), _p(n_active))
    return Grouping(counts, offsets, perm, inv_perm, active, int(n_active[0]))


def expert_ffn(x, w_gate, w_up, w_down):
    """One SwiGLU expert on every row of x: (W_down (silu(W_gate x) * (W_up x)))."""
    x = _np(x, np.uint16)
    wg, wu, wd = _np(w_gate, np.uint16), _np(w_up, np.uint16), _np(w_down, np.uint16)
    T, H = x.shape
    I = wg.shape[0]
    assert wg.shape == (I, H) and wu.shape == (I, H) and wd.shape == (H, I)
    y = np.empty((T, H), np.float64)
    _load().oracle_expert_ffn(_p(x), _p(wg), _p(wu), _p(wd), T, H, I, _p(y))
    return y


def _layer_common(x, w_gate, w_up, w_down, shared, topk_idx, topk_w, shared_scale):
    x = _np(x, np.uint16)
    wg, wu, wd = _np(w_gate, np.uint16), _np(w_up, np.uint16), _np(w_down, np.uint16)
    T, H = x.shape
    E, I, H2 = wg.shape
    assert H2 == H and wu.shape == (E, I, H) and wd.shape == (E, H, I)
    idx = _np(topk_idx, np.int32)
    w = _np(topk_w, np.float64)
    k = idx.shape[1]
    assert idx.shape == (T, k) and w.shape == (T, k)
    if shared is not None:
        sg, su, sd = (_np(s, np.uint16) for s in shared)
        I_s = sg.shape[0]
        assert sg.shape == (I_s, H) and su.shape == (I_s, H) and sd.shape == (H, I_s)
    else:
        sg = su = sd = None
        I_s = 0
    ss = _np(shared_scale, np.float64)
    keep = (x, wg, wu, wd, sg, su, sd, idx, w, ss)
    args = [_p(x), T, H, E, k, I, I_s, _p(wg), _p(wu), _p(wd), _p(sg), _p(su), _p(sd),
            _p(idx), _p(w), _p(ss)]
    return args, keep, T, H


def layer(x, w_gate, w_up, w_down, topk_idx, topk_w, shared=None, shared_scale=None,
          rows=None):
    """out[t] = sum_j w[t,j] * FFN_{idx[t,j]}(x[t]) + s[t] * FFN_shared(x[t]); fp64.

    ``shared`` is (ws_gate [I_s,H], ws_up [I_s,H], ws_down [H,I_s]) or None;
    ``shared_scale`` is s[T] or None (= 1).  ``rows`` optionally restricts the evaluation
    to a list of token ids (the layer is token-wise); the output then has len(rows) rows.
    """
    args, keep, T, H = _layer_common(x, w_gate, w_up, w_down, shared, topk_idx, topk_w,
                                     shared_scale)
    r = None if rows is None else _np(np.asarray(rows), np.int32)
    n = T if r is None else int(r.shape[0])
    out = np.empty((n, H), np.float64)
    _load().oracle_layer(*args, _p(r), n, _p(out))
    del keep
    return out


def layer_dense_masked(x, w_gate, w_up, w_down, topk_idx, topk_w, shared=None,
                       shared_scale=None):
    """Brute force for tiny inputs: all E experts on every token, then a dense mask."""
    args, keep, T, H = _layer_common(x, w_gate, w_up, w_down, shared, topk_idx, topk_w,
                                     shared_scale)
    out = np.empty((T, H), np.float64)
    _load().oracle_layer_dense_masked(*args, _p(out))
    del keep
    return out


def verify_layer(x, weights: dict, cfg: dict, logits=None, rows=None):
    """Whole layer from inputs: logits (or the fp32 ``logits`` given) -> top-k -> FFNs.

    ``cfg`` keys: top_k, score_fn, renormalize, routed_scale, shared_gate.
    ``weights`` keys: w_router, router_bias, w_gate, w_up, w_down, ws_gate, ws_up, ws_down,
    w_shared_gate (absent / None where unused).  Returns a dict with every intermediate.
    """
    z = router_logits(x, weights["w_router"], weights.get("router_bias")) if logits is None \
        else _np(logits, np.float32)
    idx, w = route_topk(z, cfg["top_k"], cfg["score_fn"], cfg["renormalize"],
                        cfg.get("routed_scale", 1.0))
    shared = None
    s = None
    if weights.get("ws_gate") is not None:
        shared = (weights["ws_gate"], weights["ws_up"], weights["ws_down"])
        if cfg.get("shared_gate", 0):
            s = shared_gate(x, weights["w_shared_gate"])
    out = layer(x, weights["w_gate"], weights["w_up"], weights["w_down"], idx, w, shared, s,
                rows)
    return {"logits": z, "topk_idx": idx, "topk_w": w, "shared_scale": s, "out": out}
