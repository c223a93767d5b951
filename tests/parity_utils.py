"""Helpers shared by the GPU parity tests: run the CUDA layer, run the oracle, compare."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2505_19645_b200 import workloads as wl

# Output tolerance (bf16 inputs, fp32 accumulation on the GPU, fp64 oracle):
#   max |err| <= 2e-2 * max |ref|   and   mean |err| / mean |ref| <= 5e-3
MAX_ERR_FRAC = 2e-2
MEAN_REL_ERR = 5e-3
# gate weights: expf on the GPU against exp in fp64
GATE_W_ATOL = 1e-5


def oracle_cfg(shape: wl.LayerShape) -> dict:
    return dict(top_k=shape.top_k, score_fn=shape.score_fn, renormalize=shape.renormalize,
                routed_scale=shape.routed_scale, shared_gate=shape.shared_gate)


def to_host(w: dict) -> dict:
    return {k: (None if v is None else v.cpu()) for k, v in w.items()}


def assert_output_close(got: np.ndarray, ref: np.ndarray, what: str = "out"):
    err = np.abs(got.astype(np.float64) - ref)
    max_ref = np.abs(ref).max()
    mean_ref = np.abs(ref).mean()
    assert np.isfinite(got).all(), what + ": non-finite values"
    assert max_ref > 0, what + ": reference is identically zero"
    assert err.max() <= MAX_ERR_FRAC * max_ref, \
        "%s: max|err| %.3e > %.1e * max|ref| %.3e" % (what, err.max(), MAX_ERR_FRAC, max_ref)
    assert err.mean() <= MEAN_REL_ERR * mean_ref, \
        "%s: mean|err|/mean|ref| = %.3e > %.1e" % (what, err.mean() / mean_ref, MEAN_REL_ERR)
    return err.max() / max_ref, err.mean() / mean_ref


def check_grouping(dbg: dict, idx_ref: np.ndarray, E: int):
    """Bit-exact comparison of the GPU grouping with the oracle's on the same indices."""
    g = oracle.permute(idx_ref, E)
    np.testing.assert_array_equal(dbg["counts"], g.counts)
    np.testing.assert_array_equal(dbg["offsets"], g.offsets)
    np.testing.assert_array_equal(dbg["perm"], g.perm)
    np.testing.assert_array_equal(dbg["inv_perm"], g.inv_perm)
    np.testing.assert_array_equal(dbg["active"], g.active)
    assert int(dbg["n_active"][0]) == g.n_active
    return g


def run_gpu_layer(shape, w_dev, x_dev, B, gamma, ws=None):
    from paper_2505_19645_b200 import api

    cfg = api.make_config(shape)
    cw = api.make_weights(w_dev)
    T = B * (gamma + 1)
    assert x_dev.shape[0] == T
    if ws is None:
        ws = api.alloc_workspace(cfg, T)
    out = torch.empty_like(x_dev)
    dbg = api.alloc_debug(cfg, T)
    api.moe_verify_layer(cfg, cw, x_dev, B, gamma, out, ws, dbg)
    api.moe_check(ws)
    host = {k: v.cpu().numpy() for k, v in dbg.items()}
    return out, host


def check_layer_against_oracle(shape, w_dev, x_dev, B, gamma, rows=None, w_host=None):
    """Full parity check of one moe_verify_layer call; returns the error fractions."""
    out_dev, dbg = run_gpu_layer(shape, w_dev, x_dev, B, gamma)
    if w_host is None:
        w_host = to_host(w_dev)
    x_host = x_dev.cpu()
    T = x_host.shape[0]
    cfg = oracle_cfg(shape)

    # router logits: fp32-accumulated GPU values against the fp64 oracle
    z_ref = oracle.router_logits(x_host, w_host["w_router"], w_host.get("router_bias"))
    # The rounding error of an fp32-accumulated dot product is bounded by a multiple of
    # 2^-24 * sum_i |x_i w_i| -- the size of the terms, not of their sum, which cancellation can
    # make arbitrarily small (a single expert and a single token leave one logit to compare).
    xa = np.abs(x_host.float().numpy().astype(np.float64))
    wa = np.abs(w_host["w_router"].float().numpy().astype(np.float64))
    scale = (xa @ wa.T).max()
    if w_host.get("router_bias") is not None:
        scale += np.abs(w_host["router_bias"].float().numpy()).max()
    assert np.abs(dbg["logits"] - z_ref).max() <= 1e-5 * scale

    # routing decided on the SAME fp32 logits on both sides: bit-exact indices
    idx_ref, w_ref = oracle.route_topk(dbg["logits"], shape.top_k, shape.score_fn,
                                       shape.renormalize, shape.routed_scale)
    np.testing.assert_array_equal(dbg["topk_idx"], idx_ref)
    assert np.abs(dbg["topk_w"].astype(np.float64) - w_ref).max() <= GATE_W_ATOL
    check_grouping(dbg, idx_ref, shape.n_experts)

    shared = None
    s = None
    if shape.shared_inter:
        shared = (w_host["ws_gate"], w_host["ws_up"], w_host["ws_down"])
        if shape.shared_gate:
            s = oracle.shared_gate(x_host, w_host["w_shared_gate"])
    ref = oracle.layer(x_host, w_host["w_gate"], w_host["w_up"], w_host["w_down"], idx_ref, w_ref,
                       shared, s, rows)
    got = out_dev.float().cpu().numpy()
    if rows is not None:
        got = got[np.asarray(rows)]
    fr = assert_output_close(got, ref)
    return fr, dbg
