"""Helpers shared by the GPU parity tests: run the CUDA layer, run the oracle, compare."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2505_19645_b200 import workloads as wl

__all__ = ["assert_logits_close", "assert_output_close", "check_layer_against_oracle",
           "run_gpu_layer", "to_host", "oracle_cfg", "check_grouping", "alloc_canary_workspace",
           "check_canaries", "stratified_rows"]

# Output tolerance (bf16 inputs, fp32 accumulation on the GPU, fp64 oracle):
#   max |err| <= 2e-2 * max |ref|   and   mean |err| / mean |ref| <= 5e-3
MAX_ERR_FRAC = 2e-2
MEAN_REL_ERR = 5e-3
# gate weights: expf on the GPU against exp in fp64
GATE_W_ATOL = 1e-5


# Router logits (one rule everywhere).  The GPU accumulates the dot product in fp32 in an order
# of its own; the rounding error of such a sum is bounded by a small multiple of
# 2^-24 * sum_i |x_i w_i| -- the size of the TERMS, not of their sum, which cancellation can make
# arbitrarily small (one expert and one token leave a single logit to compare, and a bound
# relative to max|z| then means nothing).  Tolerance: 1e-5 * max_{t,e} (sum_i |x_ti w_ei| + |b_e|),
# i.e. ~170 units of 2^-24 of the largest term sum.  On the benchmark shapes (Gaussian rows:
# sum|x w| ~ 0.64 sqrt(H) standard deviations of a logit) this is 3e-4 to 5e-4 of a logit's
# standard deviation, the same size as a bound of 1e-4 * max|z|.
LOGIT_RTOL_OF_TERMS = 1e-5


def assert_logits_close(z, z_ref, x_host, w_router, bias=None):
    xa = np.abs(x_host.float().numpy().astype(np.float64))
    wa = np.abs(w_router.float().numpy().astype(np.float64))
    scale = (xa @ wa.T).max()
    if bias is not None:
        scale += np.abs(bias.float().numpy()).max()
    err = np.abs(np.asarray(z, dtype=np.float64) - z_ref).max()
    assert err <= LOGIT_RTOL_OF_TERMS * scale, "logits: max|err| %.3e > %.1e * %.3e" % (
        err, LOGIT_RTOL_OF_TERMS, scale)


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


CANARY = 0xA5


def alloc_canary_workspace(api, cfg, T, tail=4096):
    """A workspace filled with a byte pattern, with `tail` extra bytes behind it.  The layout
    leaves at least 256 bytes between any two regions that no kernel may write."""
    n = api.moe_workspace_bytes(cfg, T)
    buf = torch.full((n + tail,), CANARY, dtype=torch.uint8, device="cuda")
    return buf, buf[:n]


def check_canaries(api, cfg, T, buf):
    """Every byte outside the regions a call with T tokens uses still holds the pattern (the
    compute sanitiser's stand-in: a store that strays out of its region lands in a guard)."""
    keep = torch.ones(buf.numel(), dtype=torch.bool, device="cuda")
    regions = api.workspace_regions(cfg, T)
    assert len(regions) >= 15
    for off, nbytes in regions:
        keep[off:off + nbytes] = False
    # the status region is written by the library (status word and its marker) within 256 bytes
    bad = (buf != CANARY) & keep
    if bool(bad.any()):
        where = int(torch.nonzero(bad)[0].item())
        raise AssertionError("workspace byte %d outside every region was overwritten" % where)


def run_gpu_layer(shape, w_dev, x_dev, B, gamma, ws=None):
    from paper_2505_19645_b200 import api

    cfg = api.make_config(shape)
    cw = api.make_weights(w_dev)
    T = B * (gamma + 1)
    assert x_dev.shape[0] == T
    buf = None
    if ws is None:
        buf, ws = alloc_canary_workspace(api, cfg, T)
    out = torch.empty_like(x_dev)
    dbg = api.alloc_debug(cfg, T)
    api.moe_verify_layer(cfg, cw, x_dev, B, gamma, out, ws, dbg)
    api.moe_check(ws)
    if buf is not None:
        check_canaries(api, cfg, T, buf)
    host = {k: v.cpu().numpy() for k, v in dbg.items()}
    return out, host


def stratified_rows(g, k: int, T: int, n: int, seed: int = 0):
    """Token rows for a sampled output comparison, chosen from the grouping `g` (the oracle's)
    so that the places where the kernels change behaviour are always covered: the first and the
    last sorted row of the largest and of the smallest activated group, the first and last row
    of a ragged tail segment (group size not a multiple of the 128-row segment), rows on both
    sides of a segment boundary, and for the shared expert (whose group is all T tokens) the
    first and last token of its last segment and of its last segment pair.  Filled up to `n`
    rows with a seeded random draw."""
    SEG = 128
    tok = lambda i: int(g.perm[i]) // k  # noqa: E731  sorted row -> token
    counts, offs = g.counts, g.offsets
    act = [e for e in range(len(counts)) if counts[e] > 0]
    picks = [0, T - 1]
    big = max(act, key=lambda e: counts[e])
    small = min(act, key=lambda e: counts[e])
    for e in (big, small):
        picks += [tok(offs[e]), tok(offs[e] + counts[e] - 1)]
    ragged = [e for e in act if counts[e] > SEG and counts[e] % SEG]
    tail_groups = ragged[:2] if ragged else [big]
    for e in tail_groups:
        first_tail = offs[e] + (int(counts[e]) - 1) // SEG * SEG
        picks += [tok(first_tail), tok(offs[e] + counts[e] - 1)]
        if first_tail > offs[e]:
            picks.append(tok(first_tail - 1))  # last row of the full segment before the tail
    # shared expert: segments of 128 tokens (64 between 65 and 128 tokens), paired beyond 128
    for seg in (SEG, SEG // 2):
        last_seg0 = (T - 1) // seg * seg
        last_pair0 = (T - 1) // (2 * seg) * (2 * seg)
        picks += [last_seg0, last_pair0, max(0, last_seg0 - 1)]
    rng = np.random.default_rng(seed + T)
    picks += rng.permutation(T)[:n].tolist()
    rows = []
    for t in picks:
        if 0 <= t < T and t not in rows:
            rows.append(int(t))
        if len(rows) >= n:
            break
    return sorted(rows)


def check_layer_against_oracle(shape, w_dev, x_dev, B, gamma, rows=None, w_host=None):
    """Full parity check of one moe_verify_layer call; returns the error fractions.  `rows`:
    None (every token), a list of token ids, or an int n (n stratified rows, see above)."""
    out_dev, dbg = run_gpu_layer(shape, w_dev, x_dev, B, gamma)
    if w_host is None:
        w_host = to_host(w_dev)
    x_host = x_dev.cpu()
    T = x_host.shape[0]
    cfg = oracle_cfg(shape)

    # router logits: fp32-accumulated GPU values against the fp64 oracle
    z_ref = oracle.router_logits(x_host, w_host["w_router"], w_host.get("router_bias"))
    assert_logits_close(dbg["logits"], z_ref, x_host, w_host["w_router"], w_host.get("router_bias"))

    # routing decided on the SAME fp32 logits on both sides: bit-exact indices
    idx_ref, w_ref = oracle.route_topk(dbg["logits"], shape.top_k, shape.score_fn,
                                       shape.renormalize, shape.routed_scale)
    np.testing.assert_array_equal(dbg["topk_idx"], idx_ref)
    assert np.abs(dbg["topk_w"].astype(np.float64) - w_ref).max() <= GATE_W_ATOL
    g = check_grouping(dbg, idx_ref, shape.n_experts)
    if isinstance(rows, int):
        rows = stratified_rows(g, shape.top_k, T, rows) if rows < T else None

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
