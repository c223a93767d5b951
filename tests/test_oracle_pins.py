"""Pins of the CPU oracle against things other than itself (CPU only).

Each test ties one oracle function to the mathematics or to an independent library
routine: exact enumeration of routing outcomes (Eq. N(t)), exact rational arithmetic
(Eq. T_thres, Eq. T_exp), numpy / scipy / torch fp64 routines for the special cases the
layer reduces to, dense-masked brute force, and structural invariants.
"""
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest
import scipy.special
import torch
import torch.nn.functional as F

import oracle
from paper_2505_19645_b200 import workloads as wl


def bf16_bits_to_f64(t):
    return t.to(torch.float64).numpy()


# --------------------------------------------------------------------------------------
# closed forms of Sec. 3.2
# --------------------------------------------------------------------------------------

@pytest.mark.parametrize("E,K,t", [(4, 2, 1), (4, 2, 2), (4, 2, 3), (5, 1, 3), (5, 3, 2), (6, 2, 2)])
def test_expected_active_equals_exact_enumeration(E, K, t):
    """Eq. N(t) is the exact mean of |union of t uniform K-subsets of E experts|."""
    subsets = list(itertools.combinations(range(E), K))
    total = Fraction(0)
    for choice in itertools.product(subsets, repeat=t):
        total += len(set().union(*choice))
    exact = total / (len(subsets) ** t)
    assert oracle.expected_active(E, K, t) == pytest.approx(float(exact), rel=1e-13)


def test_expected_active_special_values():
    """t=1 activates exactly K experts; K=E activates all; t=0 none (Eq. PrX)."""
    for E, K in [(8, 2), (60, 4), (64, 8), (256, 8)]:
        assert oracle.expected_active(E, K, 1) == pytest.approx(K, rel=1e-13)
        assert oracle.expected_active(E, K, 0) == 0.0
        assert oracle.expected_active(E, E, 3) == E
        # monotone and bounded by E
        prev = 0.0
        for t in range(1, 200):
            cur = oracle.expected_active(E, K, t)
            assert prev <= cur <= E and (cur > prev or E - cur < 1e-9)
            prev = cur


def test_expected_active_rational():
    for E, K, t in [(8, 2, 16), (60, 4, 16), (64, 8, 8), (256, 8, 16), (256, 8, 96)]:
        exact = E * (1 - Fraction(E - K, E) ** t)
        assert oracle.expected_active(E, K, t) == pytest.approx(float(exact), rel=1e-12)


@pytest.mark.parametrize("K,E", [(2, 8), (4, 60), (8, 64), (8, 256), (1, 2), (1, 100)])
def test_token_threshold_is_first_t_reaching_tau(K, E):
    """Eq. T_thres: the least integer t with N(t) >= tau*E, found by exact search."""
    tau = Fraction(95, 100)
    t = 1
    while 1 - Fraction(E - K, E) ** t < tau:
        t += 1
    assert oracle.token_threshold(K / E, 0.95) == t


def test_token_threshold_values():
    got = [oracle.token_threshold(r) for r in (2 / 8, 4 / 60, 8 / 64, 8 / 256)]
    assert got == [11, 44, 23, 95]


def test_mean_tokens_per_expert():
    """Eq. T_exp = t*K/N(t); rho=1 gives t (dense limit); decreasing in sparsity for t>1."""
    for E, K, t in [(8, 2, 16), (60, 4, 7), (256, 8, 96)]:
        exact = Fraction(t * K) / (E * (1 - Fraction(E - K, E) ** t))
        assert oracle.mean_tokens_per_expert(K / E, t) == pytest.approx(float(exact), rel=1e-12)
    for t in (1, 2, 17, 300):
        assert oracle.mean_tokens_per_expert(1.0, t) == pytest.approx(t)
    for t in (2, 16, 128):
        vals = [oracle.mean_tokens_per_expert(r, t) for r in (0.01, 0.05, 0.125, 0.25, 0.5, 1.0)]
        assert all(a < b for a, b in zip(vals, vals[1:]))
    # t = 1: one token per activated expert whatever the sparsity
    for r in (0.01, 0.3, 1.0):
        assert oracle.mean_tokens_per_expert(r, 1) == pytest.approx(1.0)


# --------------------------------------------------------------------------------------
# router
# --------------------------------------------------------------------------------------

def _tokens(T, H, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(T, H, generator=g).to(torch.bfloat16)


def test_router_logits_vs_numpy_matmul():
    T, H, E = 13, 96, 10
    x = _tokens(T, H, 1)
    g = torch.Generator().manual_seed(2)
    wr = (torch.randn(E, H, generator=g) * 0.02).float()
    b = torch.randn(E, generator=g).float()
    ref = x.to(torch.float64).numpy() @ wr.to(torch.float64).numpy().T
    z = oracle.router_logits(x, wr)
    np.testing.assert_allclose(z, ref.astype(np.float32), rtol=0, atol=float(np.abs(ref).max()) * 2e-7)
    zb = oracle.router_logits(x, wr, b)
    np.testing.assert_allclose(zb, (ref + b.double().numpy()).astype(np.float32), rtol=0,
                               atol=float(np.abs(ref).max() + 4) * 2e-7)
    # a transposed operand or a dropped bias would not survive this
    assert np.abs(zb - z).max() > 0.1


@pytest.mark.parametrize("E,k", [(8, 2), (60, 4), (64, 8), (256, 8), (5, 5), (3, 1)])
@pytest.mark.parametrize("score_fn", [oracle.SCORE_SOFTMAX, oracle.SCORE_SIGMOID])
@pytest.mark.parametrize("renorm", [0, 1])
def test_route_topk_vs_library(E, k, score_fn, renorm):
    rng = np.random.default_rng(E * 100 + k)
    z = rng.normal(0, 1.5, size=(37, E)).astype(np.float32)
    idx, w = oracle.route_topk(z, k, score_fn, renorm, 1.0)
    order = np.argsort(-z.astype(np.float64), axis=1, kind="stable")[:, :k]
    np.testing.assert_array_equal(idx, order.astype(np.int32))
    if score_fn == oracle.SCORE_SOFTMAX:
        p = scipy.special.softmax(z.astype(np.float64), axis=1)
    else:
        p = scipy.special.expit(z.astype(np.float64))
    ref = np.take_along_axis(p, order, axis=1)
    if renorm:
        ref = ref / ref.sum(axis=1, keepdims=True)
    np.testing.assert_allclose(w, ref, rtol=1e-12, atol=0)
    # invariants: distinct, in range, positive, descending logits, sums
    for t in range(z.shape[0]):
        assert len(set(idx[t])) == k and idx[t].min() >= 0 and idx[t].max() < E
        sel = z[t, idx[t]]
        assert np.all(sel[:-1] >= sel[1:])
    assert np.all(w > 0)
    if renorm:
        np.testing.assert_allclose(w.sum(1), 1.0, rtol=1e-12)
    elif score_fn == oracle.SCORE_SOFTMAX:
        assert np.all(w.sum(1) <= 1.0 + 1e-12)
        if k == E:
            np.testing.assert_allclose(w.sum(1), 1.0, rtol=1e-12)


def test_route_topk_scale_and_two_expert_softmax():
    """softmax over all E then renormalised over the 2 selected = softmax over those 2 logits."""
    rng = np.random.default_rng(5)
    z = rng.normal(0, 2, size=(50, 8)).astype(np.float32)
    idx, w = oracle.route_topk(z, 2, oracle.SCORE_SOFTMAX, 1, 1.0)
    sel = np.take_along_axis(z.astype(np.float64), idx.astype(np.int64), axis=1)
    np.testing.assert_allclose(w, scipy.special.softmax(sel, axis=1), rtol=1e-12)
    _, w25 = oracle.route_topk(z, 2, oracle.SCORE_SOFTMAX, 1, 2.5)
    np.testing.assert_allclose(w25, 2.5 * w, rtol=1e-15)


def test_route_topk_ties_take_lower_index():
    z = np.zeros((3, 9), np.float32)
    idx, w = oracle.route_topk(z, 4, oracle.SCORE_SOFTMAX, 0, 1.0)
    np.testing.assert_array_equal(idx, np.tile(np.arange(4, dtype=np.int32), (3, 1)))
    np.testing.assert_allclose(w, 1.0 / 9.0, rtol=1e-15)
    z = np.array([[1.0, 3.0, 3.0, 0.5, 3.0, 1.0]], np.float32)
    idx, _ = oracle.route_topk(z, 5, oracle.SCORE_SIGMOID, 1, 1.0)
    np.testing.assert_array_equal(idx[0], [1, 2, 4, 0, 5])
    # a difference of one fp32 ulp is not a tie
    a = np.float32(1.0)
    b = np.nextafter(a, np.float32(2.0))
    idx, _ = oracle.route_topk(np.array([[a, b, a]], np.float32), 2, oracle.SCORE_SOFTMAX, 1, 1.0)
    np.testing.assert_array_equal(idx[0], [1, 0])


# --------------------------------------------------------------------------------------
# grouping
# --------------------------------------------------------------------------------------

@pytest.mark.parametrize("T,k,E", [(1, 2, 8), (16, 2, 8), (33, 4, 60), (7, 8, 256), (50, 3, 3)])
def test_permute_vs_stable_argsort(T, k, E):
    rng = np.random.default_rng(T * 7 + E)
    idx = np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
    g = oracle.permute(idx, E)
    flat = idx.reshape(-1)
    A = T * k
    np.testing.assert_array_equal(g.counts, np.bincount(flat, minlength=E))
    np.testing.assert_array_equal(g.offsets, np.concatenate([[0], np.cumsum(g.counts)]))
    np.testing.assert_array_equal(g.perm, np.argsort(flat, kind="stable"))
    inv = np.empty(A, np.int64)
    inv[g.perm] = np.arange(A)
    np.testing.assert_array_equal(g.inv_perm, inv)
    act = np.nonzero(g.counts)[0]
    assert g.n_active == len(act)
    np.testing.assert_array_equal(g.active[:g.n_active], act)
    assert np.all(g.active[g.n_active:] == -1)
    # invariants
    assert g.counts.sum() == A and g.offsets[E] == A
    assert sorted(g.perm.tolist()) == list(range(A))
    experts_sorted = flat[g.perm]
    assert np.all(np.diff(experts_sorted) >= 0)
    for e in range(E):
        seg = g.perm[g.offsets[e]:g.offsets[e + 1]]
        assert np.all(np.diff(seg) > 0)


# --------------------------------------------------------------------------------------
# expert FFN and layer
# --------------------------------------------------------------------------------------

def _torch_ffn(x, wg, wu, wd):
    x, wg, wu, wd = (a.to(torch.float64) for a in (x, wg, wu, wd))
    return F.linear(F.silu(F.linear(x, wg)) * F.linear(x, wu), wd)


def test_expert_ffn_vs_torch_fp64():
    T, H, I = 5, 64, 96
    shape = wl.small_shape("t", H, 1, 1, I)
    w = wl.make_weights(shape, 11)
    x = wl.make_tokens(shape, T, 12)
    # larger weights so that silu is exercised away from its linear region
    wg = (w["w_gate"][0].float() * 20).to(torch.bfloat16)
    y = oracle.expert_ffn(x, wg, w["w_up"][0], w["w_down"][0])
    ref = _torch_ffn(x, wg, w["w_up"][0], w["w_down"][0]).numpy()
    np.testing.assert_allclose(y, ref, rtol=1e-10, atol=1e-14)
    # non-square on purpose: a transposed weight would not even have the right shape,
    # and swapping gate/up changes the result
    y_swapped = oracle.expert_ffn(x, w["w_up"][0], wg, w["w_down"][0])
    assert np.abs(y_swapped - y).max() > 1e-4 * np.abs(y).max()


def _tiny_case(seed, H=32, E=6, k=3, I=48, Is=0, score=wl.SCORE_SOFTMAX, renorm=1, sgate=0, T=7):
    shape = wl.small_shape("t", H, E, k, I, Is, score, renorm, sgate)
    w = wl.make_weights(shape, seed)
    # scale up so that outputs are well away from zero
    for key in ("w_gate", "w_up", "w_down", "ws_gate", "ws_up", "ws_down", "w_shared_gate"):
        if w[key] is not None:
            w[key] = (w[key].float() * 10).to(torch.bfloat16)
    w["w_router"] = w["w_router"] * 20
    x = wl.make_tokens(shape, T, seed + 1)
    cfg = dict(top_k=k, score_fn=score, renormalize=renorm, routed_scale=1.0, shared_gate=sgate)
    return shape, w, x, cfg


def _torch_dense_layer(shape, w, x, idx, wts, s):
    """Dense mixture in torch fp64: every expert on every token, masked sum."""
    T = x.shape[0]
    out = torch.zeros(T, shape.hidden, dtype=torch.float64)
    mask = torch.zeros(T, shape.n_experts, dtype=torch.float64)
    mask.scatter_(1, torch.from_numpy(idx.astype(np.int64)), torch.from_numpy(wts))
    for e in range(shape.n_experts):
        out += mask[:, e:e + 1] * _torch_ffn(x, w["w_gate"][e], w["w_up"][e], w["w_down"][e])
    if shape.shared_inter:
        sh = _torch_ffn(x, w["ws_gate"], w["ws_up"], w["ws_down"])
        out += sh * (torch.from_numpy(s)[:, None] if s is not None else 1.0)
    return out.numpy()


@pytest.mark.parametrize("variant", [
    dict(),                                                       # softmax, renorm
    dict(renorm=0, Is=40, sgate=1),                               # Qwen-style shared expert
    dict(score=wl.SCORE_SIGMOID, renorm=1, Is=24, sgate=0),       # DeepSeek-style
    dict(E=4, k=4),                                               # dense limit rho = 1
    dict(E=1, k=1, T=3),                                          # a plain FFN
])
def test_layer_equals_dense_masked_and_torch(variant):
    shape, w, x, cfg = _tiny_case(21, **variant)
    res = oracle.verify_layer(x, w, cfg)
    idx, wts, s = res["topk_idx"], res["topk_w"], res["shared_scale"]
    shared = (w["ws_gate"], w["ws_up"], w["ws_down"]) if shape.shared_inter else None
    brute = oracle.layer_dense_masked(x, w["w_gate"], w["w_up"], w["w_down"], idx, wts, shared, s)
    scale = np.abs(brute).max()
    assert scale > 1e-3
    np.testing.assert_allclose(res["out"], brute, rtol=0, atol=1e-6 * scale)
    ref = _torch_dense_layer(shape, w, x, idx, wts, s)
    np.testing.assert_allclose(res["out"], ref, rtol=0, atol=1e-10 * scale)
    if shape.shared_gate:
        sref = torch.sigmoid(x.double() @ w["w_shared_gate"].double()).numpy()
        np.testing.assert_allclose(s, sref, rtol=1e-12)
        assert 0.02 < s.min() and s.max() < 0.98 and s.std() > 0.01


def test_single_expert_is_plain_ffn():
    shape, w, x, cfg = _tiny_case(3, E=1, k=1, T=4)
    res = oracle.verify_layer(x, w, cfg)
    np.testing.assert_allclose(res["topk_w"], 1.0)
    ref = _torch_ffn(x, w["w_gate"][0], w["w_up"][0], w["w_down"][0]).numpy()
    np.testing.assert_allclose(res["out"], ref, rtol=1e-10, atol=1e-14)


def test_dense_limit_is_softmax_mixture():
    """k = E with softmax: out = sum_e softmax(z)_e * FFN_e(x) (the rho = 1 limit)."""
    shape, w, x, cfg = _tiny_case(4, E=5, k=5, T=4)
    res = oracle.verify_layer(x, w, cfg)
    p = torch.softmax(torch.from_numpy(res["logits"]).double(), dim=1)
    ref = sum(p[:, e:e + 1] * _torch_ffn(x, w["w_gate"][e], w["w_up"][e], w["w_down"][e])
              for e in range(5)).numpy()
    np.testing.assert_allclose(res["out"], ref, rtol=0, atol=1e-10 * np.abs(ref).max())


def test_layer_structural_properties():
    shape, w, x, cfg = _tiny_case(8, Is=16, sgate=1, renorm=0, T=9)
    res = oracle.verify_layer(x, w, cfg)
    # token-wise: permuting the rows permutes the outputs, a row sample equals the full rows
    p = np.random.default_rng(0).permutation(x.shape[0])
    res_p = oracle.verify_layer(x[torch.from_numpy(p)], w, cfg)
    np.testing.assert_array_equal(res_p["out"], res["out"][p])
    np.testing.assert_array_equal(res_p["topk_idx"], res["topk_idx"][p])
    rows = [5, 0, 7]
    sub = oracle.verify_layer(x, w, cfg, rows=rows)
    np.testing.assert_array_equal(sub["out"], res["out"][rows])
    # zero down-projections: only the gated shared expert remains
    w0 = dict(w)
    w0["w_down"] = torch.zeros_like(w["w_down"])
    res0 = oracle.verify_layer(x, w0, cfg)
    sh = _torch_ffn(x, w["ws_gate"], w["ws_up"], w["ws_down"]).numpy() * res["shared_scale"][:, None]
    np.testing.assert_allclose(res0["out"], sh, rtol=0, atol=1e-10 * np.abs(sh).max())
    # the routed part is linear in the gate weights
    r2 = oracle.layer(x, w["w_gate"], w["w_up"], w["w_down"], res["topk_idx"], 2 * res["topk_w"])
    r1 = oracle.layer(x, w["w_gate"], w["w_up"], w["w_down"], res["topk_idx"], res["topk_w"])
    np.testing.assert_allclose(r2, 2 * r1, rtol=1e-12, atol=1e-18)


def test_layer_uses_given_logits():
    shape, w, x, cfg = _tiny_case(9, T=5)
    z = np.zeros((5, shape.n_experts), np.float32)
    z[:, 4] = 2.0
    z[:, 1] = 1.0
    z[:, 5] = 0.5
    res = oracle.verify_layer(x, w, cfg, logits=z)
    np.testing.assert_array_equal(res["topk_idx"], np.tile(np.array([4, 1, 5], np.int32), (5, 1)))


# --------------------------------------------------------------------------------------
# activation statistics of the synthetic "balanced routing" against Eq. N(t)
# --------------------------------------------------------------------------------------

def _nact_variance(E, k, T):
    u = (1 - k / E) ** T
    v = ((E - k) * (E - k - 1) / (E * (E - 1))) ** T
    return E * u + E * (E - 1) * v - (E * u) ** 2


@pytest.mark.parametrize("E,k,T", [(8, 2, 16), (60, 4, 16), (64, 8, 8), (256, 8, 16), (256, 8, 96)])
def test_uniform_routing_matches_expected_active(E, k, T):
    """iid logits make each token's top-k set a uniform k-subset: Eq. N(t) is the exact mean.

    The standard error uses the exact variance of the number of occupied experts,
    Var = E*u + E*(E-1)*v - (E*u)^2 with u = (1-k/E)^T and
    v = ((E-k)(E-k-1)/(E(E-1)))^T (pairwise-miss probability).
    """
    seeds = 300
    counts = []
    rng = np.random.default_rng(E * 1000 + T)
    for s in range(seeds):
        z = rng.normal(size=(T, E)).astype(np.float32)
        idx, _ = oracle.route_topk(z, k, oracle.SCORE_SOFTMAX, 0, 1.0)
        grp = oracle.permute(idx, E)
        assert grp.counts.sum() == T * k
        counts.append(grp.n_active)
    mean = float(np.mean(counts))
    se = math.sqrt(_nact_variance(E, k, T) / seeds)
    assert abs(mean - oracle.expected_active(E, k, T)) < 3.5 * se
    # the sample variance agrees with the exact variance too (chi-square, loose)
    assert np.var(counts, ddof=1) == pytest.approx(_nact_variance(E, k, T), rel=0.35)
    # measured tokens per activated expert tracks Eq. T_exp
    texp = T * k / mean
    assert texp == pytest.approx(oracle.mean_tokens_per_expert(k / E, T), rel=0.03)


@pytest.mark.parametrize("E,k,T", [(60, 4, 16), (64, 8, 8)])
def test_synthetic_balanced_router_is_close_to_uniform(E, k, T):
    """The workload recipe (Gaussian router matrix on Gaussian tokens) is balanced up to the
    spread of the router rows' norms: mean activated experts within 3% of Eq. N(t)."""
    H, seeds = 1024, 60
    counts = []
    for s in range(seeds):
        shape = wl.small_shape("r", H, E, k, 32)
        g = torch.Generator().manual_seed(1000 + s)
        wr = (torch.randn(E, H, generator=g) * 0.02).float()
        x = wl.make_tokens(shape, T, s)
        idx, _ = oracle.route_topk(oracle.router_logits(x, wr), k, oracle.SCORE_SOFTMAX, 0, 1.0)
        counts.append(oracle.permute(idx, E).n_active)
    assert float(np.mean(counts)) == pytest.approx(oracle.expected_active(E, k, T), rel=0.03)


def test_single_token_activates_exactly_k():
    for E, k in [(8, 2), (60, 4), (256, 8)]:
        z = np.random.default_rng(E).normal(size=(1, E)).astype(np.float32)
        idx, _ = oracle.route_topk(z, k, oracle.SCORE_SOFTMAX, 0, 1.0)
        assert oracle.permute(idx, E).n_active == k


def test_closed_forms_against_golden_file():
    """tests/golden/closed_form_values.txt: Eq. N(t) and Eq. T_thres at the benchmark shapes."""
    import os

    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "closed_form_values.txt")
    n_rows = 0
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        kind, E, K, arg, val = line.split()
        if kind == "N":
            assert oracle.expected_active(int(E), int(K), int(arg)) == pytest.approx(float(val), abs=2e-9)
        else:
            assert oracle.token_threshold(int(K) / int(E), float(arg)) == int(val)
        n_rows += 1
    assert n_rows == 9
