"""The analytical layer-time model (Sec. 3.4, Eq. G(t), Algorithm 1) and its bounded fit."""
import math

import numpy as np
import pytest

from paper_2505_19645_b200 import model_fit as mf
from paper_2505_19645_b200 import workloads as wl

RIDGE = 255.0


def _grid():
    rows = [(B * (g + 1), K, 64) for K in wl.SPARSITY_TOP_KS for g in wl.SPARSITY_GAMMAS
            for B in wl.SPARSITY_BATCHES]
    arr = np.array(rows, dtype=np.float64)
    return {"t": arr[:, 0], "K": arr[:, 1], "E": arr[:, 2]}


def test_roofline_curve_is_exponential_then_its_tangent():
    s, tp = 1.02, 80.0
    assert mf.roofline_curve(0.0, tp, s) == pytest.approx(1.0)
    assert mf.roofline_curve(37.0, tp, s) == pytest.approx(1.02 ** 37)
    # value and first derivative agree at the transition point (Eq. G(t))
    eps = 1e-4
    left = (mf.roofline_curve(tp, tp, s) - mf.roofline_curve(tp - eps, tp, s)) / eps
    right = (mf.roofline_curve(tp + eps, tp, s) - mf.roofline_curve(tp, tp, s)) / eps
    assert left == pytest.approx(right, rel=1e-4)
    assert left == pytest.approx(math.log(s) * s ** tp, rel=1e-4)
    # linear beyond: equal increments
    a, b, c = (float(mf.roofline_curve(t, tp, s)) for t in (100.0, 150.0, 200.0))
    assert b - a == pytest.approx(c - b)
    # and below the exponential it continues (a tangent of a convex curve)
    assert float(mf.roofline_curve(200.0, tp, s)) < s ** 200.0


def test_expected_active_and_tokens_per_expert_closed_forms():
    # one token activates exactly K experts; many tokens activate all of them
    assert mf.expected_active(60, 4, 1) == pytest.approx(4.0)
    assert mf.expected_active(60, 4, 10_000) == pytest.approx(60.0)
    # exact enumeration for two tokens: E - E * ((E-K)/E)^2
    assert mf.expected_active(8, 2, 2) == pytest.approx(8 - 8 * (6 / 8) ** 2)
    # the dense limit rho = 1: every expert sees every token
    assert mf.mean_tokens_per_expert(16, 16, 37) == pytest.approx(37.0)
    # T_exp * N = t * K (every token is counted K times)
    t = np.arange(1, 200)
    assert np.allclose(mf.mean_tokens_per_expert(64, 8, t) * mf.expected_active(64, 8, t), t * 8)


def test_layer_time_reduces_to_its_terms():
    p = [10.0, 0.0, 2.0, 0.0, 0.5, 1.01]
    # only the expert-loading term: bias + k2 * N(t)
    assert mf.layer_time(p, 5, 8, 64, RIDGE) == pytest.approx(10.0 + 2.0 * mf.expected_active(64, 8, 5))
    p = [0.0, 3.0, 0.0, 0.0, 0.5, 1.01]
    assert mf.layer_time(p, 50, 8, 64, RIDGE) == pytest.approx(3.0 * 1.01 ** 50)
    p = [0.0, 0.0, 0.0, 7.0, 0.5, 1.01]
    t_exp = float(mf.mean_tokens_per_expert(64, 8, 50))
    assert mf.layer_time(p, 50, 8, 64, RIDGE) == pytest.approx(7.0 * 1.01 ** t_exp)


def test_fit_reproduces_noise_free_data():
    data = _grid()
    true = np.array([120.0, 3.0, 9.5, 40.0, 0.5, 1.01])
    data["us"] = mf.layer_time(true, data["t"], data["K"], data["E"], RIDGE)
    lo, hi = mf.default_bounds(440e6, 55e6, 6.4e12)
    x, cost = mf.fit(data, RIDGE, lo, hi)
    # root-mean-square residual below 0.1 % of the typical layer time
    assert math.sqrt(mf.mse(x, data, RIDGE)) < 1e-3 * float(np.mean(data["us"]))
    assert np.all(x >= lo) and np.all(x <= hi)


def test_fit_matches_a_library_trust_region_solver():
    """Same residuals, same bounds, same starts: the hand-written projected
    Levenberg-Marquardt reaches the cost that scipy's trust-region-reflective solver finds."""
    from scipy.optimize import least_squares

    data = _grid()
    rng = np.random.default_rng(0)
    true = np.array([120.0, 3.0, 9.5, 40.0, 0.5, 1.01])
    clean = mf.layer_time(true, data["t"], data["K"], data["E"], RIDGE)
    data["us"] = clean * (1.0 + 0.01 * rng.standard_normal(clean.size))
    lo, hi = mf.default_bounds(440e6, 55e6, 6.4e12)
    x, cost = mf.fit(data, RIDGE, lo, hi)
    best = None
    for lam in (0.3, 0.6, 0.9):
        for s in (1.002, 1.01, 1.05):
            x0 = np.clip([100.0, 1.0, 10.0, 1.0, lam, s], lo, np.minimum(hi, 1e9))
            r = least_squares(lambda p: mf._residuals(p, data, RIDGE), x0, bounds=(lo, hi), method="trf")
            if best is None or r.cost < best.cost:
                best = r
    assert cost <= best.cost * (1.0 + 1e-4)
    # fitting a strided sample still describes all points (the paper's Table "m vs MSE")
    sel = {k: v[::11] for k, v in data.items()}
    xs, _ = mf.fit(sel, RIDGE, lo, hi)
    assert mf.mse(xs, data, RIDGE) < 4.0 * mf.mse(x, data, RIDGE) + 1.0


def test_bounds_follow_the_bytes():
    lo, hi = mf.default_bounds(440e6, 55e6, 6.4e12)
    assert lo[0] == pytest.approx(68.75) and hi[0] == pytest.approx(5 * 68.75)
    assert lo[2] == pytest.approx(1e6 * 55e6 / 6.4e12) and hi[2] == pytest.approx(5 * lo[2])
    assert (lo[4], hi[4], hi[5]) == (0.2, 1.0, 2.0) and lo[5] > 1.0
