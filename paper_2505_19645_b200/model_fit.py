"""The paper's analytical model of the target model's forward time (Sec. 3.4), restricted to
the MoE FFN layer this package measures, and its bounded least-squares fit (Algorithm 1).

For t = B*(gamma+1) tokens, E experts and K experts per token the modelled layer time is

    time(t) = bias + k1*G(t) + k2*N(t) + k3*G(T_exp(t))

with N(t) the expected number of activated experts (Eq. N(t)), T_exp(t) = t*K/N(t) the mean
tokens per activated expert (Eq. T_exp) and G(t; lam*RP, s) the smooth roofline curve of
Eq. G(t): s**t up to the transition point lam*RP and its tangent line beyond.  The six
parameters (bias, k1, k2, k3, lam, s) are fitted to measured layer times by minimising
half the sum of squared residuals inside box bounds, as the paper does for its ten-parameter
speed-up model; draft model, rejection sampling and attention terms have no counterpart in
a single FFN layer and are left out.

The optimiser is a projected Levenberg-Marquardt iteration written out here (forward
difference Jacobian, damping adapted per step, iterates clipped to the box), started from
several points; it uses numpy only.  Measurements are the "sweep" rows that bench.py prints.

    python -m paper_2505_19645_b200.model_fit RESULT.json [RESULT.json ...]
"""
from __future__ import annotations

import json
import math
import os
import sys

import numpy as np

PARAM_NAMES = ("bias", "k1", "k2", "k3", "lam", "s")


def expected_active(E: float, K: float, t):
    """Eq. N(t): E * (1 - ((E - K) / E) ** t)."""
    t = np.asarray(t, dtype=np.float64)
    return E * (1.0 - ((E - K) / E) ** t)


def mean_tokens_per_expert(E: float, K: float, t):
    """Eq. T_exp: t * K / N(t) = rho * t / (1 - (1 - rho) ** t) with rho = K / E."""
    t = np.asarray(t, dtype=np.float64)
    return t * K / expected_active(E, K, t)


def roofline_curve(t, transition: float, s: float):
    """Eq. G(t): s**t for t <= transition, the tangent at the transition beyond it."""
    t = np.asarray(t, dtype=np.float64)
    at = s ** transition
    return np.where(t <= transition, s ** np.minimum(t, transition),
                    at * (1.0 + math.log(s) * (t - transition)))


def layer_time(params, t, K, E, ridge: float):
    """Modelled layer time (the target-model lines of Algorithm 1 without the dense and
    attention parts that a single FFN layer does not have)."""
    bias, k1, k2, k3, lam, s = params
    t = np.asarray(t, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    E = np.asarray(E, dtype=np.float64)
    n_act = expected_active(E, K, t)
    t_exp = t * K / n_act
    return (bias + k1 * roofline_curve(t, lam * ridge, s) + k2 * n_act
            + k3 * roofline_curve(t_exp, lam * ridge, s))


def default_bounds(fixed_bytes: float, expert_bytes: float, bandwidth: float):
    """Box bounds in the spirit of Appendix "Fitting Details": bias and k2 between the
    time the bytes need at peak bandwidth and five times that, k1 and k3 non-negative,
    lam in [0.2, 1], s in (1, 2].  Times in microseconds, bandwidth in bytes per second.
    A layer without fixed (shared-expert, router) bytes still has launch latency, so the
    upper bound of bias never falls below 100 us."""
    bias_min = 1e6 * fixed_bytes / bandwidth
    k2_min = 1e6 * expert_bytes / bandwidth
    lo = np.array([bias_min, 0.0, k2_min, 0.0, 0.2, 1.0 + 1e-9])
    hi = np.array([max(5.0 * bias_min, 100.0), np.inf, 5.0 * k2_min, np.inf, 1.0, 2.0])
    return lo, hi


def _residuals(params, data, ridge):
    return layer_time(params, data["t"], data["K"], data["E"], ridge) - data["us"]


def least_squares_box(fun, x0, lo, hi, max_iter: int = 400, tol: float = 1e-12):
    """Minimise 0.5*||fun(x)||^2 subject to lo <= x <= hi by projected Levenberg-Marquardt."""
    x = np.clip(np.asarray(x0, dtype=np.float64), lo, hi)
    r = fun(x)
    cost = 0.5 * float(r @ r)
    mu = 1e-2
    for _ in range(max_iter):
        # forward-difference Jacobian, stepping into the box
        J = np.empty((r.size, x.size))
        for j in range(x.size):
            h = 1e-6 * max(1.0, abs(x[j]))
            if x[j] + h > hi[j]:
                h = -h
            xp = x.copy()
            xp[j] += h
            J[:, j] = (fun(xp) - r) / h
        g = J.T @ r
        # variables pinned at a bound by the gradient do not move this step
        free = ~(((x <= lo) & (g > 0)) | ((x >= hi) & (g < 0)))
        if not free.any() or np.linalg.norm(g[free]) < tol:
            break
        Jf = J[:, free]
        A = Jf.T @ Jf
        improved = False
        for _ in range(30):
            step = np.linalg.solve(A + mu * np.diag(np.maximum(np.diag(A), 1e-12)), -g[free])
            xn = x.copy()
            xn[free] = np.clip(x[free] + step, lo[free], hi[free])
            rn = fun(xn)
            cn = 0.5 * float(rn @ rn)
            if np.isfinite(cn) and cn < cost:
                improved = True
                break
            mu *= 4.0
        if not improved:
            break
        done = cost - cn <= tol * max(cost, 1.0)
        x, r, cost = xn, rn, cn
        mu = max(mu / 3.0, 1e-12)
        if done:
            break
    return x, cost


def fit(data, ridge: float, lo, hi, starts=None):
    """Best of several starts.  data: dict of equal-length arrays t, K, E, us."""
    data = {k: np.asarray(v, dtype=np.float64) for k, v in data.items()}
    if starts is None:
        span = float(data["us"].max() - data["us"].min()) + 1.0
        starts = []
        for lam in (0.3, 0.6, 0.9):
            for s in (1.002, 1.01, 1.05):
                g_hi = s ** (lam * ridge)
                starts.append([max(lo[0], min(hi[0], float(data["us"].min()) / 2)),
                               span / (4 * g_hi), min(hi[2], max(lo[2], 2 * lo[2])),
                               span / (4 * g_hi), lam, s])
    best = None
    for x0 in starts:
        x, cost = least_squares_box(lambda p: _residuals(p, data, ridge), x0, lo, hi)
        if best is None or cost < best[1]:
            best = (x, cost)
    return best


def mse(params, data, ridge: float) -> float:
    r = _residuals(params, {k: np.asarray(v, dtype=np.float64) for k, v in data.items()}, ridge)
    return float(np.mean(r * r))


def load_sweeps(paths):
    """Rows (t, K, E, us) of the sweeps in bench.py result files, sorted as the paper sorts
    its measurements: by K, then gamma, then batch size."""
    rows = []
    shape = None
    for p in paths:
        line = open(p).read().strip().splitlines()[-1]
        d = json.loads(line)
        # every sweep of the line (bench.py --config X --sweeps config carries one)
        for sw in d["sweeps"].values():
            shape = sw["shape"]
            K, E = shape["top_k"], shape["n_experts"]
            for pt in sw["rows"]:
                rows.append((K, pt["gamma"], pt["B"], pt["T"], E, pt["us"]))
    rows.sort()
    arr = np.array(rows, dtype=np.float64)
    return {"K": arr[:, 0], "gamma": arr[:, 1], "B": arr[:, 2], "t": arr[:, 3], "E": arr[:, 4],
            "us": arr[:, 5]}, shape


def main(argv):
    if not argv:
        print(__doc__)
        return 2
    data, shape = load_sweeps(argv)
    try:
        peaks = json.load(open(os.path.join(os.path.dirname(os.path.dirname(
            os.path.abspath(__file__))), "MEASURED_PEAKS.json")))
    except OSError:
        peaks = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}  # earlier measurement on this GPU type
    bw = peaks["hbm_gbs"] * 1e9
    ridge = peaks["bf16_tflops"] * 1e12 / bw  # flop per byte = token rows at 2-byte weights
    H, I, Is, E = shape["hidden"], shape["inter"], shape["shared_inter"], shape["n_experts"]
    lo, hi = default_bounds(6.0 * H * Is + 4.0 * E * H, 6.0 * H * I, bw)
    cols = {k: data[k] for k in ("t", "K", "E", "us")}
    n = len(cols["t"])
    print("measurements: %d, ridge point %.0f rows" % (n, ridge))
    print("%5s %6s %10s   %s" % ("m", "stride", "MSE (us^2)", "  ".join(PARAM_NAMES)))
    for stride in (25, 16, 11, 8, 4, 2, 1):
        sel = {k: v[::stride] for k, v in cols.items()}
        x, _ = fit(sel, ridge, lo, hi)
        print("%5d %6d %10.2f   %s" % (len(sel["t"]), stride, mse(x, cols, ridge),
                                       "  ".join("%.4g" % v for v in x)))
    return 0


if __name__ == "__main__":
    sys.exit(main(sys.argv[1:]))
