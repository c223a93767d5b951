"""GPU parity of the single stages (through the C ABI) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_19645_b200 import workloads as wl
from parity_utils import GATE_W_ATOL, assert_logits_close, assert_output_close

pytestmark = pytest.mark.gpu


def _api():
    from paper_2505_19645_b200 import api
    return api


@pytest.mark.parametrize("E,k", [(8, 2), (60, 4), (64, 8), (256, 8), (512, 16), (5, 5), (1, 1), (33, 3)])
@pytest.mark.parametrize("score_fn,renorm", [(0, 0), (0, 1), (1, 1), (1, 0)])
def test_route_topk_bit_exact(E, k, score_fn, renorm):
    api = _api()
    T = 203
    rng = np.random.default_rng(E * 31 + k)
    z = rng.normal(0, 1.5, size=(T, E)).astype(np.float32)
    # crafted ties: constant rows, duplicated values, one-ulp differences
    z[0, :] = 0.25
    z[1, :] = np.float32(1.0)
    if E > 2:
        z[1, E // 2] = np.nextafter(np.float32(1.0), np.float32(2.0))
        z[2, :] = np.round(z[2, :])          # many exact duplicates
        z[3, ::2] = z[3, 0]
    shape = wl.small_shape("r", 64, E, k, 64, 0, score_fn, renorm, 0, 1.0 if E != 60 else 2.5)
    cfg = api.make_config(shape)
    zd = torch.from_numpy(z).cuda()
    idx = torch.empty((T, k), dtype=torch.int32, device="cuda")
    w = torch.empty((T, k), dtype=torch.float32, device="cuda")
    api.moe_route_topk(cfg, zd, idx, w)
    torch.cuda.synchronize()
    idx_ref, w_ref = oracle.route_topk(z, k, score_fn, renorm, shape.routed_scale)
    np.testing.assert_array_equal(idx.cpu().numpy(), idx_ref)
    assert np.abs(w.cpu().numpy().astype(np.float64) - w_ref).max() <= GATE_W_ATOL * shape.routed_scale


@pytest.mark.parametrize("E,k", [(8, 2), (60, 4), (256, 8)])
def test_route_topk_stays_in_bounds_on_non_finite_logits(E, k):
    """Logits are finite by contract; NaN / Inf rows may come out in any order, but the
    selection must still be k distinct experts inside [0, E): nothing downstream indexes out
    of bounds."""
    api = _api()
    T = 64
    rng = np.random.default_rng(E + k)
    z = rng.normal(0, 1, size=(T, E)).astype(np.float32)
    z[0, :] = np.nan
    z[1, ::2] = np.nan
    z[2, :] = -np.inf
    z[3, :] = np.inf
    z[4, 0] = np.nan
    z[5, -1] = np.inf
    z[6, : E // 2] = -np.inf
    shape = wl.small_shape("nf", 64, E, k, 64, 0, 0, 1, 0)
    cfg = api.make_config(shape)
    idx = torch.full((T, k), -7, dtype=torch.int32, device="cuda")
    w = torch.empty((T, k), dtype=torch.float32, device="cuda")
    api.moe_route_topk(cfg, torch.from_numpy(z).cuda(), idx, w)
    torch.cuda.synchronize()
    got = idx.cpu().numpy()
    assert got.min() >= 0 and got.max() < E
    for t in range(T):
        assert len(set(got[t].tolist())) == k
    # finite rows are unaffected by their neighbours
    idx_ref, _ = oracle.route_topk(z[7:], k, 0, 1, 1.0)
    np.testing.assert_array_equal(got[7:], idx_ref)


@pytest.mark.parametrize("T,k,E,mode", [
    (1, 2, 8, "rand"), (16, 2, 8, "rand"), (640, 4, 60, "rand"), (1280, 8, 64, "rand"),
    (4096, 8, 256, "rand"), (300, 1, 512, "rand"), (257, 4, 60, "one"), (100, 8, 8, "all"),
    (777, 6, 200, "skew"),
])
def test_permute_bit_exact(T, k, E, mode):
    api = _api()
    rng = np.random.default_rng(T + E)
    if mode == "one":      # every token picks the same k experts: E-k experts stay empty
        idx = np.tile(np.array([7, 3, 59, 20][:k], np.int32), (T, 1))
    elif mode == "all":    # k = E
        idx = np.stack([rng.permutation(E) for _ in range(T)]).astype(np.int32)
    elif mode == "skew":
        p = 1.0 / np.arange(1, E + 1) ** 1.2
        p /= p.sum()
        idx = np.stack([rng.choice(E, size=k, replace=False, p=p) for _ in range(T)]).astype(np.int32)
    else:
        idx = np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
    shape = wl.small_shape("p", 64, E, k, 64)
    cfg = api.make_config(shape)
    g = api.alloc_grouping(cfg, T)
    for t in (g.counts, g.offsets, g.perm, g.inv_perm, g.active, g.n_active):
        t.fill_(-77)
    api.moe_permute(cfg, torch.from_numpy(idx).cuda(), g)
    torch.cuda.synchronize()
    ref = oracle.permute(idx, E)
    np.testing.assert_array_equal(g.counts.cpu().numpy(), ref.counts)
    np.testing.assert_array_equal(g.offsets.cpu().numpy(), ref.offsets)
    np.testing.assert_array_equal(g.perm.cpu().numpy(), ref.perm)
    np.testing.assert_array_equal(g.inv_perm.cpu().numpy(), ref.inv_perm)
    np.testing.assert_array_equal(g.active.cpu().numpy(), ref.active)
    assert int(g.n_active.item()) == ref.n_active
    assert int(g.counts.sum().item()) == T * k


@pytest.mark.parametrize("T,H,E,bias,gate", [(1, 256, 8, False, False), (37, 2048, 60, False, True),
                                             (130, 7168, 256, True, False), (9, 96, 3, True, True),
                                             # two row blocks per CTA: many experts x many tokens,
                                             # an odd number of row blocks, a ragged token tile
                                             (700, 512, 256, True, False), (1000, 256, 200, False, True),
                                             # few tokens, long rows: clusters of CTAs split H
                                             (1, 4096, 8, False, False), (5, 7168, 256, True, False),
                                             (16, 4096, 60, False, True), (3, 4128, 17, True, True)])
def test_router_logits(T, H, E, bias, gate):
    api = _api()
    shape = wl.small_shape("l", H, E, 1, 64, 64 if gate else 0, 0, 0, 1 if gate else 0)
    w = wl.make_weights(shape, 5, "cuda", zipf_s=1.2 if bias else None)
    x = wl.make_tokens(shape, T, 6, "cuda")
    cfg, cw = api.make_config(shape), api.make_weights(w)
    z = torch.empty((T, E), dtype=torch.float32, device="cuda")
    s = torch.empty((T,), dtype=torch.float32, device="cuda") if gate else None
    api.moe_router_logits(cfg, cw, x, z, s)
    torch.cuda.synchronize()
    z_ref = oracle.router_logits(x.cpu(), w["w_router"].cpu(),
                                 None if not bias else w["router_bias"].cpu())
    assert_logits_close(z.cpu().numpy(), z_ref, x.cpu(), w["w_router"].cpu(),
                        None if not bias else w["router_bias"].cpu())
    if gate:
        s_ref = oracle.shared_gate(x.cpu(), w["w_shared_gate"].cpu())
        assert np.abs(s.cpu().numpy() - s_ref).max() <= 1e-5


@pytest.mark.parametrize("T,H,E,k,I,Is", [
    (5, 64, 4, 2, 96, 0),          # single partial chunk
    (77, 160, 6, 3, 224, 96),      # ragged rows, row tails (H % 64 != 0, I % 32 == 0), shared
    (150, 256, 2, 2, 128, 0),      # experts with > 32 rows: several segments per expert
])
def test_grouped_swiglu_and_combine(T, H, E, k, I, Is):
    api = _api()
    shape = wl.small_shape("f", H, E, k, I, Is, 0, 1, 0)
    w = wl.make_weights(shape, 21, "cuda")
    for key in ("w_gate", "w_up", "w_down", "ws_gate", "ws_up", "ws_down"):
        if w[key] is not None:
            w[key] = (w[key].float() * 8).to(torch.bfloat16)
    x = wl.make_tokens(shape, T, 22, "cuda")
    cfg, cw = api.make_config(shape), api.make_weights(w)
    rng = np.random.default_rng(3)
    idx = np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
    wts = rng.uniform(0.1, 1.0, size=(T, k)).astype(np.float32)
    g = api.alloc_grouping(cfg, T)
    api.moe_permute(cfg, torch.from_numpy(idx).cuda(), g)
    ws = api.alloc_workspace(cfg, T)
    y = torch.empty((T * k, H), dtype=torch.bfloat16, device="cuda")
    ys = torch.empty((T, H), dtype=torch.bfloat16, device="cuda") if Is else None
    api.moe_grouped_swiglu(cfg, cw, x, g, y, ys, ws)
    out = torch.empty((T, H), dtype=torch.bfloat16, device="cuda")
    scale = torch.from_numpy(rng.uniform(0.2, 0.9, size=(T,)).astype(np.float32)).cuda() if Is else None
    api.moe_combine(cfg, y, g.inv_perm, torch.from_numpy(wts).cuda(), ys, scale, out)
    api.moe_check(ws)

    wh = {kk: (None if v is None else v.cpu()) for kk, v in w.items()}
    xh = x.cpu()
    # per sorted row: y[i] = FFN_{expert(i)}(x[token(i)])
    perm = g.perm.cpu().numpy()
    y_ref = np.empty((T * k, H))
    for e in range(E):
        rows = [i for i in range(T * k) if idx.reshape(-1)[perm[i]] == e]
        if rows:
            toks = torch.from_numpy(perm[rows] // k)
            y_ref[rows] = oracle.expert_ffn(xh[toks], wh["w_gate"][e], wh["w_up"][e], wh["w_down"][e])
    assert_output_close(y.float().cpu().numpy(), y_ref, "y")
    shared = (wh["ws_gate"], wh["ws_up"], wh["ws_down"]) if Is else None
    if Is:
        ys_ref = oracle.expert_ffn(xh, *shared)
        assert_output_close(ys.float().cpu().numpy(), ys_ref, "shared_y")
    ref = oracle.layer(xh, wh["w_gate"], wh["w_up"], wh["w_down"], idx, wts.astype(np.float64),
                       shared, None if scale is None else scale.cpu().numpy().astype(np.float64))
    assert_output_close(out.float().cpu().numpy(), ref, "out")


def test_invalid_arguments_are_rejected_before_launch():
    api = _api()
    shape = wl.small_shape("e", 64, 4, 2, 64)
    w = wl.make_weights(shape, 1, "cuda")
    x = wl.make_tokens(shape, 4, 2, "cuda")
    cfg, cw = api.make_config(shape), api.make_weights(w)
    out = torch.empty_like(x)
    ws = api.alloc_workspace(cfg, 4)
    lib = api.load_library()
    import ctypes
    call = lambda c, B, g, wsb: lib.moe_verify_layer(  # noqa: E731
        ctypes.byref(c), ctypes.byref(cw), x.data_ptr(), B, g, out.data_ptr(), None, ws.data_ptr(), wsb, None)
    assert call(cfg, 4, 0, ws.numel()) == 0
    assert call(cfg, 0, 0, ws.numel()) == 1            # T < 1
    assert call(cfg, 4, 0, 16) == 3                    # workspace too small
    bad = api.make_config(wl.small_shape("e", 64, 4, 5, 64))
    assert call(bad, 4, 0, ws.numel()) == 1            # k > E
    bad = api.make_config(wl.small_shape("e", 72, 4, 2, 64))
    assert call(bad, 4, 0, ws.numel()) == 1            # H % 32 != 0
    assert lib.moe_verify_layer(ctypes.byref(cfg), ctypes.byref(cw), x.data_ptr() + 2, 1, 0,
                                out.data_ptr(), None, ws.data_ptr(), ws.numel(), None) == 1  # misaligned
    torch.cuda.synchronize()
