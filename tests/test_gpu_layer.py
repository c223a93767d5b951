"""GPU parity of moe_verify_layer (through the C ABI) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_19645_b200 import workloads as wl
from parity_utils import check_layer_against_oracle, run_gpu_layer, to_host, assert_output_close

pytestmark = pytest.mark.gpu


def test_tiny_config_full_parity():
    """Config 1: hidden 256, 8 experts top-2, intermediate 512, B=4, gamma=3, seed 0."""
    shape = wl.CONFIGS["tiny"]
    w = wl.make_weights(shape, wl.config_seed("tiny"), "cuda")
    x = wl.make_tokens(shape, 16, wl.point_seed("tiny", 4, 3), "cuda")
    (mx, mean), dbg = check_layer_against_oracle(shape, w, x, 4, 3)
    assert dbg["counts"].sum() == 32


@pytest.mark.parametrize("name,H,E,k,I,Is,score,renorm,sgate,B,gamma,zipf", [
    ("softmax-renorm", 256, 8, 2, 512, 0, 0, 1, 0, 7, 2, None),
    ("qwen-like", 512, 60, 4, 352, 1408, 0, 0, 1, 13, 4, None),        # 65 tokens, shared + gate
    ("qwen-like-1tok", 512, 60, 4, 352, 1408, 0, 0, 1, 1, 0, None),    # T = 1
    ("dsv3-like", 1024, 256, 8, 256, 256, 1, 1, 0, 16, 5, None),       # sigmoid, 96 tokens
    ("dsv3-like-zipf", 1024, 256, 8, 256, 256, 1, 1, 0, 32, 3, 1.0),   # skewed popularity
    ("mixtral-like", 512, 8, 2, 1792, 0, 0, 1, 0, 64, 2, None),        # 48 rows per expert
    ("ragged", 160, 6, 3, 224, 96, 0, 1, 0, 11, 6, None),              # row tails everywhere
    ("dense-limit", 128, 4, 4, 256, 0, 0, 1, 0, 5, 1, None),           # k = E
    # few experts with long reductions: the routed down pass is cut into k chunks
    ("ksplit-routed", 256, 4, 2, 4096, 0, 0, 1, 0, 10, 3, None),       # four planes of y
    ("ksplit-odd", 384, 8, 2, 2176, 0, 0, 1, 0, 3, 2, None),           # two chunks, ragged second
    ("dense-contrast", 256, 1, 1, 3072, 3072, 0, 0, 1, 65, 1, None),   # E = k = 1, 130 rows
    # small batches (one routing launch) at the expert counts that select other code paths
    ("dsv3-like-small", 1024, 256, 8, 256, 256, 1, 1, 0, 4, 3, None),  # 16 tokens, 256 experts
    ("e512-small", 256, 512, 4, 128, 0, 0, 1, 0, 5, 1, 1.0),           # the expert limit, skewed
    ("e512-warp", 256, 512, 4, 128, 128, 1, 1, 0, 2, 3, 1.0),          # 32 assignments: sorted by one warp
    ("e8-warp-dup", 128, 8, 2, 256, 0, 0, 1, 0, 3, 4, None),           # 30 assignments on 8 experts
    ("e24-32tok", 256, 24, 16, 128, 128, 0, 0, 1, 8, 3, None),         # 32 tokens x top-16: 512 assignments
    ("e24-33tok", 256, 24, 16, 128, 128, 0, 0, 1, 11, 2, None),        # one token more: the long chain
    # large batches (T * E >= 128 K): router logits on tcgen05 (three bf16 planes, k chunks)
    ("tc-logits-gate", 512, 60, 4, 128, 128, 0, 0, 1, 550, 3, None),   # 2200 tokens, gate row (R = 61)
    ("tc-logits-2pairs", 512, 300, 4, 64, 0, 1, 1, 0, 200, 2, 1.0),    # two pairs of row blocks, bias
    ("tc-logits-ragged", 544, 130, 2, 64, 64, 0, 1, 1, 337, 2, None),  # 1011 tokens, half k box, R = 131
])
def test_layer_parity_small_shapes(name, H, E, k, I, Is, score, renorm, sgate, B, gamma, zipf):
    shape = wl.small_shape(name, H, E, k, I, Is, score, renorm, sgate)
    w = wl.make_weights(shape, 100 + E, "cuda", zipf_s=zipf)
    T = B * (gamma + 1)
    x = wl.make_tokens(shape, T, 200 + T, "cuda")
    check_layer_against_oracle(shape, w, x, B, gamma)


SCHEDULING_CASES = [
    ("rr-shared", 512, 60, 4, 352, 1408, 13, 4),     # shared expert with a k-split down pass
    ("rr-segments", 256, 4, 2, 384, 256, 100, 3),    # 200 rows per expert: segment pairs, 4 shared segments
    ("rr-ragged", 160, 6, 3, 224, 96, 11, 6),        # tiles shorter than a box, k tails
]


@pytest.mark.parametrize("name,H,E,k,I,Is,B,gamma", SCHEDULING_CASES)
def test_scheduling_mode_case(name, H, E, k, I, Is, B, gamma):
    """One case of the scheduling-mode test below (in this process: the host's own choice)."""
    shape = wl.small_shape(name, H, E, k, I, Is, 0, 0, 1)
    w = wl.make_weights(shape, 300 + E, "cuda")
    T = B * (gamma + 1)
    x = wl.make_tokens(shape, T, 400 + T, "cuda")
    check_layer_against_oracle(shape, w, x, B, gamma)


def _run_child(env_extra, k_expr):
    import os
    import subprocess
    import sys

    env = dict(os.environ, **env_extra)
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run(
        [sys.executable, "-m", "pytest", os.path.join(root, "tests", "test_gpu_layer.py"), "-q", "-x",
         "-m", "gpu", "-k", k_expr],
        env=env, cwd=root, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]
    assert "passed" in r.stdout


@pytest.mark.parametrize("mode", ["0", "1"])
def test_layer_parity_in_both_scheduling_modes(mode):
    """The FFN kernels hand out the routed work either as chunks of consecutive tiles or as
    single (segment pair, tile) items; MOE_FF_RR (a test hook the library reads once per
    process) forces one of the two, so the cases run in a child process per mode."""
    _run_child({"MOE_FF_RR": mode}, "scheduling_mode_case")


# One to four tokens with at most 32 assignments take the one-launch kernel (logits, routing,
# expert FFNs and combine behind grid barriers); MOE_SMALL_FUSED=0 keeps them on the kernel chain.
FEW_TOKEN_CASES = [
    ("few-qwen", 512, 60, 4, 352, 1408, 0, 0, 1, 1, 0, None),        # T = 1, shared expert + gate
    ("few-qwen-4", 512, 60, 4, 352, 1408, 0, 0, 1, 2, 1, None),      # T = 4
    ("few-dsv3", 1024, 256, 8, 256, 256, 1, 1, 0, 1, 3, None),       # sigmoid, 32 assignments
    ("few-dsv3-3", 1024, 256, 8, 256, 256, 1, 1, 0, 3, 0, 1.0),      # T = 3, skewed, bias
    ("few-mixtral", 512, 8, 2, 1792, 0, 0, 1, 0, 1, 2, None),        # no shared expert
    ("few-dup", 256, 4, 2, 384, 256, 0, 1, 0, 2, 1, None),           # 8 assignments on 4 experts: up to 4 rows each
    ("few-dense", 128, 4, 4, 256, 0, 0, 1, 0, 4, 0, None),           # k = E: every group has all 4 rows
    ("few-ragged", 160, 6, 3, 224, 96, 0, 1, 0, 1, 1, None),         # rows shorter than a lane step
    ("few-chunks", 384, 8, 2, 4352, 2176, 0, 0, 1, 3, 0, None),      # down projection in 3 and 2 column chunks, ragged last
    ("few-e512", 256, 512, 16, 128, 128, 1, 1, 0, 1, 1, 1.0),        # the expert limit, top-16 x 2 tokens
    ("few-k16-3tok", 256, 24, 16, 128, 128, 0, 0, 1, 3, 0, None),    # 48 assignments: stays on the chain
    ("few-dense-contrast", 256, 1, 1, 3072, 3072, 0, 0, 1, 2, 1, None),  # E = k = 1
]


@pytest.mark.parametrize("name,H,E,k,I,Is,score,renorm,sgate,B,gamma,zipf", FEW_TOKEN_CASES)
def test_few_token_case(name, H, E, k, I, Is, score, renorm, sgate, B, gamma, zipf):
    shape = wl.small_shape(name, H, E, k, I, Is, score, renorm, sgate)
    w = wl.make_weights(shape, 500 + E, "cuda", zipf_s=zipf)
    T = B * (gamma + 1)
    x = wl.make_tokens(shape, T, 600 + T, "cuda")
    check_layer_against_oracle(shape, w, x, B, gamma)


def test_few_tokens_take_one_launch():
    from paper_2505_19645_b200 import api

    shape = wl.small_shape("few-launch", 512, 60, 4, 352, 1408, 0, 0, 1)
    w = wl.make_weights(shape, 21, "cuda")
    x = wl.make_tokens(shape, 4, 22, "cuda")
    out_a, dbg_a = run_gpu_layer(shape, w, x, 2, 1)
    assert api.moe_last_launch_count() == 1
    out_b, dbg_b = run_gpu_layer(shape, w, x, 4, 0)
    assert torch.equal(out_a, out_b)
    for key in dbg_a:
        np.testing.assert_array_equal(dbg_a[key], dbg_b[key])
    # the fifth token moves the call to the kernel chain
    x5 = wl.make_tokens(shape, 5, 23, "cuda")
    run_gpu_layer(shape, w, x5, 5, 0)
    assert api.moe_last_launch_count() > 1


def test_one_workspace_serves_calls_of_every_size_in_turn():
    """The one-launch kernel's barrier word and counters live in the workspace and are never
    cleared: each call tags them with its own epoch.  Calls of one to five tokens (the last on
    the kernel chain) alternate on ONE workspace, which starts out filled with a byte pattern;
    every call must reproduce what a fresh workspace gives, and the status stays clear."""
    from paper_2505_19645_b200 import api

    shape = wl.small_shape("reuse", 512, 60, 4, 352, 1408, 0, 0, 1)
    w = wl.make_weights(shape, 31, "cuda")
    cfg, cw = api.make_config(shape), api.make_weights(w)
    xs = {T: wl.make_tokens(shape, T, 40 + T, "cuda") for T in (1, 2, 3, 4, 5)}
    want = {T: run_gpu_layer(shape, w, xs[T], T, 0)[0] for T in xs}
    ws = torch.full((api.moe_workspace_bytes(cfg, 5),), 0xA5, dtype=torch.uint8, device="cuda")
    for rep in range(6):
        for T in (1, 4, 5, 2, 3, 1):
            out = torch.empty_like(xs[T])
            api.moe_verify_layer(cfg, cw, xs[T], T, 0, out, ws)
            assert torch.equal(out, want[T]), (rep, T)
    api.moe_check(ws)


def test_kernel_chain_on_the_same_few_tokens():
    """The same cases with the one-launch kernel switched off (a test hook read once per
    process, hence the child process)."""
    _run_child({"MOE_SMALL_FUSED": "0"}, "test_few_token_case")


def test_layer_depends_on_token_count_only_and_is_deterministic():
    """layer(B, gamma) == layer(B*(gamma+1), 0) bit for bit; two runs and a run on another
    stream give identical routing, grouping and outputs."""
    shape = wl.small_shape("det", 512, 60, 4, 352, 704, 0, 0, 1)
    w = wl.make_weights(shape, 7, "cuda")
    x = wl.make_tokens(shape, 60, 8, "cuda")
    out_a, dbg_a = run_gpu_layer(shape, w, x, 12, 4)
    out_b, dbg_b = run_gpu_layer(shape, w, x, 60, 0)
    out_c, dbg_c = run_gpu_layer(shape, w, x, 20, 2)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        out_d, dbg_d = run_gpu_layer(shape, w, x, 12, 4)
    s.synchronize()
    for o, d in ((out_b, dbg_b), (out_c, dbg_c), (out_d, dbg_d)):
        assert torch.equal(out_a, o)
        for key in dbg_a:
            np.testing.assert_array_equal(dbg_a[key], d[key])


def test_zero_down_projection_leaves_shared_term():
    shape = wl.small_shape("z", 256, 8, 2, 128, 192, 0, 1, 1)
    w = wl.make_weights(shape, 9, "cuda")
    for key in ("ws_gate", "ws_up", "ws_down", "w_shared_gate"):
        w[key] = (w[key].float() * 8).to(torch.bfloat16)
    w["w_down"].zero_()
    x = wl.make_tokens(shape, 24, 10, "cuda")
    out, _ = run_gpu_layer(shape, w, x, 6, 3)
    wh = to_host(w)
    s = oracle.shared_gate(x.cpu(), wh["w_shared_gate"])
    ref = oracle.expert_ffn(x.cpu(), wh["ws_gate"], wh["ws_up"], wh["ws_down"]) * s[:, None]
    assert_output_close(out.float().cpu().numpy(), ref)


def test_row_permutation_equivariance():
    shape = wl.small_shape("perm", 256, 16, 4, 128, 0, 0, 0, 0)
    w = wl.make_weights(shape, 11, "cuda")
    x = wl.make_tokens(shape, 40, 12, "cuda")
    p = torch.randperm(40, generator=torch.Generator().manual_seed(0)).cuda()
    out, dbg = run_gpu_layer(shape, w, x, 40, 0)
    out_p, dbg_p = run_gpu_layer(shape, w, x[p].contiguous(), 40, 0)
    np.testing.assert_array_equal(dbg_p["topk_idx"], dbg["topk_idx"][p.cpu().numpy()])
    assert torch.equal(out_p, out[p])


@pytest.mark.parametrize("wide", ["0", "1"])
def test_layer_parity_in_both_ring_geometries(wide):
    """The FFN kernels run with segments of up to 128 token rows (two k boxes per weight slot,
    two sets of accumulators) or of up to 256 (one k box, one set); MOE_FF_WIDE (a test hook
    read once per process) forces one of the two on every call, also where the host would
    choose the other: the scheduling cases and a few small shapes in a child process each."""
    _run_child({"MOE_FF_WIDE": wide},
               "scheduling_mode_case or (small_shapes and (qwen-like or dense-contrast or "
               "ksplit-routed or ragged or e24-33tok or dsv3-like-zipf))")


def test_layer_parity_with_plain_stream_ordering():
    """MOE_NO_PDL=1 (read once per process) launches every kernel with plain stream ordering:
    the kernels then run one after the other and every progress counter is complete when its
    reader starts.  Runs a few of the cases above in a child process."""
    _run_child({"MOE_NO_PDL": "1"},
               "small_shapes and (qwen-like or mixtral-like or ksplit-routed)")


def test_wait_limit_expiry_is_reported_and_the_context_stays_usable():
    """Every wait inside the kernels has a limit.  The self-test runs the down pass's wait for
    a progress counter, and the one-launch layer's wait for its grid-wide counters, each on a
    word nothing advances: each gives up after its limit, the kernel raises
    the workspace's status word and returns, moe_check reports MOE_ERR_TIMEOUT, nothing
    faults, and the same workspace serves a correct layer call right after.  The word is
    sticky: a layer call enqueued behind the failed wait does not erase the report, and the
    report is made exactly once."""
    import time
    from paper_2505_19645_b200 import api

    shape = wl.small_shape("limit", 512, 60, 4, 352, 1408, 0, 0, 1)
    w = wl.make_weights(shape, 160, "cuda")
    x = wl.make_tokens(shape, 65, 265, "cuda")
    cfg, cw = api.make_config(shape), api.make_weights(w)
    ws = api.alloc_workspace(cfg, 65)
    api.moe_check(ws)   # a workspace no call has touched yet reports nothing
    run_gpu_layer(shape, w, x, 13, 4, ws=ws)
    t0 = time.perf_counter()
    api.moe_selftest_wait_limit(ws, 20000)  # 20 ms
    with pytest.raises(api.MoeError) as err:
        api.moe_check(ws)
    waited = time.perf_counter() - t0
    assert err.value.status == 5  # MOE_ERR_TIMEOUT
    assert 0.035 < waited < 1.0   # two waits of 20 ms: the tile kernels' and the one-launch layer's
    assert int(ws[12:16].view(torch.int32).item()) == 1   # the second wait gave up too
    api.moe_check(ws)   # reported once
    x3 = wl.make_tokens(shape, 3, 268, "cuda")
    out3, _ = run_gpu_layer(shape, w, x3, 3, 0, ws=ws)   # the one-launch layer on the same workspace
    ref3, _ = run_gpu_layer(shape, w, x3, 3, 0)
    assert torch.equal(out3, ref3)
    # a failure in an earlier call of a queue is still seen after later calls
    out = torch.empty_like(x)
    api.moe_selftest_wait_limit(ws, 2000)
    api.moe_verify_layer(cfg, cw, x, 13, 4, out, ws)
    api.moe_verify_layer(cfg, cw, x, 13, 4, out, ws)
    with pytest.raises(api.MoeError) as err:
        api.moe_check(ws)
    assert err.value.status == 5
    out, _ = run_gpu_layer(shape, w, x, 13, 4, ws=ws)   # runs normally, nothing to report
    ref, _ = run_gpu_layer(shape, w, x, 13, 4)
    assert torch.equal(out, ref)
    check_layer_against_oracle(shape, w, x, 13, 4)


# ---- full-size shapes in the launch configuration the benchmark times -------------------
# Routing and grouping are checked on every token; the outputs on 16 token rows that the
# oracle evaluates one by one (the layer is token-wise, so a row check is exact).  The rows
# are not drawn at random: they are picked from the grouping so that the first and last row of
# the largest group, a ragged tail segment, both sides of a segment boundary and the ends of
# the shared expert's last segment pair are always among them (parity_utils.stratified_rows).

_FULL = {}   # weights of one config at a time, on the device and on the host
N_ROWS = 16


def _full_weights(name, zipf):
    if _FULL.get("name") != name:
        _FULL.clear()
        torch.cuda.empty_cache()
        shape = wl.CONFIGS[name]
        need = 2.2 * 6 * shape.hidden * shape.inter * shape.n_experts   # bytes, with head room
        free, _ = torch.cuda.mem_get_info()
        import psutil
        if free < need or psutil.virtual_memory().available < need:
            pytest.skip("needs %.0f GB of device and of host memory" % (need / 1e9))
        w = wl.make_weights(shape, wl.config_seed(name), "cuda")
        _FULL.update(name=name, dev=w, host=to_host(w))
    w_dev, w_host = dict(_FULL["dev"]), dict(_FULL["host"])
    if zipf is not None:   # the skew variant differs in the router bias only
        shape = wl.CONFIGS[name]
        b = wl.zipf_router_bias(shape.n_experts, shape.hidden, zipf, wl.config_seed(name), "cpu")
        w_host["router_bias"] = b
        w_dev["router_bias"] = b.cuda()
    return w_dev, w_host


def _full_size(name, B, gamma, zipf=None):
    shape = wl.CONFIGS[name]
    w_dev, w_host = _full_weights(name, zipf)
    T = B * (gamma + 1)
    x = wl.make_tokens(shape, T, wl.point_seed(name, B, gamma), "cuda")
    fr, dbg = check_layer_against_oracle(shape, w_dev, x, B, gamma, rows=N_ROWS, w_host=w_host)
    return fr, dbg


def test_zipf_bias_is_the_only_difference_of_the_skew_variant():
    shape = wl.small_shape("zb", 64, 16, 2, 64)
    a = wl.make_weights(shape, 3, "cuda")
    b = wl.make_weights(shape, 3, "cuda", zipf_s=1.1)
    for key in a:
        if key != "router_bias":
            assert (a[key] is None and b[key] is None) or torch.equal(a[key], b[key])
    assert torch.equal(b["router_bias"].cpu(), wl.zipf_router_bias(16, 64, 1.1, 3, "cpu"))


@pytest.mark.parametrize("B,gamma", [(1, 0), (4, 0), (4, 1), (32, 3), (128, 4), (1024, 3)])
def test_full_size_qwen15_shape(B, gamma):
    _full_size("qwen1.5-moe-a2.7b", B, gamma)


@pytest.mark.parametrize("B,gamma,zipf", [(1, 0, None), (8, 2, None), (64, 4, 1.2), (256, 4, None),
                                          (256, 4, 1.2), (512, 3, None), (1024, 3, None)])
def test_full_size_qwen2_57b_shape(B, gamma, zipf):
    """Up to the top of the config's grid (T = 1280, also with Zipf(1.2) popularity) and the two
    extra token counts 2048 and 4096."""
    _full_size("qwen2-57b-a14b", B, gamma, zipf)


@pytest.mark.parametrize("B,gamma", [(1, 0), (16, 2), (256, 4)])
def test_full_size_mixtral_shape(B, gamma):
    _full_size("mixtral-8x7b", B, gamma)


@pytest.mark.parametrize("B,gamma,zipf", [(1, 0, None), (16, 3, None), (128, 3, None), (64, 3, 1.0),
                                          (512, 5, None), (512, 5, 1.0), (512, 3, None),
                                          (1024, 3, None)])
def test_full_size_deepseek_v3_shape(B, gamma, zipf):
    """The largest shape (22.6 GB of expert weights): bottom, middle and top (T = 3072) of its
    grid, the Zipf(1.0) variant in the middle and at the top, and T = 2048 / 4096."""
    fr, dbg = _full_size("deepseek-v3", B, gamma, zipf)
    if zipf is not None and B * (gamma + 1) >= 256:
        # skew shows: the most popular expert holds several times the mean share
        assert dbg["counts"].max() > 3 * dbg["counts"].mean()


def test_full_size_weights_are_released():
    _FULL.clear()
    torch.cuda.empty_cache()
