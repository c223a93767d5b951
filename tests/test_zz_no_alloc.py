"""moe_grouped_swiglu_static: the FFN step with its scratch inside the library.

It exists for callers that cannot allocate device memory where they run the layer (a server
whose memory plan is frozen, a plugin inside another framework's allocator) and so cannot
pass a workspace.  It must give what moe_grouped_swiglu gives.  Collected last on purpose:
a run that stops at the first failure has then already been through every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_19645_b200 import workloads as wl
from parity_utils import assert_output_close

pytestmark = pytest.mark.gpu


def _case(api, shape, T, seed):
    w = wl.make_weights(shape, seed, "cuda")
    for key in ("w_gate", "w_up", "w_down", "ws_gate", "ws_up", "ws_down"):
        if w[key] is not None:
            w[key] = (w[key].float() * 8).to(torch.bfloat16)
    x = wl.make_tokens(shape, T, seed + 1, "cuda")
    cfg, cw = api.make_config(shape), api.make_weights(w)
    rng = np.random.default_rng(seed)
    idx = np.stack([rng.permutation(shape.n_experts)[:shape.top_k] for _ in range(T)]).astype(np.int32)
    g = api.alloc_grouping(cfg, T)
    api.moe_permute(cfg, torch.from_numpy(idx).cuda(), g)
    return w, x, cfg, cw, g, idx


def _oracle_rows(shape, w, x, g, idx):
    """y[i] = FFN_{expert(i)}(x[token(i)]) for every sorted row i, and the shared expert's
    output for every token, from the CPU oracle."""
    T, k, H = x.shape[0], shape.top_k, shape.hidden
    wh = {key: (None if v is None else v.cpu()) for key, v in w.items()}
    xh = x.cpu()
    perm = g.perm.cpu().numpy()
    flat = idx.reshape(-1)
    y_ref = np.empty((T * k, H))
    for e in range(shape.n_experts):
        rows = [i for i in range(T * k) if flat[perm[i]] == e]
        if rows:
            toks = torch.from_numpy(perm[rows] // k)
            y_ref[rows] = oracle.expert_ffn(xh[toks], wh["w_gate"][e], wh["w_up"][e], wh["w_down"][e])
    ys_ref = None
    if shape.shared_inter:
        ys_ref = oracle.expert_ffn(xh, wh["ws_gate"], wh["ws_up"], wh["ws_down"])
    return y_ref, ys_ref


def _both(api, shape, T, seed):
    w, x, cfg, cw, g, idx = _case(api, shape, T, seed)
    A, H = T * shape.top_k, shape.hidden
    mk = lambda n: torch.full((n, H), float("nan"), dtype=torch.bfloat16, device="cuda")  # noqa: E731
    has_shared = shape.shared_inter > 0
    # existing entry point, caller-provided workspace
    ws = api.alloc_workspace(cfg, T)
    y_ref, ys_ref = mk(A), (mk(T) if has_shared else None)
    api.moe_grouped_swiglu(cfg, cw, x, g, y_ref, ys_ref, ws)
    api.moe_check(ws)
    # new entry point, nothing allocated by or for the call beyond inputs and outputs
    y, ys = mk(A), (mk(T) if has_shared else None)
    before = torch.cuda.memory_allocated()
    api.moe_grouped_swiglu_static(cfg, cw, x, g, y, ys)
    api.moe_check_static()   # synchronises; raises if a bounded wait gave up inside the call
    # (torch's counter sees torch's allocator only; that the call itself allocates nothing is
    # a property of its source: no cudaMalloc, no allocating library routine)
    assert torch.cuda.memory_allocated() == before
    # against the CPU oracle directly ...
    y_orc, ys_orc = _oracle_rows(shape, w, x, g, idx)
    assert_output_close(y.float().cpu().numpy(), y_orc, "y vs oracle")
    if has_shared:
        assert_output_close(ys.float().cpu().numpy(), ys_orc, "shared_y vs oracle")
    # ... and against the entry point it is a variant of
    assert_output_close(y.float().cpu().numpy(), y_ref.float().cpu().numpy().astype(np.float64), "y")
    assert torch.equal(y, y_ref)          # same kernels, same order: identical bits
    if has_shared:
        assert_output_close(ys.float().cpu().numpy(), ys_ref.float().cpu().numpy().astype(np.float64),
                            "shared_y")
        assert torch.equal(ys, ys_ref)


def test_static_scratch_matches_workspace_variant_twice_in_a_row():
    from paper_2505_19645_b200 import api

    # two calls in a row share the array: the second (other shape, fewer tokens, ragged
    # segments) must not be disturbed by what the first left behind
    _both(api, wl.small_shape("s1", 256, 8, 2, 512, 384, 0, 1, 0), 150, 31)
    _both(api, wl.small_shape("s2", 160, 6, 3, 224, 0, 0, 1, 0), 41, 32)


def test_static_scratch_rejects_oversized_requests():
    from paper_2505_19645_b200 import api

    shape = wl.small_shape("big", 256, 8, 2, 2048, 0, 0, 1, 0)
    T = 2048                                  # 2*A*inter = 16 MiB > 8 MiB
    w, x, cfg, cw, g, _ = _case(api, shape, T, 33)
    y = torch.empty((T * 2, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(api.MoeError) as e:
        api.moe_grouped_swiglu_static(cfg, cw, x, g, y, None)
    assert e.value.status == 3                # MOE_ERR_WORKSPACE
    torch.cuda.synchronize()


def test_static_scratch_status_word_is_reported_through_moe_check_static():
    """A caller of the static entry point owns no workspace, so the status word of a bounded
    wait that gave up lives inside the library's array and is read with moe_check_static.  The
    self-test makes the progress-counter wait run out on that word (nothing faults): the
    report arrives once, and the next static call is unaffected."""
    from paper_2505_19645_b200 import api

    api.moe_check_static()
    api.moe_selftest_wait_limit_static(5000)   # 5 ms
    with pytest.raises(api.MoeError) as e:
        api.moe_check_static()
    assert e.value.status == 5                # MOE_ERR_TIMEOUT
    api.moe_check_static()                    # reported once
    _both(api, wl.small_shape("s3", 256, 8, 2, 512, 384, 0, 1, 0), 70, 34)
