"""CPU-only checks of the C-ABI library: it loads, exports every declared symbol, and
rejects bad arguments on the host before anything could be launched."""
import ctypes
import os
import re

import pytest

from paper_2505_19645_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in os.listdir(inc):
        if not f.endswith(".h"):
            continue
        text = open(os.path.join(inc, f)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        for m in re.finditer(r"\b(moe_[a-z_0-9]+)\s*\(", text):
            names.add(m.group(1))
    return sorted(names)


def test_library_loads_and_exports_every_declared_symbol():
    from paper_2505_19645_b200 import api

    lib = api.load_library()
    declared = _declared_functions()
    assert len(declared) >= 9
    for name in declared:
        assert hasattr(lib, name), "missing export " + name
    assert sorted(set(api.EXPORTS) - set(declared)) == []


def test_status_strings():
    from paper_2505_19645_b200 import api

    assert api.status_string(0) == "ok"
    assert "workspace" in api.status_string(3)


def test_workspace_bytes_and_host_side_validation():
    from paper_2505_19645_b200 import api

    lib = api.load_library()
    shape = wl.CONFIGS["qwen1.5-moe-a2.7b"]
    cfg = api.make_config(shape)
    n1, n2 = api.moe_workspace_bytes(cfg, 1), api.moe_workspace_bytes(cfg, 640)
    # at least h [A,I], y [A,H], shared h and y
    assert n2 > 640 * (4 * (1408 + 2048) + 5632 + 2048) * 2 and n1 < n2
    assert api.moe_workspace_bytes(cfg, 0) == 0
    bad = api.make_config(wl.small_shape("b", 64, 4, 5, 64))
    assert api.moe_workspace_bytes(bad, 8) == 0
    bad = api.make_config(wl.small_shape("b", 64, 600, 2, 64))
    assert api.moe_workspace_bytes(bad, 8) == 0
    # null pointers are refused with MOE_ERR_INVALID_ARG without touching a device
    w = api.CWeights()
    st = lib.moe_verify_layer(ctypes.byref(cfg), ctypes.byref(w), None, 1, 0, None, None, None, 0, None)
    assert st == 1
    st = lib.moe_route_topk(ctypes.byref(cfg), None, 4, None, None, None)
    assert st == 1
    st = lib.moe_permute(ctypes.byref(cfg), None, 4, None, None, None, None, None, None, None)
    assert st == 1


def test_workspace_bytes_never_shrink_with_the_token_count():
    """A workspace sized for max_tokens must serve every smaller call, also where the small
    calls keep several partial planes of the routed output."""
    from paper_2505_19645_b200 import api

    for name in ("qwen2-57b-a14b", "mixtral-8x7b", "deepseek-v3"):
        for shape in (wl.CONFIGS[name], wl.dense_contrast(wl.CONFIGS[name]),
                      wl.with_top_k(wl.CONFIGS[name], 1)):
            cfg = api.make_config(shape)
            sizes = [api.moe_workspace_bytes(cfg, t) for t in range(1, 700, 7)]
            assert all(a <= b for a, b in zip(sizes, sizes[1:])), shape.name
            A, H = 694 * shape.top_k, shape.hidden
            assert sizes[-1] >= A * (H + shape.inter) * 2


def test_workload_variants_keep_the_active_parameters():
    base = wl.CONFIGS["qwen2-57b-a14b"]
    dense = wl.dense_contrast(base)
    assert (dense.n_experts, dense.top_k) == (1, 1)
    assert dense.top_k * dense.inter == base.top_k * base.inter
    assert dense.shared_inter == base.shared_inter and dense.hidden == base.hidden
    for k in wl.SPARSITY_TOP_KS:
        v = wl.with_top_k(base, k)
        assert v.top_k == k and v.n_experts == base.n_experts and v.inter == base.inter
    assert len(wl.SPARSITY_BATCHES) == 19 and base.top_k in wl.SPARSITY_TOP_KS


def test_missing_library_fails_loudly(monkeypatch):
    from paper_2505_19645_b200 import api

    monkeypatch.setattr(api, "_lib", None)
    monkeypatch.setattr(api, "LIB_PATH", os.path.join(ROOT, "no_such_dir", "libmoe_verify.so"))
    with pytest.raises(ImportError):
        api.load_library()


def test_workspace_regions_are_disjoint_aligned_and_guarded():
    """Every region starts 256-byte aligned, lies inside moe_workspace_bytes and is followed
    by at least 256 bytes that belong to no region (the canary gaps of the GPU tests)."""
    from paper_2505_19645_b200 import api

    for name, T in (("tiny", 16), ("qwen1.5-moe-a2.7b", 1), ("qwen2-57b-a14b", 1280),
                    ("deepseek-v3", 3072)):
        cfg = api.make_config(wl.CONFIGS[name])
        total = api.moe_workspace_bytes(cfg, T)
        regions = api.workspace_regions(cfg, T)
        assert len(regions) == 24
        end = 0
        for i, (off, n) in enumerate(regions):
            assert off % 256 == 0
            assert off >= end + (256 if i else 0), (name, i)   # (an unused region has 0 bytes)
            end = off + n
        assert end + 256 <= total
        assert regions[0] == (0, 256)   # the status region leads the workspace


def test_workspace_size_never_shrinks_as_tokens_grow():
    """A workspace sized for max_tokens serves every call with fewer tokens: the layout of a
    call with T tokens must fit moe_workspace_bytes(T') for every T' >= T (regions that only
    small or only large calls use must not make the total dip in between)."""
    from paper_2505_19645_b200 import api

    for name in ("tiny", "qwen1.5-moe-a2.7b", "qwen2-57b-a14b", "mixtral-8x7b", "deepseek-v3"):
        cfg = api.make_config(wl.CONFIGS[name])
        sizes = [api.moe_workspace_bytes(cfg, T) for T in list(range(1, 70)) + [127, 128, 129, 511, 512, 513, 2048]]
        assert all(b >= a for a, b in zip(sizes, sizes[1:])), name


def test_per_device_set_up_state_is_kept_per_ordinal(tmp_path):
    """State the CUDA runtime keeps per device (the FFN kernels' shared-memory opt-in, the
    address of the built-in scratch array) is tracked per device ordinal by DeviceOnce: marking
    one ordinal must not mark another.  Compiled from the library's own header."""
    import subprocess

    src = tmp_path / "once.cpp"
    src.write_text('''
#include "device_once.h"
int main() {
    moe::DeviceOnce once;
    if (once.done(0) || once.done(1)) return 1;
    once.mark(0);
    if (!once.done(0)) return 2;
    if (once.done(1)) return 3;          // a second GPU still needs its own set-up
    once.mark(1);
    if (!once.done(1) || !once.done(0)) return 4;
    once.mark(-1); once.mark(1000);       // out of the table: ignored, never "done"
    if (once.done(-1) || once.done(1000)) return 5;
    moe::DeviceOnce other;
    if (other.done(0)) return 6;          // one object per piece of state
    return 0;
}
''')
    exe = tmp_path / "once"
    subprocess.run(["g++", "-std=c++17", "-I", os.path.join(ROOT, "paper_2505_19645_b200", "csrc"),
                    str(src), "-o", str(exe)], check=True)
    assert subprocess.run([str(exe)]).returncode == 0
