"""Host code of the library and the C oracle under AddressSanitizer / UndefinedBehaviorSanitizer
(CPU only).  The compute sanitiser is not available for the device code, so the GPU tests rely on
canary regions and bounded waits; the host side -- argument validation, workspace layout, the
launch heuristics that run inside it -- and the oracle are checked here with the compilers' own
sanitisers, in child processes with the run-times preloaded."""
import os
import shutil
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CSRC = os.path.join(ROOT, "paper_2505_19645_b200", "csrc")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")


def _runtime(name):
    path = subprocess.run(["gcc", "-print-file-name=" + name], capture_output=True, text=True).stdout.strip()
    return path if os.path.isabs(path) and os.path.exists(path) else None


def _env():
    asan, ubsan = _runtime("libasan.so"), _runtime("libubsan.so")
    if not asan or not ubsan:
        pytest.skip("sanitizer run-times not installed")
    return dict(os.environ, LD_PRELOAD=asan + ":" + ubsan,
                ASAN_OPTIONS="detect_leaks=0:protect_shadow_gap=0",
                UBSAN_OPTIONS="print_stacktrace=1:halt_on_error=1")


HOST_SCRIPT = r'''
import ctypes, sys
sys.path.insert(0, %(root)r)
from paper_2505_19645_b200 import api, workloads as wl
api.LIB_PATH = %(lib)r
lib = api.load_library()
for name in wl.CONFIG_ORDER:
    for shape in (wl.CONFIGS[name], wl.dense_contrast(wl.CONFIGS[name]), wl.with_top_k(wl.CONFIGS[name], 1)):
        cfg = api.make_config(shape)
        for T in (1, 31, 32, 33, 64, 65, 128, 129, 511, 512, 513, 1280, 3072, 4096):
            n = api.moe_workspace_bytes(cfg, T)
            regs = api.workspace_regions(cfg, T)
            assert n > 0 and regs and regs[-1][0] + regs[-1][1] <= n
w = api.CWeights()
cfg = api.make_config(wl.CONFIGS["tiny"])
assert lib.moe_verify_layer(ctypes.byref(cfg), ctypes.byref(w), None, 1, 0, None, None, None, 0, None) == 1
assert lib.moe_route_topk(ctypes.byref(cfg), None, 4, None, None, None) == 1
assert lib.moe_permute(ctypes.byref(cfg), None, 4, None, None, None, None, None, None, None) == 1
assert lib.moe_combine(ctypes.byref(cfg), None, None, None, None, None, 4, None, None) == 1
assert api.moe_workspace_bytes(api.make_config(wl.small_shape("b", 64, 600, 2, 64)), 8) == 0
print("host paths clean")
'''


def test_library_host_paths_under_asan_and_ubsan(tmp_path):
    if not os.path.exists(NVCC):
        pytest.skip("nvcc not found")
    env = _env()
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-O1", "-g", "-std=c++17", "-Xcompiler",
             "-fPIC,-fsanitize=address,-fsanitize=undefined,-fno-omit-frame-pointer",
             "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    procs, objs = [], []
    for f in sorted(os.listdir(CSRC)):
        if f.endswith(".cu"):
            obj = str(tmp_path / (f[:-3] + ".o"))
            objs.append(obj)
            procs.append(subprocess.Popen([NVCC] + flags + ["-c", os.path.join(CSRC, f), "-o", obj]))
    assert all(p.wait() == 0 for p in procs)
    lib = str(tmp_path / "libmoe_san.so")
    subprocess.run([NVCC, "-shared", "-o", lib] + objs + ["-gencode", "arch=compute_100a,code=sm_100a",
                   "-Xcompiler", "-fsanitize=address,-fsanitize=undefined"], check=True)
    r = subprocess.run([sys.executable, "-c", HOST_SCRIPT % {"root": ROOT, "lib": lib}], env=env,
                       capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "host paths clean" in r.stdout, r.stdout[-1500:] + r.stderr[-3000:]
    assert "runtime error" not in r.stderr and "AddressSanitizer" not in r.stderr, r.stderr[-3000:]


ORACLE_SCRIPT = r'''
import sys
import numpy as np
sys.path.insert(0, %(root)r)
import oracle
oracle._LIB = %(lib)r
oracle._lib = None
oracle.build = lambda force=False: %(lib)r
import torch
from paper_2505_19645_b200 import workloads as wl
shape = wl.small_shape("s", 96, 6, 3, 160, 64, 0, 1, 1)
w = wl.make_weights(shape, 3, "cpu", zipf_s=1.1)
x = wl.make_tokens(shape, 9, 4, "cpu")
cfg = dict(top_k=3, score_fn=0, renormalize=1, routed_scale=1.0, shared_gate=1)
r = oracle.verify_layer(x, w, cfg)
g = oracle.permute(r["topk_idx"], 6)
d = oracle.layer_dense_masked(x, w["w_gate"], w["w_up"], w["w_down"], r["topk_idx"], r["topk_w"],
                              (w["ws_gate"], w["ws_up"], w["ws_down"]), r["shared_scale"])
assert np.allclose(d, r["out"], rtol=1e-9, atol=1e-12) and int(g.counts.sum()) == 27
assert oracle.verify_layer(x, w, cfg, rows=[0, 8])["out"].shape == (2, 96)
assert oracle.token_threshold(4 / 60) == 44 and abs(oracle.expected_active(8, 2, 1) - 2) < 1e-12
print("oracle clean")
'''


def test_oracle_under_asan_and_ubsan(tmp_path):
    env = _env()
    lib = str(tmp_path / "libmoe_oracle_san.so")
    subprocess.run(["gcc", "-O1", "-g", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-fsanitize=address",
                    "-fsanitize=undefined", "-fno-omit-frame-pointer", "-o", lib,
                    os.path.join(ROOT, "oracle", "moe_oracle.c"), "-lm"], check=True)
    r = subprocess.run([sys.executable, "-c", ORACLE_SCRIPT % {"root": ROOT, "lib": lib}], env=env,
                       capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "oracle clean" in r.stdout, r.stdout[-1500:] + r.stderr[-3000:]
    assert "runtime error" not in r.stderr and "AddressSanitizer" not in r.stderr, r.stderr[-3000:]
