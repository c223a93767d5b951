#!/usr/bin/env python
"""Benchmark of the MoE verify layer (one pass of the whole hot path per step).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--config NAME] [--B B] [--gamma G] [--zipf S] [--sweeps all|config|none]

Prints ONE JSON line.  Headline workload (value, roofline, e2e, cpu_baseline): the
DeepSeek-V3-shaped layer -- the largest of the five benchmark shapes that fits one GPU -- at
B=32 sequences x (gamma=3)+1 tokens.  With no --config the same line carries, under "sweeps",
the (B, gamma) grids of all five shapes, the Zipf(1.2) variant of the Qwen2-57B-A14B shape, the
Zipf(1.0) variant of the DeepSeek-V3 shape and the extra token counts 2048 and 4096 on those two
shapes: per point the layer time, tokens/s, roofline fraction, the cost ratio T(B,gamma)/T(B,0)
and the activation statistics of Sec. 3.2 / 3.3 (activated experts against Eq. N(t), tokens per
activated expert against Eq. T_exp, whether T is beyond the threshold of Eq. T_thres).
Inputs are seeded and synthetic.  N > 1 runs N independent replicas (weak scaling).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2505_19645_b200 import replicas, workloads as wl  # noqa: E402

L2_FLUSH_BYTES = 512 << 20
NOMINAL_HBM_GBS = 7700.0      # HBM3e, HGX B200 data sheet
NOMINAL_BF16_TFLOPS = 2250.0  # dense bf16, data sheet
DEFAULT_CONFIG = "deepseek-v3"
DEFAULT_B, DEFAULT_GAMMA = 32, 3
T_THRES_TAU = 0.95            # Eq. T_thres: tokens for N(t) >= tau * E
# Sweeps of the default run: (key, config, Zipf exponent or None).  The two shapes with a skew
# variant also get the token counts 2048 and 4096 as extra rows (B = 512 and 1024 at gamma = 3).
ALL_SWEEPS = [("tiny", "tiny", None), ("qwen1.5-moe-a2.7b", "qwen1.5-moe-a2.7b", None),
              ("qwen2-57b-a14b", "qwen2-57b-a14b", None),
              ("qwen2-57b-a14b-zipf1.2", "qwen2-57b-a14b", 1.2),
              ("mixtral-8x7b", "mixtral-8x7b", None), ("deepseek-v3", "deepseek-v3", None),
              ("deepseek-v3-zipf1.0", "deepseek-v3", 1.0)]
EXTRA_POINTS = {"qwen2-57b-a14b": [(512, 3), (1024, 3)], "deepseek-v3": [(512, 3), (1024, 3)]}
# DRAM bytes of one gate/up launch as counted by ncu, with the hash of the kernel source they
# were taken on (written by --record-traffic from an ncu CSV; see the file for the command)
TRAFFIC_RECORD = os.path.join(ROOT, "profiles", "gate_up_dram_traffic.txt")
KERNEL_SOURCES = ["paper_2505_19645_b200/csrc/ffn_fused.cu", "paper_2505_19645_b200/csrc/common.cuh"]


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


# ---- algorithmic bytes / flops (activated experts only) ---------------------------------

def layer_bytes(shape, T, n_active):
    H, E, I, Is = shape.hidden, shape.n_experts, shape.inter, shape.shared_inter
    return n_active * 6 * H * I + 6 * H * Is + E * H * 4 + 2 * T * H * 2


def layer_flops(shape, T):
    H, E, k, I, Is = shape.hidden, shape.n_experts, shape.top_k, shape.inter, shape.shared_inter
    return T * k * 6 * H * I + T * 6 * H * Is + 2 * T * H * E


def gate_up_bytes(shape, T, n_active):
    """Gate/up kernel: both projections of every activated expert, once, plus the tokens."""
    H, I, Is = shape.hidden, shape.inter, shape.shared_inter
    return n_active * 4 * H * I + 4 * H * Is + T * H * 2


def gate_up_flops(shape, T):
    return T * shape.top_k * 4 * shape.hidden * shape.inter + T * 4 * shape.hidden * shape.shared_inter


# ---- closed forms of Sec. 3.2 / 3.3 (reported beside the measured statistics) ----------

def expected_active(E, k, T):
    """Eq. N(t): expected number of activated experts after T tokens."""
    return E * (1.0 - ((E - k) / E) ** T)


def expected_tokens_per_expert(E, k, T):
    """Eq. T_exp: rho * T / (1 - (1 - rho)^T), rho = k / E."""
    rho = k / E
    return T if rho >= 1.0 else rho * T / (1.0 - (1.0 - rho) ** T)


def token_threshold(E, k, tau=T_THRES_TAU):
    """Eq. T_thres: smallest T with N(T) >= tau * E."""
    rho = k / E
    return 1 if rho >= 1.0 else int(math.ceil(math.log(1.0 - tau) / math.log(1.0 - rho)))


def roof_ms(shape, T, n_active, hbm_gbs, tflops):
    """Slower of the activated-expert bytes over HBM bandwidth and the flops at tensor peak."""
    t_mem = layer_bytes(shape, T, n_active) / (hbm_gbs * 1e9)
    t_flop = layer_flops(shape, T) / (tflops * 1e12)
    return 1e3 * max(t_mem, t_flop), ("hbm" if t_mem >= t_flop else "tensor")


# ---- clocks -----------------------------------------------------------------------------

class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed regions run."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []
        self.skip = 0

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines[self.skip:]:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_min_mhz": min(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons),
                "samples": len(sm)}


# ---- GPU arm ----------------------------------------------------------------------------

class LayerRunner:
    def __init__(self, shape, weights_dev, device, flush):
        from paper_2505_19645_b200 import api
        self.api = api
        self.shape = shape
        self.cfg = api.make_config(shape)
        self.cw = api.make_weights(weights_dev)
        self.keep = weights_dev
        self.device = device
        self.flush = flush

    def prepare(self, T):
        self.ws = self.api.alloc_workspace(self.cfg, T, self.device)
        self.out = torch.empty((T, self.shape.hidden), dtype=torch.bfloat16, device=self.device)

    def step(self, x, B, gamma):
        T = B * (gamma + 1)
        self.api.moe_verify_layer(self.cfg, self.cw, x, B, gamma, self.out[:T], self.ws)

    def flush_l2(self):
        self.flush.zero_()

    def time_steps(self, x, B, gamma, steps, warmup, stage=None):
        """Cold-L2 timing of `steps` layer passes; returns per-step ms (whole layer) and, if
        `stage` is given, per-step ms of that kernel."""
        api = self.api
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
              for _ in range(steps)]
        kev = None
        if stage is not None:
            kev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                   for _ in range(steps)]
            for a, b in kev:   # torch creates the CUDA event lazily on first record
                a.record()
                b.record()
        for _ in range(warmup):
            self.flush_l2()
            self.step(x, B, gamma)
        torch.cuda.synchronize()
        for i in range(steps):
            self.flush_l2()
            if kev is not None:
                api.moe_profile_stage(stage, kev[i][0], kev[i][1])
            ev[i][0].record()
            self.step(x, B, gamma)
            ev[i][1].record()
        if kev is not None:
            api.moe_profile_stage(None)
        torch.cuda.synchronize()
        api.moe_check(self.ws)   # the status word is sticky: covers every step since the last check
        layer_ms = [a.elapsed_time(b) for a, b in ev]
        kern_ms = [a.elapsed_time(b) for a, b in kev] if kev is not None else None
        return layer_ms, kern_ms

    def n_active(self, x, B, gamma):
        dbg = {"n_active": torch.zeros(1, dtype=torch.int32, device=self.device)}
        self.api.moe_verify_layer(self.cfg, self.cw, x, B, gamma, self.out[:B * (gamma + 1)],
                                  self.ws, dbg)
        torch.cuda.synchronize()
        return int(dbg["n_active"].item())

    def time_e2e(self, x_host_pinned, B, gamma, steps, warmup):
        """Host buffers: H2D of the tokens, the layer, D2H of the result inside the timed region."""
        T = x_host_pinned.shape[0]
        x_dev = torch.empty((T, self.shape.hidden), dtype=torch.bfloat16, device=self.device)
        out_host = torch.empty((T, self.shape.hidden), dtype=torch.bfloat16).pin_memory()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
              for _ in range(steps)]
        for i in range(warmup + steps):
            self.flush_l2()
            j = i - warmup
            if j >= 0:
                ev[j][0].record()
            x_dev.copy_(x_host_pinned, non_blocking=True)
            self.step(x_dev, B, gamma)
            out_host.copy_(self.out[:T], non_blocking=True)
            if j >= 0:
                ev[j][1].record()
        torch.cuda.synchronize()
        ms = [a.elapsed_time(b) for a, b in ev]
        nbytes = T * self.shape.hidden * 2
        return ms, nbytes, nbytes

    def host_us_per_call(self, x, B, gamma, calls=100, raw=False):
        """Host time of one moe_verify_layer call: `calls` calls enqueued back to back on an idle
        stream without synchronising (few enough to fit the launch queue, so the host never
        waits for the GPU), wall clock / calls; the best of five rounds.  raw: the C entry
        point called through ctypes with arguments marshalled once (what a C caller pays);
        otherwise through the Python binding, which checks and converts its tensors per call."""
        import ctypes
        T = B * (gamma + 1)
        if raw:
            lib = self.api.load_library()
            out = self.out[:T]
            cargs = (ctypes.byref(self.cfg), ctypes.byref(self.cw), ctypes.c_void_p(x.data_ptr()), B,
                     gamma, ctypes.c_void_p(out.data_ptr()), None, ctypes.c_void_p(self.ws.data_ptr()),
                     self.ws.nbytes, ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
            call = lambda: lib.moe_verify_layer(*cargs)  # noqa: E731
        else:
            call = lambda: self.step(x, B, gamma)  # noqa: E731
        best = None
        for _ in range(5):
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for _ in range(calls):
                call()
            dt = time.perf_counter() - t0
            torch.cuda.synchronize()
            best = dt if best is None else min(best, dt)
        self.api.moe_check(self.ws)
        return 1e6 * best / calls


def sweep_points(config):
    Bs, gs = wl.GRIDS[config]
    pts = [(B, g) for B in Bs for g in gs]
    have = {B * (g + 1) for B, g in pts}
    return pts, [(B, g) for B, g in EXTRA_POINTS.get(config, []) if B * (g + 1) not in have]


def run_sweep(config, shape, runner, peaks, per_pass, device, grid=None):
    """Every (B, gamma) point of the config's grid (plus the extra token counts).  A point is
    visited in three passes over the grid -- at the large shapes the part sits at its power cap,
    where the SM clock steps on the time scale of one visit -- and reported by the MEDIAN of all
    its samples; the lowest of the three pass medians and the fastest sample are kept beside it
    under their own keys."""
    if grid is None:
        grid, extra = sweep_points(config)
    else:
        extra = []
    samples = {}
    for _ in range(3):
        for (Bi, gi) in grid + extra:
            Ti = Bi * (gi + 1)
            xi = wl.make_tokens(shape, Ti, wl.point_seed(config, Bi, gi), device)
            ms, _ = runner.time_steps(xi, Bi, gi, per_pass, 3)
            samples.setdefault((Bi, gi), []).append(ms)
    E, k = shape.n_experts, shape.top_k
    t_thres = token_threshold(E, k)
    base = {}
    rows = []
    for (Bi, gi) in grid + extra:
        Ti = Bi * (gi + 1)
        xi = wl.make_tokens(shape, Ti, wl.point_seed(config, Bi, gi), device)
        na = runner.n_active(xi, Bi, gi)
        launches = runner.api.moe_last_launch_count()
        passes = samples[(Bi, gi)]
        allms = [v for r in passes for v in r]
        med = statistics.median(allms)
        best_pass = min(statistics.median(r) for r in passes)
        if gi == 0:
            base[Bi] = med
        roof, bound = roof_ms(shape, Ti, na, peaks["hbm_gbs"], peaks["bf16_tflops"])
        roof_sus, _ = roof_ms(shape, Ti, na, peaks["hbm_gbs"], peaks["bf16_tflops_sustained"])
        roof_nom, _ = roof_ms(shape, Ti, na, NOMINAL_HBM_GBS, NOMINAL_BF16_TFLOPS)
        ratio = med / base[Bi] if (Bi in base and (Bi, gi) in grid) else None
        rows.append({
            "B": Bi, "gamma": gi, "T": Ti, "extra": (Bi, gi) in extra,
            "us": round(med * 1e3, 2), "us_best_pass": round(best_pass * 1e3, 2),
            "us_min": round(min(allms) * 1e3, 2), "samples": len(allms),
            "tokens_per_s": round(Ti / (med * 1e-3), 1), "launches": launches,
            # Sec. 3.2 / 3.3 statistics: measured on this input, beside the closed forms
            "n_active": na, "n_active_expected": round(expected_active(E, k, Ti), 2),
            "t_exp": round(Ti * k / na, 3),
            "t_exp_expected": round(expected_tokens_per_expert(E, k, Ti), 3),
            "beyond_t_thres": Ti > t_thres,
            "bound": bound, "roof_us": round(roof * 1e3, 2), "roof_frac": round(roof / med, 4),
            "roof_frac_best_pass": round(roof / best_pass, 4),
            "roof_frac_of_nominal": round(roof_nom / med, 4),
            "roof_frac_sustained_tensor_peak": round(roof_sus / med, 4),
            "ratio_vs_gamma0": None if ratio is None else round(ratio, 4),
            "target_efficiency": None if ratio is None else round(1.0 / ratio, 4)})
    return {"config": config, "shape": shape.as_dict(), "t_thres": t_thres, "rows": rows}


def cpu_oracle_rate(shape, w_host, x_host, n_rows, repeats=1):
    """Times the CPU oracle (as it stands) on a seeded sample of token rows; tokens/s."""
    import numpy as np
    import oracle
    T = x_host.shape[0]
    rng = np.random.default_rng(0)
    rows = sorted(rng.choice(T, size=min(n_rows, T), replace=False).tolist())
    cfg = dict(top_k=shape.top_k, score_fn=shape.score_fn, renormalize=shape.renormalize,
               routed_scale=shape.routed_scale, shared_gate=shape.shared_gate)
    times = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        oracle.verify_layer(x_host, w_host, cfg, rows=rows)
        times.append(time.perf_counter() - t0)
    # the router runs on all T rows (cheap); the FFNs on the sample
    return len(rows) / min(times), len(rows), oracle.num_threads(), times


def host_weights(shape, seed, zipf):
    """Weights on the host for the oracle: drawn on the GPU where there is one (the same
    generator the GPU arm uses; far faster than the host generator at 22 GB) and copied."""
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    w = wl.make_weights(shape, seed, dev, zipf_s=zipf)
    return {k: (None if v is None else v.cpu()) for k, v in w.items()}


def run_reference(args):
    """--impl reference: the CPU oracle on the host cores, same workload/metric/unit."""
    rank, _, world = replicas.env_world()
    if rank != 0:
        return 0
    shape = variant_shape(args)
    T = args.B * (args.gamma + 1)
    w = host_weights(shape, wl.config_seed(args.config), args.zipf)
    x = wl.make_tokens(shape, T, wl.point_seed(args.config, args.B, args.gamma), "cpu")
    import oracle
    n_rows = min(T, max(1, oracle.num_threads()))
    for _ in range(min(args.warmup, 3)):
        cpu_oracle_rate(shape, w, x, n_rows)
    t_total = 0.0
    cores = oracle.num_threads()
    for _ in range(args.steps):
        r, n, cores, times = cpu_oracle_rate(shape, w, x, n_rows)
        t_total += times[0]
    value = n_rows * args.steps / t_total
    sample = "%d seeded token rows of the T=%d batch per step" % (n_rows, T)
    line = {
        "impl": "reference", "metric": "moe_verify_layer_tokens_per_s", "value": value,
        "unit": "tokens/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * t_total / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic (seeded)",
        "config": workload_config(args, shape, T),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0,
                "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def workload_name(args):
    return "%s-shaped MoE FFN layer, B=%d, gamma=%d (T=%d tokens)" % (
        variant_shape(args).name, args.B, args.gamma, args.B * (args.gamma + 1))


def workload_config(args, shape, T):
    """The `config` object of the JSON line: the same keys in both arms."""
    return {"workload": workload_name(args), "config": args.config, "B": args.B,
            "gamma": args.gamma, "tokens": T, "zipf": args.zipf, "shape": shape.as_dict(),
            "l2": "512 MiB buffer written between timed iterations",
            "parallelism": "replicas only"}


def variant_shape(args):
    """The config's layer shape, or its --top-k / --dense-contrast variant."""
    shape = wl.CONFIGS[args.config]
    if args.dense_contrast:
        return wl.dense_contrast(shape)
    if args.top_k is not None:
        return wl.with_top_k(shape, args.top_k)
    return shape


# ---- DRAM traffic of the gate/up kernel (ncu) ----------------------------------------------

def kernel_source_hash():
    h = hashlib.sha256()
    for rel in KERNEL_SOURCES:
        h.update(open(os.path.join(ROOT, rel), "rb").read())
    return h.hexdigest()[:16]


def recorded_traffic(workload):
    """ncu's DRAM bytes of one gate/up launch on `workload`, or None when no record exists for
    it or the kernel source has changed since the counters were taken."""
    if not os.path.exists(TRAFFIC_RECORD):
        return None
    rec = {}
    for line in open(TRAFFIC_RECORD):
        if "=" in line and not line.startswith("#"):
            key, val = line.split("=", 1)
            rec[key.strip()] = val.strip()
    if rec.get("kernel_source_sha256_16") != kernel_source_hash() or rec.get("workload") != workload:
        return None
    return int(rec["dram_bytes_read"]) + int(rec["dram_bytes_write"])


def record_traffic(csv_path, workload, command):
    """Parses an `ncu --csv --metrics dram__bytes_read.sum,dram__bytes_write.sum` log of gate/up
    launches and writes the record (mean over the captured launches)."""
    import csv
    rd, wr = [], []
    rows = [r for r in csv.reader(l for l in open(csv_path) if l.startswith('"'))]
    head = rows[0]
    i_name, i_metric, i_unit, i_val = (head.index("Kernel Name"), head.index("Metric Name"),
                                       head.index("Metric Unit"), head.index("Metric Value"))
    scale = {"byte": 1, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    for r in rows[1:]:
        if "ffn_fused_kernel<1>" not in r[i_name] and "ffn_fused_kernel<true>" not in r[i_name] \
                and "(bool)1" not in r[i_name]:
            continue
        v = float(r[i_val].replace(",", "")) * scale[r[i_unit]]
        (rd if r[i_metric] == "dram__bytes_read.sum" else wr).append(v)
    if not rd or not wr:
        raise SystemExit("no gate/up launches with dram__bytes_* in " + csv_path)
    with open(TRAFFIC_RECORD, "w") as f:
        f.write("# DRAM traffic of one ffn_fused_kernel<gate/up> launch (ncu, mean of %d launches).\n"
                "# Command: %s\n# then: python bench.py --record-traffic <that csv> [same workload flags]\n"
                % (len(rd), command))
        f.write("workload = %s\n" % workload)
        f.write("kernel_source_sha256_16 = %s\n" % kernel_source_hash())
        f.write("dram_bytes_read = %d\n" % round(sum(rd) / len(rd)))
        f.write("dram_bytes_write = %d\n" % round(sum(wr) / len(wr)))
    print("wrote", TRAFFIC_RECORD)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default=None, choices=wl.CONFIG_ORDER)
    ap.add_argument("--B", type=int, default=DEFAULT_B)
    ap.add_argument("--gamma", type=int, default=DEFAULT_GAMMA)
    ap.add_argument("--zipf", type=float, default=None)
    ap.add_argument("--top-k", type=int, default=None,
                    help="experts per token instead of the config's own (sparsity sweep)")
    ap.add_argument("--dense-contrast", action="store_true",
                    help="the rho = 1 layer with the same active parameters per token")
    ap.add_argument("--grid", default="config", choices=["config", "sparsity"],
                    help="with --config: sweep its (B, gamma) grid or the 19 batch sizes x gamma 0/2/4")
    ap.add_argument("--sweeps", default=None, choices=["all", "config", "none"],
                    help="all: every shape and variant (default without --config); config: the "
                         "headline config's own grid (default with --config); none")
    ap.add_argument("--no-sweep", action="store_true", help="same as --sweeps none")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--headline-only", action="store_true",
                    help="only the headline loop and the kernel's event pair (for profiler runs): "
                         "no end-to-end, small-batch, sweep or CPU legs")
    ap.add_argument("--sweep-steps", type=int, default=30, help="samples per sweep point")
    ap.add_argument("--record-traffic", default=None, metavar="NCU_CSV",
                    help="write the DRAM-traffic record of the gate/up kernel from an ncu CSV log")
    ap.add_argument("--ncu-command", default="(not given)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.sweeps is None:
        args.sweeps = "all" if args.config is None else "config"
    if args.headline_only:
        args.no_sweep = args.no_cpu_baseline = True
    if args.no_sweep:
        args.sweeps = "none"
    if args.config is None:
        args.config = DEFAULT_CONFIG

    if args.record_traffic:
        record_traffic(args.record_traffic, workload_name(args), args.ncu_command)
        return 0
    if args.impl == "reference":
        return run_reference(args)

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the layer has no CPU fallback")
    rank, world = replicas.init("nccl")
    _, local_rank, _ = replicas.env_world()
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    peaks = load_peaks()
    if world > 1 and args.sweeps == "all":
        args.sweeps = "none"   # the sweeps are single-GPU measurements: N GPUs are not held for them

    shape = variant_shape(args)
    B, gamma = args.B, args.gamma
    T = B * (gamma + 1)
    w_dev = wl.make_weights(shape, wl.config_seed(args.config), device, zipf_s=args.zipf)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=device)
    runner = LayerRunner(shape, w_dev, device, flush)
    runner.prepare(T)
    seed = replicas.replica_seed(wl.point_seed(args.config, B, gamma), rank)
    x = wl.make_tokens(shape, T, seed, device)
    n_act = runner.n_active(x, B, gamma)
    launches_per_step = runner.api.moe_last_launch_count()

    # ---- headline: whole layer, inputs resident in HBM --------------------------------
    # the sampler keeps running through every measured loop (layer, kernel, end to end, sweeps)
    sampler = ClockSampler(local_rank)
    sampler.start()
    runner.time_steps(x, B, gamma, 3, args.warmup)
    replicas.barrier()
    torch.cuda.synchronize()
    sampler.skip = len(sampler.lines)
    layer_ms, _ = runner.time_steps(x, B, gamma, args.steps, args.warmup)
    torch.cuda.synchronize()
    replicas.barrier()
    ms_step_local = sum(layer_ms) / len(layer_ms)
    value, ms_step = replicas.job_throughput(T, ms_step_local, device)

    # ---- dominant kernel (gate/up) with its own event pair ----------------------------
    _, kern_ms = runner.time_steps(x, B, gamma, args.steps, 3, stage="gate_up")
    k_ms = sum(kern_ms) / len(kern_ms)
    # one to four tokens may run as a single launch: the stage events then bracket the whole layer
    whole_layer = launches_per_step == 1
    gu_bytes = layer_bytes(shape, T, n_act) if whole_layer else gate_up_bytes(shape, T, n_act)
    gu_flops = layer_flops(shape, T) if whole_layer else gate_up_flops(shape, T)
    t_mem = gu_bytes / (peaks["hbm_gbs"] * 1e9)
    t_flop = gu_flops / (peaks["bf16_tflops"] * 1e12)
    if t_mem >= t_flop:
        achieved = gu_bytes / (k_ms * 1e-3) / 1e9
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": achieved / peaks["hbm_gbs"]}
    else:
        achieved = gu_flops / (k_ms * 1e-3) / 1e12
        roofline = {"bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"],
                    "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"]}
    roofline.update({"traffic": recorded_traffic(workload_name(args)),
                     "kernel": ("layer_small_kernel (whole layer in one launch)" if whole_layer
                                else "ffn_fused_kernel<gate/up + SwiGLU>"),
                     "kernel_ms": k_ms, "algorithmic_bytes": gu_bytes,
                     "peak_source": peaks["source"]})

    roof, bound = roof_ms(shape, T, n_act, peaks["hbm_gbs"], peaks["bf16_tflops"])
    roof_sus, _ = roof_ms(shape, T, n_act, peaks["hbm_gbs"], peaks["bf16_tflops_sustained"])
    roof_nom, _ = roof_ms(shape, T, n_act, NOMINAL_HBM_GBS, NOMINAL_BF16_TFLOPS)
    E, k = shape.n_experts, shape.top_k
    layer_roof = {"bound": bound, "roof_ms": roof, "frac": roof / ms_step_local,
                  "frac_of_nominal": roof_nom / ms_step_local,
                  "frac_sustained_tensor_peak": roof_sus / ms_step_local,
                  "peaks": {"hbm_gbs": peaks["hbm_gbs"], "bf16_tflops": peaks["bf16_tflops"],
                            "bf16_tflops_sustained": peaks["bf16_tflops_sustained"],
                            "source": peaks["source"], "nominal_hbm_gbs": NOMINAL_HBM_GBS,
                            "nominal_bf16_tflops": NOMINAL_BF16_TFLOPS},
                  "n_active": n_act, "n_active_expected": expected_active(E, k, T),
                  "t_exp": T * k / n_act, "t_exp_expected": expected_tokens_per_expert(E, k, T),
                  "t_thres": token_threshold(E, k), "beyond_t_thres": T > token_threshold(E, k),
                  "bytes": layer_bytes(shape, T, n_act),
                  "flops": layer_flops(shape, T), "median_ms": statistics.median(layer_ms),
                  "min_ms": min(layer_ms)}

    # ---- end to end with host buffers -------------------------------------------------
    e2e_value, h2d, d2h = None, 0, 0
    if not args.headline_only:
        x_host = x.cpu().pin_memory()
        e2e_ms, h2d, d2h = runner.time_e2e(x_host, B, gamma, args.steps, 3)
        e2e_value, _ = replicas.job_throughput(T, sum(e2e_ms) / len(e2e_ms), device)

    # ---- the latency end: one token; host time of a call ---------------------------------
    small = {}
    if rank == 0 and not args.headline_only:
        x1 = wl.make_tokens(shape, 1, wl.point_seed(args.config, 1, 0), device)
        ms1, _ = runner.time_steps(x1, 1, 0, max(20, min(args.steps, 100)), 3)
        e1, b1, _ = runner.time_e2e(x1.cpu().pin_memory(), 1, 0, max(20, min(args.steps, 100)), 3)
        small = {"T1_layer_us": round(1e3 * statistics.median(ms1), 2),
                 "T1_e2e_us": round(1e3 * statistics.median(e1), 2),
                 "T1_e2e_h2d_bytes": b1,
                 "host_us_per_call": {"T1": round(runner.host_us_per_call(x1, 1, 0), 2),
                                      "T%d" % T: round(runner.host_us_per_call(x, B, gamma), 2)},
                 "host_us_per_call_c_abi": {
                     "T1": round(runner.host_us_per_call(x1, 1, 0, raw=True), 2),
                     "T%d" % T: round(runner.host_us_per_call(x, B, gamma, raw=True), 2)},
                 "host_us_per_call_how": "perf_counter around 100 unsynchronised moe_verify_layer "
                                         "calls / 100, best of 5 rounds: through the Python binding, "
                                         "and through the C entry point with arguments marshalled once"}

    # ---- sweeps ---------------------------------------------------------------------------
    sweeps = {}
    if rank == 0 and args.sweeps != "none":
        per_pass = max(5, args.sweep_steps // 3)
        if args.sweeps == "config" and args.grid == "sparsity":
            todo = []   # the sparsity grid of one variant: rows in the old flat form below
        elif args.sweeps == "config":
            todo = [(args.config if args.zipf is None else "%s-zipf%g" % (args.config, args.zipf),
                     args.config, args.zipf)]
        else:
            todo = ALL_SWEEPS
        held = {"config": None, "w": None}   # one config's weights at a time beside the headline's

        def base_weights(cname):
            if cname == args.config and shape is wl.CONFIGS[cname]:
                return w_dev   # the headline's (the router bias is set per variant below)
            if held["config"] != cname:
                held["w"] = None
                torch.cuda.empty_cache()
                held.update(config=cname, w=wl.make_weights(wl.CONFIGS[cname], wl.config_seed(cname), device))
            return held["w"]

        for key, cname, zipf in todo:
            if args.sweeps == "config":
                cshape, w_c = shape, dict(w_dev)   # the headline's own shape (or variant) and bias
            else:
                cshape = wl.CONFIGS[cname]
                w_c = dict(base_weights(cname))
                w_c["router_bias"] = None if zipf is None else wl.zipf_router_bias(
                    cshape.n_experts, cshape.hidden, zipf, wl.config_seed(cname), device)
            r = LayerRunner(cshape, w_c, device, flush)
            grid, extra = sweep_points(cname)
            r.prepare(max(Bi * (gi + 1) for Bi, gi in grid + extra))
            sweeps[key] = run_sweep(cname, cshape, r, peaks, per_pass, device)
            sweeps[key]["zipf"] = zipf
            del r, w_c
        held["w"] = None
        torch.cuda.empty_cache()
        if args.sweeps == "config" and args.grid == "sparsity":
            grid = [(Bi, gi) for Bi in wl.SPARSITY_BATCHES for gi in wl.SPARSITY_GAMMAS]
            runner.prepare(max(Bi * (gi + 1) for Bi, gi in grid))
            key = "sparsity:" + shape.name
            sweeps[key] = run_sweep(args.config, shape, runner, peaks, per_pass, device, grid=grid)
            sweeps[key]["zipf"] = args.zipf
    clocks = sampler.stop()

    # ---- CPU oracle beside it (rank 0, N = 1) -----------------------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        w_host = {kk: (None if v is None else v.cpu()) for kk, v in w_dev.items()}
        import oracle
        n_rows = min(T, 4 * oracle.num_threads())
        x_cpu = x.cpu()
        rate, n, cores, times = cpu_oracle_rate(shape, w_host, x_cpu, n_rows)
        # repeat the sample until about 10 s of CPU work have been timed
        reps = max(1, min(200, int(10.0 / max(times[0], 1e-3))))
        t0 = time.perf_counter()
        for _ in range(reps):
            cpu_oracle_rate(shape, w_host, x_cpu, n_rows)
        dt = time.perf_counter() - t0
        cpu = {"value": n * reps / dt, "unit": "tokens/s", "cores": cores, "kind": "oracle",
               "sample": "%d seeded token rows of the T=%d batch, %d passes, %.1f s"
                         % (n, T, reps, dt)}

    if rank == 0:
        line = {
            "metric": "moe_verify_layer_tokens_per_s", "value": value, "unit": "tokens/s",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic (seeded)",
            "config": workload_config(args, shape, T),
            "roofline": roofline, "layer_roofline": layer_roof, "cpu_baseline": cpu,
            "e2e": {"value": e2e_value, "unit": "tokens/s", "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h},
            "gpu_launches": launches_per_step * args.steps, "clocks": clocks,
            "layer_us": ms_step * 1e3, "small_batch": small, "sweeps": sweeps,
        }
        print(json.dumps(line))
    replicas.shutdown()
    return 0


if __name__ == "__main__":
    sys.exit(main())
