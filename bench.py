#!/usr/bin/env python
"""Benchmark of the B200 SpMM hot path (BCSR and WCSR kernels behind the C ABI).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
                    [--only NAME [--dense-width N]] [--skip-others] [--others A,B | all] [--no-cpu]
                    [--no-e2e] [--ubench]

A step is one ``spmm_run`` (the SpMM kernel, plus the merge kernel for WCSR) on
inputs already resident in HBM.  The headline workload is the largest single-GPU
configuration, configs[2] gate (BCSR, 18944 x 3584 bf16, 64 x 64 blocks, 90 % of
the blocks zero, N = 65,536, fp32 C); the other configurations are measured the
same way.  Throughput is GFLOP/s over stored nonzeros, 2 * nnz_stored * N / t.
L2 is flushed (a 512 MB write) before every timed launch and each launch is
timed with its own pair of CUDA events on the launching stream.  With N > 1 GPUs
every rank runs an independent replica of the same workload (the path has no
exchange step); value = total flops / max time.

Output: every other workload is printed as ONE short JSON line of its own
({"other": ...}) as soon as it is measured; the LAST line of stdout is the
compact result line (metric, value, roofline, cpu_baseline, e2e, clocks and a
five-field summary of the others).

``--impl reference`` times the fp64 CPU oracle (oracle/) on the host cores on a
bounded sample of the same workload and prints the same line with
"impl": "reference".
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2604_17834_b200 import workloads as wl  # noqa: E402

METRIC = "SpMM GFLOP/s over stored nonzeros (2*nnz_stored*N/time)"
UNIT = "GFLOP/s"
MAX_LINE_BYTES = 1450      # the result line (last line of stdout)


# --------------------------------------------------------------------------- workloads


def workload_table():
    """name -> (description, builder).  builder() -> dict(kind, a, dtype, size, N, Bdist, opts)."""
    def cfg1():
        return dict(kind="bcsr", a=wl.bcsr_tiny(), dtype="bf16", size=64, N=256, Bdist=("uniform", -1.0, 1.0))

    def cfg2():
        return dict(kind="wcsr", a=wl.wcsr_irregular(), dtype="tf32", size=16, N=128, Bdist=("normal", 0.0, 1.0))

    def cfg2_alpha18():
        # configs[1] quotes "Zipf(2) ... mean 12"; Zipf(2) clipped to 5000 has mean 6, a mean of
        # 12 needs an exponent near 1.8: the literal exponent is the headline, this the second reading
        return dict(kind="wcsr", a=wl.wcsr_irregular(seed=1012, alpha=1.8), dtype="tf32", size=16, N=128,
                    Bdist=("normal", 0.0, 1.0))

    def cfg3_gate():
        return dict(kind="bcsr", a=wl.bcsr_llm(), dtype="bf16", size=64, N=65536, Bdist=("normal", 0.0, 1.0))

    def cfg3_down():
        return dict(kind="bcsr", a=wl.bcsr_llm(seed=1013, m=3584, k=18944), dtype="bf16", size=64, N=65536,
                    Bdist=("normal", 0.0, 1.0))

    def variant(base, c16=False, cm=False, dyn=False):
        """Same matrix and dense operand; C in the input's 16-bit type and / or column-major
        operands (X = B^T in, Y = C^T out: the linear-layer shape of Sec. 4.4), or tiles
        scheduled at run time through Cluster Launch Control instead of the static plan."""
        def f():
            w = base()
            w["opts"] = dict(c_type=1 if c16 else 0, layout=1 if cm else 0, schedule=1 if dyn else 0)
            return w
        return f

    def cfg4(b, d, skewed=True):
        def f():
            return dict(kind="bcsr", a=wl.bcsr_sweep(1004 + b + int(d * 1000), b=b, density=d, skewed=skewed),
                        dtype="fp16", size=b, N=4096, Bdist=("uniform", -1.0, 1.0))
        return f

    def cfg5(N):
        def f():
            if "rmat" not in _CACHE:                 # ~30 s to draw: shared by the three widths
                _CACHE["rmat"] = wl.rmat()
            return dict(kind="wcsr", a=_CACHE["rmat"], dtype="fp16", size=16, N=N, Bdist=("normal", 0.0, 1.0))
        return f

    t = {
        "cfg1_bcsr_tiny": ("configs[0] BCSR 512x512 bf16 b=64 keep 0.5, N=256", cfg1),
        "cfg2_wcsr_irregular": ("configs[1] WCSR 100000x100000 tf32 zipf(2) rows, 50% band, wh=16, N=128", cfg2),
        "cfg2_wcsr_irregular_alpha1.8": ("configs[1] with row lengths zipf(1.8) (realised mean near the quoted 12)", cfg2_alpha18),
        "cfg3_bcsr_llm_gate": ("configs[2] BCSR 18944x3584 bf16 b=64 90% blocks zero, N=65536", cfg3_gate),
        "cfg3_bcsr_llm_down": ("configs[2] BCSR 3584x18944 bf16 b=64 90% blocks zero, N=65536", cfg3_down),
        "cfg3_bcsr_llm_gate_c16": ("configs[2] gate, C written as bf16", variant(cfg3_gate, c16=True)),
        "cfg3_bcsr_llm_gate_cm": ("configs[2] gate, column-major operands (X [N][k] in, Y [N][m] out), fp32 Y",
                                  variant(cfg3_gate, cm=True)),
        "cfg3_bcsr_llm_gate_cm_c16": ("configs[2] gate as a linear layer: X [N][k] bf16 in, Y [N][m] bf16 out",
                                      variant(cfg3_gate, c16=True, cm=True)),
        "cfg3_bcsr_llm_down_cm_c16": ("configs[2] down as a linear layer: X [N][k] bf16 in, Y [N][m] bf16 out",
                                      variant(cfg3_down, c16=True, cm=True)),
        "cfg5_wcsr_rmat_n128_c16": ("configs[4] N=128, C written as fp16", variant(cfg5(128), c16=True)),
        "cfg5_wcsr_rmat_n32": ("configs[4] WCSR R-MAT 2^21 deg 16 fp16 wh=16, N=32", cfg5(32)),
        "cfg5_wcsr_rmat_n128": ("configs[4] WCSR R-MAT 2^21 deg 16 fp16 wh=16, N=128", cfg5(128)),
        "cfg5_wcsr_rmat_n256": ("configs[4] WCSR R-MAT 2^21 deg 16 fp16 wh=16, N=256", cfg5(256)),
    }
    def tall(base):
        """Same matrix with the paper's own 64-row WCSR windows (Sec. 4.1) instead of 16."""
        def f():
            w = base()
            w["size"] = 64
            return w
        return f
    def plain(base):
        """Same workload with the BCSR row groups (stacked 128-row blocks) switched off."""
        def f():
            w = base()
            w["opts"] = dict(w.get("opts", {}), stack_min_fill=-1)
            return w
        return f
    def fp8_linear(m, k, seed):
        def f():
            return dict(kind="bcsr", a=wl.bcsr_llm(seed=seed, m=m, k=k, dtype="fp8", std=0.5), dtype="fp8", size=64, N=65536,
                        Bdist=("normal", 0.0, 1.0), opts=dict(layout=1))
        return f
    t["cfg3_bcsr_llm_gate_cm_fp8"] = ("configs[2] gate shape with E4M3 weights and activations, X [N][k] in, fp32 Y [N][m] out",
                                      fp8_linear(18944, 3584, 1003))
    def fp8_rowmajor(m, k, seed):
        def f():
            return dict(kind="bcsr", a=wl.bcsr_llm(seed=seed, m=m, k=k, dtype="fp8", std=0.5), dtype="fp8", size=64, N=65536,
                        Bdist=("normal", 0.0, 1.0))
        return f
    t["cfg3_bcsr_llm_gate_fp8"] = ("configs[2] gate shape with E4M3 weights and activations, row-major operands, fp32 C",
                                   fp8_rowmajor(18944, 3584, 1003))
    t["cfg3_bcsr_llm_down_cm_fp8"] = ("configs[2] down shape with E4M3 weights and activations, X [N][k] in, fp32 Y [N][m] out",
                                      fp8_linear(3584, 18944, 1013))
    t["cfg5_wcsr_rmat_s19_n128"] = ("configs[4] recipe at 2^19 rows (a profiling-sized case: B 134 MB), N=128",
                                    lambda: dict(kind="wcsr", a=wl.rmat(scale=19), dtype="fp16", size=16, N=128, Bdist=("normal", 0.0, 1.0)))
    def lsu(base):
        """Same workload with the paper's own gather (Sec. 3.2: 128-bit loads through the load/store
        units) instead of the TMA row gather."""
        def f():
            w = base()
            w["opts"] = dict(w.get("opts", {}), gather=1)
            return w
        return f
    def ksplit(base):
        """Same workload with outlier block-rows cut into parts (opts.k_split)."""
        def f():
            w = base()
            w["opts"] = dict(w.get("opts", {}), k_split=1)
            return w
        return f
    for d in (0.1, 0.01):
        t["cfg4_bcsr_sweep_b64_d%g_ksplit" % d] = ("configs[3] b=64 skewed rows, keep %g, long block-rows cut into parts" % d,
                                                    ksplit(cfg4(64, d)))
    def tf32_sweep(b, d):
        """configs[3] shape in the value type of the paper's own BCSR evaluation (Sec. 4.1: TF32)."""
        def f():
            return dict(kind="bcsr", a=wl.bcsr_sweep(1004 + b + int(d * 1000), b=b, density=d, dtype="tf32"), dtype="tf32",
                        size=b, N=4096, Bdist=("uniform", -1.0, 1.0))
        return f
    for b in (16, 32, 64, 128):
        t["cfg4_bcsr_sweep_b%d_d0.1_tf32" % b] = ("configs[3] shape, b=%d skewed rows, keep 0.1, fp32 storage / TF32 arithmetic" % b,
                                                   tf32_sweep(b, 0.1))
    t["cfg2_wcsr_irregular_lsu_gather"] = ("configs[1], B rows gathered with 16-byte cp.async instead of TMA", lsu(cfg2))
    t["cfg5_wcsr_rmat_n128_lsu_gather"] = ("configs[4] N=128, B rows gathered with 16-byte cp.async instead of TMA", lsu(cfg5(128)))
    t["cfg2_wcsr_irregular_wh64"] = ("configs[1] with 64-row windows", tall(cfg2))
    def cfg5_fp8():
        if "rmat_fp8" not in _CACHE:
            _CACHE["rmat_fp8"] = wl.rmat(dtype="fp8")
        return dict(kind="wcsr", a=_CACHE["rmat_fp8"], dtype="fp8", size=16, N=128, Bdist=("normal", 0.0, 1.0))
    t["cfg5_wcsr_rmat_n128_fp8"] = ("configs[4] N=128 with E4M3 values (windows padded to 32 columns)", cfg5_fp8)
    t["cfg5_wcsr_rmat_n128_wh64"] = ("configs[4] N=128 with 64-row windows", tall(cfg5(128)))
    t["cfg3_bcsr_llm_gate_dyn"] = ("configs[2] gate, dynamic tile scheduling", variant(cfg3_gate, dyn=True))
    t["cfg3_bcsr_llm_down_dyn"] = ("configs[2] down, dynamic tile scheduling", variant(cfg3_down, dyn=True))
    for b in (16, 32, 64, 128):
        for d in (0.5, 0.2, 0.1, 0.05, 0.01):
            t["cfg4_bcsr_sweep_b%d_d%g" % (b, d)] = (
                "configs[3] BCSR 8192x8192 fp16 b=%d skewed rows, keep %g in the rest, N=4096" % (b, d), cfg4(b, d))
            t["cfg4_bcsr_sweep_b%d_d%g_dyn" % (b, d)] = (
                "configs[3] b=%d skewed rows, keep %g, dynamic tile scheduling" % (b, d), variant(cfg4(b, d), dyn=True))
        t["cfg4_bcsr_sweep_b%d_d0.1_plain" % b] = ("configs[3] b=%d skewed rows, keep 0.1, row groups switched off" % b,
                                                    plain(cfg4(b, 0.1)))
        if b < 128:
            def fam(b=b):
                return dict(kind="bcsr", a=wl.bcsr_families(1300 + b, b=b), dtype="fp16", size=b, N=4096,
                            Bdist=("uniform", -1.0, 1.0))
            t["cfg4_bcsr_families_b%d" % b] = (
                "configs[3] shape, b=%d, block-rows in 32 scattered families (keep 0.1, 10 %% dropped per row)" % b, fam)
            t["cfg4_bcsr_families_b%d_plain" % b] = ("the same, row groups switched off", plain(fam))
        for d in (0.05, 0.01):
            t["cfg4_bcsr_flat_b%d_d%g" % (b, d)] = (
                "configs[3] BCSR 8192x8192 fp16 b=%d flat Bernoulli(%g), N=4096" % (b, d), cfg4(b, d, False))
    return t


_CACHE = {}
# the largest single-GPU configuration: the line's value, roofline, e2e and cpu_baseline are its
HEADLINE = "cfg3_bcsr_llm_gate"
# measured by default beside the headline: one or more cases of every other configuration
DEFAULT_OTHERS = ["cfg1_bcsr_tiny", "cfg2_wcsr_irregular", "cfg3_bcsr_llm_down",
                  "cfg4_bcsr_sweep_b16_d0.1", "cfg4_bcsr_sweep_b32_d0.1", "cfg4_bcsr_sweep_b64_d0.1",
                  "cfg4_bcsr_sweep_b128_d0.1", "cfg5_wcsr_rmat_n32", "cfg5_wcsr_rmat_n128", "cfg5_wcsr_rmat_n256"]
# --others all: the variants (output type, operand layout, 8-bit inputs, 64-row windows, the
# paper's own gather, dynamic scheduling, row groups off) and more sweep points
ALL_OTHERS = DEFAULT_OTHERS + [
    "cfg2_wcsr_irregular_alpha1.8", "cfg4_bcsr_sweep_b64_d0.5", "cfg4_bcsr_sweep_b64_d0.2",
    "cfg4_bcsr_sweep_b64_d0.05", "cfg4_bcsr_sweep_b64_d0.01", "cfg4_bcsr_flat_b64_d0.05", "cfg4_bcsr_flat_b64_d0.01",
    "cfg3_bcsr_llm_gate_c16", "cfg3_bcsr_llm_gate_cm", "cfg3_bcsr_llm_gate_cm_c16",
    "cfg3_bcsr_llm_down_cm_c16", "cfg5_wcsr_rmat_n128_c16",
    "cfg3_bcsr_llm_gate_cm_fp8", "cfg3_bcsr_llm_down_cm_fp8", "cfg3_bcsr_llm_gate_fp8", "cfg2_wcsr_irregular_wh64", "cfg5_wcsr_rmat_n128_wh64",
    "cfg2_wcsr_irregular_lsu_gather", "cfg5_wcsr_rmat_n128_lsu_gather",
    "cfg4_bcsr_sweep_b64_d0.1_dyn", "cfg4_bcsr_sweep_b16_d0.1_plain", "cfg4_bcsr_sweep_b32_d0.1_plain",
    "cfg4_bcsr_sweep_b16_d0.5", "cfg4_bcsr_sweep_b32_d0.5",
    "cfg5_wcsr_rmat_n128_fp8",
    "cfg4_bcsr_families_b16", "cfg4_bcsr_families_b16_plain", "cfg4_bcsr_families_b32", "cfg4_bcsr_families_b32_plain",
    "cfg4_bcsr_sweep_b64_d0.1_ksplit", "cfg4_bcsr_sweep_b64_d0.01_ksplit",
    "cfg4_bcsr_sweep_b16_d0.1_tf32", "cfg4_bcsr_sweep_b32_d0.1_tf32", "cfg4_bcsr_sweep_b64_d0.1_tf32", "cfg4_bcsr_sweep_b128_d0.1_tf32"]

# DRAM bytes (read + write) of one launch of the dominant kernel, from the ncu captures whose
# summaries are under profiles/ (absent where no capture of that exact launch exists).
NCU_DRAM_TRAFFIC = {
    "cfg2_wcsr_irregular": 118.5e6,     # profiles/wcsr_spmm_cfg2_ncu.md
    "cfg5_wcsr_rmat_n128": 3.525e9,     # profiles/wcsr_spmm_cfg5_n128_dram.md
    "cfg5_wcsr_rmat_n256": 7.186e9,     # the same file, N = 256
    # captured at N = 16,384 (1.409 GB) and scaled by 4 to N = 65,536: one L2 slab is 2048
    # tokens, so traffic grows in proportion to N (profiles/bcsr_spmm_cfg3_n8192_ncu.md)
    "cfg3_bcsr_llm_gate": 5.64e9,
}


# --------------------------------------------------------------------------- helpers


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for nme, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nme)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def create_handle(lib, w, **opt):
    a = w["a"]
    opt = dict(w.get("opts", {}), **opt)
    t0 = time.perf_counter()
    if w["kind"] == "bcsr":
        h = lib.spmm_bcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], w["dtype"], w["size"], **opt)
    else:
        h = lib.spmm_wcsr_create_csr(a["m"], a["k"], a["row_ptr"], a["col_idx"], a["vals"], w["dtype"], w["size"], **opt)
    return h, (time.perf_counter() - t0) * 1e3


def device_B(torch, w, seed=7):
    """Seeded synthetic dense operand, generated on the device in storage dtype."""
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    k, N = w["a"]["k"], w["N"]
    tdt = {"bf16": torch.bfloat16, "fp16": torch.float16, "tf32": torch.float32, "fp8": torch.float8_e4m3fn}[w["dtype"]]
    B = torch.empty((k, N), dtype=tdt, device="cuda")
    rows = max(1, (1 << 26) // N)
    for r0 in range(0, k, rows):
        r1 = min(k, r0 + rows)
        if w["Bdist"][0] == "normal":
            x = torch.randn((r1 - r0, N), generator=g, device="cuda", dtype=torch.float32) * w["Bdist"][2] + w["Bdist"][1]
        else:
            x = torch.rand((r1 - r0, N), generator=g, device="cuda", dtype=torch.float32) * (w["Bdist"][2] - w["Bdist"][1]) + w["Bdist"][1]
        B[r0:r1] = x.to(tdt)
    return B


def roofline_of(info, ms, pk, name=None):
    """Roofline of one spmm_run: slower of tensor time for the stored flops and HBM time for the
    model bytes (A values + indices + distinct B rows touched + C).  `traffic` is the DRAM
    traffic ncu measured for the same launch, where a capture exists."""
    model_bytes = info["bytes_a"] + info["bytes_idx"] + info["bytes_b_touched"] + info["bytes_c"]
    # TF32 = half, 8-bit = twice the measured bf16 rate (nominal ratios)
    tc_peak = pk["bf16_tflops"] * {2: 0.5, 3: 2.0}.get(info["dtype"], 1.0)
    t_hbm = model_bytes / (pk["hbm_gbs"] * 1e9)
    t_tc = info["flops_stored"] / (tc_peak * 1e12)
    t = ms * 1e-3
    if t_hbm >= t_tc:
        ach = model_bytes / t / 1e9
        r = {"bound": "hbm", "achieved": ach, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": ach / pk["hbm_gbs"]}
    else:
        ach = info["flops_stored"] / t / 1e12
        r = {"bound": "tensor", "achieved": ach, "peak": tc_peak, "unit": "TFLOP/s", "frac": ach / tc_peak}
    r.update({"traffic": NCU_DRAM_TRAFFIC.get(name), "peak_source": pk["source"], "model_bytes": model_bytes,
              "t_roof_us": max(t_hbm, t_tc) * 1e6})
    return r


def time_workload(torch, lib, w, steps, warmup, flush):
    """-> dict with per-launch median / mean ms (device events), GFLOP/s, roofline, info."""
    h, create_ms = create_handle(lib, w)
    try:
        N = w["N"]
        info = lib.spmm_get_info(h, N)
        B = device_B(torch, w)
        o = w.get("opts", {})
        cdt = B.dtype if (o.get("c_type") and w["dtype"] != "tf32") else torch.float32
        if o.get("layout"):
            B = B.t().contiguous()              # X = B^T, N x k
            C = torch.empty((N, w["a"]["m"]), dtype=cdt, device="cuda")
        else:
            C = torch.empty((w["a"]["m"], N), dtype=cdt, device="cuda")
        st = torch.cuda.current_stream().cuda_stream
        for _ in range(max(3, warmup)):
            lib.spmm_run(h, B.data_ptr(), C.data_ptr(), N, st)
        torch.cuda.synchronize()
        lib.spmm_check(h)
        info = lib.spmm_get_info(h, N)          # again: the BCSR plan fields are filled by the first run
        evs = []
        for _ in range(steps):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            lib.spmm_run(h, B.data_ptr(), C.data_ptr(), N, st)
            e1.record()
            evs.append((e0, e1))
        torch.cuda.synchronize()
        lib.spmm_check(h)
        ms = np.array([a.elapsed_time(b) for a, b in evs])
        # the same launches back to back, L2 left as the previous launch left it (context: the
        # smaller working sets fit the 126 MB L2; the headline numbers are the flushed ones)
        wevs = []
        for _ in range(steps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            lib.spmm_run(h, B.data_ptr(), C.data_ptr(), N, st)
            e1.record()
            wevs.append((e0, e1))
        torch.cuda.synchronize()
        ms_warm = float(np.mean([a.elapsed_time(b) for a, b in wevs]))
        launches = 1 + (1 if (w["kind"] == "wcsr" and (info["n_split"] + info["n_empty"]) > 0) else 0)
        if w["kind"] == "bcsr" and info["n_slots"] > 0:
            launches = 2                                   # K-split: the SpMM kernel and the merge of the parts
        if w["kind"] == "bcsr" and info["n_stacked_rows"] > 0:
            # row groups: their own launch, then the remaining block-rows (if any)
            if lib.spmm_export(h, lib.X_BCSR_STACK_TILES, np.int32).size > 0:
                launches = 2 if lib.spmm_export(h, lib.X_BCSR_TILES, np.int32).size > 0 else 1
        return dict(info=info, ms_mean=float(ms.mean()), ms_median=float(np.median(ms)), ms_min=float(ms.min()), ms_warm=ms_warm,
                    create_ms=create_ms, launches_per_step=launches, B=B, C=C)
    finally:
        lib.spmm_destroy(h)


def dense_context(torch, flush, m=18944, k=3584, N=65536, steps=5):
    """Context only (Sec. 4.4 compares against the dense layer): the dense bf16 product of the
    configs[2] gate shape, Y[N][m] = X[N][k] W[m][k]^T, by torch.matmul (cuBLAS)."""
    X = torch.randn((N, k), device="cuda", dtype=torch.bfloat16)
    W = torch.randn((m, k), device="cuda", dtype=torch.bfloat16) * 0.02
    for _ in range(2):
        Y = X @ W.t()
    torch.cuda.synchronize()
    evs = []
    for _ in range(steps):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        Y = X @ W.t()
        e1.record()
        evs.append((e0, e1))
    torch.cuda.synchronize()
    ms = float(np.mean([a.elapsed_time(b) for a, b in evs]))
    del X, W, Y
    # the library's TF32 rate on an 8192^3 product, beside the nominal half-of-bf16 figure the
    # roofline of the TF32 workloads uses
    prev = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = True
    try:
        P = torch.randn((8192, 8192), device="cuda", dtype=torch.float32)
        Q = torch.randn((8192, 8192), device="cuda", dtype=torch.float32)
        for _ in range(2):
            R = P @ Q
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            R = P @ Q
        e1.record()
        torch.cuda.synchronize()
        tf32_tflops = 2.0 * 8192 ** 3 * steps / (e0.elapsed_time(e1) * 1e-3) / 1e12
        del P, Q, R
    finally:
        torch.backends.cuda.matmul.allow_tf32 = prev
    return {"what": "dense bf16 torch.matmul of the configs[2] gate shape (library GEMM, context only)",
            "ms_per_step": ms, "tflops_dense": 2.0 * m * k * N / (ms * 1e-3) / 1e12,
            "tf32_matmul_8192_tflops": tf32_tflops}


def summarize(name, desc, res, pk, N):
    info = res["info"]
    ms = res["ms_mean"]
    gf = info["flops_stored"] / (ms * 1e-3) / 1e9
    return {
        "workload": name, "description": desc, "ms_per_step": ms, "ms_median": res["ms_median"], "ms_min": res["ms_min"],
        "ms_warm_l2": res["ms_warm"],
        "gflops_stored": gf, "gflops_useful": 2.0 * info["nnz"] * N / (ms * 1e-3) / 1e9,
        "fill_ratio": info["fill_ratio"], "stored_values": info["stored_values"], "n_units": info["n_units"],
        "create_ms": res["create_ms"], "launches_per_step": res["launches_per_step"],
        "roofline": roofline_of(info, ms, pk, name),
    }


def r4(x):
    """Four significant digits: keeps the result line short."""
    return None if x is None else float("%.4g" % x)


def aggregate_over_ranks(ms_local, flops_per_rank, world, dist=None, device="cpu"):
    """Replicas-only aggregation: every rank ran the same workload on its own GPU.
    -> (max step time over ranks in ms, whole-job GFLOP/s = world * flops / max time)."""
    ms = float(ms_local)
    if world > 1:
        import torch
        t = torch.tensor([ms], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    return ms, world * flops_per_rank / (ms * 1e-3) / 1e9


# --------------------------------------------------------------------------- CPU oracle legs


def cpu_oracle_time(w, budget_s=15.0, min_s=3.0):
    """Time the oracle (as it stands, one thread) on a bounded sample: all rows x a column slab,
    repeated until about min_s seconds of work have run (mean of the repeats)."""
    from oracle import spmm_ref
    a, N, dtype = w["a"], w["N"], w["dtype"]
    nnz = int(a["row_ptr"][-1])
    # ~0.35 G multiply-add pairs per second per core with the |.| sum: size the slab for the budget
    cols = int(max(1, min(N, budget_s * 2.0e8 / max(1, nnz))))
    Bs = wl.dense(11, a["k"], cols, w["Bdist"], dtype)
    v64, B64 = wl.widen(a["vals"], dtype), wl.widen(Bs, dtype)
    times = []
    while not times or (sum(times) < min_s and len(times) < 25):
        t0 = time.perf_counter()
        spmm_ref(a["row_ptr"], a["col_idx"], v64, B64)
        times.append(time.perf_counter() - t0)
    dt = float(np.mean(times))
    return dt * (N / cols), cols, dt * len(times)


def cpu_oracle_time_all_cores(w, cores, budget_s=15.0, min_s=3.0):
    """The same routine called from `cores` threads on disjoint row ranges (cut at equal stored
    entries); every thread gets its own rows as a CSR of their own and writes its own result."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle import spmm_ref
    a, N, dtype = w["a"], w["N"], w["dtype"]
    rp = np.asarray(a["row_ptr"], dtype=np.int64)
    nnz, m = int(rp[-1]), rp.shape[0] - 1
    cols = int(max(1, min(N, budget_s * cores * 2.0e8 / max(1, nnz))))
    Bs = wl.dense(11, a["k"], cols, w["Bdist"], dtype)
    v64, B64 = wl.widen(a["vals"], dtype), np.ascontiguousarray(wl.widen(Bs, dtype), dtype=np.float64)
    cuts = np.unique(np.concatenate(([0], np.searchsorted(rp, np.linspace(0, nnz, cores + 1)[1:-1]), [m]))).astype(np.int64)
    parts = []
    for r0, r1 in zip(cuts[:-1], cuts[1:]):
        p0, p1 = int(rp[r0]), int(rp[r1])
        parts.append((rp[r0:r1 + 1] - p0, a["col_idx"][p0:p1], v64[p0:p1]))

    def one(part):
        spmm_ref(part[0], part[1], part[2], B64)

    times = []
    with ThreadPoolExecutor(max_workers=cores) as ex:
        while not times or (sum(times) < min_s and len(times) < 25):
            t0 = time.perf_counter()
            list(ex.map(one, parts))
            times.append(time.perf_counter() - t0)
    dt = float(np.mean(times))
    return dt * (N / cols), cols, dt * len(times), len(parts)


def stored_values_by_oracle(w):
    """nnz_stored of the workload's format, from the oracle's own format definitions (key pass
    only: no value array is built): BCSR stored blocks * b * b, WCSR window height * padded columns."""
    from oracle import formats
    a = w["a"]
    if w["kind"] == "bcsr":
        return formats.bcsr_block_count(a["m"], a["k"], a["row_ptr"], a["col_idx"], w["size"]) * w["size"] ** 2
    b_col = 32 // wl.elem_size(w["dtype"])
    return formats.wcsr_padded_cols(a["m"], a["k"], a["row_ptr"], a["col_idx"], w["size"], b_col) * w["size"]


def run_reference(args):
    """The oracle as it stands on the host cores; nothing of the CUDA library is imported or loaded."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    name = args.only or HEADLINE
    desc, builder = workload_table()[name]
    w = builder()
    if args.dense_width:
        w["N"] = args.dense_width
    flops_stored = 2.0 * stored_values_by_oracle(w) * w["N"]
    times = []
    for i in range(args.warmup + args.steps):
        t_full, cols, dt = cpu_oracle_time(w, budget_s=max(1.0, 60.0 / (args.warmup + args.steps)))
        if i >= args.warmup:
            times.append(t_full)
    t = float(np.mean(times))
    val = flops_stored / t / 1e9
    sample = "all %d rows x %d of %d columns per step, scaled linearly in N" % (w["a"]["m"], cols, w["N"])
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": {"workload": name, "description": desc},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- main arm


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="b200")
    ap.add_argument("--only", default=None, help="time just this workload as the headline (see workload_table)")
    ap.add_argument("--skip-others", action="store_true")
    ap.add_argument("--others", default=None, help="comma-separated workload names to measure beside the headline, or 'all'")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the end-to-end leg (profiling runs)")
    ap.add_argument("--dense-width", type=int, default=0, help="override N of the --only workload (small profiling cases)")
    ap.add_argument("--ubench", action="store_true",
                    help="run the machine-constant microbenchmarks (tcgen05.mma interval, TMA load and store rates alone "
                         "and together) instead of the workloads; one JSON line per case")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.ubench:
        from paper_2604_17834_b200 import build
        exe = build.UBENCH_OUT
        if not os.path.exists(exe):
            raise SystemExit("%s is missing: build it with `python -m paper_2604_17834_b200.build`" % exe)
        raise SystemExit(subprocess.call([exe]))

    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    from paper_2604_17834_b200 import binding as lib

    pk = peaks()
    table = workload_table()
    name = args.only or HEADLINE
    desc, builder = table[name]
    w = builder()
    if args.dense_width:
        w["N"] = args.dense_width
        desc += " [N overridden to %d]" % args.dense_width
    warmup = max(3, args.warmup)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    res = time_workload(torch, lib, w, args.steps, warmup, flush)
    barrier()
    clocks = sampler.stop()
    info = res["info"]
    ms, value = aggregate_over_ranks(res["ms_mean"], info["flops_stored"], world, dist, "cuda")
    head = summarize(name if not args.dense_width else None, desc, res, pk, w["N"])

    # end to end through the C ABI with host buffers (pinned), copies inside the timed region
    a, N = w["a"], w["N"]
    e2e = None
    if not args.no_e2e:
        Bh = torch.empty(tuple(res["B"].shape), dtype=res["B"].dtype, pin_memory=True)
        Bh.copy_(res["B"])
        Ch = torch.empty(tuple(res["C"].shape), dtype=res["C"].dtype, pin_memory=True)
        del res["B"], res["C"]
        torch.cuda.empty_cache()
        h, _ = create_handle(lib, w)
        st = torch.cuda.current_stream().cuda_stream
        e2e_steps = max(3, min(args.steps, 10))
        for _ in range(2):
            lib.spmm_run_host(h, Bh.data_ptr(), Ch.data_ptr(), N, st)
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            lib.spmm_run_host(h, Bh.data_ptr(), Ch.data_ptr(), N, st)
        torch.cuda.synchronize()
        e2e_s = (time.perf_counter() - t0) / e2e_steps
        lib.spmm_destroy(h)
        e2e_ms, e2e_value = aggregate_over_ranks(e2e_s * 1e3, info["flops_stored"], world, dist, "cuda")
        e2e = {"value": r4(e2e_value), "unit": UNIT, "ms_per_step": r4(e2e_ms), "steps": e2e_steps,
               "h2d_bytes_per_step": int(Bh.numel() * Bh.element_size()), "d2h_bytes_per_step": int(Ch.numel() * Ch.element_size())}
        del Bh, Ch
    res.pop("B", None), res.pop("C", None)
    torch.cuda.empty_cache()

    # the other configurations: one short line each, printed as soon as it is measured
    others = []
    if rank == 0 and not args.skip_others and args.only is None:
        names = ALL_OTHERS if args.others == "all" else (args.others.split(",") if args.others else DEFAULT_OTHERS)
        for nm in names:
            try:
                d2, b2 = table[nm]
                w2 = b2()
                r2 = time_workload(torch, lib, w2, max(5, args.steps // 3), 3, flush)
                r2.pop("B"), r2.pop("C")
                o = summarize(nm, d2, r2, pk, w2["N"])
                del w2
            except Exception as exc:                    # the result line must come out whatever happens here
                o = {"workload": nm, "error": "%s: %s" % (type(exc).__name__, exc)}
            torch.cuda.empty_cache()
            print(json.dumps({"other": o}), flush=True)
            others.append(o)
        if args.others == "all":
            print(json.dumps({"context": dense_context(torch, flush)}), flush=True)
            torch.cuda.empty_cache()

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        t_full, cols, dt = cpu_oracle_time(w)
        cpu = {"value": r4(info["flops_stored"] / t_full / 1e9), "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": "all %d rows x %d of %d columns (%.1f s), scaled in N" % (a["m"], cols, N, dt)}
        cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
        if cores > 1:
            tp, pcols, pdt, nparts = cpu_oracle_time_all_cores(w, cores)
            cpu["all_cores"] = {"value": r4(info["flops_stored"] / tp / 1e9), "cores": nparts,
                                "sample": "same routine, %d disjoint row ranges, %d columns (%.1f s)" % (nparts, pcols, pdt)}

    if rank == 0:
        roof = head["roofline"]
        # everything that does not fit the result line: a line of its own, before it
        print(json.dumps({"detail": {"headline": head, "cpu_baseline": cpu, "peaks": pk}}), flush=True)
        line = {
            "metric": METRIC, "value": r4(value), "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
            "ms_per_step": r4(ms), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": w["dtype"], "data": "synthetic",
            "config": {"workload": name, "description": desc, "l2": "flushed (512 MB write) before every timed launch"},
            "clocks": clocks, "e2e": e2e,
            "gpu_launches": int(res["launches_per_step"] * args.steps),
            "roofline": {"bound": roof["bound"], "achieved": r4(roof["achieved"]), "peak": roof["peak"], "unit": roof["unit"],
                         "frac": r4(roof["frac"]), "traffic": roof["traffic"], "peak_source": roof["peak_source"]},
            "cpu_baseline": None if cpu is None else {k: cpu[k] for k in ("value", "unit", "cores", "kind", "sample")},
            # per other workload: [name, ms_per_step, roofline frac]; their own lines above have the rest
            "others": [([o["workload"], "error"] if "error" in o else
                        [o["workload"], r4(o["ms_per_step"]), float("%.3g" % o["roofline"]["frac"])]) for o in others],
        }
        # the result line stays short enough to survive a tail of the output whole: the other
        # workloads' own lines above carry everything that is dropped here
        text = json.dumps(line, separators=(",", ":"))
        while len(text) > MAX_LINE_BYTES and line["others"]:
            line["others"].pop()
            text = json.dumps(line, separators=(",", ":"))
        print(text, flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
