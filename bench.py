#!/usr/bin/env python
"""Benchmark of the emulated 16-bit-format hot path on B200.

One step = one pass of the format sweep (workload "config2"): the 64 Mi-element fp32 tensor is
rounded, with range statistics, to 1/5/10, 1/8/7 and 1/6/9, each with denormals kept and
flushed, at loss scales 2^0, 2^8 and 2^15 (18 kernel launches, 8 bytes of algorithmic traffic
per element and launch).  `value` is the whole-job GB/s with inputs resident in HBM; `e2e` is
the same metric through the host-buffer entry point (copies inside the timed region).  The
contraction half of the path is timed in the same run on the BERT-large FC stack (workload
"config5", its ten seeded steps: 4 layers x fwd/dgrad/wgrad each, fresh tensors and per-tensor
statistics every step) and reported under `gemm` and again inside `roofline`; the convolution
layers of config4 under `conv`, the one-pass layer output R(R(acc)+R(B)) under `epilogue` and the
FMAC-8 product (Algorithm 1) under `fmac8`.

    python bench.py --gpus N --steps K --warmup W          # this library
    python bench.py --impl reference ...                    # the CPU oracle on a bounded sample
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2103_15940_b200 import workloads  # noqa: E402

METRIC = "quantize+stats GB/s"
UNIT = "GB/s"
BYTES_PER_ELEMENT = 8  # 4 read + 4 written


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while a region is timed."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        names = {nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap",
                 nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
                 nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
                 nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
                 nv.nvmlClocksThrottleReasonHwPowerBrakeSlowdown: "hw_power_brake"}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.004)

    def __enter__(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def nvml_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ------------------------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on a bounded sample of the same workload
# ------------------------------------------------------------------------------------------------
def oracle_sweep(x: np.ndarray, threads: int = 1) -> float:
    """Runs the 18 sweep configurations on x with the oracle; returns seconds."""
    import oracle
    t0 = time.perf_counter()
    for _, e, m, den, scale in workloads.config2_runs():
        oracle.quantize_stats(x, e, m, den, scale, threads=threads)
    return time.perf_counter() - t0


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_sample = 1 << 20
    x = workloads.config2_tensor(n=n_sample)
    for _ in range(args.warmup):
        oracle_sweep(x[: 1 << 16])
    secs = [oracle_sweep(x) for _ in range(args.steps)]
    total = sum(secs)
    value = args.steps * 18 * n_sample * BYTES_PER_ELEMENT / total / 1e9
    sample = f"18 sweep runs on the first {n_sample} elements of the config2 tensor per step"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u32", "data": "synthetic",
            "config": {"workload": "config2 format sweep (bounded sample)", "elements": n_sample, "runs_per_step": 18},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# this library
# ------------------------------------------------------------------------------------------------
def max_over_ranks(torch, dist, value: float, device) -> float:
    """The slowest rank's time: what a multi-GPU number is computed from (dist is None for one rank)."""
    if dist is None:
        return value
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world: int, steps: int, step_bytes: int, total_ms: float) -> float:
    """GB/s over all ranks: every rank ran `steps` sweeps of `step_bytes` on its own replica."""
    return world * steps * step_bytes / total_ms / 1e6


def time_events(torch, fn, iters):
    """Per-call device times (ms) of fn(), CUDA events on the current stream."""
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
    for a, b in evs:
        a.record()
        fn()
        b.record()
    torch.cuda.synchronize()
    return [a.elapsed_time(b) for a, b in evs]


def gemm_section(torch, qf, dev, peaks, reps=3, steps=workloads.CONFIG5_STEPS):
    """The BERT-large FC stack over its ten seeded steps.  Every step has fresh tensors; per step and
    layer X, W and dY (loss scale 2^16) are rounded to 1/6/9 with a statistics record of their own
    (accumulate = 0), then the forward, data-gradient and weight-gradient products run: 12 rounding
    passes and 12 products per step, 120 + 120 over the workload.  Timed twice with CUDA events per
    step: the whole step, and its products alone (the contraction half of the metric)."""
    from concurrent.futures import ThreadPoolExecutor
    fmt = qf.make_format(6, 9, 1)
    n_layers = len(workloads.CONFIG5_LAYERS)
    keys = [(s_, l_) for s_ in range(steps) for l_ in range(n_layers)]
    with ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as pool:   # host-side generation only
        host = dict(zip(keys, pool.map(lambda k: workloads.config5_layer(k[1], step=k[0]), keys)))
    grad_fmt = qf.make_format(6, 9, 1, host[(0, 0)]["grad_scale"])
    raw, q, outs, jobs = {}, {}, [], {}
    flops_per_step, rounded_bytes_per_step, ws_bytes = 0.0, 0, 256
    for l_ in range(n_layers):
        tokens, d_in = host[(0, l_)]["X"].shape
        d_out = host[(0, l_)]["W"].shape[1]
        outs.append((torch.empty(tokens, d_out, dtype=torch.float32, device=dev),
                     torch.empty(tokens, d_in, dtype=torch.float32, device=dev),
                     torch.empty(d_in, d_out, dtype=torch.float32, device=dev)))
        flops_per_step += 3 * 2.0 * tokens * d_in * d_out
    for k in keys:
        raw[k] = {n_: torch.from_numpy(host[k][n_]).to(dev) for n_ in ("X", "W", "dY")}
        q[k] = {n_: torch.empty_like(v) for n_, v in raw[k].items()}
        Y, dX, dW = outs[k[1]]
        jobs[k] = ((qf.make_matrix(q[k]["X"]), qf.make_matrix(q[k]["W"]), Y, Y.shape[1]),
                   (qf.make_matrix(q[k]["dY"]), qf.make_matrix(q[k]["W"], True), dX, dX.shape[1]),
                   (qf.make_matrix(q[k]["X"], True), qf.make_matrix(q[k]["dY"]), dW, dW.shape[1]))
        for a, b, _, _ in jobs[k]:
            ws_bytes = max(ws_bytes, qf.qfmt_gemm_workspace_bytes(a, b))
        if k[0] == 0:
            rounded_bytes_per_step += BYTES_PER_ELEMENT * sum(v.numel() for v in raw[k].values())
    sample_A, sample_B = host[(0, 0)]["X"], host[(0, 0)]["W"]
    del host
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)  # the recommended size (split-K partials)
    records = torch.zeros(steps, n_layers, 3, qf.STATS_WORDS, dtype=torch.int64, device=dev)

    def rounding(s_):
        for l_ in range(n_layers):
            k = (s_, l_)
            for i, (n_, f) in enumerate((("X", fmt), ("W", fmt), ("dY", grad_fmt))):
                qf.qfmt_quantize_stats(raw[k][n_], q[k][n_], raw[k][n_].numel(), f, records[s_, l_, i], 0)

    def products(s_):
        for l_ in range(n_layers):
            for a, b, C, ldc in jobs[(s_, l_)]:
                qf.qfmt_gemm(a, b, C, ldc, fmt, ws, ws.numel())

    def whole(s_):
        rounding(s_)
        products(s_)

    for _ in range(2):  # warm-up over the whole workload (also fills the rounded operands)
        for s_ in range(steps):
            whole(s_)
    assert qf.qfmt_device_status(ws) == qf.QFMT_OK
    rec = records.cpu().numpy().view(np.uint64)
    for (s_, l_) in keys:
        for i, n_ in enumerate(("X", "W", "dY")):
            assert int(rec[s_, l_, i, 256]) == raw[(s_, l_)][n_].numel() == int(rec[s_, l_, i, :256].sum())
    step_ms = [statistics.median(v) for v in zip(*[[time_events(torch, lambda s_=s_: whole(s_), 1)[0]
                                                     for s_ in range(steps)] for _ in range(reps)])]
    gemm_ms = [statistics.median(v) for v in zip(*[[time_events(torch, lambda s_=s_: products(s_), 1)[0]
                                                     for s_ in range(steps)] for _ in range(reps)])]
    denormal_fraction_dY = [float(rec[s_, :, 2, 258].sum()) / float(rec[s_, :, 2, 256].sum()) for s_ in range(steps)]
    # library TF32 GEMM on the same box, same run: a second view of the tensor-pipe denominator
    torch.backends.cuda.matmul.allow_tf32 = True
    a = torch.randn(8192, 8192, device=dev)
    b = torch.randn(8192, 8192, device=dev)
    c = torch.empty(8192, 8192, device=dev)
    for _ in range(3):
        torch.matmul(a, b, out=c)
    lib_ms = min(time_events(torch, lambda: torch.matmul(a, b, out=c), 5))
    lib_tf32 = 2.0 * 8192 ** 3 / lib_ms / 1e9
    del a, b, c
    total_gemm_ms, total_step_ms = sum(gemm_ms), sum(step_ms)
    achieved = steps * flops_per_step / total_gemm_ms / 1e9
    peak = peaks["bf16_tflops"] * (1.1 / 2.25)  # TF32 dense is nominally 1.1/2.25 of bf16 dense
    # the fp64 oracle on this machine's host cores (OpenMP over outputs): 2^18 sampled outputs of the first product
    import oracle
    hA, _ = oracle.quantize_stats(sample_A, 6, 9, 1, 1.0, want_stats=False)
    hB, _ = oracle.quantize_stats(sample_B, 6, 9, 1, 1.0, want_stats=False)
    rng = np.random.default_rng(0)
    ii, jj = rng.integers(0, hA.shape[0], size=1 << 18), rng.integers(0, hB.shape[1], size=1 << 18)
    t0 = time.perf_counter()
    oracle.gemm_sampled(hA, hB, ii, jj)
    cpu_s = time.perf_counter() - t0
    cpu = {"value": 2.0 * ii.size * hA.shape[1] / cpu_s / 1e12, "unit": "TFLOP/s", "cores": os.cpu_count(),
           "kind": "oracle", "seconds": cpu_s,
           "sample": f"{ii.size} sampled outputs of the {hA.shape[0]} x {hB.shape[1]} x {hA.shape[1]} forward product "
                     "(step 0, QKV layer), full-K fp64 dot products"}
    return {"metric": "emulated GEMM TFLOP/s", "value": achieved, "unit": "TFLOP/s", "cpu_baseline": cpu,
            "workload": f"config5 BERT-large FC stack, {steps} seeded steps x 4 layers x fwd/dgrad/wgrad, 1/6/9, fresh "
                        "tensors per step (5.6 GB of operands: larger than L2), per-tensor statistics every step",
            "steps": steps, "ms_per_step": total_gemm_ms / steps, "per_step_gemm_ms": gemm_ms,
            "per_step_whole_ms": step_ms, "total_gemm_ms": total_gemm_ms, "total_whole_ms": total_step_ms,
            "whole_step_gemm_tflops": steps * flops_per_step / total_step_ms / 1e9,
            "rounding_gbs": steps * rounded_bytes_per_step / max(total_step_ms - total_gemm_ms, 1e-9) / 1e6,
            "denormal_fraction_of_dY_per_step": denormal_fraction_dY,
            "gemms_per_step": 3 * n_layers, "gpu_launches_per_step": 6 * n_layers,
            "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                         "frac": achieved / peak, "traffic": None,
                         "peak_source": f"bf16 {peaks['source']} burst x 1.1/2.25 (nominal TF32:bf16 ratio)",
                         "frac_of_sustained": achieved / (peaks["bf16_tflops_sustained"] * (1.1 / 2.25)),
                         "library_tf32_same_run": lib_tf32, "frac_of_library_tf32": achieved / lib_tf32,
                         "nominal_tf32_dense": 1100.0, "frac_of_nominal": achieved / 1100.0}}


def conv_section(torch, qf, dev, peaks, reps=5):
    """The two ResNet-50-shaped layers of config4 (batch 128, 14x14): NCHW tensors are rounded to
    1/6/9 into channels-last by the transposing pass, then fwd, dgrad and wgrad run as implicit GEMMs."""
    out = {"metric": "emulated conv TFLOP/s", "unit": "TFLOP/s", "layers": {}}
    total_flops, total_ms, launches = 0.0, 0.0, 0
    for tag, sh in (("3x3", workloads.CONV3X3), ("1x1", workloads.CONV1X1)):
        cfg = workloads.config4(sh)
        n, ci, h, w, co, r, s_, pad = sh.n, sh.c_in, sh.h, sh.w, sh.c_out, sh.r, sh.s, sh.pad
        g = qf.qfmt_conv_t(n, ci, h, w, co, r, s_, pad, pad)
        fmt = qf.make_format(6, 9, 1)

        def cl(x, scale=1.0):
            b, c, hh, ww = x.shape
            d_in = torch.from_numpy(x).to(dev)
            d_out = torch.empty(b * hh * ww * c, dtype=torch.float32, device=dev)
            qf.qfmt_quantize_stats_transpose(d_in, d_out, b, c, hh * ww, qf.make_format(6, 9, 1, scale))
            return d_out
        X, Wt, dY = cl(cfg["X"]), cl(cfg["W"]), cl(cfg["dY"], cfg["grad_scale"])
        jobs = []
        for op, P, Q, numel in ((qf.QFMT_CONV_FWD, X, Wt, n * h * w * co), (qf.QFMT_CONV_DGRAD, dY, Wt, n * h * w * ci),
                                (qf.QFMT_CONV_WGRAD, dY, X, co * r * s_ * ci)):
            wb = qf.qfmt_conv_workspace_bytes(op, g)
            jobs.append((op, P, Q, torch.empty(numel, dtype=torch.float32, device=dev),
                         torch.zeros(wb, dtype=torch.uint8, device=dev), wb))

        def step():
            for op, P, Q, O, ws, wb in jobs:
                qf.qfmt_conv(op, g, P, Q, O, fmt, ws, wb)
        for _ in range(3):
            step()
        for j in jobs:
            assert qf.qfmt_device_status(j[4]) == qf.QFMT_OK
        ms = statistics.median(time_events(torch, step, reps))
        flops = 3 * 2.0 * n * h * w * co * ci * r * s_
        out["layers"][tag] = {"ms_per_step": ms, "tflops": flops / ms / 1e9}
        total_flops += flops
        total_ms += ms
        # three products + the split-K reduction of the filter gradient; forward and data gradient of the 3x3 layer
        # run under the balanced schedule, whose hand-over words a one-block kernel clears before each of them
        launches += 4 + (2 if tag == "3x3" else 0)
    peak = peaks["bf16_tflops"] * (1.1 / 2.25)
    out.update({"value": total_flops / total_ms / 1e9, "ms_per_step": total_ms, "gpu_launches_per_step": launches,
                "workload": "config4: 3x3 (256->256) and 1x1 (1024->256) layers, fwd+dgrad+wgrad, 1/6/9, channels-last",
                "roofline": {"bound": "tensor", "achieved": total_flops / total_ms / 1e9, "peak": peak, "unit": "TFLOP/s",
                             "frac": total_flops / total_ms / 1e9 / peak, "traffic": None}})
    return out


def epilogue_section(torch, qf, dev, peaks, reps=20):
    """Layer output Y = R(R(acc) + R(B)) with statistics of Y, one pass: the forward output of the
    config5 FFN-up layer (8192 x 4096, the library's own product as `acc`), 1/6/9."""
    c = workloads.config5_layer(2, step=0)
    fmt = qf.make_format(6, 9, 1)
    X, W = torch.from_numpy(c["X"]).to(dev), torch.from_numpy(c["W"]).to(dev)
    qf.qfmt_quantize_stats(X, X, X.numel(), fmt)
    qf.qfmt_quantize_stats(W, W, W.numel(), fmt)
    rows, cols = X.shape[0], W.shape[1]
    acc = torch.empty(rows, cols, dtype=torch.float32, device=dev)
    a, b = qf.make_matrix(X), qf.make_matrix(W)
    ws = torch.zeros(max(256, qf.qfmt_gemm_workspace_bytes(a, b)), dtype=torch.uint8, device=dev)
    qf.qfmt_gemm(a, b, acc, cols, fmt, ws, ws.numel())
    assert qf.qfmt_device_status(ws) == qf.QFMT_OK
    bias = torch.from_numpy(workloads.normal_tensor(workloads.rng_for(4, 1000), (cols,), 0.02)).to(dev)
    out = torch.empty_like(acc)
    st = torch.zeros(qf.STATS_WORDS, dtype=torch.int64, device=dev)

    def step():
        qf.qfmt_bias_quantize_stats(acc, cols, bias, out, cols, rows, cols, fmt, st)
    for _ in range(3):
        step()
    ms = statistics.median(time_events(torch, step, reps))
    assert int(st.cpu()[256]) == rows * cols
    achieved = rows * cols * BYTES_PER_ELEMENT / ms / 1e6
    # the same pass writing packed 16-bit codes: 4 B read + 2 B written per element
    codes = torch.empty(rows, cols, dtype=torch.int16, device=dev)

    def step_codes():
        qf.qfmt_bias_quantize_stats_pack16(acc, cols, bias, codes, cols, rows, cols, fmt, st)
    for _ in range(3):
        step_codes()
    ms_codes = statistics.median(time_events(torch, step_codes, reps))
    codes_gbs = rows * cols * 6 / ms_codes / 1e6
    to_codes = {"ms": ms_codes, "value": codes_gbs, "unit": "GB/s",
                "roofline": {"bound": "hbm", "achieved": codes_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                             "frac": codes_gbs / peaks["hbm_gbs"], "traffic": None,
                             "algorithmic_bytes_per_launch": rows * cols * 6}}
    del codes
    # the whole forward layer through qfmt_linear_forward: default plan (GEMM, then the pass above in place)
    # and with the epilogue inside the GEMM kernel (K = 1024)
    wb = qf.qfmt_linear_forward_workspace_bytes(a, b)
    ws2 = torch.zeros(wb, dtype=torch.uint8, device=dev)

    def layer():
        qf.qfmt_linear_forward(a, b, bias, out, cols, fmt, st, 0, ws2, wb)

    def gemm_only():
        qf.qfmt_gemm(a, b, acc, cols, fmt, ws, ws.numel())
    timings = {}
    for name, policy in (("two_kernels", 0), ("in_kernel", 1)):
        qf.qfmt_linear_fusion_policy(policy)
        for _ in range(3):
            layer()
        assert qf.qfmt_device_status(ws2) == qf.QFMT_OK
        timings[name] = statistics.median(time_events(torch, layer, reps))
    qf.qfmt_linear_fusion_policy(0)
    for _ in range(3):
        gemm_only()
    gemm_ms = statistics.median(time_events(torch, gemm_only, reps))
    flops = 2.0 * rows * cols * X.shape[1]
    linear = {"workload": f"config5 FFN-up forward layer, {rows} x {cols} x {X.shape[1]}, Y = R(R(XW) + R(B)) with statistics",
              "ms": timings["two_kernels"], "tflops": flops / timings["two_kernels"] / 1e9, "gemm_alone_ms": gemm_ms,
              "epilogue_in_gemm_kernel_ms": timings["in_kernel"]}
    return {"metric": "layer output R(R(acc)+R(B)) + stats GB/s", "value": achieved, "unit": "GB/s", "linear_forward": linear,
            "to_packed_codes": to_codes,
            "workload": f"config5 FFN-up forward output, {rows} x {cols}, 1/6/9 (268 MB moved per launch, larger than L2)",
            "ms_per_step": ms, "gpu_launches_per_step": 2,  # the pass and the one-block kernel that clears its record
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": achieved / peaks["hbm_gbs"], "traffic": NCU_EPILOGUE_TRAFFIC_BYTES_PER_LAUNCH,
                         "peak_source": f"copy bandwidth, {peaks['source']}",
                         "algorithmic_bytes_per_launch": rows * cols * BYTES_PER_ELEMENT}}


def step5_section(torch, qf, dev, peaks, reps=5):
    """One training step of the config5 BERT-large FC stack with everything the path does per step:
    for each of the four layers the operands are rounded to 1/6/9 with per-tensor statistics (X, W, and
    dY with the device-resident loss scale), the forward layer output is Y = R(R(XW) + R(B)) with
    statistics, the two gradient products follow, and the loss-scale controller reads the gradients'
    overflow counts -- all enqueued on one stream, nothing returns to the host."""
    fmt = qf.make_format(6, 9, 1)
    state = qf.qfmt_dls_t(2.0 ** 16, 2.0, 0.5, 1.0, 2.0 ** 24, 2000, 0, 0, 0, 0, 0)
    d_state = torch.from_numpy(np.frombuffer(bytes(state), dtype=np.uint8).copy()).to(dev)
    layers, flops, bytes_rounded = [], 0.0, 0
    for li in range(len(workloads.CONFIG5_LAYERS)):
        c = workloads.config5_layer(li, step=0)
        raw = {k: torch.from_numpy(c[k]).to(dev) for k in ("X", "W", "dY")}
        q = {k: torch.empty_like(v) for k, v in raw.items()}
        tokens, d_in = c["X"].shape
        d_out = c["W"].shape[1]
        bias = torch.from_numpy(workloads.normal_tensor(workloads.rng_for(4, 2000 + li), (d_out,), 0.02)).to(dev)
        Y = torch.empty(tokens, d_out, dtype=torch.float32, device=dev)
        dX = torch.empty(tokens, d_in, dtype=torch.float32, device=dev)
        dW = torch.empty(d_in, d_out, dtype=torch.float32, device=dev)
        fwd = (qf.make_matrix(q["X"]), qf.make_matrix(q["W"]))
        dg = (qf.make_matrix(q["dY"]), qf.make_matrix(q["W"], True))
        wg = (qf.make_matrix(q["X"], True), qf.make_matrix(q["dY"]))
        wb = max(qf.qfmt_linear_forward_workspace_bytes(*fwd), qf.qfmt_gemm_workspace_bytes(*dg),
                 qf.qfmt_gemm_workspace_bytes(*wg), 256)
        layers.append((raw, q, bias, Y, dX, dW, fwd, dg, wg, torch.zeros(wb, dtype=torch.uint8, device=dev), wb,
                       d_out, d_in))
        flops += 3 * 2.0 * tokens * d_in * d_out
        bytes_rounded += BYTES_PER_ELEMENT * (sum(v.numel() for v in raw.values()) + tokens * d_out)
    stats = torch.zeros(len(layers), 4, qf.STATS_WORDS, dtype=torch.int64, device=dev)   # X, W, -, Y per layer
    grad_stats = torch.zeros(len(layers), qf.STATS_WORDS, dtype=torch.int64, device=dev)

    def step():
        for li, (raw, q, bias, Y, dX, dW, fwd, dg, wg, ws, wb, d_out, d_in) in enumerate(layers):
            qf.qfmt_quantize_stats(raw["X"], q["X"], raw["X"].numel(), fmt, stats[li, 0])
            qf.qfmt_quantize_stats(raw["W"], q["W"], raw["W"].numel(), fmt, stats[li, 1])
            qf.qfmt_quantize_stats_dls(raw["dY"], q["dY"], raw["dY"].numel(), fmt, d_state, grad_stats[li])
            qf.qfmt_linear_forward(fwd[0], fwd[1], bias, Y, d_out, fmt, stats[li, 3], 0, ws, wb)
            qf.qfmt_gemm(dg[0], dg[1], dX, d_in, fmt, ws, wb)
            qf.qfmt_gemm(wg[0], wg[1], dW, d_out, fmt, ws, wb)
        qf.qfmt_dls_update(d_state, grad_stats, len(layers))
    for _ in range(3):
        step()
    for l in layers:
        assert qf.qfmt_device_status(l[9]) == qf.QFMT_OK
    ms = statistics.median(time_events(torch, step, reps))
    final = qf.qfmt_dls_t.from_buffer_copy(d_state.cpu().numpy().tobytes())
    return {"metric": "config5 training step, ms", "value": ms, "unit": "ms", "higher_is_better": False,
            "workload": "config5 step: 4 layers x (round X, W, dY with statistics; Y = R(R(XW)+R(B)) with statistics; "
                        "dgrad; wgrad) + loss-scale controller, 1/6/9, loss scale 2^16 kept on the device",
            "ms_per_step": ms, "gemm_tflops_over_whole_step": flops / ms / 1e9,
            "rounded_bytes_per_step": bytes_rounded, "gpu_launches_per_step": 8 * len(layers) + 1,
            "steps_seen_by_controller": int(final.n_steps), "steps_skipped": int(final.n_skipped),
            "loss_scale": float(final.scale)}


def config13_section(torch, qf, dev, peaks, reps=5):
    """The two remaining workloads.  config1: the small reference case (A 256x512, B 512x256 rounded to
    1/6/9 with statistics, C = A B), latency-bound: time per pass.  config3: the BERT-base FC layer in four
    variants (1/6/9 and 1/5/10, denormals kept and flushed): X, W and dY (loss scale 2^10) rounded with
    statistics, then forward, data-gradient and weight-gradient products."""
    out = {}
    c1 = workloads.config1()
    e, m = c1["fmt"]
    fmt = qf.make_format(e, m, c1["denormals"], c1["loss_scale"])
    rA, rB = torch.from_numpy(c1["A"]).to(dev), torch.from_numpy(c1["B"]).to(dev)
    qA, qB = torch.empty_like(rA), torch.empty_like(rB)
    st = torch.zeros(2, qf.STATS_WORDS, dtype=torch.int64, device=dev)
    C = torch.empty(256, 256, dtype=torch.float32, device=dev)
    a, b = qf.make_matrix(qA), qf.make_matrix(qB)
    ws = torch.zeros(max(256, qf.qfmt_gemm_workspace_bytes(a, b)), dtype=torch.uint8, device=dev)

    def pass1():
        qf.qfmt_quantize_stats(rA, qA, rA.numel(), fmt, st[0])
        qf.qfmt_quantize_stats(rB, qB, rB.numel(), fmt, st[1])
        qf.qfmt_gemm(a, b, C, 256, fmt, ws, ws.numel())
    for _ in range(3):
        pass1()
    assert qf.qfmt_device_status(ws) == qf.QFMT_OK
    ms = statistics.median(time_events(torch, pass1, 20))
    # the same pass replayed from a CUDA graph: what remains once the host-side launch cost is gone
    graph_ms = None
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            pass1()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            pass1()
        for _ in range(3):
            graph.replay()
        graph_ms = statistics.median(time_events(torch, graph.replay, 20))
        torch.cuda.synchronize()
    except Exception as exc:  # capture is an extra, not part of the path
        graph_ms = None
        out["config1_graph_error"] = str(exc)[:200]
    out["config1"] = {"workload": "config1: round A 256x512 and B 512x256 to 1/6/9 with statistics, C = A B",
                      "ms_per_pass": ms, "ms_per_pass_cuda_graph": graph_ms, "gpu_launches_per_pass": 3,
                      "gemm_gflop": 2.0 * 256 * 256 * 512 / 1e9,
                      "note": "latency-bound (three small launches): time only, no roofline fraction"}

    c3 = workloads.config3()
    raw = {k: torch.from_numpy(c3[k]).to(dev) for k in ("X", "W", "dY")}
    q = {k: torch.empty_like(v) for k, v in raw.items()}
    tokens, d_in = c3["X"].shape
    d_out = c3["W"].shape[1]
    Y = torch.empty(tokens, d_out, dtype=torch.float32, device=dev)
    dX = torch.empty(tokens, d_in, dtype=torch.float32, device=dev)
    dW = torch.empty(d_in, d_out, dtype=torch.float32, device=dev)
    prods = ((qf.make_matrix(q["X"]), qf.make_matrix(q["W"]), Y, d_out),
             (qf.make_matrix(q["dY"]), qf.make_matrix(q["W"], True), dX, d_in),
             (qf.make_matrix(q["X"], True), qf.make_matrix(q["dY"]), dW, d_out))
    wb = max([256] + [qf.qfmt_gemm_workspace_bytes(pa, pb) for pa, pb, _, _ in prods])
    ws3 = torch.zeros(wb, dtype=torch.uint8, device=dev)
    st3 = torch.zeros(3, qf.STATS_WORDS, dtype=torch.int64, device=dev)
    variants = c3["variants"]

    def rounding():
        for (e_, m_), den in variants:
            for i, (name, scale) in enumerate((("X", 1.0), ("W", 1.0), ("dY", c3["grad_scale"]))):
                qf.qfmt_quantize_stats(raw[name], q[name], raw[name].numel(), qf.make_format(e_, m_, den, scale), st3[i])

    def products():
        for (e_, m_), den in variants:
            f = qf.make_format(e_, m_, den)
            for pa, pb, Cc, ldc in prods:
                qf.qfmt_gemm(pa, pb, Cc, ldc, f, ws3, wb)
    for _ in range(3):
        rounding()
        products()
    assert qf.qfmt_device_status(ws3) == qf.QFMT_OK
    r_ms = statistics.median(time_events(torch, rounding, reps))
    p_ms = statistics.median(time_events(torch, products, reps))
    r_bytes = len(variants) * BYTES_PER_ELEMENT * sum(v.numel() for v in raw.values())
    flops = len(variants) * 3 * 2.0 * tokens * d_in * d_out
    tf = flops / p_ms / 1e9
    peak = peaks["bf16_tflops"] * (1.1 / 2.25)
    out["config3"] = {"workload": f"config3 BERT-base FC layer ({tokens} x {d_in} x {d_out}), 4 variants: 12 rounding passes with "
                                  "statistics, 12 products",
                      "rounding_ms": r_ms, "rounding_gbs": r_bytes / r_ms / 1e6,
                      "rounding_note": "tensors of 9-50 MB, smaller than L2: not an HBM figure",
                      "products_ms": p_ms, "gemm_tflops": tf, "gpu_launches_per_step": 24,
                      "roofline": {"bound": "tensor", "achieved": tf, "peak": peak, "unit": "TFLOP/s", "frac": tf / peak,
                                   "traffic": None}}
    return out


def pack16_section(torch, qf, dev, peaks, d_in, n, reps=20):
    """16-bit storage on the config2 tensor: the rounding pass writing packed codes (4 B read + 2 B
    written per element) and the expansion back to fp32 containers (2 B read + 4 B written)."""
    codes = torch.empty(n, dtype=torch.int16, device=dev)
    out = torch.empty(n, dtype=torch.float32, device=dev)
    st = torch.zeros(qf.STATS_WORDS, dtype=torch.int64, device=dev)
    fmt = qf.make_format(6, 9, 1, 2.0 ** 8)
    res = {}
    for name, fn in (("pack", lambda: qf.qfmt_quantize_stats_pack16(d_in, codes, n, fmt, st)),
                     ("unpack", lambda: qf.qfmt_unpack16(codes, out, n, fmt))):
        for _ in range(3):
            fn()
        ms = statistics.median(time_events(torch, fn, reps))
        gbs = n * 6 / ms / 1e6
        res[name] = {"ms": ms, "value": gbs, "unit": "GB/s",
                     "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                  "frac": gbs / peaks["hbm_gbs"], "traffic": None,
                                  "algorithmic_bytes_per_launch": n * 6}}
    assert int(st.cpu()[256]) == n
    return {"metric": "quantize+stats to packed 16-bit codes GB/s", "value": res["pack"]["value"], "unit": "GB/s",
            "workload": f"config2 tensor, {n} elements, 1/6/9 with loss scale 2^8 (6 B per element)",
            "gpu_launches_per_step": 2, "roofline": res["pack"]["roofline"], "runs": res}


def gemm16_section(torch, qf, dev, peaks, reps=5):
    """One step of the BERT-large FC stack (12 products: forward, activation gradient, weight
    gradient of 4 layers) on packed 16-bit operands: the rounding pass writes the codes of X, W and
    dY (1/5/10 as binary16 words, 1/8/7 as bfloat16 words), qfmt_gemm_packed16 contracts them in
    the layouts they are stored in."""
    out = {"metric": "emulated GEMM on packed 16-bit operands TFLOP/s", "unit": "TFLOP/s", "runs": {},
           "workload": "config5 BERT-large FC stack, one step: 4 layers x fwd/dgrad/wgrad, operands as packed codes; "
                       "whole_step_ms adds the rounding of X, W, dY to codes with statistics, the layer output as codes "
                       "with statistics and the loss-scale controller (gradient scale 2^16 given by the host)"}
    layers = []
    for layer in range(len(workloads.CONFIG5_LAYERS)):
        c = workloads.config5_layer(layer, step=0)
        layers.append(({k: torch.from_numpy(c[k]).to(dev) for k in ("X", "W", "dY")}, c["grad_scale"]))
    for tag, e, m in (("1/5/10 binary16", 5, 10), ("1/8/7 bfloat16", 8, 7)):
        fmt = qf.make_format(e, m, 1)
        jobs, flops, ws_bytes, pack_ms = [], 0.0, 256, 0.0
        st = torch.zeros(qf.STATS_WORDS, dtype=torch.int64, device=dev)
        for fp32, grad_scale in layers:
            t = {}
            for name, scale in (("X", 1.0), ("W", 1.0), ("dY", grad_scale)):
                src = fp32[name]
                codes = torch.empty(src.shape, dtype=torch.int16, device=dev)
                f = qf.make_format(e, m, 1, scale)
                qf.qfmt_quantize_stats_pack16(src, codes, src.numel(), f, st)
                pack_ms += statistics.median(time_events(
                    torch, lambda: qf.qfmt_quantize_stats_pack16(src, codes, src.numel(), f, st), 3))
                t[name] = codes
            tokens, d_in = fp32["X"].shape
            d_out = fp32["W"].shape[1]
            for A, ta, B, tb, M, N, K in ((t["X"], False, t["W"], False, tokens, d_out, d_in),
                                          (t["dY"], False, t["W"], True, tokens, d_in, d_out),
                                          (t["X"], True, t["dY"], False, d_in, d_out, tokens)):
                C = torch.empty(M, N, dtype=torch.float32, device=dev)
                jobs.append((qf.make_matrix(A, ta), qf.make_matrix(B, tb), C, N, (A, B)))
                ws_bytes = max(ws_bytes, qf.qfmt_gemm_packed16_workspace_bytes(jobs[-1][0], jobs[-1][1]))
                flops += 2.0 * M * N * K
        ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)

        def step(which=jobs):
            for a, b, C, N, _ in which:
                qf.qfmt_gemm_packed16(a, b, C, N, fmt, ws, ws.numel())
        for _ in range(3):
            step()
        assert qf.qfmt_device_status(ws) == qf.QFMT_OK
        ms = statistics.median(time_events(torch, step, reps))
        tf = flops / ms / 1e9
        # the whole step with codes as the only stored form: per layer X, W and dY are rounded to codes with
        # statistics, the forward product gets Y = R(R(XW) + R(B)) written as codes with statistics, the two
        # gradient products follow; the loss-scale controller reads the gradients' records at the end
        n_layers = len(layers)
        rec = torch.zeros(n_layers, 4, qf.STATS_WORDS, dtype=torch.int64, device=dev)
        grad_rec = torch.zeros(n_layers, qf.STATS_WORDS, dtype=torch.int64, device=dev)
        state = qf.qfmt_dls_t(2.0 ** 16, 2.0, 0.5, 1.0, 2.0 ** 24, 2000, 0, 0, 0, 0, 0)
        d_state = torch.from_numpy(np.frombuffer(bytes(state), dtype=np.uint8).copy()).to(dev)
        extras = []
        for li, (fp32, grad_scale) in enumerate(layers):
            d_out = fp32["W"].shape[1]
            bias = torch.from_numpy(workloads.normal_tensor(workloads.rng_for(4, 2000 + li), (d_out,), 0.02)).to(dev)
            extras.append((bias, torch.empty(fp32["X"].shape[0], d_out, dtype=torch.int16, device=dev),
                           qf.make_format(e, m, 1, grad_scale)))

        def whole_step():
            for li, (fp32, _) in enumerate(layers):
                bias, y_codes, gfmt = extras[li]
                (a0, b0, C0, N0, (cX, cW)), (a1, b1, C1, N1, (cG, _)), (a2, b2, C2, N2, _) = jobs[3 * li:3 * li + 3]
                qf.qfmt_quantize_stats_pack16(fp32["X"], cX, cX.numel(), fmt, rec[li, 0])
                qf.qfmt_quantize_stats_pack16(fp32["W"], cW, cW.numel(), fmt, rec[li, 1])
                qf.qfmt_quantize_stats_pack16(fp32["dY"], cG, cG.numel(), gfmt, grad_rec[li])
                qf.qfmt_gemm_packed16(a0, b0, C0, N0, fmt, ws, ws.numel())
                qf.qfmt_bias_quantize_stats_pack16(C0, N0, bias, y_codes, N0, C0.shape[0], N0, fmt, rec[li, 3])
                qf.qfmt_gemm_packed16(a1, b1, C1, N1, fmt, ws, ws.numel())
                qf.qfmt_gemm_packed16(a2, b2, C2, N2, fmt, ws, ws.numel())
            qf.qfmt_dls_update(d_state, grad_rec, n_layers)
        for _ in range(3):
            whole_step()
        assert qf.qfmt_device_status(ws) == qf.QFMT_OK
        whole_ms = statistics.median(time_events(torch, whole_step, reps))
        del extras
        out["runs"][tag] = {"ms_per_step": ms, "tflops": tf, "rounding_to_codes_ms": pack_ms, "gemms_per_step": len(jobs),
                            "whole_step_ms": whole_ms, "whole_step_gemm_tflops": flops / whole_ms / 1e9,
                            "whole_step_launches": 7 * n_layers + 1,
                            "gpu_launches_per_step": len(jobs),
                            "roofline": {"bound": "tensor", "achieved": tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                                         "frac": tf / peaks["bf16_tflops"], "traffic": None,
                                         "peak_source": f"bf16 {peaks['source']} burst"}}
        del jobs, ws
    first = out["runs"]["1/5/10 binary16"]
    out.update({"value": first["tflops"], "ms_per_step": first["ms_per_step"], "roofline": first["roofline"]})
    return out


# FMAC-8 is plain-ALU work.  Peak = SMs x 4 schedulers x 32 lanes x max SM clock / (scheduler cycles one
# warp-wide multiply-add must cost).  General kernel: per FMAC FMAC8_FLOAT_OPS float-pipe instructions (two
# directed fused multiply-adds, add and subtract of the rounding constant)
# (one per cycle) and FMAC8_INT_OPS integer-pipe instructions (one per two cycles: 16 lanes per
# scheduler), counted in the kernel's inner loop; the bound is the larger of the issue slots and the
# integer pipe.  Native kernel (binary16, bfloat16): one fma.rn.f16x2 / fma.rn.bf16x2 per two FMACs, two cycles each on this part (the
# float pipe's busy cycles are twice its instruction count for a stream of them).
SM_COUNT, LANES_PER_SM = 148, 128
FMAC8_FLOAT_OPS, FMAC8_INT_OPS = 4.0, 6.0


def fmac8_section(torch, qf, dev, peaks, clock_mhz, reps=3):
    """Algorithm 1 (FMAC-8) on the config3 forward product (4096 x 3072 x 768): 1/6/9 on the general
    ALU kernel, 1/5/10 and 1/8/7 on the native 16-bit FMA kernel; output statistics taken in the kernel."""
    cfg = workloads.config3()
    M, K = cfg["X"].shape
    N = cfg["W"].shape[1]
    out = {"metric": "FMAC-8 product TFMAC/s", "unit": "TFMAC/s",
           "workload": f"config3 forward product {M} x {N} x {K}, FMAC-8 accumulation, statistics of the output", "runs": {}}
    clk = clock_mhz * 1e6
    cyc_general = max(FMAC8_FLOAT_OPS + FMAC8_INT_OPS, 2.0 * FMAC8_INT_OPS)
    peaks_t = {"general": SM_COUNT * LANES_PER_SM * clk / cyc_general / 1e12,
               "binary16": SM_COUNT * LANES_PER_SM * clk * 2 / 2.0 / 1e12}
    for tag, e, m, path, kind in (("1/6/9 general", 6, 9, 0, "general"), ("1/5/10 binary16", 5, 10, 0, "binary16"),
                                  ("1/8/7 bfloat16", 8, 7, 0, "binary16")):
        fmt = qf.make_format(e, m, 1)
        X, W = torch.from_numpy(cfg["X"]).to(dev), torch.from_numpy(cfg["W"]).to(dev)
        qf.qfmt_quantize_stats(X, X, X.numel(), fmt)
        qf.qfmt_quantize_stats(W, W, W.numel(), fmt)
        C = torch.empty(M, N, dtype=torch.float32, device=dev)
        st = torch.zeros(qf.STATS_WORDS, dtype=torch.int64, device=dev)
        a, b = qf.make_matrix(X), qf.make_matrix(W)

        def step():
            qf.qfmt_gemm_fmac8(a, b, C, N, fmt, st, 0, path)
        step()
        ms = statistics.median(time_events(torch, step, reps))
        assert int(st.cpu()[256]) == M * N
        tf = M * N * K / ms / 1e9
        out["runs"][tag] = {"ms": ms, "tfmac_per_s": tf, "denormal_fraction_of_output": int(st.cpu()[258]) / (M * N),
                            "roofline": {"bound": "alu", "achieved": tf, "peak": peaks_t[kind], "unit": "TFMAC/s",
                                         "frac": tf / peaks_t[kind], "traffic": None,
                                         "peak_source": "derived: SMs x lanes x max SM clock / cycles per FMAC (see comment)"}}
    # FMAC-8 in a convolution layer: the config4 3x3 layer (batch 128, 256 -> 256 channels at 14 x 14), forward
    sh = workloads.CONV3X3
    cfg4 = workloads.config4(sh)
    g = qf.qfmt_conv_t(sh.n, sh.c_in, sh.h, sh.w, sh.c_out, sh.r, sh.s, sh.pad, sh.pad)
    fmacs = float(sh.n * sh.h * sh.w) * sh.c_out * sh.c_in * sh.r * sh.s
    out["conv"] = {"workload": "config4 3x3 layer forward (25088 x 256 x 2304 as a product), FMAC-8 accumulation, "
                               "channels-last, statistics of the output", "runs": {}}
    for tag, e, m, kind in (("1/6/9 general", 6, 9, "general"), ("1/5/10 binary16", 5, 10, "binary16")):
        fmt = qf.make_format(e, m, 1)
        tensors = []
        for x in (cfg4["X"], cfg4["W"]):
            b_, c_, hh, ww = x.shape
            d_in = torch.from_numpy(x).to(dev)
            d_cl = torch.empty(b_ * hh * ww * c_, dtype=torch.float32, device=dev)
            qf.qfmt_quantize_stats_transpose(d_in, d_cl, b_, c_, hh * ww, fmt)
            tensors.append(d_cl)
        Y = torch.empty(sh.n * sh.h * sh.w * sh.c_out, dtype=torch.float32, device=dev)
        st = torch.zeros(qf.STATS_WORDS, dtype=torch.int64, device=dev)

        def conv_step():
            qf.qfmt_conv_fmac8(qf.QFMT_CONV_FWD, g, tensors[0], tensors[1], Y, fmt, st, 0, 0)
        conv_step()
        ms = statistics.median(time_events(torch, conv_step, reps))
        assert int(st.cpu()[256]) == Y.numel()
        tf = fmacs / ms / 1e9
        out["conv"]["runs"][tag] = {"ms": ms, "tfmac_per_s": tf,
                                    "roofline": {"bound": "alu", "achieved": tf, "peak": peaks_t[kind], "unit": "TFMAC/s",
                                                 "frac": tf / peaks_t[kind], "traffic": None,
                                                 "peak_source": "derived: SMs x lanes x max SM clock / cycles per FMAC (see comment)"}}
    first = out["runs"]["1/6/9 general"]
    out.update({"value": first["tfmac_per_s"], "ms_per_step": first["ms"], "gpu_launches_per_step": 1,
                "roofline": first["roofline"]})
    return out


def run_library(args):
    import torch
    import paper_2103_15940_b200 as qf

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    qf.lib()  # fail loudly if the CUDA library has not been built
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group(backend="nccl", device_id=dev)

    peaks = measured_peaks()
    n = workloads.CONFIG2_N
    runs = workloads.config2_runs()
    x_host = workloads.config2_tensor()
    d_in = torch.from_numpy(x_host).to(dev)
    d_out = torch.empty_like(d_in)
    d_stats = torch.zeros(len(runs), qf.STATS_WORDS, dtype=torch.int64, device=dev)
    fmts = [qf.make_format(e, m, den, s) for _, e, m, den, s in runs]

    def step():
        for i, f in enumerate(fmts):
            qf.qfmt_quantize_stats(d_in, d_out, n, f, d_stats[i], 0)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    launch_ms = []
    barrier()
    with ClockSampler(nvml_index(local_rank)) as clocks:
        t_begin = torch.cuda.Event(enable_timing=True)
        t_end = torch.cuda.Event(enable_timing=True)
        pairs = []
        t_begin.record()
        for _ in range(args.steps):
            for i, f in enumerate(fmts):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                qf.qfmt_quantize_stats(d_in, d_out, n, f, d_stats[i], 0)
                b.record()
                pairs.append((a, b))
        t_end.record()
        barrier()
    total_ms = t_begin.elapsed_time(t_end)
    launch_ms = [a.elapsed_time(b) for a, b in pairs]
    total_ms = max_over_ranks(torch, dist, total_ms, dev)
    step_bytes = len(runs) * n * BYTES_PER_ELEMENT
    value = whole_job_value(world, args.steps, step_bytes, total_ms)

    # sanity: the timed kernels did the work (denormal counts of the last step are plausible)
    st = d_stats.cpu().numpy().view(np.uint64)
    assert int(st[0, 256]) == n and int(st[:, 258].max()) > 0

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (quantize+stats): algorithmic bytes / mean launch time
    mean_launch_ms = statistics.mean(launch_ms)
    achieved = n * BYTES_PER_ELEMENT / mean_launch_ms / 1e6
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH,
                "peak_source": f"copy bandwidth, {peaks['source']}", "algorithmic_bytes_per_launch": n * BYTES_PER_ELEMENT,
                "mean_launch_us": 1e3 * mean_launch_ms, "nominal_hbm_gbs": 7700.0, "frac_of_nominal": achieved / 7700.0}

    sections = set(args.sections.split(","))
    e2e = gemm = cpu = conv = None
    extra = {}
    if "epilogue" in sections:
        extra["epilogue"] = epilogue_section(torch, qf, dev, peaks)
    if "config13" in sections:
        extra.update(config13_section(torch, qf, dev, peaks))
    if "step5" in sections:
        extra["step5"] = step5_section(torch, qf, dev, peaks)
    if "pack16" in sections:
        extra["pack16"] = pack16_section(torch, qf, dev, peaks, d_in, n)
    if "gemm16" in sections:
        extra["gemm16"] = gemm16_section(torch, qf, dev, peaks)
    if "fmac8" in sections:
        extra["fmac8"] = fmac8_section(torch, qf, dev, peaks, clocks.summary()["sm_max_mhz"] or 1965)
    if "e2e" in sections:
        e2e = e2e_section(torch, qf, dev, x_host, fmts, n, step_bytes, args)
    if "gemm" in sections:
        gemm = gemm_section(torch, qf, dev, peaks)
    if "conv" in sections:
        conv = conv_section(torch, qf, dev, peaks)
    if "cpu" in sections:
        # the CPU oracle on this machine's host cores: one thread on a quarter of the tensor, and every core
        # (pieces in parallel, records summed) on the whole tensor
        n_cpu = 1 << 24
        cpu_secs = oracle_sweep(x_host[:n_cpu])
        cpu_value = len(runs) * n_cpu * BYTES_PER_ELEMENT / cpu_secs / 1e9
        cores = os.cpu_count() or 1
        all_secs = oracle_sweep(x_host, threads=cores)
        cpu = {"value": cpu_value, "unit": UNIT, "cores": 1, "kind": "oracle", "seconds": cpu_secs,
               "host_cores_available": cores,
               "sample": f"the 18 sweep runs on the first {n_cpu} of {n} elements",
               "all_cores": {"value": len(runs) * n * BYTES_PER_ELEMENT / all_secs / 1e9, "unit": UNIT, "cores": cores,
                             "kind": "oracle", "seconds": all_secs,
                             "sample": f"the 18 sweep runs on all {n} elements, {cores} pieces in parallel"}}
    return finish(args, world, value, total_ms, n, runs, clocks, e2e, roofline, cpu, gemm, conv, dist, extra)


def e2e_section(torch, qf, dev, x_host, fmts, n, step_bytes, args):
    """End to end through the host-buffer entry point (pinned host memory, copies timed)."""
    runs = fmts
    h_in = torch.from_numpy(x_host).pin_memory()
    h_out = torch.empty(n, dtype=torch.float32).pin_memory()
    h_stats = torch.zeros(qf.STATS_WORDS, dtype=torch.int64).pin_memory()
    wb = qf.qfmt_quantize_stats_host_work_bytes(n)
    d_work = torch.empty(wb, dtype=torch.uint8, device=dev)
    e2e_steps = max(1, min(args.steps, 2))
    qf.qfmt_quantize_stats_host(h_in, h_out, n, fmts[0], h_stats, d_work, wb)
    e2e_ms = time_events(torch, lambda: [qf.qfmt_quantize_stats_host(h_in, h_out, n, f, h_stats, d_work, wb)
                                         for f in fmts], e2e_steps)
    e2e_value = step_bytes / statistics.mean(e2e_ms) / 1e6
    e2e = {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": len(runs) * n * 4,
           "d2h_bytes_per_step": len(runs) * (n * 4 + qf.STATS_WORDS * 8), "steps": e2e_steps}
    del d_work, h_in, h_out
    return e2e


def finish(args, world, value, total_ms, n, runs, clocks, e2e, roofline, cpu, gemm, conv, dist, extra):
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u32", "data": "synthetic",
            "config": {"workload": "config2 format sweep: 64 Mi fp32 elements x 18 (format, denormal mode, loss scale) runs",
                       "elements": n, "runs_per_step": len(runs), "l2": "inputs larger than L2 (256 MiB in, 256 MiB out)",
                       "multi_gpu": "replicas only: every rank runs the whole sweep on its own copy"},
            "clocks": clocks.summary(), "e2e": e2e, "gpu_launches": args.steps * len(runs),
            "roofline": roofline, "cpu_baseline": cpu, "gemm": gemm, "conv": conv}
    line.update(extra)
    # The metric has two halves.  The contraction half (and the other tensor-bound workloads) is repeated
    # inside `roofline` and `cpu_baseline`, next to the rounding pass's own figures.
    def brief(section):
        r = section["roofline"]
        keep = {k: r[k] for k in ("bound", "achieved", "peak", "unit", "frac", "peak_source", "frac_of_sustained",
                                  "library_tf32_same_run", "frac_of_library_tf32", "frac_of_nominal") if k in r}
        keep["workload"] = section["workload"]
        return keep
    if gemm is not None:
        roofline["gemm"] = brief(gemm)
        if cpu is not None:
            cpu["gemm"] = gemm["cpu_baseline"]
    if conv is not None:
        roofline["conv"] = brief(conv)
    if "config3" in line:
        roofline["config3"] = brief(line["config3"])
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


# dram__bytes_read.sum + dram__bytes_write.sum per launch of the quantize+stats kernel on the 64 Mi-element
# tensor, from one ncu capture of that kernel (read + write).  A figure here belongs to the kernel as it was
# when the counters were taken: it is set to None as soon as that kernel's code changes, until re-taken.
NCU_TRAFFIC_BYTES_PER_LAUNCH = 268463872 + 218982144
# the same for the layer-output kernel on the 8192 x 4096 product
NCU_EPILOGUE_TRAFFIC_BYTES_PER_LAUNCH = 134294528 + 84735232


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="library", choices=["library", "reference"])
    ap.add_argument("--sections", default="quantize,e2e,gemm,conv,config13,epilogue,step5,pack16,gemm16,fmac8,cpu",
                    help="comma list of what to measure besides the timed sweep (quantize is always timed): "
                         "e2e, gemm, conv, config13, epilogue, step5, pack16, fmac8, cpu; profiling captures use a subset")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_library(args)


if __name__ == "__main__":
    main()
