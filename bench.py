#!/usr/bin/env python
"""Benchmark of the fused Gated MLP (libgmlp) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--shard rows|dff] [--no-extra]
    python bench.py --impl reference ...          # times the CPU oracle on the host cores

One "step" is one pass of the whole hot path (optional RMSNorm, gate/up GEMM with the SiLU
product epilogue, down GEMM) over one batch of synthetic, seeded input.  Rank 0 prints ONE
JSON line.  ``value`` is whole-job tokens/s with the inputs resident in HBM; ``e2e`` is the
same metric through the host-buffer entry point (host->device copy of X and device->host
copy of Y inside the timed region).  The line also carries the roofline of the dominant
kernel (measured with CUDA events around that kernel), the CPU oracle timed on the host
cores, the SM clocks sampled during the timed region, and, unless --no-extra, the same
measurements for every other stated workload under "workloads", with a compact "summary"
of all of them as the last key.

The primary workload is the largest stated single-GPU configuration (the 70B-shaped prefill).
A region of exactly K steps is timed between a barrier + synchronize on both sides; it is
repeated until about half a second of steps has run and the median region is reported (min
and max beside it), so that the number belongs to the clock the GPU settles at under load.

With N > 1 the script starts N ranks itself (or runs under torchrun when that set
WORLD_SIZE).  --shard rows (default): every rank runs the same workload on its own rows (rows
are independent, weights replicated, no collective on the data path): weak scaling.
--shard dff: d_ff is cut over the ranks (per-GPU weight bytes fall as 1 / N), each rank
computes an fp32 partial product and the ranks exchange ONE all-reduce of M x d_model
floats per step: strong scaling, the cut that helps a handful of tokens.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

PRIMARY = "llama3-70b-prefill-M4096-outliers"
PRIMARY_DFF = "llama3-8b-decode-M8"             # default workload of --shard dff
# every stated configuration (decode first), then one unstated mid-M shape of the 8B layer
STATED = ["llama3-8b-decode-M8", "llama3-8b-prefill-M2048-rmsnorm", "llama3-70b-prefill-M4096-outliers",
          "ragged-M1-plain", "ragged-M7-plain", "ragged-M129-plain", "ragged-M1000-plain", "ragged-M8192-plain",
          "ragged-M1-norm", "ragged-M7-norm", "ragged-M129-norm", "ragged-M1000-norm", "ragged-M8192-norm", "tiny"]
UNSTATED = ["llama3-8b-batch-M64"]
L2_BYTES = 126 * 1024 * 1024
NOMINAL = {"bf16_tflops": 2250.0, "hbm_gbs": 8000.0}       # dense bf16 peak and "about 8 TB/s": the stated targets' denominators
MIN_TIMED_S = 0.5                                            # steps timed per workload, all regions together
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu captures
# summarised under profiles/ (skinny_cluster_gemm_decode_M8.md, umma_pair_gemm_chunked_prefill8b_M2048.md,
# bench_prefill70b_launch_list.md; the M = 64 figure from the same two-counter capture as the decode one)
NCU_TRAFFIC_BYTES = {
    ("llama3-8b-decode-M8", "gate_up"): 235.0e6 + 3.2e6,
    ("llama3-8b-prefill-M2048-rmsnorm", "gate_up"): 256.8e6 + 52.6e6,
    ("llama3-70b-prefill-M4096-outliers", "gate_up"): 3966.1e6 + 233.4e6,     # captured at full size (row tiles in groups of eight)
    ("llama3-8b-batch-M64", "gate_up"): 235.5e6 + 3.1e6,
    # the small-M schedule's one-kernel form: the weights, read once (the partial Y stay in L2 for the kernel that adds them)
    ("ragged-M7-plain", "fused"): 69.31e6 + 0.47e6,
    ("ragged-M7-norm", "fused"): 69.31e6 + 0.47e6,
    ("ragged-M1-plain", "fused"): 69.28e6 + 0.42e6,
    ("ragged-M1-norm", "fused"): 69.28e6 + 0.42e6,
}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons in the background during a timed region."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def cpu_oracle_rate(inp, rows, min_seconds: float):
    """Times the oracle as it stands on `rows`, repeating whole passes until min_seconds have elapsed."""
    import oracle
    w = inp.workload
    args = (inp.bits("X"), inp.bits("Wg"), inp.bits("Wu"), inp.bits("Wd"))
    kw = dict(rows=rows, gamma=inp.bits("gamma") if w.rmsnorm else None, eps=w.eps, rmsnorm=w.rmsnorm)
    oracle.build()
    done, t0 = 0, time.perf_counter()
    while True:
        oracle.gmlp_rows(*args, **kw)
        done += len(rows)
        dt = time.perf_counter() - t0
        if dt >= min_seconds:
            break
    return done / dt, done, dt, oracle.max_threads()


def run_reference(args):
    """--impl reference: the CPU oracle, as it stands, on the host cores; one step = one bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2606_26344_b200 import inputs as I
    w = I.WORKLOADS[args.workload or PRIMARY]
    inp = I.make_inputs(w)
    rows = I.sample_rows(w, inp.outlier_rows)
    n_rows = min(len(rows), 8)
    rows = rows[:n_rows]
    X, Wg, Wu, Wd = (inp.bits(n) for n in ("X", "Wg", "Wu", "Wd"))
    kw = dict(rows=rows, gamma=inp.bits("gamma") if w.rmsnorm else None, eps=w.eps, rmsnorm=w.rmsnorm)
    oracle.build()
    for _ in range(args.warmup):
        oracle.gmlp_rows(X, Wg, Wu, Wd, **kw)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.gmlp_rows(X, Wg, Wu, Wd, **kw)
    dt = time.perf_counter() - t0
    value = n_rows * args.steps / dt
    cores = oracle.max_threads()
    sample = f"{n_rows} rows of the workload per step (rows are independent), fp64, OpenMP over rows"
    print(json.dumps({
        "impl": "reference", "metric": "gated_mlp_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "M": w.M, "d_model": w.d_model, "d_ff": w.d_ff, "rmsnorm": w.rmsnorm},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def fractions(w, ms, peaks):
    """Roofline of the whole path: the slower of the FLOPs at the bf16 peak and the algorithmic bytes at the HBM
    bandwidth, against the measured peaks (burst and, for a tensor-bound shape, sustained) and the nominal ones."""
    t = ms * 1e-3
    t_tensor = w.flops / (peaks["bf16_tflops"] * 1e12)
    t_hbm = w.min_bytes / (peaks["hbm_gbs"] * 1e9)
    bound = "tensor" if t_tensor >= t_hbm else "hbm"
    out = {"bound": bound, "frac": max(t_tensor, t_hbm) / t,
           "frac_nominal": max(w.flops / (NOMINAL["bf16_tflops"] * 1e12), w.min_bytes / (NOMINAL["hbm_gbs"] * 1e9)) / t,
           "denominators": f"frac: measured {peaks['bf16_tflops']} TFLOP/s burst, {peaks['hbm_gbs']} GB/s copy ({peaks['source']}); "
                           f"frac_nominal: {NOMINAL['bf16_tflops']} TFLOP/s, {NOMINAL['hbm_gbs']} GB/s"}
    if bound == "tensor":
        out["frac_sustained"] = w.flops / (peaks["bf16_tflops_sustained"] * 1e12) / t
    return out


def timed_regions(run_step, steps, barrier, stream, est_ms, max_regions=40):
    """Regions of exactly `steps` steps, each between a barrier + synchronize on both sides and its own pair of
    events, repeated until MIN_TIMED_S of steps have run (at least three regions).  Returns the per-step time of
    every region, in milliseconds."""
    import torch
    n = max(3, min(max_regions, int(math.ceil(MIN_TIMED_S * 1e3 / max(est_ms * steps, 1e-6)))))
    out = []
    k = 0
    for _ in range(n):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            run_step(k)
            k += 1
        e1.record(stream)
        barrier()
        out.append(e0.elapsed_time(e1) / steps)
    return out


def measure_workload(w, steps, warmup, dev, peaks, dist=None, want_e2e=True, sample_clocks=True, clock_roll=0.6,
                     autotune=False, exact_steps=True):
    """Times one workload on this rank's GPU.  `exact_steps`: regions of exactly `steps` steps (the primary line);
    otherwise a region is stretched to about 0.1 s of steps."""
    import torch
    from paper_2606_26344_b200 import gmlp, inputs as I

    inp = I.make_inputs(w)
    X, Wg, Wu, Wd = (t.to(dev) for t in (inp.X, inp.Wg, inp.Wu, inp.Wd))
    gamma = inp.gamma.to(dev) if inp.gamma is not None else None
    Y = torch.empty_like(X)
    stream = torch.cuda.current_stream(dev)
    tuned = None
    if autotune:
        # empirical schedule selection on this shape first (library-owned workspace), then AUTO follows it
        gmlp.autotune(gmlp.make_args(X, Wg, Wu, Wd, Y, gamma, w.eps, w.rmsnorm, gmlp.VARIANT_AUTO, None, stream), 20)
        tuned = gmlp.autotune_query(w.M, w.d_model, w.d_ff)
    variant = gmlp.pick_variant(w.M, w.d_model, w.d_ff)
    ws = gmlp.alloc_workspace(w.M, w.d_model, w.d_ff, w.rmsnorm)
    a = gmlp.make_args(X, Wg, Wu, Wd, Y, gamma, w.eps, w.rmsnorm, gmlp.VARIANT_AUTO, ws, stream)
    weight_bytes = 3 * w.d_model * w.d_ff * 2
    fits_l2 = weight_bytes < L2_BYTES
    flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev) if fits_l2 else None

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    # Weights that would stay in L2 are timed cold: several copies of the weights are used in rotation, enough that a
    # copy has left L2 before its turn comes again (2.5 x L2 of other weights pass in between), steps back to back
    # like the large workloads - programmatic dependent launch overlaps a step's launch and ramp with its
    # predecessor's tail, as in a model that runs layer after layer.
    rot, keep = [a], []
    if fits_l2:
        n_sets = int(-(-2.5 * L2_BYTES // weight_bytes)) + 1
        for _ in range(n_sets - 1):
            wg, wu, wd = Wg.clone(), Wu.clone(), Wd.clone()
            keep.append((wg, wu, wd))
            rot.append(gmlp.make_args(X, wg, wu, wd, Y, gamma, w.eps, w.rmsnorm, gmlp.VARIANT_AUTO, ws, stream))
    n_sets = len(rot)

    def run_step(k):
        gmlp.forward_ex(rot[k % n_sets])

    for k in range(max(warmup, 2 * n_sets)):
        run_step(k)
    torch.cuda.synchronize(dev)
    st = gmlp.device_status()
    if st != 0:
        raise RuntimeError(f"device status {st:#x} after warm-up")
    t0 = time.perf_counter()
    for k in range(10):
        run_step(k)
    torch.cuda.synchronize(dev)
    est_ms = (time.perf_counter() - t0) * 1e3 / 10

    # The clocks are sampled over an untimed pre-roll of the same steps (which also brings the GPU to the power state
    # it holds under this load), every timed region, and a short post-roll: one stretch of identical load.
    sampler = ClockSampler(dev.index or 0) if (sample_clocks and clock_roll > 0) else None

    def roll(seconds):
        t_end = time.perf_counter() + seconds
        k = 0
        while time.perf_counter() < t_end:
            for _ in range(20):
                run_step(k)
                k += 1
            torch.cuda.synchronize(dev)

    if sampler:
        sampler.start()
        roll(clock_roll)
    region_steps = steps if exact_steps else max(steps, int(math.ceil(100.0 / max(est_ms, 1e-3))))
    gmlp.reset_launch_count()
    run_step(0)
    launches_per_step = gmlp.launch_count()
    per_step = timed_regions(run_step, region_steps, barrier, stream, est_ms)
    ms = statistics.median(per_step)
    isolated_ms = None
    if fits_l2:
        # the same step alone: L2 overwritten before it, one pair of events around it (launch latency and ramp exposed)
        iso = []
        for _ in range(10):
            flush.fill_(1)
            i0, i1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            i0.record(stream)
            gmlp.forward_ex(a)
            i1.record(stream)
            iso.append((i0, i1))
        torch.cuda.synchronize(dev)
        isolated_ms = sum(x.elapsed_time(y) for x, y in iso) / len(iso)
    if sampler:
        roll(min(clock_roll, 0.2))
    clocks = sampler.stop() if sampler else None
    if clocks is not None:
        clocks["window"] = f"pre-roll {clock_roll} s + the timed regions + post-roll of the same steps"

    # per-kernel durations, in a loop of their own (an event between two kernels stops the second from
    # overlapping the first's tail, so these are stand-alone kernel times, like a profiler's)
    n_prof = max(3, min(int(math.ceil(150.0 / max(est_ms, 1e-3))), 50))
    if flush is None:
        for _ in range(3):
            gmlp.forward_ex(a)
        gmlp.profile_enable(True)
        for _ in range(n_prof):
            gmlp.forward_ex(a)
        kern_ms = gmlp.profile_read()
    else:
        acc = {}
        for _ in range(min(n_prof, 20)):
            gmlp.profile_enable(True)
            flush.fill_(1)
            gmlp.forward_ex(a)
            for k, v in gmlp.profile_read().items():
                acc.setdefault(k, []).append(v)
        kern_ms = {k: sum(v) / len(v) for k, v in acc.items()}
    gmlp.profile_enable(False)

    res = {"name": w.name, "M": w.M, "d_model": w.d_model, "d_ff": w.d_ff, "rmsnorm": w.rmsnorm,
           "variant": {1: "simt", 2: "stream", 3: "umma", 4: "skinny", 5: "pair", 6: "tensor", 7: "fused"}.get(variant, str(variant)),
           "ms_per_step": ms, "ms_min": min(per_step), "ms_max": max(per_step), "regions": len(per_step),
           "steps_per_region": region_steps, "tokens_per_s": w.M / (ms * 1e-3), "tflops": w.flops / (ms * 1e-3) / 1e12,
           "gbps_min_bytes": w.min_bytes / (ms * 1e-3) / 1e9, "launches": launches_per_step * region_steps, "clocks": clocks,
           "kernel_ms": kern_ms,
           "l2": f"weights fit L2: {n_sets} copies in rotation, steps back to back" if fits_l2
                 else "inputs larger than L2; steps back to back"}
    if tuned is not None:
        res["autotuned"] = {"variant": tuned[0], "gate_up_pair": tuned[1], "down_pair": tuned[2]}
    if isolated_ms is not None:
        res["ms_step_alone"] = isolated_ms      # L2 overwritten before the step, events around that one step
    res["roofline_path"] = fractions(w, ms, peaks)

    # roofline of the dominant kernel (gate/up: two thirds of the FLOPs and of the weight bytes)
    if "gate_up" in kern_ms:
        kms = kern_ms["gate_up"] * 1e-3
        if res["roofline_path"]["bound"] == "tensor":
            flops = 4 * w.M * w.d_model * w.d_ff
            ach = flops / kms / 1e12
            # a kernel timed inside a long run of steps under the power cap is held against the sustained figure
            long_run = est_ms * n_prof > 100.0
            peak = peaks["bf16_tflops_sustained"] if long_run else peaks["bf16_tflops"]
            res["roofline"] = {"kernel": "gate_up", "bound": "tensor", "achieved": ach, "peak": peak,
                               "unit": "TFLOP/s", "frac": ach / peak, "frac_burst": ach / peaks["bf16_tflops"],
                               "frac_nominal": ach / NOMINAL["bf16_tflops"],
                               "traffic": NCU_TRAFFIC_BYTES.get((w.name, "gate_up")), "algorithmic_flops": flops,
                               "peak_source": peaks["source"] + (" (sustained bf16: the kernel is timed inside a long run)"
                                                                 if long_run else " (burst bf16)")}
        else:
            nbytes = 2 * (2 * w.d_model * w.d_ff + w.M * w.d_model + w.M * w.d_ff)
            ach = nbytes / kms / 1e9
            res["roofline"] = {"kernel": "gate_up", "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"],
                               "unit": "GB/s", "frac": ach / peaks["hbm_gbs"], "frac_nominal": ach / NOMINAL["hbm_gbs"],
                               "traffic": NCU_TRAFFIC_BYTES.get((w.name, "gate_up")), "algorithmic_bytes": nbytes,
                               "peak_source": peaks["source"] + " (copy)"}

    elif "fused" in kern_ms:
        # the small-M schedule's one-kernel form: all three weight matrices stream through one kernel, which also writes
        # the slices' partial Y (fp32); the sum over the slices is a second, tiny kernel
        kms = kern_ms["fused"] * 1e-3
        slices = (w.d_ff + 127) // 128
        nbytes = 2 * (3 * w.d_model * w.d_ff + w.M * w.d_model) + 4 * slices * w.M * w.d_model
        ach = nbytes / kms / 1e9
        res["roofline"] = {"kernel": "fused", "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"],
                           "unit": "GB/s", "frac": ach / peaks["hbm_gbs"], "frac_nominal": ach / NOMINAL["hbm_gbs"],
                           "traffic": NCU_TRAFFIC_BYTES.get((w.name, "fused")), "algorithmic_bytes": nbytes,
                           "peak_source": peaks["source"] + " (copy)"}

    if "roofline" in res and not fits_l2 and res["roofline"]["bound"] == "hbm":
        # The same kernel in a chain of its own launches: programmatic dependent launch overlaps a launch's ramp with
        # its predecessor's tail, as it does inside the timed steps, so this is the kernel's rate in steady state
        # (the figure above is one launch between two events, like a profiler's).  Two events around the loop; the
        # RMSNorm prologue, a kernel of its own, is left out.
        Hc = torch.empty(w.M, w.d_ff, dtype=torch.bfloat16, device=dev)
        n_chain = max(20, min(steps, 100))
        for _ in range(5):
            gmlp.gate_up(X, Wg, Wu, Hc, stream=stream)
        torch.cuda.synchronize(dev)
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record(stream)
        for _ in range(n_chain):
            gmlp.gate_up(X, Wg, Wu, Hc, stream=stream)
        c1.record(stream)
        torch.cuda.synchronize(dev)
        chain_ms = c0.elapsed_time(c1) / n_chain
        r = res["roofline"]
        ach_c = r["algorithmic_bytes"] / (chain_ms * 1e-3) / 1e9
        r["chained"] = {"achieved": ach_c, "frac": ach_c / r["peak"], "ms_per_launch": chain_ms, "launches": n_chain,
                        "how": "launches of this kernel back to back on one stream, two events around the loop"}
        del Hc

    if want_e2e:
        # End to end through the host-buffer entry point: every step copies its X from pinned host memory and its Y
        # back.  Two lanes (stream + staging buffers + workspace each) alternate, so that a step's copies overlap the
        # other lane's kernels, as a server with two batches in flight would run it.
        lanes = []
        for _ in range(2):
            st_l = torch.cuda.Stream(device=dev)
            Xs, Ys = torch.empty_like(X), torch.empty_like(X)
            ws_l = gmlp.alloc_workspace(w.M, w.d_model, w.d_ff, w.rmsnorm)
            lanes.append({"stream": st_l, "Xh": inp.X.clone().pin_memory(), "Yh": torch.empty_like(inp.X).pin_memory(),
                          "keep": (Xs, Ys, ws_l),
                          "args": gmlp.make_args(Xs, Wg, Wu, Wd, Ys, gamma, w.eps, w.rmsnorm, gmlp.VARIANT_AUTO, ws_l, st_l)})
        # the same regime as the resident number: an untimed pre-roll of the same host-buffer steps, then at least
        # MIN_TIMED_S of them between the two events
        n_e2e = max(4, steps, int(math.ceil(MIN_TIMED_S * 1e3 / max(ms, 1e-3))))
        n_e2e = min(n_e2e, 20000)
        for i in range(max(6, int(math.ceil(clock_roll * 1e3 / max(ms, 1e-3))))):
            ln = lanes[i % 2]
            gmlp.forward_host(ln["args"], ln["Xh"], ln["Yh"])
        barrier()
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        t0.record(stream)
        for ln in lanes:
            ln["stream"].wait_event(t0)
        for i in range(n_e2e):
            ln = lanes[i % 2]
            gmlp.forward_host(ln["args"], ln["Xh"], ln["Yh"])
        for ln in lanes:
            done = torch.cuda.Event()
            done.record(ln["stream"])
            stream.wait_event(done)
        t1.record(stream)
        barrier()
        e2e_ms = t0.elapsed_time(t1) / n_e2e
        nb = w.M * w.d_model * 2
        res["e2e"] = {"value": w.M / (e2e_ms * 1e-3), "unit": "tokens/s", "ms_per_step": e2e_ms,
                      "h2d_bytes_per_step": nb, "d2h_bytes_per_step": nb, "steps": n_e2e, "lanes": 2}
    del keep
    res["_inputs"] = inp
    return res


def measure_dff_sharded(w, steps, warmup, dev, peaks, dist, rank, world, clock_roll=0.6):
    """--shard dff: this rank holds columns [a, b) of W_gate / W_up and rows [a, b) of W_down.  A step is the rank's
    fp32 partial product (one call of the library), ONE all-reduce of M x d_model floats over the ranks, and the
    single rounding to bf16 (gmlp_sum_partials).  Every rank ends with the whole Y."""
    import torch
    from paper_2606_26344_b200 import gmlp, inputs as I, sharding

    inp = I.make_inputs(w)
    a0, a1 = sharding.dff_range(w.d_ff, rank, world)
    X = inp.X.to(dev)
    Wg, Wu = inp.Wg[:, a0:a1].contiguous().to(dev), inp.Wu[:, a0:a1].contiguous().to(dev)
    Wd = inp.Wd[a0:a1].contiguous().to(dev)
    gamma = inp.gamma.to(dev) if inp.gamma is not None else None
    stream = torch.cuda.current_stream(dev)
    P = torch.zeros(w.M, w.d_model, dtype=torch.float32, device=dev)
    Y = torch.empty_like(X)
    use_dist = dist if world > 1 else None

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    def run_step(_k):
        sharding.forward_dff_sharded(X, Wg, Wu, Wd, use_dist, gamma, w.eps, w.rmsnorm, stream, P=P, Y=Y)

    for k in range(max(warmup, 3)):
        run_step(k)
    torch.cuda.synchronize(dev)
    t0 = time.perf_counter()
    for k in range(10):
        run_step(k)
    torch.cuda.synchronize(dev)
    est_ms = (time.perf_counter() - t0) * 1e3 / 10
    sampler = ClockSampler(dev.index or 0) if clock_roll > 0 else None
    if sampler:
        sampler.start()
        t_end = time.perf_counter() + clock_roll
        while time.perf_counter() < t_end:
            for k in range(20):
                run_step(k)
            torch.cuda.synchronize(dev)
    gmlp.reset_launch_count()
    run_step(0)
    launches_per_step = gmlp.launch_count()
    per_step = timed_regions(run_step, steps, barrier, stream, est_ms)
    clocks = sampler.stop() if sampler else None
    ms = statistics.median(per_step)
    # end to end: X from pinned host memory on every rank, Y back to the host on rank 0
    Xh, Yh = inp.X.clone().pin_memory(), torch.empty_like(inp.X).pin_memory()
    n_e2e = max(4, min(steps, 50))
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for k in range(n_e2e):
        X.copy_(Xh, non_blocking=True)
        run_step(k)
        if rank == 0:
            Yh.copy_(Y, non_blocking=True)
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1) / n_e2e
    nb = w.M * w.d_model * 2
    return {"ms_per_step": ms, "ms_min": min(per_step), "ms_max": max(per_step), "regions": len(per_step),
            "launches": launches_per_step * steps, "clocks": clocks, "slice": [a0, a1],
            "allreduce_bytes": w.M * w.d_model * 4 if world > 1 else 0,
            "weight_bytes_per_gpu": 3 * w.d_model * (a1 - a0) * 2,
            "e2e": {"ms_per_step": e2e_ms, "unit": "tokens/s", "h2d_bytes_per_step": nb, "d2h_bytes_per_step": nb},
            "_inputs": inp}


def measure_rmsnorm_matmul(dev, sizes=(2048, 4096, 8192), iters=10):
    """RMSNorm+MatMul over the paper's {2K,4K,8K}^3 sweep: rewritten schedule (row scale in the GEMM epilogue, RMS
    branch overlapped) against the unfused one (RMSNorm kernel, then GEMM).  Times in microseconds, CUDA events."""
    import math
    import torch
    from paper_2606_26344_b200 import gmlp
    g = torch.Generator(device="cpu").manual_seed(0)
    rows = []
    for M in sizes:
        for K in sizes:
            X = torch.randn(M, K, generator=g).bfloat16().to(dev)
            for N in sizes:
                W = (torch.randn(K, N, generator=g) * K ** -0.5).bfloat16().to(dev)
                Z = torch.empty(M, N, dtype=torch.bfloat16, device=dev)
                t = {}
                for name, unf in (("rewritten", False), ("unfused", True)):
                    for _ in range(3):
                        gmlp.rmsnorm_matmul(X, W, Z, unfused=unf)
                    torch.cuda.synchronize(dev)
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    for _ in range(iters):
                        gmlp.rmsnorm_matmul(X, W, Z, unfused=unf)
                    e1.record()
                    torch.cuda.synchronize(dev)
                    t[name] = e0.elapsed_time(e1) / iters * 1e3
                rows.append({"M": M, "K": K, "N": N, "rewritten_us": t["rewritten"], "unfused_us": t["unfused"],
                             "speedup": t["unfused"] / t["rewritten"],
                             "rewritten_tflops": 2.0 * M * K * N / t["rewritten"] / 1e6})
                del W, Z
            del X
    sp = [r["speedup"] for r in rows]
    return {"shapes": "{2K,4K,8K}^3 as MxKxN", "timing": "back-to-back calls, operands may stay in L2",
            "geomean_speedup_rewritten_over_unfused": math.exp(sum(math.log(v) for v in sp) / len(sp)),
            "min_speedup": min(sp), "max_speedup": max(sp),
            "best_rewritten_tflops": max(r["rewritten_tflops"] for r in rows), "table": rows}


def measure_matmul_add_rmsnorm(dev, sizes=(2048, 4096, 8192), iters=10):
    """MatMul+Add+RMSNorm over the paper's {2K,4K,8K}^3 sweep: fused schedule (residual and sum of squares in the
    GEMM epilogue, light normalise pass) against the three operators run one after the other.  Microseconds."""
    import math
    import torch
    from paper_2606_26344_b200 import gmlp
    g = torch.Generator(device="cpu").manual_seed(0)
    rows = []
    for M in sizes:
        for K in sizes:
            X = torch.randn(M, K, generator=g).bfloat16().to(dev)
            for N in sizes:
                W = (torch.randn(K, N, generator=g) * K ** -0.5).bfloat16().to(dev)
                R = torch.randn(M, N, generator=g).bfloat16().to(dev)
                gam = (0.5 + torch.rand(N, generator=g)).bfloat16().to(dev)
                S, Z = torch.empty_like(R), torch.empty_like(R)
                t = {}
                for name, unf in (("fused", False), ("unfused", True)):
                    ws = gmlp.mmaddnorm_workspace(M, N, unf, dev)
                    a = gmlp.make_mmaddnorm_args(X, W, R, S, Z, gam, 1e-5, unf, ws)
                    for _ in range(3):
                        gmlp.matmul_add_rmsnorm_ex(a)
                    torch.cuda.synchronize(dev)
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    for _ in range(iters):
                        gmlp.matmul_add_rmsnorm_ex(a)
                    e1.record()
                    torch.cuda.synchronize(dev)
                    t[name] = e0.elapsed_time(e1) / iters * 1e3
                    del ws
                rows.append({"M": M, "K": K, "N": N, "fused_us": t["fused"], "unfused_us": t["unfused"],
                             "speedup": t["unfused"] / t["fused"], "fused_tflops": 2.0 * M * K * N / t["fused"] / 1e6})
                del W, R, S, Z
            del X
    sp = [r["speedup"] for r in rows]
    return {"shapes": "{2K,4K,8K}^3 as MxKxN", "timing": "back-to-back calls, operands may stay in L2",
            "geomean_speedup_fused_over_unfused": math.exp(sum(math.log(v) for v in sp) / len(sp)),
            "min_speedup": min(sp), "max_speedup": max(sp),
            "best_fused_tflops": max(r["fused_tflops"] for r in rows), "table": rows}


def measure_qkv(dev, iters=10):
    """QKV projection on grouped-query attention shapes: one launch over the three weight matrices against three
    GEMM launches.  Microseconds, CUDA events."""
    import math
    import torch
    from paper_2606_26344_b200 import gmlp
    g = torch.Generator(device="cpu").manual_seed(0)
    rows = []
    for (K, Nq, Nkv, label) in ((2048, 2048, 512, "2048-wide, 4:1 groups"), (4096, 4096, 1024, "8B attention block"),
                                (8192, 8192, 1024, "70B attention block")):
        Ws = [(torch.randn(K, n, generator=g) * K ** -0.5).bfloat16().to(dev) for n in (Nq, Nkv, Nkv)]
        for M in (128, 512, 2048, 4096, 8192):
            X = torch.randn(M, K, generator=g).bfloat16().to(dev)
            Q = torch.empty(M, Nq, dtype=torch.bfloat16, device=dev)
            Ko, V = (torch.empty(M, Nkv, dtype=torch.bfloat16, device=dev) for _ in range(2))
            t = {}
            for name, sep in (("fused", False), ("separate", True)):
                a = gmlp.make_qkv_args(X, Ws[0], Ws[1], Ws[2], Q, Ko, V, sep)
                for _ in range(3):
                    gmlp.qkv_proj_ex(a)
                torch.cuda.synchronize(dev)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(iters):
                    gmlp.qkv_proj_ex(a)
                e1.record()
                torch.cuda.synchronize(dev)
                t[name] = e0.elapsed_time(e1) / iters * 1e3
            rows.append({"shape": label, "M": M, "K": K, "Nq": Nq, "Nkv": Nkv, "fused_us": t["fused"],
                         "separate_us": t["separate"], "speedup": t["separate"] / t["fused"],
                         "fused_tflops": 2.0 * M * K * (Nq + 2 * Nkv) / t["fused"] / 1e6})
            del X, Q, Ko, V
        del Ws
    sp = [r["speedup"] for r in rows]
    return {"timing": "back-to-back calls, operands may stay in L2",
            "geomean_speedup_fused_over_separate": math.exp(sum(math.log(v) for v in sp) / len(sp)),
            "min_speedup": min(sp), "max_speedup": max(sp),
            "best_fused_tflops": max(r["fused_tflops"] for r in rows), "table": rows}


def measure_gqa(dev, peaks, iters=10):
    """Group Query Attention forward (no mask, head dimension 128) on grouped-query blocks; 4*M*S*D*Hq flops."""
    import torch
    from paper_2606_26344_b200 import gmlp
    g = torch.Generator(device="cpu").manual_seed(0)
    rows = []
    for (Hq, Hkv, label) in ((32, 8, "8B attention block"), (64, 8, "70B attention block")):
        for T in (512, 2048, 4096, 8192):
            Q = torch.randn(T, Hq * 128, generator=g).bfloat16().to(dev)
            K = torch.randn(T, Hkv * 128, generator=g).bfloat16().to(dev)
            V = torch.randn(T, Hkv * 128, generator=g).bfloat16().to(dev)
            O = torch.empty_like(Q)
            res = {}
            for causal in (False, True):
                a = gmlp.make_gqa_args(Q, K, V, O, Hq, Hkv, causal=causal)
                for _ in range(3):
                    gmlp.gqa_attention_ex(a)
                torch.cuda.synchronize(dev)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(iters):
                    gmlp.gqa_attention_ex(a)
                e1.record()
                torch.cuda.synchronize(dev)
                res[causal] = e0.elapsed_time(e1) / iters * 1e3
            us = res[False]
            tf = 4.0 * T * T * 128 * Hq / us / 1e6
            tf_causal = 4.0 * (T * (T + 1) / 2) * 128 * Hq / res[True] / 1e6        # visible (query, key) pairs only
            rows.append({"shape": label, "M": T, "S": T, "n_q_heads": Hq, "n_kv_heads": Hkv, "us": us, "tflops": tf,
                         "frac_of_bf16_peak": tf / peaks["bf16_tflops"], "causal_us": res[True],
                         "causal_tflops": tf_causal})
            del Q, K, V, O
    return {"timing": "back-to-back calls", "peak": peaks["bf16_tflops"], "peak_source": peaks["source"] + " (burst bf16)",
            "best_tflops": max(r["tflops"] for r in rows), "table": rows}


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launch_ranks(n: int) -> int:
    """--gpus N without a launcher: start N ranks of this script (one per GPU) under torch.distributed.run on this
    node and pass their exit code on.  Rank 0 of those prints the JSON line."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(free_port()), os.path.abspath(__file__), *sys.argv[1:]]
    return subprocess.call(cmd)


def summary_entry(r):
    rp = r.get("roofline_path", {})
    rk = r.get("roofline") or {}
    clk = r.get("clocks") or {}
    return {"name": r["name"], "ms": round(r["ms_per_step"], 5), "bound": rp.get("bound"),
            "frac_path": round(rp.get("frac", 0.0), 4), "frac_path_nominal": round(rp.get("frac_nominal", 0.0), 4),
            **({"frac_path_sustained": round(rp["frac_sustained"], 4)} if "frac_sustained" in rp else {}),
            "frac_kernel": round(rk["frac"], 4) if "frac" in rk else None, "sm_mhz": clk.get("sm_mhz"),
            "reasons": clk.get("reasons")}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="gmlp", choices=["gmlp", "reference"])
    ap.add_argument("--workload", default=None, help=f"primary workload (default {PRIMARY}; {PRIMARY_DFF} with --shard dff)")
    ap.add_argument("--shard", default="rows", choices=["rows", "dff"],
                    help="rows: ranks take disjoint rows, no collective (weak scaling); dff: d_ff cut over the ranks, "
                         "one all-reduce of M x d_model floats per step (strong scaling)")
    ap.add_argument("--no-extra", action="store_true", help="time only the primary workload")
    ap.add_argument("--op", default="gmlp", choices=["gmlp", "rmsnorm_matmul", "matmul_add_rmsnorm", "qkv", "gqa"],
                    help="rmsnorm_matmul / matmul_add_rmsnorm / qkv / gqa: print only that operator's sweep "
                         "(one JSON line) and exit")
    ap.add_argument("--autotune", action="store_true",
                    help="run gmlp_autotune on each workload's shape before timing it (default: the built-in rule)")
    ap.add_argument("--cpu-seconds", type=float, default=10.0, help="least CPU time spent on the oracle baseline (0 = skip)")
    ap.add_argument("--clock-roll", type=float, default=0.6,
                    help="seconds of untimed identical steps before the timed regions while clocks are sampled "
                         "(0 = no clock sampling; for runs under a profiler)")
    ap.add_argument("--stub-measure", action="store_true",
                    help="test hook: no GPU work at all - the ranks rendezvous over gloo, report a constant step time and "
                         "rank 0 prints the line marked \"data\": \"stub\" (checks the launch path on a CPU-only machine)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(launch_ranks(args.gpus))

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    wname = args.workload or (PRIMARY_DFF if args.shard == "dff" else PRIMARY)
    parallelism = (f"dp{world} (rows sharded, no collective)" if args.shard == "rows"
                   else f"tp{world} (d_ff sharded, one all-reduce of M x d_model fp32 per step)")
    scaling = "weak" if args.shard == "rows" else "strong"

    import torch
    from paper_2606_26344_b200 import inputs as I, sharding
    w = I.WORKLOADS[wname]

    if args.stub_measure:
        import torch.distributed as dist_mod
        if world > 1:
            dist_mod.init_process_group("gloo")
            dist_mod.barrier()
        ms = sharding.max_over_ranks(1.0 + 0.25 * rank, dist_mod if world > 1 else None)
        units = w.M * (world if args.shard == "rows" else 1)
        if rank == 0:
            print(json.dumps({"metric": "gated_mlp_tokens_per_s", "value": units / (ms * 1e-3), "unit": "tokens/s",
                              "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
                              "higher_is_better": True, "scaling": scaling, "vs_baseline": None, "dtype": "bf16",
                              "data": "stub", "config": {"workload": w.name, "parallelism": parallelism}}))
        if world > 1:
            dist_mod.barrier()
            dist_mod.destroy_process_group()
        return

    from paper_2606_26344_b200 import build as B
    from paper_2606_26344_b200 import gmlp
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    if rank == 0:
        B.build_libgmlp()
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist = dist_mod
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    if dist is not None:
        dist.barrier()
    gmlp.lib()
    peaks = load_peaks()
    warmup = max(args.warmup, 3)

    if args.op != "gmlp":
        if rank == 0:
            fn = {"rmsnorm_matmul": measure_rmsnorm_matmul, "matmul_add_rmsnorm": measure_matmul_add_rmsnorm,
                  "qkv": measure_qkv, "gqa": lambda d: measure_gqa(d, peaks)}[args.op]
            print(json.dumps({"op": args.op, **fn(dev)}))
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return

    if args.shard == "dff":
        res = measure_dff_sharded(w, args.steps, warmup, dev, peaks, dist, rank, world, clock_roll=args.clock_roll)
        ms = sharding.max_over_ranks(res["ms_per_step"], dist, dev)
        e2e_ms = sharding.max_over_ranks(res["e2e"]["ms_per_step"], dist, dev)
        if rank == 0:
            line = {
                "metric": "gated_mlp_tokens_per_s", "value": w.M / (ms * 1e-3), "unit": "tokens/s", "n_gpus": world,
                "steps": args.steps, "warmup": warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": scaling,
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": w.name, "M": w.M, "d_model": w.d_model, "d_ff": w.d_ff, "rmsnorm": w.rmsnorm,
                           "parallelism": parallelism, "d_ff_slice_rank0": res["slice"],
                           "weight_bytes_per_gpu": res["weight_bytes_per_gpu"], "allreduce_bytes_per_step": res["allreduce_bytes"]},
                "timing": {"ms_min": res["ms_min"], "ms_max": res["ms_max"], "regions": res["regions"],
                           "how": "median over regions of exactly `steps` steps, max over ranks"},
                "tflops": w.flops / (ms * 1e-3) / 1e12,
                "roofline_path": fractions(w, ms, peaks),
                "e2e": {"value": w.M / (e2e_ms * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": res["e2e"]["h2d_bytes_per_step"],
                        "d2h_bytes_per_step": res["e2e"]["d2h_bytes_per_step"]},
                "gpu_launches": res["launches"], "clocks": res["clocks"], "peaks": peaks,
            }
            print(json.dumps(line))
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return

    res = measure_workload(w, args.steps, warmup, dev, peaks, dist=dist, clock_roll=args.clock_roll,
                           autotune=args.autotune, exact_steps=True)
    ms = sharding.max_over_ranks(res["ms_per_step"], dist, dev)          # the slowest rank bounds the step
    res["e2e"]["ms_per_step"] = sharding.max_over_ranks(res["e2e"]["ms_per_step"], dist, dev)
    res["e2e"]["value"] = sharding.job_throughput(w.M, world, res["e2e"]["ms_per_step"])
    value = sharding.job_throughput(w.M, world, ms)

    extras = []
    if not args.no_extra and world == 1:
        for name in [n for n in STATED + UNSTATED if n != w.name]:
            try:
                r = measure_workload(I.WORKLOADS[name], args.steps, 3, dev, peaks, want_e2e=False, sample_clocks=True,
                                     clock_roll=min(args.clock_roll, 0.3), autotune=args.autotune, exact_steps=False)
                r.pop("_inputs", None)
                extras.append(r)
            except Exception as exc:  # a failed extra must not hide the primary number
                extras.append({"name": name, "error": repr(exc)})
            torch.cuda.empty_cache()

    rmsmm = None
    if not args.no_extra and world == 1:
        try:
            rmsmm = measure_rmsnorm_matmul(dev, iters=5)
            rmsmm.pop("table")
        except Exception as exc:
            rmsmm = {"error": repr(exc)}

    if rank != 0:
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return

    inp = res.pop("_inputs")
    rows = I.sample_rows(w, inp.outlier_rows)          # the rows the parity tests compare: all, or the 256 seeded ones
    if world == 1 and args.cpu_seconds > 0:
        cpu_rate, cpu_rows, cpu_dt, cores = cpu_oracle_rate(inp, rows, args.cpu_seconds)
        cpu = {"value": cpu_rate, "unit": "tokens/s", "cores": cores, "kind": "oracle",
               "sample": f"{cpu_rows} row evaluations of this workload (its {len(rows)} parity rows per pass, "
                         f"{cpu_dt:.1f} s in all); fp64, OpenMP over rows"}
    else:
        cpu = None

    line = {
        "metric": "gated_mlp_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": scaling, "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "M": w.M, "d_model": w.d_model, "d_ff": w.d_ff, "rmsnorm": w.rmsnorm,
                   "schedule": res["variant"], "l2": res["l2"], "parallelism": parallelism},
        "timing": {"ms_min": res["ms_min"], "ms_max": res["ms_max"], "regions": res["regions"],
                   "how": "median over regions of exactly `steps` steps, each between barrier + synchronize; "
                          "regions repeat until 0.5 s of steps have run, after a pre-roll of the same load"},
        "tflops": world * w.flops / (ms * 1e-3) / 1e12,
        "gbps_min_bytes": world * w.min_bytes / (ms * 1e-3) / 1e9,
        "roofline_path": res["roofline_path"],
        "roofline": res.get("roofline"),
        "kernel_ms": res["kernel_ms"],
        "cpu_baseline": cpu,
        "e2e": {k: res["e2e"][k] for k in ("value", "unit", "h2d_bytes_per_step", "d2h_bytes_per_step")},
        "gpu_launches": res["launches"],
        "clocks": res["clocks"],
        "peaks": peaks,
        "workloads": extras,
        "rmsnorm_matmul": rmsmm,
        "summary": [summary_entry(r) for r in [dict(res, name=w.name)] + [e for e in extras if "error" not in e]],
    }
    print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
