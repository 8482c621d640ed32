#!/usr/bin/env python
"""Benchmark of the SLoPe 2:4-sparse linear-layer path on B200.

A step = one pass of the whole hot path over one batch of synthetic input, for every
linear layer of the workload: first-pass prune + compress, double prune, [adapter T = X L],
forward, [adapter backward], input gradient, masked weight gradient -- every stage a
hand-written kernel behind the C ABI.  The LAST line of stdout (rank 0) is one compact JSON
object (at most 2000 characters: headline, clocks, roofline, dense comparison, e2e, CPU baseline); the
per-stage table and, with --extras, the probe suite go to a side file.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload KEY] [--impl reference] [--extras]

N > 1 (under torchrun) runs N independent replicas (the path has no exchange step).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2608_24070_b200 import inputs as si  # noqa: E402

METRIC = "SLoPe linear fwd+bwd TFLOP/s (dense-equivalent)"
UNIT = "TFLOP/s"
DEFAULT_WORKLOAD = "c4_llama7b_adapter"


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16": p["bf16_tflops"], "bf16_sustained": p["bf16_tflops_sustained"],
                "src": "measured"}
    return {"hbm_gbs": 6650.0, "bf16": 1590.0, "bf16_sustained": 1400.0, "src": "fallback"}


# ------------------------------------------------------------------------------ flop accounting
def layer_flops(b, d_in, d_out, r):
    """Dense-equivalent and executed FLOPs of one layer's fwd + dX + dW (+ adapter GEMMs)."""
    main = 2.0 * b * d_in * d_out
    adapter = 6.0 * b * r * (d_in + d_out)         # T, +T R, dT, dL, dR, +dT L^T
    return 3 * main + adapter, 2 * main + adapter


def workload_flops(wl, b):
    de = ex = 0.0
    for lay in wl.layers:
        a, c = layer_flops(b, lay.d_in, lay.d_out, wl.rank)
        de += a
        ex += c
    return de, ex


# ------------------------------------------------------------------------------ clocks sampler
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t_begin=None, t_end=None):
        """Summary of the samples taken between the two host timestamps (the timed region)."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = [r for (t, r) in self.rows if (t_begin is None or t >= t_begin) and (t_end is None or t <= t_end)]
        if len(rows) < 3:
            rows = [r for (_, r) in self.rows]
        for row in rows:
            f = [x.strip() for x in row.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_mhz_min": min(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "power_w_max": max(power) if power else None,
                "samples": len(sm), "window": "samples taken inside the timed region", "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------ the CUDA arm
class LayerState:
    def __init__(self, B, torch, wl, idx, b, dev):
        lay = wl.layers[idx]
        self.name, self.d_in, self.d_out, self.r, self.b = lay.name, lay.d_in, lay.d_out, wl.rank, b
        t = si.layer_tensors(wl, idx, tokens=b)
        self.W = B.bf16_from_bits(t["W"], dev)
        self.X = B.bf16_from_bits(t["X"], dev)
        self.dY = B.bf16_from_bits(t["dY"], dev)
        self.L = B.bf16_from_bits(t["L"], dev) if self.r else None
        self.R = B.bf16_from_bits(t["R"], dev) if self.r else None
        self.Wc_vals, self.Wc_meta, self.mask1 = B.alloc_compressed(self.d_out, self.d_in, dev)
        self.WTc_vals, self.WTc_meta, _ = B.alloc_compressed(self.d_in, self.d_out, dev)
        self.mask2 = torch.empty_like(self.mask1)
        bf = torch.bfloat16
        self.Y = torch.empty((b, self.d_out), dtype=bf, device=dev)
        self.dX = torch.empty((b, self.d_in), dtype=bf, device=dev)
        self.dWc = torch.empty((self.d_out, self.d_in // 2), dtype=bf, device=dev)
        if self.r:
            self.T = torch.empty((b, self.r), dtype=bf, device=dev)
            self.dT = torch.empty((b, self.r), dtype=bf, device=dev)
            self.dL = torch.empty((self.d_in, self.r), dtype=bf, device=dev)
            self.dR = torch.empty((self.r, self.d_out), dtype=bf, device=dev)
            self.ws = torch.empty(max(B.slope_adapter_workspace_bytes(b, self.d_out, self.d_in, self.r),
                                      B.slope_bwd_dw_adapter_workspace_bytes(b, self.d_out, self.d_in, self.r)),
                                  dtype=torch.uint8, device=dev)


OPS = ("prune_24_double", "adapter_T", "linear_fwd", "adapter_bwd", "linear_bwd_dx", "linear_bwd_dw_masked")


FUSED_ADAPTER_GRADS = False     # True: dL, dR ride in the weight-gradient launch (measured: no faster, see --fused-adapter-grads)


def run_layer(B, s: LayerState, rec=None):
    """All stages of one layer; `rec(op)` brackets a stage with CUDA events when timing per stage."""
    def stage(op, fn):
        if rec is None:
            fn()
        else:
            rec(op, s, fn)

    # both pruning passes in one launch (same outputs as slope_prune_24 + slope_double_prune, W read
    # once); the second-pass mask is an optional diagnostic output that no kernel of the step reads
    stage("prune_24_double", lambda: B.slope_prune_24_double(s.W, s.Wc_vals, s.Wc_meta, s.mask1, s.WTc_vals,
                                                             s.WTc_meta, None))
    if s.r:
        stage("adapter_T", lambda: B.slope_adapter_fwd_bwd(0, s.X, None, s.L, None, s.b, s.d_out, s.d_in, s.r, T=s.T))
        stage("linear_fwd", lambda: B.slope_linear_fwd(s.X, s.Wc_vals, s.Wc_meta, s.d_out, s.Y, s.T, s.R))
        if FUSED_ADAPTER_GRADS:     # dT here; dL and dR come out of the weight-gradient launch below
            stage("adapter_bwd", lambda: B.slope_adapter_fwd_bwd(2, None, s.dY, None, s.R, s.b, s.d_out, s.d_in, s.r,
                                                                 dT=s.dT))
        else:
            stage("adapter_bwd", lambda: B.slope_adapter_fwd_bwd(1, s.X, s.dY, s.L, s.R, s.b, s.d_out, s.d_in, s.r,
                                                                 T=s.T, dT=s.dT, dL=s.dL, dR=s.dR, workspace=s.ws))
        stage("linear_bwd_dx", lambda: B.slope_linear_bwd_dx(s.dY, s.WTc_vals, s.WTc_meta, s.d_in, s.dX, s.dT, s.L))
        if FUSED_ADAPTER_GRADS:
            stage("linear_bwd_dw_masked", lambda: B.slope_linear_bwd_dw_adapter(s.dY, s.X, s.T, s.dT, s.mask1, s.dWc,
                                                                                 s.dL, s.dR, s.ws))
            return
    else:
        stage("linear_fwd", lambda: B.slope_linear_fwd(s.X, s.Wc_vals, s.Wc_meta, s.d_out, s.Y))
        stage("linear_bwd_dx", lambda: B.slope_linear_bwd_dx(s.dY, s.WTc_vals, s.WTc_meta, s.d_in, s.dX))
    stage("linear_bwd_dw_masked", lambda: B.slope_linear_bwd_dw_masked(s.dY, s.X, s.mask1, s.dWc))


def stage_ms_by_graph(torch, B, layers, replays=5):
    """Device time of every op without the launch gaps that per-call events add: per op one CUDA graph
    holding that op's launches of all layers back to back (each layer has its own buffers, together far
    larger than L2, so the launches run cold as in the step), median of `replays` replays."""
    class Collect:
        def __init__(self):
            self.calls = {}

        def __call__(self, op, s, fn):
            self.calls.setdefault(op, []).append(fn)

    col = Collect()
    for s in layers:
        run_layer(B, s, rec=col)                 # collects the closures, launches nothing
    side = torch.cuda.Stream()
    out = {}
    for op, fns in col.calls.items():
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            for fn in fns:
                fn()
            side.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                for fn in fns:
                    fn()
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        ts = []
        for _ in range(replays):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); graph.replay(); e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        out[op] = round(statistics.median(ts), 4)
    return out


def cpu_baseline_sample(wl, seconds_hint=15.0):
    """Time the oracle, as it stands, on the workload: in full where that takes about half a
    minute at the oracle's ~0.02 TFLOP/s (the two small configurations), else on a bounded sample
    of the first layer, with the flop-scaled extrapolation to a whole step as a separate key."""
    import oracle

    oracle.build()
    b, r = wl.tokens, wl.rank
    step_flops = sum(6.0 * b * l.d_in * l.d_out + 6.0 * b * r * (l.d_in + l.d_out) for l in wl.layers)
    full = step_flops / 0.02e12 <= 2.0 * seconds_hint
    flops, dt, what = 0.0, 0.0, []
    for li, lay in enumerate(wl.layers if full else wl.layers[:1]):
        t = si.layer_tensors(wl, li, tokens=b)
        _, _, mask1 = oracle.prune24(t["W"])
        _, _, mask2 = oracle.double_prune(t["W"], mask1)
        rows = np.arange(b) if full else si.sample_indices(b, 1024, 1)
        orows = np.arange(lay.d_out) if full else si.sample_indices(lay.d_out, 1024, 2)
        t0 = time.perf_counter()
        oracle.fwd_rows(t["X"], t["W"], mask1, rows, t.get("L"), t.get("R"))
        oracle.dx_rows(t["dY"], t["W"], mask2, rows, t.get("L"), t.get("R"))
        oracle.dw_rows(t["dY"], t["X"], mask1, orows)
        dt += time.perf_counter() - t0
        flops += (2 * len(rows) * (2.0 * lay.d_in * lay.d_out + 2.0 * r * (lay.d_in + lay.d_out))
                  + len(orows) * 2.0 * b * lay.d_in)
        what.append(f"{lay.name} {lay.d_in}->{lay.d_out} b={b}: fwd+dX {len(rows)} token rows, dW {len(orows)} rows")
    value = flops / dt / 1e12
    return {"value": round(value, 6), "unit": UNIT, "cores": oracle.max_threads(), "kind": "oracle", "seconds": round(dt, 2),
            "sample": ("whole workload: " if full else "bounded sample: ") + "; ".join(what),
            "full_workload": full,
            "extrapolated_step_seconds": round(step_flops / (value * 1e12), 1),
            "extrapolation": "flop-scaled: dense-equivalent FLOPs of one step (fwd + dX + dW + adapter terms of every layer) "
                             "/ the measured rate; equals the measured time when the whole workload was run"}


def run_reference(args, rank):
    """The reference arm: the fp64 CPU oracle on the machine's host cores (there is no other
    implementation of the paper to run)."""
    if rank != 0:
        return
    wl = si.WORKLOADS[args.workload]
    import oracle

    oracle.build()
    lay = wl.layers[0]
    b = wl.tokens
    t = si.layer_tensors(wl, 0, tokens=b)
    _, _, mask1 = oracle.prune24(t["W"])
    _, _, mask2 = oracle.double_prune(t["W"], mask1)
    n_rows = 128
    rows = si.sample_indices(b, n_rows, 1)
    orows = si.sample_indices(lay.d_out, n_rows, 2)
    r = wl.rank
    flops = (2 * len(rows) * (2.0 * lay.d_in * lay.d_out + 2.0 * r * (lay.d_in + lay.d_out))
             + len(orows) * 2.0 * b * lay.d_in)

    def step():
        oracle.fwd_rows(t["X"], t["W"], mask1, rows, t.get("L"), t.get("R"))
        oracle.dx_rows(t["dY"], t["W"], mask2, rows, t.get("L"), t.get("R"))
        oracle.dw_rows(t["dY"], t["X"], mask1, orows)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    val = flops * args.steps / dt / 1e12
    sample = (f"each step: layer '{lay.name}' {lay.d_in}->{lay.d_out}, b={b}: fwd+dX on {len(rows)} token rows, "
              f"masked dW on {len(orows)} d_out rows")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.key, "tokens": b, "rank": r, "note": "bounded sample of the workload per step"},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.max_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }), flush=True)


def replica_max_ms(torch, dist, ms_local, device):
    """Replicas only: the job's time is the slowest rank's device time."""
    if dist is None:
        return float(ms_local)
    tt = torch.tensor([ms_local], device=device, dtype=torch.float64)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return float(tt.item())


def replica_throughput(world, flops_per_replica, ms_step):
    """Whole-job dense-equivalent TFLOP/s of `world` independent replicas."""
    return world * flops_per_replica / (ms_step * 1e-3) / 1e12


def replica_e2e(torch, dist, e2e_local, world, flops_per_replica, device):
    """End-to-end record of `world` replicas from each rank's own: the slowest rank's time, all
    replicas' work and bytes."""
    ms = replica_max_ms(torch, dist, e2e_local["ms_per_step"], device)
    out = dict(e2e_local)
    out.update(ms_per_step=round(ms, 3), value=round(replica_throughput(world, flops_per_replica, ms), 2),
               h2d_bytes_per_step=world * e2e_local["h2d_bytes_per_step"],
               d2h_bytes_per_step=world * e2e_local["d2h_bytes_per_step"])
    return out


GEMM_SOURCES = ("gemm_kernels.cuh", "ptx.cuh", "slope_lib.cu")     # the GEMM kernels, their PTX wrappers, the kernel choice


def kernel_sources_sha256():
    """Hash of the CUDA sources that decide what the two tensor-core kernels do: the ncu-recorded
    DRAM traffic below is reported only while it describes the kernels that actually ran."""
    import hashlib

    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2608_24070_b200", "csrc")
    for name in GEMM_SOURCES:
        with open(os.path.join(csrc, name), "rb") as f:
            h.update(name.encode() + b"\0" + f.read())
    return h.hexdigest()


# dram__bytes_read.sum + dram__bytes_write.sum per launch of the two tensor-core kernels, from a
# one-pass ncu capture (--clock-control none) of this benchmark's own workload at full size: the 21
# GEMM launches of one step of c4_llama7b_adapter at 16384 tokens.  `sources` is kernel_sources_sha256() of the build that was captured; a build with other
# sources reports traffic = null (tests/test_bench_line.py fails until the capture is refreshed or
# cleared).
NCU_TRAFFIC = {
    "sources": "e850cb677486eadb7dcfe7bb186a34c258c3387ea56bcab297d207fbd978d0fa",
    "captured_tokens": 16384,
    "sparse_bytes_per_launch": 493554889,     # mean over the 14 sparse GEMM launches of one step
    "dense_bytes_per_launch": 1389503488,     # mean over the 7 weight-gradient launches of one step
}


def recorded_traffic(kind, wl_key, tokens):
    if NCU_TRAFFIC["sources"] is None or wl_key not in ("c3_llama7b", "c4_llama7b_adapter"):
        return None, "no ncu capture recorded for this workload"
    if NCU_TRAFFIC["sources"] != kernel_sources_sha256():
        return None, "stale: the kernels changed since the recorded ncu capture"
    v = NCU_TRAFFIC[f"{kind}_bytes_per_launch"]
    if v is None:
        return None, "no ncu capture recorded for this kernel"
    scale = tokens / NCU_TRAFFIC["captured_tokens"]
    return round(v * scale), f"ncu {NCU_TRAFFIC['captured_tokens']} tok x{scale:g}, src {NCU_TRAFFIC['sources'][:8]}"


SM_COUNT = 148
DENSE_FLOP_PER_CLK_SM = 8192            # dense bf16 tcgen05: 2 * 4096 MAC per clock and SM
DATASHEET_SPARSE_TFLOPS = 4500.0
DATASHEET_DENSE_TFLOPS = 2250.0


def algorithmic_bytes(op, b, d_in, d_out, r):
    """Minimum HBM bytes of one launch (activations in and out, compressed weight, adapter operands)."""
    w = 1.125 * d_in * d_out
    if op == "linear_fwd":
        return 2.0 * b * d_in + w + 2.0 * b * d_out + (2.0 * b * r + 2.0 * r * d_out if r else 0.0)
    if op == "linear_bwd_dx":
        return 2.0 * b * d_out + w + 2.0 * b * d_in + (2.0 * b * r + 2.0 * r * d_in if r else 0.0)
    if op == "linear_bwd_dw_masked":
        return 2.0 * b * (d_in + d_out) + w
    return 0.0


LINE_LIMIT = 2000


def compact_line(out):
    """The one line the driver parses: short enough to survive a few-KB tail of stdout.  If a workload
    with many layers makes it too long, the least important detail goes first (it stays in the side
    file); a line that is still too long is an error."""
    out = dict(out)
    trims = (
        lambda o: o.get("cpu_baseline") and o["cpu_baseline"].update(sample=o["cpu_baseline"]["sample"][:60] + "..."),
        lambda o: o.pop("stage_ms", None),
        lambda o: o.pop("roofline_other", None),
    )
    line = json.dumps(out, separators=(",", ":"))
    for trim in trims:
        if len(line) <= LINE_LIMIT:
            break
        if out.get("cpu_baseline"):
            out["cpu_baseline"] = dict(out["cpu_baseline"])
        trim(out)
        line = json.dumps(out, separators=(",", ":"))
    if len(line) > LINE_LIMIT:
        raise SystemExit(f"bench line grew to {len(line)} characters; move detail to the side file")
    return line


def headline(args, wl, b, world, value, ms_step, executed_tflops, launches, clocks_full, roofline, other,
             ms_step_staged, stage_ms, kernel_mhz=None):
    """The compact record (pure function of measured numbers: also exercised without a GPU)."""
    clocks = None
    if clocks_full is not None:
        clocks = {k: clocks_full.get(k) for k in ("sm_mhz", "sm_mhz_min", "sm_max_mhz", "power_w_max", "reasons")}
        clocks["kernel_mhz"] = kernel_mhz
    adapter_ms = stage_ms.get("adapter_T", 0.0) + stage_ms.get("adapter_bwd", 0.0)
    return {
        "impl": "slope", "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms_step, 4), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": wl.key, "tokens": b, "rank": wl.rank, "parallelism": "replicas" if world > 1 else "1 GPU",
                   "l2": "inputs > L2",
                   "step": f"prune x2, adapters, fwd, dX, masked dW x {len(wl.layers)} layers"},
        "executed_tflops": round(executed_tflops, 2),
        "gpu_launches": int(launches), "clocks": clocks, "roofline": roofline,
        "roofline_other": None if other is None else {k: other[k] for k in (
            "kernel", "achieved", "peak", "frac", "frac_sustained", "frac_kernel_clock", "kernel_ms_per_step")},
        "ms_per_step_staged": round(ms_step_staged, 4),
        "stage_ms": stage_ms,
        "adapter_share": round(adapter_ms / sum(stage_ms.values()), 4) if stage_ms else None,
    }


def attach_extras(out, dl, e2e, cb):
    """Dense comparison, end-to-end run and CPU baseline, cut down to what the line carries."""
    if dl is not None:
        out["dense_layer"] = {"cublas_ms": dl["dense_ms"], "inhouse_ms": dl["inhouse_dense_ms"], "slope_ms": dl["slope_ms"],
                              "speedup": dl["speedup"], "speedup_vs_inhouse": dl["speedup_vs_inhouse_dense"]}
    out["e2e"] = None if e2e is None else {k: e2e[k] for k in ("value", "unit", "ms_per_step", "h2d_bytes_per_step",
                                                                 "d2h_bytes_per_step")}
    out["cpu_baseline"] = None if cb is None else {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample",
                                                                       "full_workload", "seconds")}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(si.WORKLOADS))
    ap.add_argument("--impl", default="slope", choices=["slope", "reference"])
    ap.add_argument("--tokens", type=int, default=0, help="override the workload's token count (profiling only)")
    ap.add_argument("--no-extras", action="store_true",
                    help="only the timed step: skip the per-stage pass' side file, dense comparison, e2e and CPU baseline")
    ap.add_argument("--extras", action="store_true",
                    help="also run the probe suite (per-op medians over 200 launches, burst, optimizer tail, N:M, "
                         "inference forward, decode block, shape sweep, small configurations, decoder block) and "
                         "write it to the side file")
    ap.add_argument("--side-file", default=os.path.join(ROOT, "bench_extras.json"),
                    help="where the per-stage table and the probe results go (not printed)")
    ap.add_argument("--fused-adapter-grads", action="store_true",
                    help="compute dL, dR inside the weight-gradient launch (slope_linear_bwd_dw_adapter) instead of by "
                         "their own launches; for comparison (measured: the step is no faster)")
    ap.add_argument("--cusparselt-context", action="store_true",
                    help="with --extras: also time the forward GEMMs through torch's semi-structured sparse matmul "
                         "(cuSPARSELt, the library the paper builds on); context only")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "slope" and not args.tokens else args.warmup

    global FUSED_ADAPTER_GRADS
    FUSED_ADAPTER_GRADS = args.fused_adapter_grads
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    from paper_2608_24070_b200 import binding as B
    from paper_2608_24070_b200 import build as _build

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the SLoPe path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod

        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)
    if local_rank == 0:
        _build.build()                # no-op when libslope.so is newer than its sources
    if dist is not None:
        dist.barrier()
    B.lib()

    pk = peaks()
    wl = si.WORKLOADS[args.workload]
    b = args.tokens or wl.tokens
    layers = [LayerState(B, torch, wl, i, b, dev) for i in range(len(wl.layers))]
    de_flops, ex_flops = workload_flops(wl, b)
    stream = torch.cuda.current_stream()

    def step(rec=None):
        for s in layers:
            run_layer(B, s, rec)

    def barrier():
        if dist is not None:
            dist.barrier()

    def check_status(where):
        st = B.slope_poll_status()
        if st != 0:
            raise SystemExit(f"device status after {where}: {B.slope_status_string(st)}")

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    check_status("warm-up")

    # ---------------- timed region: exactly K steps, nothing but the library's launches between the
    # two events (per-stage events would sit between the programmatic dependent launches), device
    # time, max over ranks
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = B.slope_launch_count()
    barrier()
    torch.cuda.synchronize()
    B.slope_kernel_clock_mhz(0), B.slope_kernel_clock_mhz(1)        # start the in-kernel clock averages here
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_begin = time.time()
    ev0.record(stream)
    for _ in range(args.steps):
        step()
    ev1.record(stream)
    torch.cuda.synchronize()
    t_end = time.time()
    barrier()
    launches = B.slope_launch_count() - launches0
    ms_total = replica_max_ms(torch, dist, ev0.elapsed_time(ev1), dev)
    check_status("the timed region")
    # the mean SM clock inside the sparse / dense tile-kernel launches of the timed region (the power
    # limiter moves it within microseconds; nvidia-smi's samples average over all kernels of the step)
    kernel_mhz = {"sparse": round(B.slope_kernel_clock_mhz(0), 1), "dense": round(B.slope_kernel_clock_mhz(1), 1)}
    ms_step = ms_total / args.steps
    value = replica_throughput(world, de_flops, ms_step)

    # ---------------- stage pass: the same K steps again, every call bracketed by CUDA events on the
    # launching stream; per (layer, op) the MEDIAN over the K launches.  The clock sampler keeps
    # running, so the clocks below cover both passes (same load).
    events = []

    def rec(op, s, fn):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        fn()
        e1.record(stream)
        events.append((op, s, e0, e1))

    ev2, ev3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev2.record(stream)
    for _ in range(args.steps):
        step(rec)
    ev3.record(stream)
    torch.cuda.synchronize()
    t_end_stage = time.time()
    ms_step_staged = ev2.elapsed_time(ev3) / args.steps
    check_status("the stage pass")
    if rank == 0:
        time.sleep(0.1)
    clocks_full = sampler.stop(t_begin, t_end_stage) if rank == 0 else None

    per_layer_op = {}
    for op, s, e0, e1 in events:
        per_layer_op.setdefault((s.name, op), []).append(e0.elapsed_time(e1))
    by_name = {s.name: s for s in layers}

    def op_flops(op, s):
        m = 2.0 * s.b * s.d_in * s.d_out
        return {"linear_fwd": m + 2.0 * s.b * s.r * s.d_out, "linear_bwd_dx": m + 2.0 * s.b * s.r * s.d_in,
                "linear_bwd_dw_masked": m}.get(op, 0.0)

    sm_mhz = (clocks_full or {}).get("sm_mhz")
    stage_rows, per_op_ms = [], {op: 0.0 for op in OPS}
    tot = {"sparse": [0.0, 0.0, 0.0, 0], "dense": [0.0, 0.0, 0.0, 0]}        # flops, seconds, bytes, launches
    for (name, op), lst in per_layer_op.items():
        s = by_name[name]
        ms = statistics.median(lst)
        per_op_ms[op] += ms
        row = {"layer": name, "d_in": s.d_in, "d_out": s.d_out, "op": op, "ms_median": round(ms, 4),
               "ms_mean": round(statistics.mean(lst), 4), "launches": len(lst)}
        fl = op_flops(op, s)
        n_el = s.d_in * s.d_out
        if fl:
            kind = "dense" if op == "linear_bwd_dw_masked" else "sparse"
            nbytes = algorithmic_bytes(op, s.b, s.d_in, s.d_out, s.r)
            t = tot[kind]
            t[0] += fl; t[1] += ms * 1e-3; t[2] += nbytes; t[3] += 1
            tf = fl / (ms * 1e-3) / 1e12
            burst = pk["bf16"] * (1.0 if kind == "dense" else 2.0)
            t_star = max(fl / (burst * 1e12), nbytes / (pk["hbm_gbs"] * 1e9))
            row.update({"tflops_dense_eq": round(tf, 1), "tflops_executed": round(tf if kind == "dense" else tf / 2, 1),
                        "frac_of_burst_peak": round(tf / burst, 4), "roofline_frac_t_star": round(t_star / (ms * 1e-3), 4)})
        elif op == "prune_24_double":
            # W in (2 B), two compressed copies out (1 + 1/8 B each), first mask out (1/8 B)
            gbs = 4.375 * n_el / (ms * 1e-3) / 1e9
            row.update({"gbs": round(gbs, 1), "frac_of_hbm_peak": round(gbs / pk["hbm_gbs"], 4)})
        elif op in ("adapter_T", "adapter_bwd"):
            # T = X L streams X once; the backward streams dY once for dT (X and dY for dL, dR ride in the dW launch
            # when the library fuses them)
            small = 2.0 * s.r * (s.b + s.d_in + s.d_out)
            nbytes = 2.0 * s.b * s.d_in + small if op == "adapter_T" else 2.0 * s.b * (s.d_in + 2 * s.d_out) + 3 * small
            gbs = nbytes / (ms * 1e-3) / 1e9
            row.update({"gbs": round(gbs, 1), "frac_of_hbm_peak": round(gbs / pk["hbm_gbs"], 4)})
        stage_rows.append(row)

    def roofline_of(kind, kernel, peak_burst, peak_sustained, datasheet, flop_per_clk_sm):
        fl, sec, nbytes, n = tot[kind]
        if not sec:
            return None
        tf = fl / sec / 1e12
        traffic, source = recorded_traffic(kind, wl.key, b)
        r = {"kernel": kernel, "bound": "tensor", "achieved": round(tf, 1), "peak": round(peak_burst, 1),
             "unit": "TFLOP/s", "frac": round(tf / peak_burst, 4), "traffic": traffic,
             "algorithmic_bytes": round(nbytes / n), "traffic_source": source,
             "peak_source": ("2x " if kind == "sparse" else "") + f"{pk['src']} burst cuBLAS",
             "frac_sustained": round(tf / peak_sustained, 4), "frac_datasheet": round(tf / datasheet, 4),
             "frac_clock": round(fl / sec / (sm_mhz * 1e6 * SM_COUNT * flop_per_clk_sm), 4) if sm_mhz else None,
             "frac_kernel_clock": round(fl / sec / (kernel_mhz[kind] * 1e6 * SM_COUNT * flop_per_clk_sm), 4)
             if kernel_mhz[kind] else None,
             "tflop_per_step": round(fl / 1e12, 4), "kernel_ms_per_step": round(sec * 1e3, 4), "launches_per_step": n}
        return r

    roofline_sparse = roofline_of(
        "sparse", "sparse_gemm_quad/pair_kernel (fwd, dX)",
        2.0 * pk["bf16"], 2.0 * pk["bf16_sustained"], DATASHEET_SPARSE_TFLOPS, 2 * DENSE_FLOP_PER_CLK_SM)
    roofline_dense = roofline_of(
        "dense", "dense_gemm_pair_kernel (masked dW)",
        pk["bf16"], pk["bf16_sustained"], DATASHEET_DENSE_TFLOPS, DENSE_FLOP_PER_CLK_SM)
    sparse_dominant = tot["sparse"][1] >= tot["dense"][1]
    roofline = roofline_sparse if sparse_dominant else roofline_dense
    other = roofline_dense if sparse_dominant else roofline_sparse
    stage_ms = {k: round(v, 3) for k, v in per_op_ms.items() if v > 0}

    line_roofline = {k: v for k, v in roofline.items() if k not in ("launches_per_step",)}
    out = headline(args, wl, b, world, value, ms_step, world * ex_flops / (ms_step * 1e-3) / 1e12, launches,
                   clocks_full, line_roofline, other, ms_step_staged, stage_ms, kernel_mhz)

    side = {"headline": dict(out), "clocks": clocks_full, "roofline_sparse": roofline_sparse,
            "roofline_dense": roofline_dense, "stages": stage_rows}
    if rank == 0 and not args.no_extras and world == 1:
        dl = dense_comparison(torch, B, layers, stream)
        side["dense_layer"] = dl
        sg = stage_ms_by_graph(torch, B, layers)
        side["stage_ms_graph"] = {"what": "ms per step and op from one CUDA graph per op (all layers back to back, no events "
                                          "between launches), median of 5 replays", **sg,
                                  "adapter_share": round((sg.get("adapter_T", 0.0) + sg.get("adapter_bwd", 0.0)) /
                                                         sum(sg.values()), 4)}
        if args.extras:
            side["per_op_200"] = per_op_probe(torch, B, layers, stream, pk)
            side["hbm_kernels_cold"] = hbm_kernel_probe(torch, B, pk)
            side["optimizer_tail"] = optimizer_tail_probe(torch, B, layers, stream, pk)
            side["burst"] = burst_probe(torch, B, layers, stream, pk)
            side["inference_forward"] = inference_forward_probe(torch, B, wl, pk)
            side["decode_block"] = decode_block_probe(torch, B)
            side["nm_masked_dense"] = nm_probe(torch, B, layers, stream, pk)
            side["forward_speedup_by_shape"] = forward_shape_sweep(torch, B, stream)
            side["small_configs_hot_cold"] = small_config_probe(torch, B, stream, pk)
            side["decoder_block_c5"] = decoder_block_probe(torch)
            if args.cusparselt_context:
                side["cusparselt_context"] = cusparselt_context(torch, B, layers, stream)
        e2e = e2e_run(torch, B, layers, de_flops, max(2, min(args.steps, 5)))
        side["e2e"] = e2e
        cb = cpu_baseline_sample(wl)
        side["cpu_baseline"] = cb
        attach_extras(out, dl, e2e, cb)
    elif world > 1 and not args.no_extras:
        # N replicas: every rank runs the host-buffer step on its own GPU and PCIe link; the job's
        # end-to-end figure is all replicas' work over the slowest rank's time (no CPU baseline, no
        # dense comparison at N > 1)
        e2e = replica_e2e(torch, dist, e2e_run(torch, B, layers, de_flops, max(2, min(args.steps, 5))), world, de_flops, dev)
        if rank == 0:
            side["e2e"] = e2e
            attach_extras(out, None, e2e, None)
    elif rank == 0:
        attach_extras(out, None, None, None)
    if rank == 0:
        if not args.no_extras:
            try:
                os.makedirs(os.path.dirname(args.side_file), exist_ok=True)
                with open(args.side_file, "w") as f:
                    json.dump(side, f, indent=1)
            except OSError as ex:
                print(f"side file not written: {ex}", file=sys.stderr)
        print(compact_line(out), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def per_op_probe(torch, B, layers, stream, pk, launches=200, warm=20):
    """Every op of every distinct layer shape timed alone: `warm` untimed launches, then `launches`
    launches each bracketed by its own pair of CUDA events; median per op (the activations of one
    launch are larger than L2, so consecutive launches do not find them there)."""
    rows, seen = [], set()
    for s in layers:
        if (s.d_in, s.d_out) in seen:
            continue
        seen.add((s.d_in, s.d_out))
        calls = {"prune_24": lambda s=s: B.slope_prune_24(s.W, s.Wc_vals, s.Wc_meta, s.mask1),
                 "double_prune": lambda s=s: B.slope_double_prune(s.W, s.mask1, s.WTc_vals, s.WTc_meta, None),
                 "prune_24_double": lambda s=s: B.slope_prune_24_double(s.W, s.Wc_vals, s.Wc_meta, s.mask1, s.WTc_vals,
                                                                        s.WTc_meta, None),
                 "linear_bwd_dw_masked": lambda s=s: B.slope_linear_bwd_dw_masked(s.dY, s.X, s.mask1, s.dWc)}
        if s.r:
            calls["adapter_T"] = lambda s=s: B.slope_adapter_fwd_bwd(0, s.X, None, s.L, None, s.b, s.d_out, s.d_in, s.r, T=s.T)
            calls["linear_fwd"] = lambda s=s: B.slope_linear_fwd(s.X, s.Wc_vals, s.Wc_meta, s.d_out, s.Y, s.T, s.R)
            calls["adapter_bwd"] = lambda s=s: B.slope_adapter_fwd_bwd(1, s.X, s.dY, s.L, s.R, s.b, s.d_out, s.d_in, s.r,
                                                                      T=s.T, dT=s.dT, dL=s.dL, dR=s.dR, workspace=s.ws)
            calls["linear_bwd_dx"] = lambda s=s: B.slope_linear_bwd_dx(s.dY, s.WTc_vals, s.WTc_meta, s.d_in, s.dX, s.dT, s.L)
        else:
            calls["linear_fwd"] = lambda s=s: B.slope_linear_fwd(s.X, s.Wc_vals, s.Wc_meta, s.d_out, s.Y)
            calls["linear_bwd_dx"] = lambda s=s: B.slope_linear_bwd_dx(s.dY, s.WTc_vals, s.WTc_meta, s.d_in, s.dX)
        for op, fn in calls.items():
            for _ in range(warm):
                fn()
            evs = []
            for _ in range(launches):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream); fn(); e1.record(stream)
                evs.append((e0, e1))
            torch.cuda.synchronize()
            ms = statistics.median(e0.elapsed_time(e1) for e0, e1 in evs)
            row = {"d_in": s.d_in, "d_out": s.d_out, "tokens": s.b, "op": op, "ms_median": round(ms, 4)}
            if op.startswith("linear"):
                fl = 2.0 * s.b * s.d_in * s.d_out
                peak = pk["bf16"] * (1.0 if op == "linear_bwd_dw_masked" else 2.0)
                nbytes = algorithmic_bytes(op, s.b, s.d_in, s.d_out, s.r)
                t_star = max(fl / (peak * 1e12), nbytes / (pk["hbm_gbs"] * 1e9))
                row.update({"tflops_dense_eq": round(fl / ms / 1e9, 1), "frac_of_burst_peak": round(fl / ms / 1e9 / peak, 4),
                            "roofline_frac_t_star": round(t_star / (ms * 1e-3), 4)})
            elif op in ("prune_24", "double_prune", "prune_24_double"):
                nbytes = (4.375 if op == "prune_24_double" else 3.25) * s.d_in * s.d_out
                row.update({"gbs": round(nbytes / ms / 1e6, 1), "frac_of_hbm_peak": round(nbytes / ms / 1e6 / pk["hbm_gbs"], 4)})
            rows.append(row)
    return {"what": f"median of {launches} launches after {warm} warm-ups, each launch between its own CUDA events; "
                    f"peaks: dense {pk['bf16']} TFLOP/s burst ({pk['src']}), sparse := 2 x dense", "rows": rows}


def hbm_kernel_probe(torch, B, pk, sets=3, launches=12, replays=5):
    """The HBM-bound kernels (both pruning passes separately and in one launch, the optimizer tail)
    timed COLD and without launch gaps: a CUDA graph of `launches` back-to-back launches that cycle
    through `sets` separate buffer sets (inputs and outputs of one set are 60-450 MB, so a set has left
    the 126 MB L2 long before its turn comes again), best of `replays` replays.  Events around single
    launches of 15-50 us kernels add 5-15 us of launch gap each, which is what the per-stage table of
    the step shows for them."""
    dev = torch.device("cuda")
    side = torch.cuda.Stream()

    def graph_us(calls):
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            for fn in calls[:sets]:
                fn()
            side.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                for fn in calls:
                    fn()
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        best = float("inf")
        for _ in range(replays):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); graph.replay(); e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        return best * 1e3 / len(calls)

    rows = []
    for d_out, d_in in ((4096, 4096), (11008, 4096), (4096, 11008), (13824, 5120)):
        n = d_out * d_in
        bufs = []
        for i in range(sets):
            W = B.bf16_from_bits(si.gaussian_bf16((d_out, d_in), 0.02, si.seed_for(7, i, "W")), dev)
            vals, meta, mask1 = B.alloc_compressed(d_out, d_in, dev)
            valsT, metaT, _ = B.alloc_compressed(d_in, d_out, dev)
            B.slope_prune_24_double(W, vals, meta, mask1, valsT, metaT, None)
            bufs.append({"W": W, "vals": vals, "meta": meta, "mask1": mask1, "valsT": valsT, "metaT": metaT,
                         "g": torch.randn_like(vals), "out": torch.empty_like(vals), "newT": torch.empty_like(valsT)})
        ops = {
            "prune_24": (lambda q: B.slope_prune_24(q["W"], q["vals"], q["meta"], q["mask1"]), 3.25),
            "double_prune": (lambda q: B.slope_double_prune(q["W"], q["mask1"], q["valsT"], q["metaT"], None), 3.25),
            "prune_24_double": (lambda q: B.slope_prune_24_double(q["W"], q["vals"], q["meta"], q["mask1"], q["valsT"],
                                                                  q["metaT"], None), 4.375),
            "sparse_add": (lambda q: B.slope_sparse_add(q["g"], q["vals"], 1.0 / 1024.0, 0.01, q["out"]), 3.0),
            "update_sparse_matrix": (lambda q: B.slope_update_sparse_matrix(q["vals"], q["mask1"], q["metaT"], q["newT"]),
                                     2.25),
        }
        for op, (fn, bytes_per_el) in ops.items():
            us = graph_us([lambda fn=fn, q=bufs[i % sets]: fn(q) for i in range(launches)])
            gbs = bytes_per_el * n / us / 1e3
            rows.append({"op": op, "d_out": d_out, "d_in": d_in, "us": round(us, 2), "bytes_per_element": bytes_per_el,
                         "gbs": round(gbs, 1), "frac_of_hbm_peak": round(gbs / pk["hbm_gbs"], 4)})
        del bufs
    st = B.slope_poll_status()
    if st != 0:
        raise SystemExit(f"device status after the HBM kernel probe: {B.slope_status_string(st)}")
    return {"what": f"us per launch from a CUDA graph of {launches} launches cycling through {sets} buffer sets (cold), best "
                    f"of {replays} replays; algorithmic bytes per weight element as listed; HBM peak {pk['hbm_gbs']} GB/s "
                    f"({pk['src']})", "rows": rows}


def optimizer_tail_probe(torch, B, layers, stream, pk, reps=20):
    """Algorithm 1's optimizer tail on the largest layer: sparseAdd (g = dWc/gamma + alpha*Wc) and
    updateSparseMatrix (refresh the transposed copy), HBM-bound, against the measured HBM peak."""
    s = max(layers, key=lambda l: l.d_in * l.d_out)
    n = s.d_in * s.d_out
    g = torch.empty_like(s.dWc)
    new_t = torch.empty_like(s.WTc_vals)
    calls = {
        "sparse_add": (lambda: B.slope_sparse_add(s.dWc, s.Wc_vals, 1.0 / 1024.0, 0.01, g), 3.0 * n),
        "update_sparse_matrix": (lambda: B.slope_update_sparse_matrix(s.Wc_vals, s.mask1, s.WTc_meta, new_t),
                                 2.25 * n),
    }
    rows = []
    for op, (fn, nbytes) in calls.items():
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        gbs = nbytes / (ms * 1e-3) / 1e9
        rows.append({"op": op, "layer": s.name, "d_in": s.d_in, "d_out": s.d_out, "ms": round(ms, 4),
                     "algorithmic_bytes": int(nbytes), "gbs": round(gbs, 1),
                     "frac_of_hbm_peak": round(gbs / pk["hbm_gbs"], 4)})
    return {"what": f"{reps} back-to-back launches, CUDA events; bytes: sparse_add 3 B and update 2.25 B per weight "
                    f"element; HBM peak {pk['hbm_gbs']} GB/s ({pk['src']}); the working set of sparse_add "
                    f"({3 * n / 1e6:.0f} MB) partly lives in the 126 MB L2 across launches", "rows": rows}


def forward_shape_sweep(torch, B, stream, tokens=2048, reps=20):
    """The setting of the paper's per-shape speedup figure (attention d -> d, upsample d -> 4d and
    downsample 4d -> d matrices, batch 2048): forward GEMM, slope_linear_fwd against torch.matmul on
    the dense weight, back-to-back launches timed with CUDA events, interleaved."""
    dev = torch.device("cuda")
    rows = []
    for d in (1024, 2048, 4096, 8192):
        for kind, d_in, d_out in (("attention", d, d), ("upsample", d, 4 * d), ("downsample", 4 * d, d)):
            W = B.bf16_from_bits(si.gaussian_bf16((d_out, d_in), 0.02, si.seed_for(8, 0, "W")), dev)
            X = B.bf16_from_bits(si.gaussian_bf16((tokens, d_in), 1.0, si.seed_for(8, 0, "X")), dev)
            vals, meta, _ = B.alloc_compressed(d_out, d_in, dev)
            B.slope_prune_24(W, vals, meta, None)
            Y = torch.empty((tokens, d_out), dtype=torch.bfloat16, device=dev)

            def timed(fn):
                for _ in range(3):
                    fn()
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for _ in range(reps):
                    fn()
                e1.record(stream)
                torch.cuda.synchronize()
                return e0.elapsed_time(e1) / reps * 1e3

            us_dense = timed(lambda: torch.matmul(X, W.t(), out=Y))
            us_sparse = timed(lambda: B.slope_linear_fwd(X, vals, meta, d_out, Y))
            flop = 2.0 * tokens * d_in * d_out
            rows.append({"kind": kind, "d_in": d_in, "d_out": d_out, "tokens": tokens, "dense_us": round(us_dense, 1),
                         "slope_us": round(us_sparse, 1), "speedup": round(us_dense / us_sparse, 3),
                         "slope_tflops_dense_eq": round(flop / us_sparse / 1e6, 1)})
            del W, X, vals, meta, Y
    return {"what": f"forward only, {tokens} tokens, {reps} back-to-back launches each (includes host launch overhead "
                    f"for the smallest shapes), torch.matmul (cuBLAS) dense against slope_linear_fwd", "rows": rows}


def small_config_probe(torch, B, stream, pk, min_launches=48):
    """The two small configurations (one 512 x 512 layer with 256 tokens; GPT-2-small with 8192 tokens),
    every op of every layer, device time per launch from a CUDA graph of back-to-back launches (no host
    overhead; includes the ~1 us gap between dependent kernels): "hot" = all launches on one buffer set
    (operands stay in L2), "cold" = the launches cycle through enough separate buffer sets (at least 4,
    together more than 160 MB) that every operand has left L2 when its turn comes again.
    Roofline time t* = max(dense-equivalent FLOP / peak, bytes / HBM peak)."""
    dev = torch.device("cuda")
    side = torch.cuda.Stream()

    def graph_us(calls):
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            for fn in calls[:4]:
                fn()
            side.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                for fn in calls:
                    fn()
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        best = float("inf")
        for _ in range(5):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); graph.replay(); e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        return best * 1e3 / len(calls)

    rows = []
    for key in ("c1_single_512", "c2_gpt2_small"):
        wl = si.WORKLOADS[key]
        for idx, lay in enumerate(wl.layers):
            n_w = lay.d_in * lay.d_out
            act = 2.0 * wl.tokens * (lay.d_in + lay.d_out)
            set_bytes = 2.0 * n_w * 2.25 + 2.0 * act                      # W + both compressed copies, X, dY, Y, dX
            nsets = int(min(128, max(4, -(-160e6 // set_bytes))))
            sets = []
            for _ in range(nsets):
                s = LayerState(B, torch, wl, idx, wl.tokens, dev)
                B.slope_prune_24(s.W, s.Wc_vals, s.Wc_meta, s.mask1)
                B.slope_double_prune(s.W, s.mask1, s.WTc_vals, s.WTc_meta, None)
                sets.append(s)
            flop = 2.0 * wl.tokens * n_w
            ops = {
                "prune_24": (lambda s: B.slope_prune_24(s.W, s.Wc_vals, s.Wc_meta, s.mask1), 0.0, 3.25 * n_w, None),
                "double_prune": (lambda s: B.slope_double_prune(s.W, s.mask1, s.WTc_vals, s.WTc_meta, None), 0.0,
                                 3.25 * n_w, None),
                "linear_fwd": (lambda s: B.slope_linear_fwd(s.X, s.Wc_vals, s.Wc_meta, s.d_out, s.Y), flop,
                               act + 1.125 * n_w, 2.0 * pk["bf16"]),
                "linear_bwd_dx": (lambda s: B.slope_linear_bwd_dx(s.dY, s.WTc_vals, s.WTc_meta, s.d_in, s.dX), flop,
                                  act + 1.125 * n_w, 2.0 * pk["bf16"]),
                "linear_bwd_dw_masked": (lambda s: B.slope_linear_bwd_dw_masked(s.dY, s.X, s.mask1, s.dWc), flop,
                                         act + 1.125 * n_w, pk["bf16"]),
            }
            launches = nsets * max(1, -(-min_launches // nsets))
            for op, (fn, fl, nbytes, peak_tf) in ops.items():
                hot = graph_us([lambda fn=fn: fn(sets[0])] * launches)
                cold = graph_us([lambda fn=fn, s=sets[i % nsets]: fn(s) for i in range(launches)])
                t_star = max(fl / (peak_tf * 1e12) if peak_tf else 0.0, nbytes / (pk["hbm_gbs"] * 1e9)) * 1e6
                rows.append({"workload": key, "layer": lay.name, "d_in": lay.d_in, "d_out": lay.d_out,
                             "tokens": wl.tokens, "op": op, "buffer_sets": nsets, "hot_us": round(hot, 2),
                             "cold_us": round(cold, 2), "roofline_us": round(t_star, 2),
                             "roofline_frac_cold": round(t_star / cold, 3),
                             "tflops_dense_eq_cold": round(fl / cold / 1e6, 1) if fl else None})
            del sets
    st = B.slope_poll_status()
    if st != 0:
        raise SystemExit(f"device status after the small-config probe: {B.slope_status_string(st)}")
    return {"what": f"us per launch from CUDA graphs of >= {min_launches} launches (best of 5 replays); hot = one buffer "
                    f"set, cold = cycling through buffer_sets sets (> 160 MB together); t* from burst peaks (dense "
                    f"{pk['bf16']} TFLOP/s, sparse := 2x, HBM {pk['hbm_gbs']} GB/s)", "rows": rows}


def nm_probe(torch, B, layers, stream, pk, reps=10):
    """General N:M pruning to masked-dense matrices on the largest layer: both passes and the
    gradient mask, HBM-bound, against the measured HBM peak (2 B in + 2 B out per element, plus
    the 1/8 B mask read and / or written)."""
    s = max(layers, key=lambda l: l.d_in * l.d_out)
    n_el = s.d_in * s.d_out
    WR = torch.empty_like(s.W)
    WRC = torch.empty_like(s.W)
    m1 = torch.empty_like(s.mask1)
    m2 = torch.empty_like(s.mask1)
    rows = []
    for n, m in ((1, 2), (2, 4), (2, 8), (4, 16)):
        calls = {
            "prune_nm": (lambda: B.slope_prune_nm(s.W, n, m, WR, m1), 4.125 * n_el),
            "double_prune_nm": (lambda: B.slope_double_prune_nm(WR, m1, n, m, WRC, m2), 4.25 * n_el),
        }
        if (n, m) == (2, 4):
            calls["apply_mask"] = (lambda: B.slope_apply_mask(s.W, m1, WRC), 4.125 * n_el)
        for op, (fn, nbytes) in calls.items():
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(reps):
                fn()
            e1.record(stream)
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / reps
            gbs = nbytes / (ms * 1e-3) / 1e9
            rows.append({"op": op, "pattern": f"{n}:{m}", "d_in": s.d_in, "d_out": s.d_out, "ms": round(ms, 4),
                         "algorithmic_bytes": int(nbytes), "gbs": round(gbs, 1),
                         "frac_of_hbm_peak": round(gbs / pk["hbm_gbs"], 4)})
    return {"what": f"{reps} back-to-back launches on the largest layer ({n_el * 2 / 1e6:.0f} MB dense, working set of "
                    f"one call > L2), CUDA events; HBM peak {pk['hbm_gbs']} GB/s ({pk['src']})", "rows": rows}


def inference_forward_probe(torch, B, wl, pk, copies=12, reps=5):
    """Forward only at decode sizes (8 and 64 tokens), without and with adapters (the workload's
    rank, else 64 = 1.56 % of 4096, and 256 = 6.25 %): the GEMM is a stream of compressed weights
    from HBM.  Each shape is timed as a CUDA graph of `copies` launches over distinct weight
    copies (together larger than L2), best of `reps` replays; cuBLAS on the dense bf16 weight
    in the same harness for comparison."""
    dev = torch.device("cuda")
    shapes = []
    for lay in wl.layers:
        if (lay.d_in, lay.d_out) not in shapes:
            shapes.append((lay.d_in, lay.d_out))
    ranks = [0, wl.rank if wl.rank else 64, 256]

    def time_graph(fn):
        side = torch.cuda.Stream()
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            fn(); fn()
            side.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                fn()
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        best = float("inf")
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); graph.replay(); e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        return best * 1e3 / copies                         # microseconds per layer call

    rows = []
    for d_in, d_out in shapes[:3]:
        W = B.bf16_from_bits(si.gaussian_bf16((d_out, d_in), 0.02, si.seed_for(9, 0, "W")), dev)
        vals, meta, _ = B.alloc_compressed(d_out, d_in, dev)
        B.slope_prune_24(W, vals, meta, None)
        Wc = [(vals.clone(), meta.clone()) for _ in range(copies)]
        Wd = [W.clone() for _ in range(copies)]
        for b in (1, 8, 64, 512, 2048):
            X = B.bf16_from_bits(si.gaussian_bf16((b, d_in), 1.0, si.seed_for(9, 0, "X")), dev)
            Y = torch.empty((b, d_out), dtype=torch.bfloat16, device=dev)
            us_dense = time_graph(lambda: [torch.matmul(X, w.t(), out=Y) for w in Wd])
            for r in ranks:
                if r:
                    L = B.bf16_from_bits(si.gaussian_bf16((d_in, r), 0.01, si.seed_for(9, 0, "L")), dev)
                    R = B.bf16_from_bits(si.gaussian_bf16((r, d_out), 0.01, si.seed_for(9, 0, "R")), dev)
                    T = torch.empty((b, r), dtype=torch.bfloat16, device=dev)

                    def run():
                        for v, m in Wc:
                            B.slope_linear_fwd_adapter(X, v, m, d_out, L, R, T, Y)

                    def run_two_calls():
                        for v, m in Wc:
                            B.slope_adapter_fwd_bwd(0, X, None, L, None, b, d_out, d_in, r, T=T)
                            B.slope_linear_fwd(X, v, m, d_out, Y, T, R)
                    us_two = time_graph(run_two_calls)
                else:
                    def run():
                        for v, m in Wc:
                            B.slope_linear_fwd(X, v, m, d_out, Y)
                    us_two = None
                us = time_graph(run)
                nbytes = d_in * d_out * 1.125 + 2.0 * b * (d_in + d_out) + 2.0 * r * (d_in + d_out) + 4.0 * b * r
                gbs = nbytes / (us * 1e-6) / 1e9
                rows.append({"d_in": d_in, "d_out": d_out, "tokens": b, "rank": r, "us": round(us, 2),
                             "algorithmic_bytes": int(nbytes), "gbs": round(gbs, 1),
                             "frac_of_hbm_peak": round(gbs / pk["hbm_gbs"], 4),
                             "cublas_dense_us": round(us_dense, 2), "speedup_vs_cublas_dense": round(us_dense / us, 3),
                             "separate_adapter_call_us": None if us_two is None else round(us_two, 2)})
        del Wc, Wd
    st = B.slope_poll_status()
    if st != 0:
        raise SystemExit(f"device status after the inference probe: {B.slope_status_string(st)}")
    return {"what": f"forward only (with adapters: slope_linear_fwd_adapter, T = X L and the sparse GEMM with the fused "
                    f"T R term as an overlapped pair of launches; separate_adapter_call_us = slope_adapter_fwd_bwd(0) "
                    f"then slope_linear_fwd), CUDA graph of {copies} calls over distinct "
                    f"weight copies, best of {reps} replays, us per call; bytes: 1.125 B per weight element "
                    f"(values + metadata) + activations + adapter factors; HBM peak {pk['hbm_gbs']} GB/s "
                    f"({pk['src']}); cuBLAS reads the dense bf16 weight (2 B per element, no adapter)",
            "rows": rows}


def decode_block_probe(torch, B, blocks=4, reps=5):
    """decode_block_width for LLaMA-7B and LLaMA-13B widths."""
    return {"llama7b": decode_block_width(torch, B, 4096, 11008, blocks, reps),
            "llama13b": decode_block_width(torch, B, 5120, 13824, blocks, reps)}


def decode_block_width(torch, B, d, ffn, blocks=4, reps=5):
    """The linears of a LLaMA-style decoder block (width d, hidden ffn) at decode sizes, in the order
    a block runs them and each fed by a real predecessor in the stream: q, k, v stacked along d_out
    (d -> 3d), o, gate and up stacked (d -> 2 ffn), down; `blocks` blocks with their own weights (> L2
    together) in one CUDA graph.  Stacking is exact for both pruning passes.  The activations between
    the linears are stand-ins of the right shape (attention and the gate are not part of this
    library).  With adapters every linear is one slope_linear_fwd_adapter call; cuBLAS runs the
    dense bf16 weights without adapters."""
    dev = torch.device("cuda")
    shapes = [("qkv", d, 3 * d), ("o", d, d), ("gate_up", d, 2 * ffn), ("down", ffn, d)]
    gen = torch.Generator(device="cuda").manual_seed(si.seed_for(8, 0, "W"))
    mk = lambda shape, sigma: (torch.randn(shape, device="cuda", generator=gen) * sigma).bfloat16()
    dense, sparse, adapters = [], [], {64: [], 256: []}
    for _ in range(blocks):
        dl, sl = [], []
        for name, d_in, d_out in shapes:
            W = mk((d_out, d_in), 0.02)
            vals, meta, _ = B.alloc_compressed(d_out, d_in, dev)
            B.slope_prune_24(W, vals, meta, None)
            dl.append(W)
            sl.append((vals, meta, d_out))
        dense.append(dl)
        sparse.append(sl)
    for r in adapters:
        adapters[r] = [(mk((d_in, r), 0.01), mk((r, d_out), 0.01)) for _, d_in, d_out in shapes]

    def time_graph(fn):
        side = torch.cuda.Stream()
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            fn(); fn()
            side.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                fn()
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        best = float("inf")
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); graph.replay(); e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        return best * 1e3 / blocks                          # microseconds per block

    rows = []
    for b in (1, 8):
        X = {w: mk((b, w), 1.0) for w in (d, ffn)}
        Y = {n: torch.empty((b, d_out), dtype=torch.bfloat16, device=dev) for n, _, d_out in shapes}

        def run_dense():
            for dl in dense:
                for (name, d_in, d_out), W in zip(shapes, dl):
                    torch.matmul(X[d_in], W.t(), out=Y[name])

        def run_sparse():
            for sl in sparse:
                for (name, d_in, d_out), (vals, meta, _) in zip(shapes, sl):
                    B.slope_linear_fwd(X[d_in], vals, meta, d_out, Y[name])

        us_dense, us_sparse = time_graph(run_dense), time_graph(run_sparse)
        row = {"tokens": b, "cublas_dense_us_per_block": round(us_dense, 1), "slope_us_per_block": round(us_sparse, 1),
               "speedup": round(us_dense / us_sparse, 3)}
        for r, facs in adapters.items():
            T = torch.empty((b, r), dtype=torch.bfloat16, device=dev)

            def run_adapter():
                for sl in sparse:
                    for (name, d_in, d_out), (vals, meta, _), (L, R) in zip(shapes, sl, facs):
                        B.slope_linear_fwd_adapter(X[d_in], vals, meta, d_out, L, R, T, Y[name])

            us = time_graph(run_adapter)
            row[f"slope_rank{r}_us_per_block"] = round(us, 1)
            row[f"speedup_rank{r}"] = round(us_dense / us, 3)
        rows.append(row)
    st = B.slope_poll_status()
    if st != 0:
        raise SystemExit(f"device status after the decode block probe: {B.slope_status_string(st)}")
    weight_bytes = sum(d_in * d_out for _, d_in, d_out in shapes)
    return {"what": f"the four linears of a LLaMA-style decoder block of width {d} / {ffn} at decode sizes (q, k, v stacked; gate, up stacked), "
                    f"{blocks} blocks with their own weights in one CUDA graph, us per block, best of {reps} replays; "
                    f"compressed weights {weight_bytes * 1.125 / 1e6:.0f} MB per block against {weight_bytes * 2 / 1e6:.0f} MB dense",
            "rows": rows}


def burst_probe(torch, B, layers, stream, pk, launches=8):
    """Context only, not the headline: the GEMM kernels timed alone in short bursts after an idle
    pause, i.e. before the 1 kW power cap pulls the SM clock down, against the burst peaks."""
    rows = []
    seen = set()
    for s in layers:
        if (s.d_in, s.d_out) in seen:
            continue
        seen.add((s.d_in, s.d_out))
        calls = {
            "linear_fwd": lambda s=s: B.slope_linear_fwd(s.X, s.Wc_vals, s.Wc_meta, s.d_out, s.Y),
            "linear_bwd_dx": lambda s=s: B.slope_linear_bwd_dx(s.dY, s.WTc_vals, s.WTc_meta, s.d_in, s.dX),
            "linear_bwd_dw_masked": lambda s=s: B.slope_linear_bwd_dw_masked(s.dY, s.X, s.mask1, s.dWc),
        }
        for op, fn in calls.items():
            fn()
            torch.cuda.synchronize()
            time.sleep(0.5)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(launches):
                fn()
            e1.record(stream)
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / launches
            tf = 2.0 * s.b * s.d_in * s.d_out / (ms * 1e-3) / 1e12
            peak = pk["bf16"] if op == "linear_bwd_dw_masked" else 2.0 * pk["bf16"]
            rows.append({"layer": s.name, "d_in": s.d_in, "d_out": s.d_out, "op": op, "ms": round(ms, 4),
                         "tflops_dense_eq": round(tf, 1), "frac_of_burst_peak": round(tf / peak, 4)})
    return {"what": f"{launches} back-to-back launches after a 0.5 s idle pause, CUDA events; peaks: dense {pk['bf16']}"
                    f" TFLOP/s burst ({pk['src']}), sparse := 2 x dense", "rows": rows}


def dense_comparison(torch, B, layers, stream, reps=5):
    """fwd+bwd of the same layers as dense bf16 GEMMs, once through torch.matmul (cuBLAS) and once
    through this library's own dense tcgen05 kernels, interleaved with the SLoPe stages
    fwd/dX/dW (no pruning, no adapter) in the same process."""
    totals = {"cublas": 0.0, "inhouse": 0.0, "slope": 0.0}
    rows = []
    for s in layers:
        Wd = s.W
        Yd = torch.empty_like(s.Y)
        dXd = torch.empty_like(s.dX)
        dWd = torch.empty_like(s.W)

        def cublas():
            Y = torch.matmul(s.X, Wd.t())
            dX = torch.matmul(s.dY, Wd)
            dW = torch.matmul(s.dY.t(), s.X)
            del Y, dX, dW

        def inhouse():
            B.slope_dense_linear_fwd(s.X, Wd, Yd)
            B.slope_dense_linear_bwd_dx(s.dY, Wd, dXd)
            B.slope_dense_linear_bwd_dw(s.dY, s.X, dWd)

        def slope():
            B.slope_linear_fwd(s.X, s.Wc_vals, s.Wc_meta, s.d_out, s.Y)
            B.slope_linear_bwd_dx(s.dY, s.WTc_vals, s.WTc_meta, s.d_in, s.dX)
            B.slope_linear_bwd_dw_masked(s.dY, s.X, s.mask1, s.dWc)

        arms = {"cublas": cublas, "inhouse": inhouse, "slope": slope}
        times = {k: [] for k in arms}
        for _ in range(reps + 1):
            evs = {}
            for k, fn in arms.items():
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                fn()
                e1.record(stream)
                evs[k] = (e0, e1)
            torch.cuda.synchronize()
            for k, (e0, e1) in evs.items():
                times[k].append(e0.elapsed_time(e1))
        med = {k: statistics.median(v[1:]) for k, v in times.items()}
        for k in totals:
            totals[k] += med[k]
        rows.append({"layer": s.name, "dense_ms": round(med["cublas"], 4), "inhouse_dense_ms": round(med["inhouse"], 4),
                     "slope_ms": round(med["slope"], 4), "speedup": round(med["cublas"] / med["slope"], 3),
                     "speedup_vs_inhouse_dense": round(med["inhouse"] / med["slope"], 3)})
        del Yd, dXd, dWd
    return {"what": "dense layer Y=XW^T, dX=dY W, dW=dY^T X through torch.matmul (cuBLAS) and through the library's own "
                    "dense tcgen05 kernels (slope_dense_linear_*) vs slope fwd+dX+masked dW, same shapes, interleaved",
            "dense_ms": round(totals["cublas"], 4), "inhouse_dense_ms": round(totals["inhouse"], 4),
            "slope_ms": round(totals["slope"], 4), "speedup": round(totals["cublas"] / totals["slope"], 3),
            "speedup_vs_inhouse_dense": round(totals["inhouse"] / totals["slope"], 3), "layers": rows}


def decoder_block_probe(torch, reps=5):
    """c5_llama13b_block as one decoder-block training step with real data flow (normalisation ->
    q, k, v -> causal attention -> o -> residual -> normalisation -> gate, up -> SiLU * up -> down
    -> residual; forward + backward, no optimizer).  The seven linears run through the library
    (rank-128 adapters) or, for the all-dense arm, through torch (cuBLAS); normalisation,
    attention, gate and residuals are torch in both arms.  Linear calls are bracketed by CUDA
    events inside the step, so their sum is reported next to the whole-block time."""
    from paper_2608_24070_b200 import block_harness as H

    wl = si.WORKLOADS["c5_llama13b_block"]
    batch, seq, heads, r = 4, 2048, 40, wl.rank
    tokens, d = batch * seq, wl.layers[0].d_in
    gen = torch.Generator(device="cuda").manual_seed(si.seed_for(5, 0, "W"))
    mk = lambda shape, sigma: (torch.randn(shape, device="cuda", generator=gen) * sigma).bfloat16()
    arms = {"slope": {}, "dense": {}}
    for l in wl.layers:
        W = mk((l.d_out, l.d_in), 0.02)
        arms["slope"][l.name] = H.SlopeLinear(W, mk((l.d_in, r), 0.01), mk((r, l.d_out), 0.01), max_tokens=tokens)
        arms["dense"][l.name] = H.DenseLinear(W)
        del W
    x, dout = mk((tokens, d), 1.0), mk((tokens, d), 1.0)
    block_ms = {k: [] for k in arms}
    linear_ms = {k: [] for k in arms}
    for _ in range(reps + 2):
        for k, layers in arms.items():
            timers = []
            for lay in layers.values():
                lay.timers = timers
                if k == "dense":
                    lay.W.grad = None
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            H.block_step(x, dout, layers, batch, seq, heads)
            e1.record()
            torch.cuda.synchronize()
            block_ms[k].append(e0.elapsed_time(e1))
            linear_ms[k].append(H.elapsed_ms(timers))
    med = lambda v: statistics.median(v[2:])
    res = {k: {"linears_ms": round(med(linear_ms[k]), 4), "block_ms": round(med(block_ms[k]), 4)} for k in arms}
    return {"what": "one decoder-block step (forward + backward) at LLaMA-13B width: 8192 tokens = 4 x 2048, 40 heads, "
                    "seven linears through the library with rank-128 adapters vs the same block with dense torch "
                    "(cuBLAS) linears and no adapters; non-linear glue is torch in both; seeded torch.randn inputs; "
                    "median of %d steps after 2 warm-ups, arms interleaved" % reps,
            **res,
            "speedup_linears": round(res["dense"]["linears_ms"] / res["slope"]["linears_ms"], 3),
            "speedup_block": round(res["dense"]["block_ms"] / res["slope"]["block_ms"], 3)}


def cusparselt_context(torch, B, layers, stream, reps=10):
    """Context, not a target: the forward GEMM of each distinct layer shape through
    torch.sparse.to_sparse_semi_structured + F.linear (cuSPARSELt), next to slope_linear_fwd, with
    the relative error of both against torch.matmul on the same masked dense weight."""
    rows, seen = [], set()
    try:
        from torch.sparse import to_sparse_semi_structured
        version = torch.backends.cusparselt.version() if torch.backends.cusparselt.is_available() else None
    except Exception as ex:                                 # noqa: BLE001
        return {"unavailable": f"{type(ex).__name__}: {ex}"}
    for s in layers:
        if (s.d_in, s.d_out) in seen:
            continue
        seen.add((s.d_in, s.d_out))
        try:
            shifts = torch.arange(8, device=s.W.device, dtype=torch.uint8)
            keep = ((s.mask1.unsqueeze(-1) >> shifts) & 1).bool().view(s.d_out, s.d_in)     # slope_prune_24's mask
            Wp = (s.W * keep).contiguous()
            Ws = to_sparse_semi_structured(Wp)
            ref = torch.matmul(s.X, Wp.t()).float()

            def timed(fn):
                fn()
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for _ in range(reps):
                    y = fn()
                e1.record(stream)
                torch.cuda.synchronize()
                return e0.elapsed_time(e1) / reps, y

            ms_lib, y_lib = timed(lambda: torch.nn.functional.linear(s.X, Ws))
            ms_own, _ = timed(lambda: (B.slope_linear_fwd(s.X, s.Wc_vals, s.Wc_meta, s.d_out, s.Y), s.Y)[1])
            flop = 2.0 * s.b * s.d_in * s.d_out
            rows.append({"d_in": s.d_in, "d_out": s.d_out, "tokens": s.b,
                         "cusparselt_ms": round(ms_lib, 4), "cusparselt_tflops_dense_eq": round(flop / ms_lib / 1e9, 1),
                         "cusparselt_rel_err_vs_dense": round(float((y_lib.float() - ref).norm() / ref.norm()), 5),
                         "slope_fwd_ms": round(ms_own, 4), "slope_tflops_dense_eq": round(flop / ms_own / 1e9, 1),
                         "slope_rel_err_vs_dense": round(float((s.Y.float() - ref).norm() / ref.norm()), 5)})
            del Ws, Wp, ref, y_lib
        except Exception as ex:                             # noqa: BLE001
            rows.append({"d_in": s.d_in, "d_out": s.d_out, "failed": f"{type(ex).__name__}: {str(ex)[:200]}"})
    return {"what": f"forward GEMM through torch.sparse.to_sparse_semi_structured + F.linear (cuSPARSELt {version}) vs "
                    f"slope_linear_fwd, {reps} back-to-back launches each, CUDA events; both on slope_prune_24's mask, "
                    f"errors against torch.matmul on the masked dense weight", "rows": rows}


def e2e_run(torch, B, layers, de_flops, steps):
    """Same step with HOST buffers: every step copies each layer's X and dY from pinned host
    memory, runs the path through the C ABI, and reads the compressed weight gradient back.
    Copies run on their own streams so that layer i+1's inputs travel while layer i computes;
    every copy and every kernel of a step lies inside the timed region."""
    compute = torch.cuda.current_stream()
    h2d_stream, d2h_stream = torch.cuda.Stream(), torch.cuda.Stream()
    host = {}
    for s in layers:
        for nm, t in (("X", s.X), ("dY", s.dY)):
            key = (nm, tuple(t.shape))
            if key not in host:
                host[key] = t.cpu().pin_memory()
        for nm in ("dWc", "dL", "dR") if s.r else ("dWc",):
            t = getattr(s, nm)
            key = (nm, tuple(t.shape))
            if key not in host:
                host[key] = torch.empty(t.shape, dtype=t.dtype).pin_memory()
    h2d = sum(2 * (s.X.numel() + s.dY.numel()) for s in layers)
    d2h = sum(2 * (s.dWc.numel() + (s.dL.numel() + s.dR.numel() if s.r else 0)) for s in layers)
    n = len(layers)
    arrived = [torch.cuda.Event() for _ in range(n)]       # inputs of layer i are on the device
    consumed = [torch.cuda.Event() for _ in range(n)]      # layer i's kernels are done with its inputs
    read_back = [torch.cuda.Event() for _ in range(n)]     # layer i's gradient has left the device
    for ev in consumed + read_back:
        ev.record(compute)

    def step():
        for i, s in enumerate(layers):
            with torch.cuda.stream(h2d_stream):
                h2d_stream.wait_event(consumed[i])
                s.X.copy_(host[("X", tuple(s.X.shape))], non_blocking=True)
                s.dY.copy_(host[("dY", tuple(s.dY.shape))], non_blocking=True)
                arrived[i].record(h2d_stream)
        for i, s in enumerate(layers):
            compute.wait_event(arrived[i])
            compute.wait_event(read_back[i])
            run_layer(B, s)
            consumed[i].record(compute)
            with torch.cuda.stream(d2h_stream):
                d2h_stream.wait_event(consumed[i])
                for nm in ("dWc", "dL", "dR") if s.r else ("dWc",):
                    t = getattr(s, nm)
                    host[(nm, tuple(t.shape))].copy_(t, non_blocking=True)
                read_back[i].record(d2h_stream)

    def drain():
        compute.wait_stream(h2d_stream)
        compute.wait_stream(d2h_stream)

    step()
    drain()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(compute)
    for _ in range(steps):
        step()
    drain()
    e1.record(compute)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    return {"value": round(de_flops / (ms * 1e-3) / 1e12, 2), "unit": UNIT, "ms_per_step": round(ms, 3),
            "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": steps,
            "note": "pinned host X, dY -> device per layer (copy stream, overlapped with compute), C-ABI kernels, "
                    "the layer's parameter gradients (compressed dW, dL, dR) -> pinned host; Y and dX stay on the "
                    "device on purpose: they are the next / previous layer's input, not a result the host reads"}


if __name__ == "__main__":
    main()
