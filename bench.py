#!/usr/bin/env python
"""Benchmark of the per-example clipping path: clipped+noised gradient examples/s.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4] [--impl reference]

A "step" is one pass of the whole path (per-layer squared norms -> clip factors
-> clipped sums -> noise) over one batch of synthetic inputs shaped like the
paper's workloads.  The headline workload is the largest single-GPU
configuration: the sequence-model layers at B = 128, T = 256 in bf16 (cfg4).
The other configurations (the two MLPs, the CNN in both precisions, the
Gram-vs-materialise sweep) are timed in the same run; their step times and
roofline fractions are in the JSON line under "configs" (compact, printed last)
and, with per-kernel detail, under "workloads".  Rank 0 prints ONE JSON line.

Timing: CUDA events on the launching stream, max over ranks.  Models with T > 1
layers (hundreds of microseconds per step): one step = one replay of a CUDA
graph that holds ONE dpclip_step_streams call (the library forks over four
streams inside the call); events around every step, the L2 flushed by a 256 MB
write between steps (outside the events).  All-T=1 models (one launch of about
ten microseconds per step): the K timed steps are recorded back to back into
one CUDA graph, step i working on its own copy i % R of the inputs and outputs
with R copies adding up to more than twice the L2, and one event pair brackets
the K steps -- the steady state of a training loop, without a graph-launch
latency charged to every step.  The per-step-graph figure is reported beside it
("single_step_graph_ms_per_step"), and so is the measured floor of an empty
launch of the same shape ("launch_floor_us").
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import workloads  # noqa: E402

METRIC = "clipped+noised gradient examples/sec"
UNIT = "examples/s"
FFMA_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12        # 148 SMs x 128 fp32 lanes x 2 flop x 1.965 GHz


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# ---------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.samples = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append((time.time(), line.strip()))

    def stop(self, t0=None, t1=None):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        mhz, mx, reasons = [], None, set()
        for ts, line in self.samples:
            if t0 is not None and not (t0 - 0.05 <= ts <= t1 + 0.15):
                continue
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                mhz.append(float(parts[0])); mx = float(parts[1])
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=float(np.median(mhz)) if mhz else None, sm_max_mhz=mx, reasons=sorted(reasons),
                    samples=len(mhz))


# ---------------------------------------------------------------------------
# algorithmic work per kernel launch
# ---------------------------------------------------------------------------
def elt_bytes(dtype):
    return 4 if dtype == "f32" else 2


def layer_work(w, spec, kind):
    """(algorithmic bytes, flops) of one launch of `kind` on one layer: every
    input element read once, every output written once; flops of the exact
    form the kernel evaluates."""
    es = elt_bytes(w.dtype)
    inp = w.B * spec.T * (spec.d_in + spec.d_out) * es
    P = spec.d_in * spec.d_out + (spec.d_out if spec.has_bias else 0)
    if kind == "norm_t1":
        return inp + 4 * w.B, 2 * w.B * (spec.d_in + spec.d_out)
    if kind == "norm_simt" or kind == "norm_mat":
        return inp + 4 * w.B, 2 * w.B * spec.T * spec.d_in * spec.d_out
    if kind == "norm_gram":
        return inp + 4 * w.B, w.B * spec.T * (spec.T + 1) * (spec.d_in + spec.d_out)
    if kind == "grad":
        return inp + 4 * P, 2 * w.B * spec.T * spec.d_in * spec.d_out
    if kind == "noise":
        return 8 * P, 0
    raise ValueError(kind)


def step_algorithmic_bytes(w):
    """Two passes over the inputs (norms, then the clipped sum: the factor of
    an example depends on all its layers) + every output written once."""
    return 2 * w.input_bytes() + 4 * w.n_params


TF32X3_PER_BF16 = (1.1 / 2.25) / 3.0      # nominal tf32 : bf16 dense ratio, three tf32 MMAs per fp32 product


def step_algorithmic_flops(w):
    """The cheaper exact norm form per layer (closed form for T = 1; symmetric Gram or one materialised
    product for T > 1) + the one clipped-sum product per layer."""
    norm = grad = 0.0
    for s in w.layers:
        if s.T == 1:
            norm += 2.0 * w.B * (s.d_in + s.d_out)
        else:
            norm += min(float(w.B) * s.T * (s.T + 1) * (s.d_in + s.d_out), 2.0 * w.B * s.T * s.d_in * s.d_out)
        grad += 2.0 * w.B * s.T * s.d_in * s.d_out
    return norm, grad


def step_roofline(w, peaks):
    """Lower bound of a whole step: max(algorithmic bytes / HBM bandwidth, algorithmic flops / the peak of the
    engine the contractions run on).  Bytes: every input twice (norm pass, clipped-sum pass) + every output
    once.  Engine: bf16 -> the tensor cores (burst and sustained figures both given; the burst one binds
    harder and is the one `frac` uses, since clocks stay at their maximum in these sub-millisecond steps);
    fp32 -> the tensor cores as error-compensated tf32 (measured bf16 peak x nominal tf32:bf16 / 3)."""
    nbytes = step_algorithmic_bytes(w)
    f_norm, f_grad = step_algorithmic_flops(w)
    flops = f_norm + f_grad
    t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9)
    if w.dtype == "bf16":
        engine, peak, peak_sus = "tensor bf16", peaks["bf16_tflops"], peaks["bf16_tflops_sustained"]
    else:
        engine = "tensor 3xtf32"
        peak, peak_sus = peaks["bf16_tflops"] * TF32X3_PER_BF16, peaks["bf16_tflops_sustained"] * TF32X3_PER_BF16
    t_eng, t_eng_sus = flops / (peak * 1e12), flops / (peak_sus * 1e12)
    return dict(bytes=int(nbytes), flops=flops, engine=engine, t_hbm_us=t_hbm * 1e6, t_engine_burst_us=t_eng * 1e6,
                t_engine_sustained_us=t_eng_sus * 1e6, bound="hbm" if t_hbm >= t_eng else "tensor",
                roof_us=max(t_hbm, t_eng) * 1e6, roof_sustained_us=max(t_hbm, t_eng_sus) * 1e6)


# ---------------------------------------------------------------------------
# device arm
# ---------------------------------------------------------------------------
def to_dev(x, dtype, torch):
    t = torch.from_numpy(x).cuda()
    return t if dtype == "f32" else t.to(torch.bfloat16)


def make_plan(dp, w, layers, torch):
    return dp.StepPlan([dp.Layer(to_dev(A, w.dtype, torch), to_dev(Z, w.dtype, torch), s.has_bias)
                        for (A, Z), s in zip(layers, w.layers)])


def time_steps(torch, fn, steps, warmup, flush):
    """Per-step device times (ms): events around each step, L2 flush between."""
    for _ in range(warmup):
        flush(); fn()
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for s, e in ev:
        flush()
        s.record(); fn(); e.record()
    torch.cuda.synchronize()
    return [s.elapsed_time(e) for s, e in ev]


L2_BYTES = 126 << 20


def time_steps_rotating(torch, dp, w, layers, steps, warmup, flush):
    """Launch-bound small models: K steps back to back in ONE CUDA graph, step i working on input/output
    set i % R, with R sets whose total footprint is at least twice the L2 (or R = K distinct sets and a
    flush before the region), so every step finds its inputs in HBM; one event pair around the K steps.
    This is the steady state of a training loop (kernels queued back to back) without the per-replay
    launch latency that per-step events around single-step graphs would add to every step."""
    footprint = w.input_bytes() + 4 * w.n_params
    R = int(min(steps, max(2, -(-2 * L2_BYTES // footprint))))
    plans = [make_plan(dp, w, layers, torch) for _ in range(R)]
    for pl in plans:
        pl.run(w.C, w.sigma, 1)
    torch.cuda.synchronize()
    for i in range(warmup):
        plans[i % R].run(w.C, w.sigma, 1)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for i in range(steps):
            plans[i % R].run(w.C, w.sigma, 1)
    graph.replay()                                   # untimed: uploads the graph
    torch.cuda.synchronize()
    reps = []
    for _ in range(3):
        flush()
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record(); graph.replay(); e.record()
        torch.cuda.synchronize()
        reps.append(s.elapsed_time(e))
    for pl in plans:
        assert dp.dpclip_read_status(pl.workspace) == 0
    total = float(np.median(reps))
    return [total / steps] * steps, dict(sets=R, set_bytes=int(footprint), region_ms=reps)


def kernel_breakdown(torch, dp, w, plan, steps, flush, C, sigma):
    """Second, instrumented pass of the same steps: one event pair around every
    entry-point call, to attribute the step time to kernels."""
    acc = {}

    def timed(key, fn):
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record(); fn(); e.record()
        acc.setdefault(key, []).append((s, e))

    # what dpclip_step does: layers whose norms go by the Gram identity share a launch, and so do the clipped
    # sums of layers of one shape; the grouped calls report which layers they took
    taken_n = taken_g = [False] * len(w.layers)
    for it in range(steps + 1):
        flush()
        box = {}
        timed(("norm_gram_group", -2), lambda: box.update(t=dp.dpclip_gram_layers_sqnorms(plan)))
        taken_n = box["t"]
        for l, (y, spec) in enumerate(zip(plan.layers, w.layers)):
            if taken_n[l]:
                continue
            m = dp.dpclip_pick_method(w.B, spec.T, spec.d_in, spec.d_out, None, None, plan.dtype_code)
            kind = {dp.DPCLIP_T1: "norm_t1", dp.DPCLIP_SIMT: "norm_simt", dp.DPCLIP_GRAM: "norm_gram",
                    dp.DPCLIP_MATERIALIZE: "norm_mat"}[m]
            timed((kind, l), lambda: dp.dpclip_layer_sqnorms(y.A, y.Zbar, spec.has_bias, plan.sq_layers[l],
                                                             plan.workspace))
        timed(("factors", -1), lambda: dp.dpclip_factors(plan.sq_layers, C, plan.clip, plan.norms))
        timed(("grad_group", -3), lambda: box.update(g=dp.dpclip_same_shape_layers_clipped_grad_noise(plan, C, sigma, 1, 0)))
        taken_g = box["g"]
        for l, (y, spec) in enumerate(zip(plan.layers, w.layers)):
            if taken_g[l]:
                continue
            # the clipped sum with its noise, as the step launches it (noise folded into the last pass over the output)
            timed(("grad", l), lambda: dp.dpclip_clipped_grad_noise(y.A, y.Zbar, plan.clip, plan.gW[l], plan.gb[l], sigma, C,
                                                                    1, 2 * l, 2 * l + 1, plan.workspace))
    if not any(taken_n):
        acc.pop(("norm_gram_group", -2))
    if not any(taken_g):
        acc.pop(("grad_group", -3))
    kernel_breakdown.groups = {"norm_gram_group": [l for l, t in enumerate(taken_n) if t],
                               "grad_group": [l for l, t in enumerate(taken_g) if t]}
    torch.cuda.synchronize()
    out = {}
    for key, evs in acc.items():
        ts = [s.elapsed_time(e) for s, e in evs[1:]]            # first iteration is warm-up
        out[key] = float(np.mean(ts))
    return out


kernel_breakdown.groups = {}          # members of the grouped launches of the last breakdown


# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu captures
# summarised under profiles/ (same workload, same launch configuration); None where not captured
NCU_TRAFFIC_BYTES = {
    ("mlp_784_1000_1000_10_b128", "t1_all_grads_tf32_kernel"): 2.55e6,   # profiles/fused_t1_mlp_784_1000_1000_10_b128.txt
    ("mlp_784_1000_1000_10_b128", "t1_all_grads_kernel"): 2.54e6,
    ("seq_b128_t256_d512_bf16", "norm_gram_group"): 775.4e6,          # profiles/tc_kernels_seq_b128_t256.txt
    # zta_pair_kernel 772.8 + 24.2 MB, reduce_segments_kernel 50.5 + 0.5 MB (cold-cache capture: inside a step the
    # reduce finds the partial tiles in L2)
    ("seq_b128_t256_d512_bf16", "grad_group"): 848.0e6,
}


def roofline_fused_t1(w, step_ms, peaks):
    """All-T=1 models run inside one dpclip_step call.  Models whose rows TMA can address take the
    one-launch tensor-core kernel (t1_all_grads_tf32_kernel<true, T>: norms, factors, clipped sums, noise;
    fp32 as error-compensated tf32, bf16 as one kind::f16 instruction per 16 rows); others take two launches
    (t1_all_norms_kernel + t1_all_grads_kernel on the fp32 ALUs).  The kernel time is taken as the whole
    step's device time, which can only understate it.  The contraction peak for fp32-by-3xtf32 is the
    measured bf16 peak x the nominal tf32:bf16 ratio / 3; for bf16 it is the measured bf16 peak."""
    flops = sum(2.0 * w.B * s.d_in * s.d_out for s in w.layers)
    # algorithmic bytes of the step: inputs twice (norms, clipped sums) + outputs once.  The one-launch kernel
    # fetches its inputs from HBM once (the second pass hits L2), so its DRAM traffic is below this figure.
    nbytes = step_algorithmic_bytes(w)
    quantum = 4 if w.dtype == "f32" else 8
    on_tensor = all(s.d_in % quantum == 0 and (s.d_out % quantum == 0 or s.d_out <= 16) for s in w.layers)
    kernel = "t1_all_grads_tf32_kernel" if on_tensor else "t1_all_grads_kernel"
    if on_tensor:
        peak_tf = peaks["bf16_tflops"] * (TF32X3_PER_BF16 if w.dtype == "f32" else 1.0)
    else:
        peak_tf = FFMA_PEAK_TFLOPS
    t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9)
    t_alu = flops / (peak_tf * 1e12)
    if t_hbm >= t_alu:
        ach = nbytes / (step_ms * 1e-3) / 1e9
        r = dict(bound="hbm", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s", frac=ach / peaks["hbm_gbs"])
    else:
        ach = flops / (step_ms * 1e-3) / 1e12
        r = dict(bound="tensor" if on_tensor else "alu", achieved=ach, peak=peak_tf, unit="TFLOP/s", frac=ach / peak_tf)
    r.update(traffic=NCU_TRAFFIC_BYTES.get((w.name, kernel)), kernel=kernel,
             kernel_ms=step_ms, share_of_step=1.0, algorithmic_bytes=nbytes, algorithmic_flops=flops,
             launches_per_step=1, hbm_frac=(nbytes / (step_ms * 1e-3) / 1e9) / peaks["hbm_gbs"],
             peak_source=peaks["source"],
             note="whole step in one kernel; time = step device time; both roofs are below any launch (see "
                  "launch_floor_us): the step is a chain of memory round trips (row loads, grid barrier, factor "
                  "loads, tile loads, output stores)")
    return r


def entry_name(w, key):
    """Layer name(s) of a breakdown entry."""
    kind, l = key
    if kind in kernel_breakdown.groups:
        return "+".join(w.layers[i].name for i in kernel_breakdown.groups[kind])
    return w.layers[l].name if l >= 0 else "all"


def roofline_group(w, key, breakdown, peaks):
    """Roofline of a launch that several layers share (bf16, tensor cores): work = the member layers' sum."""
    kind = key[0]
    base = "norm_gram" if kind == "norm_gram_group" else "grad"
    members = kernel_breakdown.groups[kind]
    nbytes = sum(layer_work(w, w.layers[i], base)[0] for i in members)
    flops = sum(layer_work(w, w.layers[i], base)[1] for i in members)
    ms = breakdown[key]
    t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9)
    t_alu = flops / (peaks["bf16_tflops"] * 1e12)
    if t_hbm >= t_alu:
        ach = nbytes / (ms * 1e-3) / 1e9
        r = dict(bound="hbm", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s", frac=ach / peaks["hbm_gbs"])
    else:
        ach = flops / (ms * 1e-3) / 1e12
        r = dict(bound="tensor", achieved=ach, peak=peaks["bf16_tflops"], unit="TFLOP/s", frac=ach / peaks["bf16_tflops"])
    name = f"{kind}[{entry_name(w, key)}]"
    r.update(traffic=NCU_TRAFFIC_BYTES.get((w.name, kind)), kernel=name, kernel_ms=ms,
             share_of_step=ms / sum(breakdown.values()), algorithmic_bytes=nbytes, algorithmic_flops=flops,
             peak_source=peaks["source"])
    return r


def _zta_layers(w):
    """Layers whose clipped sum runs on zta_tc_kernel (bf16, rows TMA can address, not narrow)."""
    if w.dtype != "bf16":
        return []
    return [l for l, s in enumerate(w.layers)
            if s.T > 1 and s.d_in % 8 == 0 and s.d_out % 8 == 0 and not (s.d_in + (1 if s.has_bias else 0) <= 32 and s.d_out <= 64)]


def roofline_zta(w, breakdown, peaks):
    """The bf16 clipped-sum kernel over ALL its launches of a step (grouped launch + per-layer launches): work =
    the layers' sum, time = the sum of the entry-point calls' device times (each call = zta_tc_kernel + the
    reduce/noise launch that follows it), launches counted."""
    members = _zta_layers(w)
    keys = [k for k in breakdown if k[0] == "grad_group" or (k[0] == "grad" and k[1] in members)]
    if not keys:
        return None
    ms = sum(breakdown[k] for k in keys)
    nbytes = sum(layer_work(w, w.layers[l], "grad")[0] for l in members)
    flops = sum(layer_work(w, w.layers[l], "grad")[1] for l in members)
    t_hbm, t_alu = nbytes / (peaks["hbm_gbs"] * 1e9), flops / (peaks["bf16_tflops"] * 1e12)
    if t_hbm >= t_alu:
        ach = nbytes / (ms * 1e-3) / 1e9
        r = dict(bound="hbm", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s", frac=ach / peaks["hbm_gbs"])
    else:
        ach = flops / (ms * 1e-3) / 1e12
        r = dict(bound="tensor", achieved=ach, peak=peaks["bf16_tflops"], unit="TFLOP/s", frac=ach / peaks["bf16_tflops"],
                 frac_of_sustained_peak=ach / peaks["bf16_tflops_sustained"])
    traffic = [NCU_TRAFFIC_BYTES.get((w.name, "grad_group" if k[0] == "grad_group" else f"grad[{w.layers[k[1]].name}]")) for k in keys]
    r.update(traffic=(sum(traffic) / len(keys) if all(t is not None for t in traffic) else None),
             kernel="zta_pair_kernel + reduce_segments_kernel (bf16 clipped sums)", launches_per_step=len(keys), kernel_ms=ms / len(keys),
             kernel_ms_total=ms, share_of_step=ms / sum(breakdown.values()), algorithmic_bytes=nbytes / len(keys),
             algorithmic_flops=flops / len(keys), peak_source=peaks["source"],
             note="per launch: averages over the kernel's launches of one step; peak = burst bf16 figure")
    return r


def roofline_for(w, breakdown, peaks):
    """Roofline of the kernel that takes the largest share of the step: the bf16 clipped-sum kernel over all its
    launches when that is the largest, else the single launch with the largest share."""
    cands = {k: v for k, v in breakdown.items() if k[0] not in ("factors",)}
    key = max(cands, key=cands.get)
    kind, l = key
    zta = roofline_zta(w, breakdown, peaks)
    if zta is not None and zta["kernel_ms_total"] >= cands[key]:
        return zta
    if kind in kernel_breakdown.groups:
        return roofline_group(w, key, breakdown, peaks)
    spec = w.layers[l]
    nbytes, flops = layer_work(w, spec, kind)
    ms = breakdown[key]
    t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9)
    # bf16 layers whose rows are 16-byte multiples run on the tcgen05 kernels; so do fp32 layers above 2^25
    # multiply-adds whose rows are 16-byte multiples (three tf32 MMAs per product), unless they are narrow
    # enough for the streaming kernel
    narrow = spec.T > 1 and spec.d_in + (1 if spec.has_bias else 0) <= 32 and spec.d_out <= 64
    tc_bf16 = w.dtype == "bf16" and spec.d_in % 8 == 0 and spec.d_out % 8 == 0
    tc_f32 = (w.dtype == "f32" and spec.d_in % 4 == 0 and spec.d_out % 4 == 0 and not narrow and
              float(w.B) * spec.T * spec.d_in * spec.d_out >= 2 ** 25)
    on_tensor = (kind in ("norm_gram", "norm_mat") or (kind == "grad" and (tc_bf16 or tc_f32))) and not narrow
    if on_tensor and w.dtype == "f32":
        alu_peak = peaks["bf16_tflops"] * TF32X3_PER_BF16 * 1e12
    else:
        alu_peak = (peaks["bf16_tflops"] if on_tensor else FFMA_PEAK_TFLOPS) * 1e12
    t_alu = flops / alu_peak
    total = sum(breakdown.values())
    if t_hbm >= t_alu:
        ach = nbytes / (ms * 1e-3) / 1e9
        r = dict(bound="hbm", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s", frac=ach / peaks["hbm_gbs"])
    else:
        ach = flops / (ms * 1e-3) / 1e12
        pk = alu_peak / 1e12
        r = dict(bound="tensor" if on_tensor else "alu", achieved=ach, peak=pk, unit="TFLOP/s", frac=ach / pk)
    r.update(traffic=NCU_TRAFFIC_BYTES.get((w.name, f"{kind}[{spec.name}]")), kernel=f"{kind}[{spec.name}]", kernel_ms=ms, share_of_step=ms / total,
             algorithmic_bytes=nbytes, algorithmic_flops=flops, peak_source=peaks["source"])
    return r


def bench_workload(torch, dp, w, steps, warmup, flush, peaks, with_e2e=True):
    layers = workloads.generate(w, seed=0)
    plan = make_plan(dp, w, layers, torch)
    n0 = dp.dpclip_launch_count()
    plan.run(w.C, w.sigma, 1)
    launches_per_step = dp.dpclip_launch_count() - n0
    # the timed step replays a CUDA graph recorded from one dpclip_step call (same kernels, no launch gaps)
    # models with T > 1 layers: per-layer calls on four streams (parallel graph branches); all-T=1 models
    # take the fused two-launch step inside one dpclip_step call
    branches = 1 if all(s.T == 1 for s in w.layers) else 4
    graph = plan.capture(w.C, w.sigma, 1, branches=branches)
    # per-call times first, while the GPU is still in the state in which the burst peaks were measured (a kernel
    # timed alone is compared with the burst figure; after the long loops below the power cap lowers the clocks)
    for _ in range(3):
        flush(); graph.replay()
    bd = kernel_breakdown(torch, dp, w, plan, min(steps, 20), flush, w.C, w.sigma)
    torch.cuda.synchronize()
    time.sleep(0.5)                  # the timed loop starts from an idle GPU (see rest() below), then its warm-up steps
    single = time_steps(torch, graph.replay, steps, warmup, flush)
    assert all(dp.dpclip_read_status(x) == 0 for x in plan.workspaces())
    rotating = None
    if branches == 1:
        times, rotating = time_steps_rotating(torch, dp, w, layers, steps, warmup, flush)
    else:
        times = single
    def rest():
        # the other launch modes are measured for comparison, each from the same starting state: half a second of
        # idle lets the power cap's running average recover after the loop before
        torch.cuda.synchronize()
        time.sleep(0.5)

    one_stream_ms = None
    if branches > 1:
        g1 = plan.capture(w.C, w.sigma, 1, branches=1)          # the same step as ONE dpclip_step call on one stream
        rest()
        one_stream_ms = float(np.mean(time_steps(torch, g1.replay, min(steps, 30), 3, flush)))
    rest()
    eager = time_steps(torch, lambda: plan.run(w.C, w.sigma, 1), min(steps, 30), 3, flush)
    rest()
    warm = time_steps(torch, graph.replay, steps, 3, lambda: None)
    # The literal inputs clip every example (the worst case for the clipped sum: stages whose factor is exactly one
    # skip the rescaling in shared memory): the same step with the threshold at the median norm and above every norm.
    clip_cases = None
    if with_e2e:
        norms = plan.norms.float()
        clip_cases = {"literal": dict(clipped_fraction=float((plan.clip < 1).float().mean().item()))}
        for name, c in (("half_clipped", float(norms.median().item())), ("unclipped", 2.0 * float(norms.max().item()))):
            g = plan.capture(c, w.sigma, 1, branches=branches)
            ms = float(np.mean(time_steps(torch, g.replay, min(steps, 20), 3, flush)))
            clip_cases[name] = dict(C=c, ms_per_step=ms, clipped_fraction=float((plan.clip < 1).float().mean().item()))
        plan.run(w.C, w.sigma, 1)
        torch.cuda.synchronize()
    res = dict(times_ms=times, warm_ms=float(np.median(warm)), eager_ms=float(np.median(eager)),
               single_graph_ms=float(np.mean(single)), rotating=rotating, one_stream_ms=one_stream_ms,
               launches_per_step=int(launches_per_step),
               breakdown={f"{k[0]}[{entry_name(w, k)}]": round(v * 1e3, 2) for k, v in bd.items()},
               roofline=(roofline_fused_t1(w, float(np.mean(times)), peaks) if branches == 1
                         else roofline_for(w, bd, peaks)))
    # whole-step lower bound: max(total algorithmic bytes / HBM, total flops / the engine used)
    res["step_roofline"] = step_roofline(w, peaks)
    res["step_roofline_us"] = res["step_roofline"]["roof_us"]
    res["clip_cases"] = clip_cases
    if with_e2e:
        host_layers = [dp.Layer(torch.from_numpy(A).to(torch.float32 if w.dtype == "f32" else torch.bfloat16).pin_memory(),
                                torch.from_numpy(Z).to(torch.float32 if w.dtype == "f32" else torch.bfloat16).pin_memory(),
                                s.has_bias) for (A, Z), s in zip(layers, w.layers)]
        # two steps in flight on two streams (each with its own device arena and pinned result buffers), the
        # way a training loop pipelines transfers: step i+1's host->device copies overlap step i's
        # device->host read.  Every step copies all its inputs in and all its results out, and the caller
        # waits for step i's results before it enqueues step i+2.
        hs = dp.HostStep(host_layers, pack_inputs=True)          # one pinned buffer per direction: one copy each way
        hs2 = dp.HostStep(host_layers, pack_inputs=True)
        slots = [(hs, torch.cuda.Stream()), (hs2, torch.cuda.Stream())]

        def e2e_steps(n):
            for i in range(n):
                h, st = slots[i % 2]
                st.synchronize()                                   # results of step i-2 have been read
                with torch.cuda.stream(st):
                    h.run(w.C, w.sigma, 1)
            for _, st in slots:
                st.synchronize()

        e2e_steps(max(2, warmup))
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        e2e_steps(steps)
        res["e2e_wall_ms"] = (time.perf_counter() - t0) * 1e3 / steps
        res["e2e_ms"] = res["e2e_wall_ms"]           # bracketed by synchronisation on both sides: host clock = device time
        # one step at a time, for comparison
        t0 = time.perf_counter()
        for _ in range(steps):
            hs.run(w.C, w.sigma, 1)
            torch.cuda.current_stream().synchronize()
        res["e2e_serial_ms"] = (time.perf_counter() - t0) * 1e3 / steps
        res["h2d"], res["d2h"] = hs.h2d_bytes, hs.d2h_bytes
    return res


def bench_elementwise(torch, dp, B, T, d, dtype, steps, flush, peaks):
    """LayerNorm gain/shift parameters (element-wise layers): the two streaming kernels, each timed alone
    with CUDA events, L2 flushed between launches.  Algorithmic bytes = Hbar and Zbar once per kernel."""
    H, Z = workloads.layernorm_pair(0, B, T, d, dtype, var_z=1.0 / (B * T))
    dH, dZ = to_dev(H, dtype, torch), to_dev(Z, dtype, torch)
    clip = torch.rand(B, device="cuda") * 0.9 + 0.1
    sq = torch.empty(B, device="cuda"); g = torch.empty(d, device="cuda"); sh = torch.empty(d, device="cuda")
    nbytes = 2 * B * T * d * (4 if dtype == "f32" else 2)
    out = dict(workload=f"layernorm_b{B}_t{T}_d{d}_{dtype}", algorithmic_bytes=nbytes)
    for name, fn in (("norm", lambda: dp.dpclip_elementwise_sqnorms(dH, dZ, True, sq)),
                     ("grad", lambda: dp.dpclip_elementwise_clipped_grad(dH, dZ, clip, g, sh))):
        ms = float(np.median(time_steps(torch, fn, steps, 3, flush)))
        ach = nbytes / (ms * 1e-3) / 1e9
        out[name] = dict(ms=ms, roofline=dict(bound="hbm", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s",
                                              frac=ach / peaks["hbm_gbs"], traffic=None, peak_source=peaks["source"]))
    return out


def bench_model_block(torch, dp, steps, flush):
    """One Transformer block through dpclip_model_step (one call, one stream, replayed as a CUDA graph): LayerNorm
    gain/shift, four bias-free d -> d attention projections, LayerNorm, d -> d_ff and d_ff -> d layers;
    B = 128, T = 256, d = 512, d_ff = 2048, bf16."""
    import dataclasses
    w = workloads.seq("bf16")
    w = dataclasses.replace(w, layers=w.layers[:6])
    dense = workloads.generate(w, 0)
    lns = [workloads.layernorm_pair(50 + k, w.B, 256, 512, "bf16", var_z=w.zbar_var) for k in range(2)]
    mk = lambda kind, A, Z, b: dp.ModelLayer(kind, to_dev(A, "bf16", torch), to_dev(Z, "bf16", torch), b)   # noqa: E731
    d = [mk(dp.DPCLIP_KIND_DENSE, A, Z, s.has_bias) for (A, Z), s in zip(dense, w.layers)]
    n = [mk(dp.DPCLIP_KIND_ELEMENTWISE, H, Z, True) for H, Z in lns]
    plan = dp.ModelPlan([n[0]] + d[:4] + [n[1]] + d[4:])
    plan.run(w.C, w.sigma, 1)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        plan.run(w.C, w.sigma, 1)
    one_stream_ms = float(np.mean(time_steps(torch, graph.replay, steps, 3, flush)))
    graph4 = plan.capture(w.C, w.sigma, 1, branches=4)
    ms = float(np.mean(time_steps(torch, graph4.replay, steps, 3, flush)))
    assert dp.dpclip_read_status(plan.workspace) == 0
    nbytes = sum(2 * 2 * y.A.numel() + 2 * 2 * y.Zbar.numel() for y in plan.layers) + 4 * plan.flat.numel()
    return dict(workload="transformer_block_b128_t256_d512_bf16", entry="dpclip_model_step", layers=plan.L,
                ms_per_step=ms, one_stream_ms_per_step=one_stream_ms, value=w.B / (ms * 1e-3), algorithmic_bytes=nbytes,
                timing="graph of per-layer calls on four streams; one_stream = the single dpclip_model_step call as a graph",
                clipped_fraction=float((plan.clip < 1).float().mean().item()))


def bench_per_layer(torch, dp, steps, flush):
    """Per-layer clipping (every layer to C / sqrt(L)) over the layers of the sequence workload: one
    dpclip_step_per_layer call replayed as a graph on one stream."""
    w = workloads.seq("bf16")
    data = workloads.generate(w, 0)
    plan = dp.StepPlan([dp.Layer(to_dev(A, "bf16", torch), to_dev(Z, "bf16", torch), s.has_bias)
                        for (A, Z), s in zip(data, w.layers)])
    Cl = [w.C / np.sqrt(plan.L)] * plan.L
    clip = torch.empty(plan.L, plan.B, device="cuda")
    dp.dpclip_step_per_layer(plan, Cl, w.sigma, 1, clip_layers=clip)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        dp.dpclip_step_per_layer(plan, Cl, w.sigma, 1, clip_layers=clip)
    ms = float(np.mean(time_steps(torch, graph.replay, steps, 3, flush)))
    assert dp.dpclip_read_status(plan.workspace) == 0
    return dict(workload="per_layer_clipping_" + w.name, entry="dpclip_step_per_layer", layers=plan.L, ms_per_step=ms,
                value=w.B / (ms * 1e-3), clipped_fraction=float((clip < 1).float().mean().item()))


def bench_model_cnn(torch, dp, dtype, steps, flush):
    """The CNN of the cnn_32x32x3 workloads with its convolutions given by their feature maps and dL/dZ in the
    channel-major layout it has in a framework (no patch matrices anywhere), dense 8192 -> 256 -> 10 on top:
    ModelPlan, graph of per-layer calls on four streams.  B = 128."""
    B = 128
    convs = [(3, 32, 32, 32), (32, 16, 16, 64), (64, 8, 8, 128)]
    layers = []
    for i, (cin, H, W, cout) in enumerate(convs):
        X, Z = workloads.conv_inputs(60 + i, B, cin, H, W, 3, 1, 1, cout, dtype, var_z=1.0 / B)
        dZ = to_dev(Z, dtype, torch).transpose(1, 2).contiguous()
        layers.append(dp.ModelLayer(dp.DPCLIP_KIND_CONV, to_dev(X, dtype, torch), dZ, True, conv=(3, 3, 1, 1),
                                    z_channel_major=True))
    rng = np.random.default_rng(63)
    for d_in, d_out in ((8192, 256), (256, 10)):
        A = np.maximum(rng.standard_normal((B, 1, d_in)), 0).astype(np.float32)
        Z = (rng.standard_normal((B, 1, d_out)) / np.sqrt(B)).astype(np.float32)
        layers.append(dp.ModelLayer(dp.DPCLIP_KIND_DENSE, to_dev(A, dtype, torch), to_dev(Z, dtype, torch), True))
    plan = dp.ModelPlan(layers)
    graph = plan.capture(1.0, 1.0, 1, branches=4)
    ms = float(np.mean(time_steps(torch, graph.replay, steps, 3, flush)))
    assert dp.dpclip_read_status(plan.workspace) == 0
    es = 4 if dtype == "f32" else 2
    nbytes = sum(2 * es * (y.A.numel() + y.Zbar.numel()) for y in plan.layers) + 4 * plan.flat.numel()
    return dict(workload=f"cnn_feature_maps_b128_{dtype}", entry="ModelPlan.capture (per-layer calls, four streams)",
                layers=plan.L, ms_per_step=ms, value=B / (ms * 1e-3), algorithmic_bytes=nbytes,
                clipped_fraction=float((plan.clip < 1).float().mean().item()))


def bench_conv_implicit(torch, dp, name, B, C, H, W, k, pad, d_out, dtype, steps, flush, peaks):
    """A convolution layer straight from its feature map (implicit im2col on the tensor cores), next to the same
    layer through the patch-matrix entry points.  Algorithmic bytes: feature map + Zbar once per kernel."""
    X, Z = workloads.conv_inputs(0, B, C, H, W, k, pad, 1, d_out, dtype, var_z=1.0 / B)
    A = workloads.im2col(X, k, pad)
    dX, dZ, dA = to_dev(X, dtype, torch), to_dev(Z, dtype, torch), to_dev(A, dtype, torch)
    T, d_in = Z.shape[1], C * k * k
    clip = torch.rand(B, device="cuda") * 0.9 + 0.1
    sq = torch.empty(B, device="cuda"); gW = torch.empty(d_out, d_in, device="cuda"); gb = torch.empty(d_out, device="cuda")
    ws = torch.empty(max(dp.dpclip_workspace_bytes(B, T, d_in, d_out, dp.DPCLIP_BF16),
                         dp.dpclip_conv_workspace_bytes(dX, dZ.transpose(1, 2).contiguous(), k, k, 1, pad, True)),
                     dtype=torch.uint8, device="cuda")
    dp.dpclip_workspace_init(ws)
    es = 4 if dtype == "f32" else 2
    nbytes = (X.size + Z.size) * es
    flops = 2.0 * B * T * d_in * d_out
    out = dict(workload=name, algorithmic_bytes=int(nbytes), patch_matrix_bytes=int((A.size + Z.size) * es))
    for kind, fn, ref in (("norm", lambda: dp.dpclip_conv_sqnorms(dX, dZ, k, k, 1, pad, True, sq, workspace=ws),
                           lambda: dp.dpclip_layer_sqnorms(dA, dZ, True, sq, ws)),
                          ("grad", lambda: dp.dpclip_conv_clipped_grad(dX, dZ, k, k, 1, pad, clip, gW, gb, workspace=ws),
                           lambda: dp.dpclip_clipped_grad(dA, dZ, clip, gW, gb, ws))):
        ms = float(np.median(time_steps(torch, fn, steps, 3, flush)))
        ms_ref = float(np.median(time_steps(torch, ref, steps, 3, flush)))
        # layers of this size take the tensor-core forms (fp32: three tf32 MMAs per product); the binding roof is the
        # larger of bytes / HBM and flops / the tensor peak of the form
        peak_tf = peaks["bf16_tflops"] * (TF32X3_PER_BF16 if dtype == "f32" else 1.0)
        t_hbm, t_mma = nbytes / (peaks["hbm_gbs"] * 1e9), flops / (peak_tf * 1e12)
        if t_hbm >= t_mma:
            ach = nbytes / (ms * 1e-3) / 1e9
            roof = dict(bound="hbm", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s", frac=ach / peaks["hbm_gbs"])
        else:
            ach = flops / (ms * 1e-3) / 1e12
            roof = dict(bound="tensor", achieved=ach, peak=peak_tf, unit="TFLOP/s", frac=ach / peak_tf)
        roof.update(traffic=None, peak_source=peaks["source"])
        out[kind] = dict(ms=ms, patch_matrix_path_ms=ms_ref, roofline=roof)
    # dL/dZ as back-propagation produces it, [B][c_out][T] (the patch-matrix path would first have to transpose it)
    dZcm = dZ.transpose(1, 2).contiguous()
    out["norm_channel_major_ms"] = float(np.median(time_steps(
        torch, lambda: dp.dpclip_conv_sqnorms(dX, dZcm, k, k, 1, pad, True, sq, z_channel_major=True, workspace=ws),
        steps, 3, flush)))
    return out


# ---------------------------------------------------------------------------
# CPU oracle legs
# ---------------------------------------------------------------------------
def oracle_sample(w, budget_s=12.0):
    """Time the oracle, as it stands, on a bounded sample of `w`: whole steps
    over the first `n` examples of the batch (n chosen so one step takes a few
    seconds), repeated until about `budget_s` of CPU time is spent."""
    import oracle
    oracle.build()
    hb = [s.has_bias for s in w.layers]
    flops_per_ex = sum(4.0 * s.T * s.d_in * s.d_out for s in w.layers)      # norm pass + clipped-sum pass
    n = int(max(1, min(w.B, 4e9 / max(flops_per_ex, 1.0))))
    layers = workloads.generate(w, seed=0, examples=n)
    t0 = time.perf_counter()
    reps = 0
    while True:
        oracle.step(layers, hb, w.C, w.sigma, 1)
        reps += 1
        dt = time.perf_counter() - t0
        if dt >= budget_s or reps >= 50:
            break
    return dict(value=n * reps / dt, unit=UNIT, cores=1, kind="oracle",
                sample=f"{reps} whole steps over the first {n} of {w.B} examples of {w.name} "
                       f"(fp64, single thread, {dt:.1f} s)"), dt / reps, n


def workload_config(w, world):
    """The `config` object of the JSON line: the same for both arms, so that their lines can be matched."""
    return dict(workload=w.name, B_per_gpu=w.B, layers=[f"{s.name}:T{s.T}:{s.d_in}->{s.d_out}" for s in w.layers],
                C=w.C, sigma=w.sigma, l2="flushed by a 256 MB write between steps",
                parallelism=f"dp{world}" if world > 1 else "single")


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = workloads.by_name(args.workload)
    total_t, total_n = 0.0, 0
    info = None
    for i in range(args.warmup + args.steps):
        info, per_step, n = oracle_sample(w, budget_s=1.0)
        if i >= args.warmup:
            total_t += per_step; total_n += n
    value = total_n / total_t
    line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=total_t / args.steps * 1e3, higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                config=workload_config(w, args.gpus), sample=info["sample"],
                cpu_baseline=dict(value=value, unit=UNIT, cores=1, kind="oracle", sample=info["sample"]),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                gpu_launches=0)
    print(json.dumps(line))


def run_sweep(args):
    """Gram vs materialise crossover of the T > 1 norm (one dense bf16 layer per point, bias on): both norm
    methods and the clipped sum at every point, each launch timed alone with CUDA events, L2 flushed between
    launches.  Inputs are drawn on the device (timing only; parity at these shapes is in the test suite).
    Prints one table line per point and a final JSON line."""
    import torch

    import paper_2009_03106_b200 as dp
    torch.cuda.set_device(0)
    dp.load_library()
    peaks = measured_peaks()
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    flush = lambda: flush_buf.fill_(1)                                           # noqa: E731
    rows = []
    print(f"{'B':>5} {'T':>5} {'d_in':>5} {'d_out':>5} | {'gram us':>9} {'mat us':>9} {'faster':>7} {'flop rule':>9} "
          f"{'auto':>6} | {'clipped sum us':>14} {'TFLOP/s':>8}")
    if args.points:
        grid_points = [tuple(int(v) for v in pt.split(",")) for pt in args.points.split(";") if pt]
    else:
        grid_points = [(B, T, d_in, d_out) for B in (256, 1024) for T in (16, 128, 512, 2048)
                       for d_in, d_out in ((1024, 1024), (1024, 4096), (4096, 1024))]
    # Measured from the lightest point to the heaviest: after a point whose launches run for milliseconds under
    # the power cap, the tensor-core kernels of the following points ran 15-30 % slower for seconds (the
    # HBM-bound Gram kernel did not), so the short points go first.  Printed in measurement order.
    if not args.points:
        grid_points.sort(key=lambda pt: pt[0] * pt[1] * pt[2] * pt[3])
    for B, T, d_in, d_out in grid_points:
        if 2 * B * T * (d_in + d_out) > 12e9:
            continue                                                    # keep the device footprint bounded
        ws = torch.empty(dp.dpclip_workspace_bytes(B, T, d_in, d_out, dp.DPCLIP_BF16), dtype=torch.uint8, device="cuda")
        dp.dpclip_workspace_init(ws)
        g = torch.Generator(device="cuda").manual_seed(B * 7919 + T)
        A = torch.randn(B, T, d_in, device="cuda", generator=g).to(torch.bfloat16)
        Z = (torch.randn(B, T, d_out, device="cuda", generator=g) * (B * T) ** -0.5).to(torch.bfloat16)
        sq = torch.empty(B, device="cuda"); clip = torch.rand(B, device="cuda", generator=g) * 0.9 + 0.1
        gW = torch.empty(d_out, d_in, device="cuda"); gb = torch.empty(d_out, device="cuda")
        n = max(3, min(args.steps, 10))
        t = {}
        for name, m in (("gram", dp.DPCLIP_GRAM), ("mat", dp.DPCLIP_MATERIALIZE)):
            t[name] = float(np.median(time_steps(torch, lambda: dp.dpclip_layer_sqnorms(A, Z, True, sq, ws, m), n, 3, flush)))
        t["grad"] = float(np.median(time_steps(torch, lambda: dp.dpclip_clipped_grad(A, Z, clip, gW, gb, ws), n, 3, flush)))
        assert dp.dpclip_read_status(ws) == 0
        rule = "gram" if T * (T + 1) * (d_in + d_out) <= 2 * T * d_in * d_out else "mat"
        auto = {dp.DPCLIP_GRAM: "gram", dp.DPCLIP_MATERIALIZE: "mat"}.get(
            dp.dpclip_pick_method(B, T, d_in, d_out, d_in, d_out, dp.DPCLIP_BF16), "other")
        tf = 2.0 * B * T * d_in * d_out / (t["grad"] * 1e-3) / 1e12
        rows.append(dict(B=B, T=T, d_in=d_in, d_out=d_out, gram_ms=t["gram"], materialize_ms=t["mat"],
                         faster="gram" if t["gram"] <= t["mat"] else "mat", flop_rule=rule, auto=auto,
                         clipped_sum_ms=t["grad"], clipped_sum_tflops=tf))
        print(f"{B:5d} {T:5d} {d_in:5d} {d_out:5d} | {t['gram'] * 1e3:9.1f} {t['mat'] * 1e3:9.1f} {rows[-1]['faster']:>7} "
              f"{rule:>9} {auto:>6} | {t['grad'] * 1e3:14.1f} {tf:8.0f}", flush=True)
        del A, Z
    noise = None
    if args.noise_n:
        # the noise kernel alone at a size where it is bandwidth-bound (8 bytes per element: read + write)
        g = torch.zeros(args.noise_n, device="cuda")
        ms = float(np.median(time_steps(torch, lambda: dp.dpclip_add_noise(g, 1.0, 1.0, 1, 0), 5, 3, flush)))
        noise = dict(n=args.noise_n, ms=ms, gbs=8.0 * args.noise_n / (ms * 1e-3) / 1e9)
        print(f"noise n={args.noise_n}: {ms * 1e3:.1f} us  {noise['gbs']:.0f} GB/s "
              f"({noise['gbs'] / peaks['hbm_gbs']:.2f} of the {peaks['source']} copy bandwidth)")
        # parameter updates with the noise folded in: SGD 12 bytes per parameter (gsum, theta in; theta out),
        # Adam 28 (gsum, theta, m, v in; theta, m, v out)
        th = torch.zeros(args.noise_n, device="cuda"); m = torch.zeros_like(th); v = torch.zeros_like(th)
        for name, nbytes, fn in (("dp_sgd_step", 12.0, lambda: dp.dpclip_dp_sgd_step(th, g, 1 / 128, 1.0, 1.0, 1, 0, 1e-3)),
                                 ("dp_adam_step", 28.0, lambda: dp.dpclip_dp_adam_step(th, m, v, g, 1 / 128, 1.0, 1.0, 1, 0, 1e-3,
                                                                                       0.9, 0.999, 1e-8, 1))):
            ms = float(np.median(time_steps(torch, fn, 5, 3, flush)))
            gbs = nbytes * args.noise_n / (ms * 1e-3) / 1e9
            noise[name] = dict(ms=ms, gbs=gbs)
            print(f"{name} n={args.noise_n}: {ms * 1e3:.1f} us  {gbs:.0f} GB/s ({gbs / peaks['hbm_gbs']:.2f} of the copy bandwidth)")
    print(json.dumps(dict(sweep="norm_method_crossover", dtype="bf16", peaks=peaks, points=rows, noise=noise)))


def launch_floors(torch, dp, steps, flush):
    """Device time per EMPTY launch with the launch shape of the one-launch T = 1 step (128 CTAs of 18 warps, its
    dynamic shared memory), plain and cooperative, measured the way the all-T=1 steps are: `steps` launches
    back to back in one CUDA graph, one event pair around them, median of three replays."""
    out = {}
    for name, coop in (("plain", False), ("cooperative", True)):
        dp.dpclip_null_launch(coop, 128)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for _ in range(steps):
                dp.dpclip_null_launch(coop, 128)
        graph.replay(); torch.cuda.synchronize()
        reps = []
        for _ in range(3):
            flush()
            s0, e0 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s0.record(); graph.replay(); e0.record()
            torch.cuda.synchronize()
            reps.append(s0.elapsed_time(e0) * 1e3 / steps)
        out[name] = round(float(np.median(reps)), 2)
        # and one launch per graph replay, events around each replay (what single_step_graph_ms_per_step pays)
        g1 = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g1):
            dp.dpclip_null_launch(coop, 128)
        out[name + "_single_graph"] = round(float(np.median(time_steps(torch, g1.replay, 20, 3, flush))) * 1e3, 2)
    return out


def sweep_points_compact(torch, dp, steps, flush, peaks):
    """The Gram-vs-materialise sweep (one dense bf16 layer with bias per point; B in {256, 1024}, T in {16, 128,
    512, 2048}, d_in x d_out in {1024x1024, 1024x4096, 4096x1024}): per point the step = norms (the method the
    library picks) + factors + clipped sum with noise, each launch timed alone with CUDA events, L2 flushed in
    between, against the point's own step roofline.  Inputs are drawn on the device (timing only; parity at these
    shapes is in the test suite).  Lightest points first (see run_sweep)."""
    pts = [(B, T, d_in, d_out) for B in (256, 1024) for T in (16, 128, 512, 2048)
           for d_in, d_out in ((1024, 1024), (1024, 4096), (4096, 1024))]
    pts.sort(key=lambda pt: pt[0] * pt[1] * pt[2] * pt[3])
    rows = []
    for B, T, d_in, d_out in pts:
        w = workloads.sweep_point(B, T, d_in, d_out)
        ws = torch.empty(dp.dpclip_workspace_bytes(B, T, d_in, d_out, dp.DPCLIP_BF16), dtype=torch.uint8, device="cuda")
        dp.dpclip_workspace_init(ws)
        g = torch.Generator(device="cuda").manual_seed(B * 7919 + T)
        A = torch.empty(B, T, d_in, device="cuda", dtype=torch.bfloat16)
        Z = torch.empty(B, T, d_out, device="cuda", dtype=torch.bfloat16)
        for i in range(0, B, 64):                                  # drawn in slabs: no 30 GB fp32 temporaries
            A[i:i + 64] = torch.randn(min(64, B - i), T, d_in, device="cuda", generator=g).to(torch.bfloat16)
            Z[i:i + 64] = (torch.randn(min(64, B - i), T, d_out, device="cuda", generator=g) * (B * T) ** -0.5).to(torch.bfloat16)
        sq = torch.empty(1, B, device="cuda"); clip = torch.empty(B, device="cuda"); nrm = torch.empty(B, device="cuda")
        gW = torch.empty(d_out, d_in, device="cuda"); gb = torch.empty(d_out, device="cuda")
        n = 3 if B * T * d_in * d_out > 1e14 / 8 else max(3, min(steps, 6))
        t_norm = float(np.median(time_steps(torch, lambda: dp.dpclip_layer_sqnorms(A, Z, True, sq[0], ws), n, 2, flush)))
        t_fac = float(np.median(time_steps(torch, lambda: dp.dpclip_factors(sq, w.C, clip, nrm), n, 2, flush)))
        t_grad = float(np.median(time_steps(
            torch, lambda: dp.dpclip_clipped_grad_noise(A, Z, clip, gW, gb, w.sigma, w.C, 1, 0, 1, ws), n, 2, flush)))
        assert dp.dpclip_read_status(ws) == 0
        roof = step_roofline(w, peaks)
        step_us = (t_norm + t_fac + t_grad) * 1e3
        meth = {dp.DPCLIP_GRAM: "gram", dp.DPCLIP_MATERIALIZE: "mat"}.get(
            dp.dpclip_pick_method(B, T, d_in, d_out, d_in, d_out, dp.DPCLIP_BF16), "other")
        rows.append(dict(B=B, T=T, d_in=d_in, d_out=d_out, norm_method=meth, norm_us=t_norm * 1e3, factors_us=t_fac * 1e3,
                         grad_us=t_grad * 1e3, step_us=step_us, roof_us=roof["roof_us"], bound=roof["bound"],
                         frac=roof["roof_us"] / step_us, value=B / (step_us * 1e-6),
                         grad_tflops=2.0 * B * T * d_in * d_out / (t_grad * 1e-3) / 1e12))
        del A, Z, gW, ws
        torch.cuda.empty_cache()
    return rows


def config_summary(name, w, r, ms):
    """One compact entry of the `configs` object."""
    sr = r["step_roofline"]
    return dict(workload=w.name, us=round(ms * 1e3, 2), ex_s=round(w.B / (ms * 1e-3), 1), bound=sr["bound"],
                roof_us=round(sr["roof_us"], 2), frac=round(sr["roof_us"] / (ms * 1e3), 4),
                frac_sustained=round(sr["roof_sustained_us"] / (ms * 1e3), 4))


# ---------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="cfg4")
    ap.add_argument("--impl", default="dpclip", choices=["dpclip", "reference"])
    ap.add_argument("--others", default="cfg1,cfg2,cfg2_bf16,cfg3_f32,cfg3_bf16,cfg4",
                    help="further workloads reported under 'configs' / 'workloads' (N=1 only; 'none' for none)")
    ap.add_argument("--no-extras", action="store_true", help="skip the sweep points and the single-feature timings")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--points", default="", help="with --sweep: only these points, 'B,T,d_in,d_out;B,T,d_in,d_out;...'")
    ap.add_argument("--noise-n", type=int, default=0, help="with --sweep: also time dpclip_add_noise on this many elements")
    ap.add_argument("--sweep", action="store_true",
                    help="instead of the benchmark line: Gram-vs-materialise sweep of the T > 1 norm (1 GPU)")
    args = ap.parse_args()
    if args.others == "none":
        args.others = ""
    args.warmup = max(args.warmup, 3) if args.impl == "dpclip" else args.warmup
    if args.impl == "reference":
        return run_reference(args)
    if args.sweep:
        return run_sweep(args)

    import torch
    import torch.distributed as dist

    import paper_2009_03106_b200 as dp

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local)
    dp.load_library()
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks = measured_peaks()
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    def flush():
        flush_buf.fill_(1)

    w = workloads.by_name(args.workload)
    sampler = ClockSampler(local) if rank == 0 else None
    if world > 1:
        from paper_2009_03106_b200 import parallel
        layers = workloads.generate(w, seed=rank)                 # every rank owns its own batch (weak scaling)
        plan = make_plan(dp, w, layers, torch)
        step = parallel.ShardedStep(plan, w.C, w.sigma, seed=1, stream_id0=0)
        n0 = dp.dpclip_launch_count(); step.run(); lps = dp.dpclip_launch_count() - n0
        dist.barrier(); torch.cuda.synchronize()
        t_wall0 = time.time()
        times = time_steps(torch, step.run, args.steps, args.warmup, flush)
        torch.cuda.synchronize(); dist.barrier()
        t_wall1 = time.time()
        tot = torch.tensor([sum(times)], device="cuda", dtype=torch.float64)
        dist.all_reduce(tot, op=dist.ReduceOp.MAX)
        total_ms = tot.item()
        res = dict(launches_per_step=int(lps), roofline=None, e2e_ms=None, how=step.describe())
    else:
        t_wall0 = time.time()
        res = bench_workload(torch, dp, w, args.steps, args.warmup, flush, peaks)
        t_wall1 = time.time()
        total_ms = sum(res["times_ms"])
    clocks = sampler.stop(t_wall0, t_wall1) if sampler else None

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    ms_per_step = total_ms / args.steps
    value = w.B * world * args.steps / (total_ms * 1e-3)
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                ms_per_step=ms_per_step, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype=w.dtype, data="synthetic",
                config=workload_config(w, world),
                gpu_launches=int(res["launches_per_step"]) * args.steps, clocks=clocks)
    if world > 1:
        line["launch"] = res["how"]
        line["e2e"] = None
        dist.destroy_process_group()
        print(json.dumps(line))
        return

    if res.get("clip_cases"):
        line["clip_cases"] = res["clip_cases"]
    if len(res["times_ms"]) >= 8 and not res.get("rotating"):
        # the timed steps in four quarters: shows whether the power cap lowered the clocks during the run
        q = np.array_split(np.asarray(res["times_ms"]), 4)
        line["ms_per_step_by_quarter"] = [round(float(x.mean()), 5) for x in q]
    sr = res["step_roofline"]
    roof = res["roofline"]
    roof["step"] = dict(sr, measured_us=ms_per_step * 1e3, frac=sr["roof_us"] / (ms_per_step * 1e3),
                        frac_sustained=sr["roof_sustained_us"] / (ms_per_step * 1e3),
                        note="whole step: max(bytes / HBM, flops / tensor peak) over the measured step time; bytes = inputs "
                             "twice + outputs once, flops = cheaper exact norm form + clipped-sum product")
    line["roofline"] = roof
    line["step_roofline_frac"] = sr["roof_us"] / (ms_per_step * 1e3)
    line["warm_l2_ms_per_step"] = res["warm_ms"]
    line["eager_ms_per_step"] = res["eager_ms"]
    line["one_stream_graph_ms_per_step"] = res.get("one_stream_ms")
    if res.get("rotating"):
        rt = res["rotating"]
        line["config"]["l2"] = (f"inputs larger than L2: step i works on input/output set i % {rt['sets']} "
                                f"({rt['set_bytes'] / 1e6:.1f} MB each), 256 MB flush write before the timed region")
        line["launch"] = (f"one CUDA graph holding the {args.steps} timed steps back to back (one dpclip_step "
                                    "call each); one event pair around the region, median of 3 regions")
        line["single_step_graph_ms_per_step"] = res["single_graph_ms"]
    else:
        line["launch"] = ("CUDA graph replay of one step = ONE dpclip_step_streams call (the library forks over 4 "
                                    "streams); events around every step")
    line["breakdown_us"] = res["breakdown"]
    line["e2e"] = dict(value=w.B / (res["e2e_ms"] * 1e-3), unit=UNIT, h2d_bytes_per_step=res["h2d"],
                       d2h_bytes_per_step=res["d2h"], ms_per_step=res["e2e_ms"],
                       serial_ms_per_step=res["e2e_serial_ms"],
                       note="dpclip_step_host per step (all inputs host->device from pinned memory, all results "
                            "device->host); two steps in flight on two streams; serial_ms_per_step = one step at a time")
    configs = {args.workload: config_summary(args.workload, w, res, ms_per_step)}
    others = {}
    for name in [n for n in args.others.split(",") if n and n != args.workload]:
        ow = workloads.by_name(name)
        r = bench_workload(torch, dp, ow, min(args.steps, 20), 3, flush, peaks, with_e2e=False)
        ms = float(np.mean(r["times_ms"]))
        configs[name] = config_summary(name, ow, r, ms)
        others[name] = dict(workload=ow.name, dtype=ow.dtype, value=ow.B / (ms * 1e-3), ms_per_step=ms,
                            warm_l2_ms_per_step=r["warm_ms"], eager_ms_per_step=r["eager_ms"], launches_per_step=r["launches_per_step"],
                            single_step_graph_ms_per_step=r["single_graph_ms"], one_stream_graph_ms_per_step=r.get("one_stream_ms"),
                            timing=("rotating sets, one graph of all timed steps" if r.get("rotating") else "flush + events per step"),
                            step_roofline=r["step_roofline"], step_roofline_frac=r["step_roofline_us"] / (ms * 1e3),
                            roofline=r["roofline"], breakdown_us=r["breakdown"])
    if args.others:
        line["launch_floor_us"] = launch_floors(torch, dp, max(args.steps, 20), flush)
        for k in ("cfg1", "cfg2", "cfg2_bf16"):
            if k in configs:
                configs[k]["launch_floor_us"] = line["launch_floor_us"]["cooperative"]
    if args.others and not args.no_extras:
        pts = sweep_points_compact(torch, dp, min(args.steps, 30), flush, peaks)
        others["cfg5_sweep"] = pts
        # compact: "B,T,d_in,d_out": [step us, fraction of the point's step roofline]
        configs["cfg5"] = {f"{r['B']},{r['T']},{r['d_in']},{r['d_out']}": [round(r["step_us"], 1), round(r["frac"], 3)]
                           for r in pts}
        for shape in ((128, 256, 512, "bf16"), (512, 512, 1024, "bf16")):
            r = bench_elementwise(torch, dp, *shape, min(args.steps, 20), flush, peaks)
            others[r["workload"]] = r
        r = bench_model_block(torch, dp, min(args.steps, 20), flush)
        others[r["workload"]] = r
        r = bench_per_layer(torch, dp, min(args.steps, 20), flush)
        others[r["workload"]] = r
        for cdt in ("f32", "bf16"):
            r = bench_model_cnn(torch, dp, cdt, min(args.steps, 20), flush)
            others[r["workload"]] = r
        for cdt in ("f32", "bf16"):
            r = bench_conv_implicit(torch, dp, "conv2_implicit_im2col_b128_" + cdt, 128, 32, 16, 16, 3, 1, 64, cdt,
                                    min(args.steps, 20), flush, peaks)
            others[r["workload"]] = r
    line["workloads"] = others
    if not args.no_cpu_baseline:
        line["cpu_baseline"], _, _ = oracle_sample(w)
    # per-configuration step times and roofline fractions: inside `roofline` (kept with the headline) and,
    # compact, as the LAST key of the line
    roof["per_config"] = {k: (v if k == "cfg5" else dict(us=v["us"], frac=v["frac"], bound=v["bound"])) for k, v in configs.items()}
    line["configs"] = configs
    print(json.dumps(line))


if __name__ == "__main__":
    main()
