#!/usr/bin/env python
"""Benchmark of the convolution-forward hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A step is one pass of the whole path over one batch of a workload: every layer of the named
network shape, each with its own resident input, weights, bias and output (the layers'
inputs are generated independently, so the working set is far larger than L2 and no L2
flush is needed between steps).  The step is captured once as a CUDA graph and the K timed
steps replay it (--no-graph: eager launches); per-layer times come from capturing every
distinct layer alone as a graph over rotating buffer sets.  The line also carries, under
`workloads`, the other throughput configurations (graph replay, per-path figures) and the
batch-1 workloads.  Prints ONE JSON line (rank 0).

N > 1 (under torchrun): the path has no exchange step; every rank runs an independent
replica on its own batch ("weak" scaling) and the line reports the aggregate.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_1901_00858_b200 import workloads  # noqa: E402

DEFAULT_WORKLOAD = "vgg16_n16"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


# ---- bookkeeping that needs no GPU (also exercised by the CPU tests) ------------------------

def layer_flops(batch: int, l) -> float:
    """2*N*K*(C/g)*R*S*P*Q: padded taps count, bias/ReLU/cast do not."""
    return 2.0 * batch * l.k * (l.c // l.group) * l.r * l.r * l.out * l.out


def layer_bytes(batch: int, l) -> float:
    """Algorithmic bytes: x read once, w once, bias once, y written once (fp16)."""
    return 2.0 * (batch * l.c * l.h * l.h + l.k * (l.c // l.group) * l.r * l.r + l.k + batch * l.k * l.out * l.out)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    return dict(FALLBACK_PEAKS, source="fallback")


def measured_traffic(workload: str, kernel: str, subset: bool):
    """DRAM bytes per launch of the dominant kernel from the committed ncu capture of this
    workload (profiles/traffic.txt: `workload kernel bytes_per_launch`), or None."""
    if subset:
        return None
    path = os.path.join(ROOT, "profiles", "traffic.txt")
    if not os.path.exists(path):
        return None
    for line in open(path):
        parts = line.split()
        if len(parts) >= 3 and not line.startswith("#") and parts[0] == workload and parts[1] == kernel:
            return float(parts[2])
    return None


def layer_roof_seconds(batch, l, peaks) -> float:
    return max(layer_flops(batch, l) / (peaks["bf16_tflops_sustained"] * 1e12),
               layer_bytes(batch, l) / (peaks["hbm_gbs"] * 1e9))


def aggregate(per_rank_flops, per_rank_images, max_seconds_per_step):
    """Whole-job throughput of independent replicas: everything all ranks processed divided
    by the slowest rank's time."""
    return {"tflops": sum(per_rank_flops) / max_seconds_per_step / 1e12,
            "images_per_s": sum(per_rank_images) / max_seconds_per_step}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self, window=None):
        """window = (t0, t1) host epoch seconds of the timed region: only samples inside it are
        used if there are at least three, else every sample taken while the bench ran."""
        import datetime
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "window": "timed region"}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = []
        for line in self.file.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rows.append((ts, float(parts[1]), float(parts[2]),
                             [nm for nm, v in zip(names, parts[5:9]) if v.lower().startswith("active")]))
            except ValueError:
                continue
        inside = [r for r in rows if window and window[0] <= r[0] <= window[1]]
        if len(inside) < 3:
            inside = rows
            out["window"] = "whole bench run (timed region shorter than three samples)"
        sm = [r[1] for r in inside]
        smax = [r[2] for r in inside]
        reasons = set(x for r in inside for x in r[3])
        self.file.close()
        try:
            os.unlink(self.file.name)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(smax), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


# ---- the oracle legs (CPU) -------------------------------------------------------------------

def oracle_pass(wl, batch):
    """One pass of every layer of the workload at `batch` images through the CPU oracle as it
    stands.  Returns (seconds, flops)."""
    import oracle
    secs, flops = 0.0, 0.0
    for li, l in enumerate(wl.expanded_unique()):
        x, w, b = workloads.make_tensors(wl.config_id, wl.batch, li, l, batch_override=batch)
        P = oracle.ConvParams(batch, l.c, l.h, l.h, l.k, l.r, l.r, l.pad, l.pad, l.stride, l.stride,
                              l.dil, l.dil, l.group)
        t0 = time.perf_counter()
        oracle.conv_fast(P, x, w, b, l.relu)
        secs += (time.perf_counter() - t0) * l.count
        flops += layer_flops(batch, l) * l.count
    return secs, flops


def cpu_baseline(wl):
    import oracle
    secs, flops = oracle_pass(wl, 1)
    batch = 1
    if secs < 5.0 and wl.batch > 1:
        batch = int(min(wl.batch, max(2, round(10.0 / max(secs, 1e-3)))))
        secs, flops = oracle_pass(wl, batch)
    return {"value": flops / secs / 1e12, "unit": "TFLOP/s", "cores": oracle.num_threads(),
            "kind": "oracle", "images_per_s": batch / secs,
            "sample": f"every layer of {wl.name} once at batch {batch} (of {wl.batch}); repeated shapes "
                      f"timed once and counted by multiplicity; {flops / 1e9:.1f} GFLOP in {secs:.1f} s"}


def run_reference(args, wl):
    """--impl reference: the CPU oracle on the machine's host cores, same metric and config; each
    step is a bounded sample (every layer of the workload at batch 1)."""
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    oracle.build()
    for _ in range(min(args.warmup, 1)):
        oracle_pass(wl, 1)
    steps = max(1, min(args.steps, 5))
    secs, flops = 0.0, 0.0
    for _ in range(steps):
        s, f = oracle_pass(wl, 1)
        secs += s
        flops += f
    val = flops / secs / 1e12
    line = {
        "impl": "reference", "metric": "conv_forward_tflops", "value": val, "unit": "TFLOP/s",
        "n_gpus": args.gpus, "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": secs / steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "sample": "every layer once at batch 1 per step"},
        "images_per_s": steps / secs,
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "kind": "oracle", "cores": oracle.num_threads(),
                         "sample": f"every layer of {wl.name} at batch 1, {steps} passes"},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---- the CUDA arm ----------------------------------------------------------------------------

def layer_roof(batch, l, peaks, tensor_key):
    return max(layer_flops(batch, l) / (peaks[tensor_key] * 1e12), layer_bytes(batch, l) / (peaks["hbm_gbs"] * 1e9))


def choose_regime(timed_seconds, clocks):
    """Which measured tensor peak a timed region is compared with: the burst figure when the
    region is shorter than a second and the clock sampler saw no power capping, else the
    sustained one (MEASURED_PEAKS.json holds both)."""
    capped = bool(clocks) and "sw_power_cap" in (clocks.get("reasons") or [])
    return "sustained" if (timed_seconds >= 1.0 or capped) else "burst"


def _geo(batch, l):
    return (batch, l.c, l.h, l.h, l.k, l.r, l.r, l.pad, l.pad, l.stride, l.stride, l.dil, l.dil, l.group)


def build_state(hgc, torch, layers, batch, gen, channels_last=False):
    """Resident tensors, one set per layer (weights registered once: steady-state inference).
    channels_last: every layer that can takes both layout flags; a layer that cannot read
    channels-last input (3-channel stems) takes the output flag alone."""
    state, n_in, n_out = [], 0, 0
    for l in layers:
        fl = 0
        if channels_last:
            d = None
            for fl in (hgc.HGC_FLAG_X_NHWC | hgc.HGC_FLAG_Y_NHWC, hgc.HGC_FLAG_Y_NHWC, 0):
                try:
                    d = hgc.ConvDesc(*_geo(batch, l), fl)
                    break
                except hgc.HgcError:
                    continue
            n_in += 1 if fl & hgc.HGC_FLAG_X_NHWC else 0
            n_out += 1 if fl & hgc.HGC_FLAG_Y_NHWC else 0
        else:
            d = hgc.ConvDesc(*_geo(batch, l))
        d.ensure_workspace()
        x = torch.empty((batch, l.c, l.h, l.h), dtype=torch.float16, device="cuda")
        x.uniform_(l.x_lo, 1.0, generator=gen)
        w = torch.empty((l.k, l.c // l.group, l.r, l.r), dtype=torch.float16, device="cuda")
        w.normal_(0.0, float(np.sqrt(2.0 / l.fan_in())), generator=gen)
        b = torch.empty((l.k,), dtype=torch.float16, device="cuda")
        b.uniform_(-0.1, 0.1, generator=gen)
        y = torch.empty((batch, l.k, l.out, l.out), dtype=torch.float16, device="cuda")
        d.set_weights(w)
        state.append((d, x, w, b, y, l))
    torch.cuda.synchronize()
    return state, n_in, n_out


def capture_step(hgc, torch, state, side):
    """The whole step as one CUDA graph on stream `side`.  Returns (graph, launches per step)."""
    graph = torch.cuda.CUDAGraph()
    c0 = hgc.kernel_launch_count()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for (d, x, w, b, y, l) in state:
                hgc.conv_forward(d, x, w, b, y, l.relu, side)
    per_step = hgc.kernel_launch_count() - c0
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        for _ in range(3):
            graph.replay()
    torch.cuda.synchronize()
    return graph, per_step


def time_replays(torch, graph, side, steps):
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(side):
        t0.record(side)
        for _ in range(steps):
            graph.replay()
        t1.record(side)
    torch.cuda.synchronize()
    return t0.elapsed_time(t1) / steps


def time_layers_as_graphs(hgc, torch, state, batch, side, replays=7):
    """Per-layer device times without launch gaps: every distinct layer shape is captured alone as
    a CUDA graph of `calls` forwards that rotate over enough (x, y) buffer sets to keep the
    footprint above twice the L2 size (at most 12 sets), and the graph is replayed `replays` times
    between events.  For layers whose input goes through the NCHW->NHWC layout pass, the pass
    is timed on its own the same way.  Returns {shape key: {"ms", "ms_min", "layout_ms", "sets"}}."""
    out = {}
    l2 = 126 << 20
    for (d, x, w, b, y, l) in state:
        key = (l.c, l.h, l.k, l.r, l.stride, l.pad, l.dil, l.group, l.relu)
        if key in out:
            continue
        per_set = (x.numel() + y.numel()) * 2
        sets = int(min(12, max(3, -(-2 * l2 // per_set))))
        xs = [x] + [torch.empty_like(x).copy_(x) for _ in range(sets - 1)]
        ys = [y] + [torch.empty_like(y) for _ in range(sets - 1)]
        calls = max(sets, 24 // sets * sets)

        def timed(fn):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                for i in range(sets):
                    fn(i)
                torch.cuda.synchronize()
                with torch.cuda.graph(g, stream=side):
                    for i in range(calls):
                        fn(i % sets)
            torch.cuda.synchronize()
            samples = []
            for _ in range(replays + 1):
                samples.append(time_replays(torch, g, side, 1) / calls)
            samples = samples[1:]
            return statistics.median(samples), min(samples)

        med, mn = timed(lambda i: hgc.conv_forward(d, xs[i], w, b, ys[i], l.relu, side))
        layout_ms = None
        info = d.plan_info() if d.path() == hgc.HGC_PATH_IGEMM else None
        if (info is not None and info["x_source"] == 0 and not info["fused_layout"]
                and not (d.params.flags & hgc.HGC_FLAG_X_NHWC) and l.c % 8 == 0):
            xt = torch.empty((batch, l.h, l.h, l.c), dtype=torch.float16, device="cuda")
            layout_ms, _ = timed(lambda i: hgc.layout_nchw_to_nhwc(xs[i], xt, batch, l.c, l.h, l.h, l.c, side))
            del xt
        out[key] = {"ms": med, "ms_min": mn, "layout_ms": layout_ms, "sets": sets}
        del xs, ys
    return out


def summarize(hgc, state, batch, layer_t, peaks, regime):
    """Per path and for the whole step: achieved TFLOP/s and GB/s from the per-layer graph times
    (a layer's layout pass counted with its path, and listed separately as `layout`)."""
    tensor_key = "bf16_tflops" if regime == "burst" else "bf16_tflops_sustained"
    by_path, layout = {}, {"ms": 0.0, "bytes": 0.0, "launches": 0}
    rows = []
    for (d, x, w, b, y, l) in state:
        key = (l.c, l.h, l.k, l.r, l.stride, l.pad, l.dil, l.group, l.relu)
        t = layer_t[key]
        p = hgc.PATH_NAMES[d.path()]
        e = by_path.setdefault(p, {"ms": 0.0, "flops": 0.0, "bytes": 0.0, "launches": 0, "roof_s": 0.0})
        e["ms"] += t["ms"]
        e["flops"] += layer_flops(batch, l)
        e["bytes"] += layer_bytes(batch, l)
        e["launches"] += 1
        e["roof_s"] += layer_roof(batch, l, peaks, tensor_key)
        if t["layout_ms"] is not None:
            layout["ms"] += t["layout_ms"]
            layout["bytes"] += 4.0 * x.numel()          # 2 bytes read + 2 written per element
            layout["launches"] += 1
        rows.append({"name": l.name, "path": p, "ms": t["ms"], "ms_min": t["ms_min"], "layout_ms": t["layout_ms"],
                     "tflops": layer_flops(batch, l) / (t["ms"] * 1e-3) / 1e12,
                     "gbs": layer_bytes(batch, l) / (t["ms"] * 1e-3) / 1e9,
                     "roof_frac": layer_roof(batch, l, peaks, tensor_key) * 1e3 / t["ms"]})
    per_path = {}
    for k, v in by_path.items():
        tf = v["flops"] / (v["ms"] * 1e-3) / 1e12
        gb = v["bytes"] / (v["ms"] * 1e-3) / 1e9
        per_path[k] = {"ms_per_step": v["ms"], "layers": v["launches"], "tflops": tf, "gbs": gb,
                       "frac_of_tensor_peak": tf / peaks[tensor_key], "frac_of_hbm_peak": gb / peaks["hbm_gbs"],
                       "roofline_frac": v["roof_s"] * 1e3 / v["ms"]}
    if layout["launches"]:
        gb = layout["bytes"] / (layout["ms"] * 1e-3) / 1e9
        per_path["layout"] = {"ms_per_step": layout["ms"], "layers": layout["launches"], "gbs": gb,
                              "frac_of_hbm_peak": gb / peaks["hbm_gbs"],
                              "note": "the NCHW->NHWC pass of the layers that need one, timed alone; its time is "
                                      "also inside those layers' path"}
    total_ms = sum(v["ms"] for v in by_path.values())
    t_roof = sum(v["roof_s"] for v in by_path.values())
    return by_path, per_path, rows, total_ms, t_roof


def measure_block_chain(hgc, torch, steps, side, rank):
    """MobileNet-v1 at batch 32 as a channels-last chain: the stem, then the 13 depthwise +
    pointwise blocks each as ONE kernel (hgc_dwpw_forward).  Same shapes, tensors per block."""
    wl = workloads.by_name("mobilenet_v1_n32")
    layers = wl.expanded()
    gen = torch.Generator(device="cuda")
    gen.manual_seed(777 + rank)
    n = wl.batch
    stem = layers[0]
    calls = []
    d0 = hgc.ConvDesc(*_geo(n, stem), hgc.HGC_FLAG_Y_NHWC)
    d0.ensure_workspace()
    x0 = torch.empty((n, stem.c, stem.h, stem.h), dtype=torch.float16, device="cuda").uniform_(0, 1, generator=gen)
    w0 = torch.empty((stem.k, stem.c, stem.r, stem.r), dtype=torch.float16, device="cuda").normal_(0, 0.27, generator=gen)
    b0 = torch.zeros(stem.k, dtype=torch.float16, device="cuda")
    y0 = torch.empty((n, stem.out, stem.out, stem.k), dtype=torch.float16, device="cuda")
    d0.set_weights(w0)
    calls.append(lambda st: hgc.conv_forward(d0, x0, w0, b0, y0, True, st))
    keep = [d0]
    flops = layer_flops(n, stem)
    for i in range(1, len(layers), 2):
        dw, pw = layers[i], layers[i + 1]
        d = hgc.DwPwDesc(n, dw.c, dw.h, dw.h, pw.k, dw.stride, hgc.HGC_FLAG_Y_NHWC)
        d.ensure_workspace()
        x = torch.empty((n, dw.h, dw.h, dw.c), dtype=torch.float16, device="cuda").uniform_(0, 1, generator=gen)
        w_dw = torch.empty((dw.c, 1, 3, 3), dtype=torch.float16, device="cuda").normal_(0, 0.47, generator=gen)
        w_pw = torch.empty((pw.k, dw.c, 1, 1), dtype=torch.float16, device="cuda").normal_(0, float(np.sqrt(2.0 / dw.c)), generator=gen)
        b_dw = torch.zeros(dw.c, dtype=torch.float16, device="cuda")
        b_pw = torch.zeros(pw.k, dtype=torch.float16, device="cuda")
        y = torch.empty((n, pw.out, pw.out, pw.k), dtype=torch.float16, device="cuda")
        d.set_weights(w_dw, w_pw)
        calls.append(lambda st, d=d, x=x, w_dw=w_dw, b_dw=b_dw, w_pw=w_pw, b_pw=b_pw, y=y:
                     hgc.dwpw_forward(d, x, w_dw, b_dw, w_pw, b_pw, y, True, True, st))
        keep.append(d)
        flops += layer_flops(n, dw) + layer_flops(n, pw)
    for c in calls:
        c(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    c0 = hgc.kernel_launch_count()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            for c in calls:
                c(side)
    per_step = hgc.kernel_launch_count() - c0
    torch.cuda.synchronize()
    ms = time_replays(torch, g, side, steps)
    ms = time_replays(torch, g, side, steps)
    for d in keep:
        d.close()
    return {"ms_per_step": ms, "steps": steps, "tflops": flops / (ms * 1e-3) / 1e12, "images_per_s": n / (ms * 1e-3),
            "launches_per_step": per_step, "launch": "cuda_graph",
            "note": "channels-last chain: stem + 13 depthwise+pointwise blocks, one kernel per block (hgc_dwpw_forward)"}


def measure_extra(hgc, torch, name, steps, peaks, side, rank):
    """One more workload for the JSON line's `workloads` object: graph replay of the step, and
    per-path figures from per-layer graph times."""
    wl = workloads.by_name(name)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(4321 + rank)
    state, _, _ = build_state(hgc, torch, wl.expanded(), wl.batch, gen)
    for _ in range(3):
        for (d, x, w, b, y, l) in state:
            hgc.conv_forward(d, x, w, b, y, l.relu, side)
    torch.cuda.synchronize()
    graph, per_step = capture_step(hgc, torch, state, side)
    host0 = time.time()
    ms = time_replays(torch, graph, side, steps)
    secs = time.time() - host0
    flops = sum(layer_flops(wl.batch, l) for (_, _, _, _, _, l) in state)
    out = {"ms_per_step": ms, "steps": steps, "tflops": flops / (ms * 1e-3) / 1e12,
           "images_per_s": wl.batch / (ms * 1e-3), "launches_per_step": per_step, "launch": "cuda_graph",
           "layers": len(state), "batch": wl.batch}
    if wl.batch > 1:
        regime = choose_regime(secs, None)
        layer_t = time_layers_as_graphs(hgc, torch, state, wl.batch, side)
        _, per_path, _, total_ms, t_roof = summarize(hgc, state, wl.batch, layer_t, peaks, regime)
        tensor_key = "bf16_tflops" if regime == "burst" else "bf16_tflops_sustained"
        t_roof_step = sum(layer_roof(wl.batch, l, peaks, tensor_key) for (_, _, _, _, _, l) in state)
        out["roofline_config"] = {"t_roof_ms": t_roof_step * 1e3, "frac": t_roof_step * 1e3 / ms, "regime": regime,
                                  "note": "sum over layers of max(flops / tensor peak, bytes / HBM peak), divided by "
                                          "the graph-replayed step time"}
        out["per_path"] = per_path
        out["sum_of_layer_ms"] = total_ms
        try:   # the same step with channels-last activations
            gen2 = torch.Generator(device="cuda")
            gen2.manual_seed(99 + rank)
            nstate, n_in, n_out = build_state(hgc, torch, wl.expanded(), wl.batch, gen2, True)
            for (d, x, w, b, y, l) in nstate:
                hgc.conv_forward(d, x, w, b, y, l.relu, side)
            torch.cuda.synchronize()
            gl, _ = capture_step(hgc, torch, nstate, side)
            out["channels_last"] = {"ms_per_step": time_replays(torch, gl, side, steps), "layers_with_channels_last_input": n_in,
                                    "layers_with_channels_last_output": n_out}
            for (d, *_r) in nstate:
                d.close()
            del nstate, gl
        except Exception as exc:
            out["channels_last"] = {"error": repr(exc)}
    for (d, *_rest) in state:
        d.close()
    del state, graph
    torch.cuda.empty_cache()
    return out


def run_ours(args, wl):
    import torch
    import torch.distributed as dist
    from paper_1901_00858_b200 import binding as hgc

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.launch_overlap:
        hgc.set_launch_overlap(True)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the CUDA path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    hgc.lib()
    peaks = load_peaks()
    stream = torch.cuda.current_stream()
    layers = wl.expanded()
    if args.only:
        layers = [l for l in layers if l.name in args.only.split(",")]
        if not layers:
            raise SystemExit(f"--only {args.only}: no such layer in {wl.name}")
    batch = args.batch if args.batch else wl.batch
    subset = bool(args.only or args.batch)

    gen = torch.Generator(device="cuda")
    gen.manual_seed(1234 + rank)
    state, n_cl_in, n_cl_out = build_state(hgc, torch, layers, batch, gen, args.layout == "channels_last")

    def one_step():
        for (d, x, w, b, y, l) in state:
            hgc.conv_forward(d, x, w, b, y, l.relu, stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    for _ in range(max(args.warmup, 3)):
        one_step()
    barrier()

    # The step is launch-bound in places (layers of 10-40 us behind a ctypes call each), so the
    # whole step is captured once as a CUDA graph and the timed steps replay it: same kernels,
    # same arguments, same order, no per-launch host cost.  --no-graph times eager launches.
    graph = None
    graph_err = None
    side = torch.cuda.Stream()
    launches_per_step = None
    if not args.no_graph:
        try:
            side.wait_stream(stream)
            graph, launches_per_step = capture_step(hgc, torch, state, side)
        except Exception as exc:  # capture not possible: say why and time eager launches
            graph = None
            graph_err = repr(exc)

    # timed region: exactly K steps between two events on the launching stream
    tstream = side if graph is not None else stream
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = hgc.kernel_launch_count()
    barrier()
    host_t0 = time.time()
    with torch.cuda.stream(tstream):
        t_start.record(tstream)
        for s in range(args.steps):
            if graph is not None:
                graph.replay()
            else:
                one_step()
        t_end.record(tstream)
    barrier()
    host_t1 = time.time()
    launches = (launches_per_step * args.steps) if graph is not None else hgc.kernel_launch_count() - launches0
    total_ms = t_start.elapsed_time(t_end)
    ms_per_step = total_ms / args.steps
    clocks = sampler.stop((host_t0, host_t1)) if rank == 0 else None

    # per-layer device times without launch gaps: every distinct layer captured alone as a graph
    layer_t = time_layers_as_graphs(hgc, torch, state, batch, side) if not args.no_graph else None

    # ---- the same step with channels-last activations (HGC_FLAG_X_NHWC / HGC_FLAG_Y_NHWC) --------
    # Not the headline (the metric is NCHW in, NCHW out): what a stack of layers that keeps its
    # activations channels-last between layers pays per step.  Layers that cannot take a flag
    # (3-channel stems on the input side) keep NCHW on that side.
    nhwc = None
    if not args.no_graph and args.layout == "nchw":
        try:
            gen2 = torch.Generator(device="cuda")
            gen2.manual_seed(99 + rank)
            nstate, n_in, n_out = build_state(hgc, torch, layers, batch, gen2, True)
            for (d, x, w, b, y, l) in nstate:
                hgc.conv_forward(d, x, w, b, y, l.relu, side)
            torch.cuda.synchronize()
            gl, _ = capture_step(hgc, torch, nstate, side)
            nms = time_replays(torch, gl, side, args.steps)
            nhwc = {"ms_per_step": nms, "layers_with_channels_last_input": n_in,
                    "layers_with_channels_last_output": n_out, "layers": len(nstate),
                    "note": "same layers, activations channels-last where the layer takes the flag; this rank"}
            for (d, *_r) in nstate:
                d.close()
            del nstate, gl
            torch.cuda.empty_cache()
        except Exception as exc:
            nhwc = {"error": repr(exc)}

    # ---- end to end through the host-buffer entry point ------------------------------------
    e2e_steps = max(1, min(args.steps, 5))
    host = []
    h2d = d2h = 0
    for (d, x, w, b, y, l) in (state if not args.no_e2e else []):
        d.ensure_workspace(host=True)
        d.set_weights(w)
        hx = torch.empty(x.shape, dtype=torch.float16).pin_memory()
        hx.copy_(x.cpu())
        hw = w.cpu().pin_memory()
        hb = b.cpu().pin_memory()
        hy = torch.empty(y.shape, dtype=torch.float16).pin_memory()
        host.append((hx, hw, hb, hy))
        h2d += (hx.numel() + hw.numel() + hb.numel()) * 2
        d2h += hy.numel() * 2
    torch.cuda.synchronize()

    # Layers are independent, so they take turns on eight streams: the device-to-host copy of
    # one layer's result runs beside the host-to-device copies of the next ones (the link is full
    # duplex); every layer's copies and kernels stay ordered within its stream.  (Measured, VGG-16
    # batch 16: 2 streams 11.7 ms per step, 4: 10.3, 8: 8.9, 13: 8.8.)
    lanes = [torch.cuda.Stream() for _ in range(8)]

    def e2e_step():
        for i, ((d, x, w, b, y, l), (hx, hw, hb, hy)) in enumerate(zip(state, host)):
            hgc.conv_forward_host(d, hx, hw, hb, hy, l.relu, lanes[i % len(lanes)])

    e2e_ms = float("nan")
    if not args.no_e2e:
        e2e_step()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for ln in lanes:
            ln.wait_stream(stream)
        for _ in range(e2e_steps):
            e2e_step()
        for ln in lanes:
            stream.wait_stream(ln)
        e1.record(stream)
        barrier()
        e2e_ms = e0.elapsed_time(e1) / e2e_steps

    # ---- the other workloads (single GPU, whole workloads only) ------------------------------
    extras = None
    if world == 1 and not subset and not args.no_graph and not args.no_extra and args.layout == "nchw":
        extras = {}
        big = [n for n in ("vgg16_n16", "mobilenet_v1_n32", "resnet50_n64") if n != wl.name]
        small = [n for n in ("vgg16_n1", "mobilenet_v1_n1") if n != wl.name]
        for name in big + small:
            try:
                extras[name] = measure_extra(hgc, torch, name, 50, peaks, side, rank)
            except Exception as exc:
                extras[name] = {"error": repr(exc)}
        try:
            extras["mobilenet_v1_n32_block_kernels"] = measure_block_chain(hgc, torch, 50, side, rank)
        except Exception as exc:
            extras["mobilenet_v1_n32_block_kernels"] = {"error": repr(exc)}

    # ---- max over ranks ---------------------------------------------------------------------
    if world > 1:
        t = torch.tensor([ms_per_step, e2e_ms], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_per_step, e2e_ms = float(t[0]), float(t[1])
        lt = torch.tensor([launches], dtype=torch.int64, device="cuda")
        dist.all_reduce(lt)
        launches = int(lt[0])

    step_flops = sum(layer_flops(batch, l) for l in layers)
    agg = aggregate([step_flops] * world, [batch] * world, ms_per_step * 1e-3)
    e2e = aggregate([step_flops] * world, [batch] * world, e2e_ms * 1e-3)

    if rank == 0:
        regime = choose_regime(total_ms * 1e-3, clocks)
        tensor_key = "bf16_tflops" if regime == "burst" else "bf16_tflops_sustained"
        t_roof_step = sum(layer_roof(batch, l, peaks, tensor_key) for l in layers)
        roof, per_path, rows = None, None, None
        if layer_t is not None:
            by_path, per_path, rows, sum_layer_ms, _ = summarize(hgc, state, batch, layer_t, peaks, regime)
            # dominant kernel path by time; its achieved rate from the per-layer graph times
            dom = max(by_path, key=lambda k: by_path[k]["ms"])
            e = by_path[dom]
            hbm_bound = e["bytes"] / (peaks["hbm_gbs"] * 1e9) > e["flops"] / (peaks[tensor_key] * 1e12)
            if dom == "depthwise" or hbm_bound:
                ach = e["bytes"] / (e["ms"] * 1e-3) / 1e9
                roof = {"bound": "hbm", "kernel": dom, "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                        "frac": ach / peaks["hbm_gbs"]}
            else:
                ach = e["flops"] / (e["ms"] * 1e-3) / 1e12
                roof = {"bound": "tensor", "kernel": dom, "achieved": ach, "peak": peaks[tensor_key], "unit": "TFLOP/s",
                        "frac": ach / peaks[tensor_key], "frac_burst": ach / peaks["bf16_tflops"],
                        "frac_sustained": ach / peaks["bf16_tflops_sustained"], "regime": regime,
                        "frac_of_step": (e["flops"] / (ms_per_step * 1e-3) / 1e12) / peaks[tensor_key]}
            roof["traffic"] = measured_traffic(wl.name, dom, subset)
            roof["peak_source"] = peaks["source"]
            roof["share_of_step"] = e["ms"] / sum_layer_ms
            roof["avg_launch_ms"] = e["ms"] / e["launches"]
            roof["timing"] = ("every distinct layer captured alone as a CUDA graph over rotating buffer sets "
                              "(median of 7 replays); a layer's layout pass is counted with its kernel")
        cpu = cpu_baseline(wl) if world == 1 and not args.no_cpu_baseline else None
        line = {
            "metric": "conv_forward_tflops", "value": agg["tflops"], "unit": "TFLOP/s", "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f16 (f32 accumulate)",
            "data": "synthetic",
            "config": {"workload": wl.name if not subset else f"{wl.name} (subset: only={args.only or 'all'}, batch={batch})",
                       "layers": len(layers), "batch_per_gpu": batch,
                       "l2": "inputs larger than L2 (every layer has its own tensors)",
                       "launch": "cuda_graph" if graph is not None else "eager",
                       "parallelism": f"replicas x{world}" if world > 1 else "single GPU",
                       **({"layout": f"channels_last ({n_cl_in} of {len(layers)} layers read, {n_cl_out} write "
                                     "channels-last activations)"} if args.layout == "channels_last" else {})},
            "images_per_s": agg["images_per_s"],
            "roofline": roof,
            "roofline_config": {"t_roof_ms": t_roof_step * 1e3, "frac": t_roof_step * 1e3 / ms_per_step, "regime": regime,
                                "frac_burst": sum(layer_roof(batch, l, peaks, "bf16_tflops") for l in layers) * 1e3 / ms_per_step,
                                "frac_sustained": sum(layer_roof(batch, l, peaks, "bf16_tflops_sustained") for l in layers) * 1e3 / ms_per_step,
                                "note": "sum over layers of max(flops / tensor peak, bytes / HBM peak), divided by the "
                                        "timed step (ms_per_step); regime = which measured tensor peak applies: burst "
                                        "for a timed region under a second without power capping, else sustained"},
            "per_path": per_path,
            "e2e": {"value": e2e["tflops"], "unit": "TFLOP/s", "ms_per_step": e2e_ms, "steps": e2e_steps,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "images_per_s": e2e["images_per_s"]},
            "gpu_launches": launches,
            "clocks": clocks,
        }
        if graph_err is not None:
            line["graph_error"] = graph_err
        if nhwc is not None:
            if "ms_per_step" in nhwc:
                nhwc["tflops"] = step_flops / (nhwc["ms_per_step"] * 1e-3) / 1e12
            line["channels_last"] = nhwc
        if extras is not None:
            line["workloads"] = extras
        if cpu is not None:
            line["cpu_baseline"] = cpu
        if args.layers and rows is not None:
            line["layers"] = rows
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ---- the two layers next to the convolution path (not part of the default run) ----------------

def run_side_op(args):
    """--op cast: FP32 -> FP16 cast of 64 Mi values (HBM bound, 6 bytes per element).
    --op bn: batch norm with batch statistics on two VGG-16 activation tensors (HBM bound, 8 bytes
    per element: three reads of x, one write of y).
    --op fc: the three inner-product layers of a VGG-16 classifier at batch 64 (25088->4096,
    4096->4096, 4096->1000; weight-streaming, HBM bound).  One JSON line each, same keys."""
    import torch
    from paper_1901_00858_b200 import binding as hgc
    import oracle
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the CUDA path has no CPU fallback")
    hgc.lib()
    peaks = load_peaks()
    stream = torch.cuda.current_stream()
    steps, warm = args.steps, max(args.warmup, 3)
    if args.op == "cast":
        count = 64 << 20
        nbuf = 3   # rotate buffers: 1.1 GB footprint, far larger than L2
        srcs = [torch.randn(count, dtype=torch.float32, device="cuda") for _ in range(nbuf)]
        dsts = [torch.empty(count, dtype=torch.float16, device="cuda") for _ in range(nbuf)]
        over = torch.zeros(1, dtype=torch.int64, device="cuda")
        step = lambda i: hgc.cast_f32_to_f16(srcs[i % nbuf], dsts[i % nbuf], overflow_count=over, stream=stream)
        step_bytes, step_flops = 6.0 * count, 0.0
        metric, unit, workload = "cast_f32_to_f16_gbs", "GB/s", "cast_64Mi"
        sample = np.random.default_rng(0).normal(0, 1, 16 << 20).astype(np.float32)
        t0 = time.perf_counter(); oracle.cast_f32_to_f16(sample); dt = time.perf_counter() - t0
        cpu = {"value": 6.0 * sample.size / dt / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle",
               "sample": f"{sample.size} values once ({dt:.2f} s)"}
    elif args.op == "bn":
        # the output of VGG-16's first block at batch 16 (16 x 64 x 224 x 224, 103 MB) and of its
        # second (16 x 128 x 112 x 112, 51 MB), alternating: 308 MB touched per pair, larger than L2
        shapes_bn = [(16, 64, 224, 224), (16, 128, 112, 112)]
        bufs = []
        for shp in shapes_bn:
            n_, c_ = shp[0], shp[1]
            hw_ = shp[2] * shp[3]
            x = (torch.rand(shp, device="cuda") * 255.0).to(torch.float16)
            y = torch.empty_like(x)
            mean = torch.empty(c_, dtype=torch.float32, device="cuda")
            var = torch.empty(c_, dtype=torch.float32, device="cuda")
            ws = torch.empty(hgc.batchnorm_workspace_bytes(n_, c_, hw_), dtype=torch.uint8, device="cuda")
            bufs.append((x, y, mean, var, ws))
        def step(i):
            for x, y, mean, var, ws in bufs:
                hgc.batchnorm_forward(x, y, 1e-5, mean, var, ws, shift_log2=-5, stream=stream)
        elems = sum(b[0].numel() for b in bufs)
        step_bytes, step_flops = 8.0 * elems, 0.0   # x read three times, y written once
        metric, unit, workload = "batchnorm_gbs", "GB/s", "vgg16_block1_block2_n16"
        sample = (np.random.default_rng(0).integers(0, 256, (8, 64, 224, 224))).astype(np.float16)
        t0 = time.perf_counter(); oracle.batchnorm(sample, 1e-5); dt = time.perf_counter() - t0
        cpu = {"value": 8.0 * sample.size / dt / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle",
               "sample": f"{sample.size} values once ({dt:.2f} s)"}
    else:
        n = 64
        shapes = [(25088, 4096), (4096, 4096), (4096, 1000)]
        layers = []
        for c, k in shapes:
            d = hgc.ConvDesc.inner_product(n, c, k)
            d.ensure_workspace()
            x = torch.rand((n, c), dtype=torch.float16, device="cuda")
            w = torch.randn((k, c), dtype=torch.float16, device="cuda") * float(np.sqrt(2.0 / c))
            b = torch.zeros(k, dtype=torch.float16, device="cuda")
            y = torch.empty((n, k), dtype=torch.float16, device="cuda")
            d.set_weights(w)
            layers.append((d, x, w, b, y))
        def step(i):
            for d, x, w, b, y in layers:
                hgc.conv_forward(d, x, w, b, y, True, stream)
        step_flops = sum(2.0 * n * c * k for c, k in shapes)
        step_bytes = sum(2.0 * (n * c + c * k + k + n * k) for c, k in shapes)
        metric, unit, workload = "inner_product_tflops", "TFLOP/s", "vgg16_classifier_n64"
        rng = np.random.default_rng(0)
        t0 = time.perf_counter()
        oracle.inner_product(rng.uniform(-1, 1, (4, 4096)).astype(np.float16),
                             rng.normal(0, 0.02, (1000, 4096)).astype(np.float16), None, True)
        dt = time.perf_counter() - t0
        cpu = {"value": 2.0 * 4 * 4096 * 1000 / dt / 1e12, "unit": "TFLOP/s", "cores": 1, "kind": "oracle",
               "sample": f"4096->1000 at batch 4 once ({dt:.2f} s)"}
    sampler = ClockSampler(0)
    sampler.start()
    for i in range(warm):
        step(i)
    torch.cuda.synchronize()
    c0 = hgc.kernel_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    host_t0 = time.time()
    e0.record(stream)
    for i in range(steps):
        step(i)
    e1.record(stream)
    torch.cuda.synchronize()
    host_t1 = time.time()
    ms = e0.elapsed_time(e1) / steps
    gbs = step_bytes / (ms * 1e-3) / 1e9
    value = gbs if args.op in ("cast", "bn") else step_flops / (ms * 1e-3) / 1e12
    line = {"metric": metric, "value": value, "unit": unit, "n_gpus": 1, "steps": steps, "warmup": warm,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32 -> f16" if args.op == "cast" else "f16 (f32 accumulate)", "data": "synthetic",
            "config": {"workload": workload, "l2": "buffers rotate over a footprint larger than L2" if args.op == "cast"
                       else ("two tensors alternate, 308 MB touched per step" if args.op == "bn"
                             else "weights (278 MB) larger than L2"), "launch": "eager"},
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm_gbs"], "traffic": None, "peak_source": peaks["source"]},
            "cpu_baseline": cpu, "gpu_launches": hgc.kernel_launch_count() - c0,
            "e2e": {"value": None, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
                    "note": "side operation: device-resident timing only"},
            "clocks": sampler.stop((host_t0, host_t1))}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--op", choices=["conv", "cast", "fc", "bn"], default="conv",
                    help="conv: the convolution path (default); cast / fc / bn: the FP32->FP16 cast, the "
                         "inner-product layer and the batch-norm layer, measured on their own")
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD,
                    help="one of: " + ", ".join(w.name for w in workloads.all_workloads()))
    ap.add_argument("--layout", choices=["nchw", "channels_last"], default="nchw",
                    help="nchw: the metric's configuration (default). channels_last: the same layers with "
                         "HGC_FLAG_X_NHWC / HGC_FLAG_Y_NHWC where a layer takes them (a chained stack)")
    ap.add_argument("--layers", action="store_true", help="add per-layer figures to the JSON line")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="time eager launches instead of replaying the step as a CUDA graph")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg (profiling runs)")
    ap.add_argument("--no-extra", action="store_true", help="skip the other workloads of the `workloads` object")
    ap.add_argument("--launch-overlap", action="store_true",
                    help="launch the library's kernels with programmatic stream serialization (hgc_set_launch_overlap)")
    ap.add_argument("--only", default="", help="comma-separated layer names: run just these layers (profiling)")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (profiling on a small case)")
    args = ap.parse_args()
    if args.op != "conv":
        if int(os.environ.get("RANK", "0")) == 0:
            run_side_op(args)
        return
    wl = workloads.by_name(args.workload)
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
