#!/usr/bin/env python
"""Benchmark of the compressed-activation backward hot path.

One step = one pass of the whole path over a set of convolution layers: for every layer,
compress the saved input X to Z (k x k average pooling) and compute the weight gradient dW
from Z and the output gradient dY.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Headline workload: the large layers the targets are stated on -- the 3x3 128-channel layer on
64 x 64 maps at batch 256 (the pooling sweep's layer, at k = 2) and the four layers of a
ResNet-50 bottleneck stage at batch 128. The ResNet-18-shaped stack at batch 64 is timed as a
secondary block of the same JSON line. Prints one JSON line (rank 0). `--impl reference` times
the CPU checker.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "compressed-wgrad TFLOP/s + compress GB/s (% B200 roofline); saved-activation bytes"
UNIT = "TFLOP/s"
K_POOL = 2
DTYPE = "bf16"
LAYOUT = "nhwc"
NOMINAL_TFLOPS = 2250.0     # dense bf16, per GPU
NOMINAL_HBM_GBS = 8000.0

# (name, N, C_in, C_out, H, W, R, S, stride, pad)
WORKLOAD = "large_layers_bf16_nhwc_k2"
LAYERS = [
    ("sweep_3x3_128ch_64x64_b256", 256, 128, 128, 64, 64, 3, 3, 1, 1),
    ("bneck_1x1_256to64_56x56_b128", 128, 256, 64, 56, 56, 1, 1, 1, 0),
    ("bneck_3x3_64ch_56x56_b128", 128, 64, 64, 56, 56, 3, 3, 1, 1),
    ("bneck_1x1_64to256_56x56_b128", 128, 64, 256, 56, 56, 1, 1, 1, 0),
    ("bneck_3x3_s2_128ch_56x56_b128", 128, 128, 128, 56, 56, 3, 3, 2, 1),
]
ROOFLINE_LAYER = 0           # the kernel behind `roofline`: wgrad_tc2_kernel on the first layer
SECONDARY_WORKLOAD = "resnet18_3x3_stack_b64_bf16_k2"
SECONDARY = [
    ("64ch_56x56", 64, 64, 64, 56, 56, 3, 3, 1, 1),
    ("128ch_28x28", 64, 128, 128, 28, 28, 3, 3, 1, 1),
    ("256ch_14x14", 64, 256, 256, 14, 14, 3, 3, 1, 1),
    ("512ch_8x8", 64, 512, 512, 8, 8, 3, 3, 1, 1),
]
N_SETS = 2            # input buffer sets of the headline workload, rotated between steps
N_SETS_SECONDARY = 4  # the small stack needs four to exceed the L2
SEED_IMAGES = 8       # images drawn per layer; the batch repeats them (kernel time does not depend on values)
TRAFFIC_RECORD = os.path.join(ROOT, "paper_2409_11902_b200", "ncu_traffic.json")


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


def kernel_source_hash():
    """sha256 over the sources of the dominant kernel: a DRAM-traffic record taken with ncu counts
    only for the binary built from exactly these files."""
    h = hashlib.sha256()
    for f in ("wgrad_tc2.cu", "tc_ptx.cuh", "tc_units.h", "ac_common.h"):
        h.update(open(os.path.join(ROOT, "paper_2409_11902_b200", "csrc", f), "rb").read())
    return h.hexdigest()


def recorded_traffic(layer_name):
    """DRAM bytes per launch from the committed ncu record, or None if the kernel's sources have
    changed since it was taken (or there is none for this layer)."""
    try:
        rec = json.load(open(TRAFFIC_RECORD))
    except (OSError, ValueError):
        return None, None
    e = rec.get(layer_name)
    if not e or e.get("source_sha256") != kernel_source_hash():
        return None, None
    return e["dram_bytes_per_launch"], e.get("profile")


def descs(table):
    import paper_2409_11902_b200 as ac
    return [(name, ac.ConvDesc(N, ci, co, H, W, R, S, (st, st), (pd, pd), K_POOL, DTYPE, LAYOUT))
            for name, N, ci, co, H, W, R, S, st, pd in table]


def host_inputs(d, seed, n_images=None):
    """Seeded inputs of one layer on the host: `n_images` images drawn by the generator (default:
    the whole batch)."""
    from paper_2409_11902_b200 import synth
    n = d.N if n_images is None else min(d.N, n_images)
    x = synth.to_layout(synth.activation(seed, (n, d.C_in, d.H, d.W), d.dtype), d.layout)
    dy = synth.to_layout(synth.grad_output(seed, (n, d.C_out, d.Ho, d.Wo), d.dtype), d.layout)
    return x, dy


def tile_batch(t, N, shift=0):
    """The first images repeated along the batch up to N images, starting `shift` images in."""
    import torch
    n = t.shape[0]
    if n >= N:
        return t[:N].contiguous()
    reps = -(-(N + shift) // n)
    return t.repeat((reps, 1, 1, 1))[shift:shift + N].contiguous()


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); pw.append(float(r[2]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "reasons": sorted(reasons), "samples": len(sm)}


def max_over_ranks(value: float, device) -> float:
    """Slowest rank's time: the step time of a job whose replicas run side by side."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tflops(world: int, flops_per_replica: int, ms: float) -> float:
    """All replicas' work over the slowest replica's time (weak scaling)."""
    return world * flops_per_replica / (ms * 1e-3) / 1e12


def layer_bytes(d):
    elt = 2
    x = d.N * d.C_in * d.H * d.W * elt
    z = d.N * d.C_in * d.Hp * d.Wp * elt
    dy = d.N * d.C_out * d.Ho * d.Wo * elt
    dw = d.C_out * d.C_in * d.R * d.S * 4
    return x, z, dy, dw


class Workload:
    """Device buffers of a list of layers (several rotating input sets) and the timed passes."""

    def __init__(self, ac, layers, host, n_sets, dev):
        import torch
        self.ac, self.layers, self.n_sets, self.dev = ac, layers, n_sets, dev
        self.sets = []
        for s in range(n_sets):
            bufs = []
            for (name, d), (x, dy) in zip(layers, host):
                bufs.append(dict(
                    x=tile_batch(x, d.N, s).to(dev), dy=tile_batch(dy, d.N, s).to(dev),
                    z=torch.empty(d.z_shape, dtype=d.torch_dtype, device=dev),
                    dw=torch.empty(d.dw_shape, dtype=torch.float32, device=dev),
                    ws=torch.empty(max(ac.ac_workspace_bytes(d), 256), dtype=torch.uint8, device=dev)))
            self.sets.append(bufs)
        self.set_bytes = sum(b[k].numel() * b[k].element_size() for b in self.sets[0] for k in ("x", "dy", "z"))
        self.side = [torch.cuda.Stream(device=dev) for _ in layers]

    def step(self, it):
        """Every layer's compress -> wgrad, back to back on the current stream."""
        ac = self.ac
        for (name, d), b in zip(self.layers, self.sets[it % self.n_sets]):
            ac.ac_compress(d, b["x"], b["z"])
            ac.ac_conv2d_wgrad_compressed(d, b["z"], b["dy"], b["dw"], b["ws"])

    def step_concurrent(self, it):
        """The same step with every layer's chain on a stream of its own (the layers of a step do
        not depend on one another). Called under graph capture (fork / join)."""
        import torch
        ac = self.ac
        cur = torch.cuda.current_stream()
        for s_, ((name, d), b) in zip(self.side, zip(self.layers, self.sets[it % self.n_sets])):
            s_.wait_stream(cur)
            with torch.cuda.stream(s_):
                ac.ac_compress(d, b["x"], b["z"])
                ac.ac_conv2d_wgrad_compressed(d, b["z"], b["dy"], b["dw"], b["ws"])
        for s_ in self.side:
            cur.wait_stream(s_)

    def check_status(self):
        for bufs in self.sets:
            for b in bufs:
                st, detail = self.ac.ac_workspace_status(b["ws"])
                assert st == 0, f"device status {st} detail {detail:#x}"

    def step_graphs(self, concurrent):
        import torch
        graphs = []
        for sidx in range(self.n_sets):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                (self.step_concurrent if concurrent else self.step)(sidx)
            graphs.append(g)
        for g in graphs:
            g.replay()
        torch.cuda.synchronize()
        return graphs

    def time_one(self, fn, reps):
        """Microseconds per call of fn(buffers): `reps` calls over the rotating buffer sets
        captured into ONE graph with nothing between them, replayed once untimed and then
        `timed_replays` times, each between two events on the launching stream: the median (the
        least is left in `last_min`)."""
        import torch
        stream = torch.cuda.current_stream()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(reps):
                fn(i % self.n_sets)
        g.replay()
        torch.cuda.synchronize()
        per_call = []
        for _ in range(self.timed_replays):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            g.replay()
            e1.record(stream)
            torch.cuda.synchronize()
            per_call.append(e0.elapsed_time(e1) * 1e3 / reps)
        per_call.sort()
        self.last_min = per_call[0]
        return per_call[len(per_call) // 2]

    timed_replays = 3      # of each per-layer graph, after one untimed replay; the median is reported, the least beside it

    def per_layer(self, reps, peaks, kernel_events=True):
        """Per layer: compress alone, the weight-gradient call alone (kernel + split-K reduce), and
        the main weight-gradient kernel alone (events recorded by the library around that launch)."""
        import torch
        ac = self.ac
        out = []
        stream = torch.cuda.current_stream()
        for li, (name, d) in enumerate(self.layers):
            t_c = self.time_one(lambda s: ac.ac_compress(d, self.sets[s][li]["x"], self.sets[s][li]["z"]), reps)
            t_c_min = self.last_min
            t_w = self.time_one(lambda s: ac.ac_conv2d_wgrad_compressed(
                d, self.sets[s][li]["z"], self.sets[s][li]["dy"], self.sets[s][li]["dw"], self.sets[s][li]["ws"]), reps)
            t_w_min = self.last_min
            t_k = None
            if kernel_events:
                try:
                    evs = [[torch.cuda.Event(enable_timing=True, external=True) for _ in range(2)] for _ in range(reps)]
                    for pair in evs:
                        for e in pair:
                            e.record(stream)          # creates the event handles before capture
                    torch.cuda.synchronize()
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g):
                        for i in range(reps):
                            b = self.sets[i % self.n_sets][li]
                            ac.ac_set_kernel_timing_events(evs[i][0], evs[i][1])
                            ac.ac_conv2d_wgrad_compressed(d, b["z"], b["dy"], b["dw"], b["ws"])
                        ac.ac_set_kernel_timing_events(None, None)
                    g.replay()
                    torch.cuda.synchronize()
                    g.replay()
                    torch.cuda.synchronize()
                    t_k = sum(a.elapsed_time(b) for a, b in evs) * 1e3 / reps
                except (RuntimeError, TypeError):
                    ac.ac_set_kernel_timing_events(None, None)
                    t_k = None
            x, z, dy, dw = layer_bytes(d)
            wbytes = z + dy + dw
            ai = d.flops / wbytes
            bound_meas = min(peaks["bf16_tflops"], ai * peaks["hbm_gbs"] / 1e3)
            bound_nom = min(NOMINAL_TFLOPS, ai * NOMINAL_HBM_GBS / 1e3)
            info = ac.ac_wgrad_plan_info(d)
            # both intervals contain the main kernel (the call also the split-K reduction, the event pair
            # also its own record nodes, which moreover keep the reduction from being brought onto the
            # GPU early): each is an upper bound of the kernel's duration, the smaller one the tighter
            t_best = min(t_k, t_w) if t_k else t_w
            out.append({
                "layer": name, "gflop": d.flops / 1e9, "x_bytes": x, "z_bytes": z,
                "compress_us": t_c, "compress_us_min": t_c_min, "compress_gbs": (x + z) / t_c / 1e3,
                "compress_frac_of_hbm_measured": (x + z) / t_c / 1e3 / peaks["hbm_gbs"],
                "compress_frac_of_hbm_nominal": (x + z) / t_c / 1e3 / NOMINAL_HBM_GBS,
                "wgrad_call_us": t_w, "wgrad_call_us_min": t_w_min, "wgrad_call_tflops": d.flops / t_w / 1e6,
                "wgrad_kernel_ms": t_best / 1e3,
                "wgrad_kernel_tflops": d.flops / t_best / 1e6,
                "wgrad_kernel_ms_source": "library event pair" if t_k and t_k <= t_w else "whole call",
                "wgrad_event_pair_us": t_k,
                "wgrad_bytes": wbytes, "arithmetic_intensity": ai,
                "bound": "tensor" if bound_meas == peaks["bf16_tflops"] else "hbm",
                "bound_tflops_measured": bound_meas, "bound_tflops_nominal": bound_nom,
                "kernel_frac_of_bound_measured": d.flops / t_best / 1e6 / bound_meas,
                "kernel_frac_of_tensor_burst": d.flops / t_best / 1e6 / peaks["bf16_tflops"],
                "kernel_frac_of_tensor_sustained": (d.flops / t_best / 1e6 / peaks["bf16_tflops_sustained"]
                                                    if peaks.get("bf16_tflops_sustained") else None),
                "kernel_frac_of_tensor_nominal": d.flops / t_best / 1e6 / NOMINAL_TFLOPS,
                "splits": info["splits"], "ctas": info["ctas"],
            })
        return out


def launches_per_step(ac, layers):
    """Kernels of this library launched per step: compress, the weight-gradient kernel and, when K
    is split, the reduction."""
    n = 0
    for _, d in layers:
        n += 2 + (1 if ac.ac_wgrad_plan_info(d)["splits"] > 1 else 0)
    return n


def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2409_11902_b200 as ac
    import __graft_entry__ as entry

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    entry.build() if rank == 0 or world == 1 else None
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
        dist.barrier()
        if rank != 0:
            entry.build()
    peaks = load_peaks()
    layers = descs(LAYERS)
    host = [host_inputs(d, seed=rank * 100 + li, n_images=SEED_IMAGES) for li, (_, d) in enumerate(layers)]
    wl = Workload(ac, layers, host, N_SETS, dev)
    stream = torch.cuda.current_stream()

    for it in range(args.warmup):
        wl.step(it)
    torch.cuda.synchronize()
    wl.check_status()
    graphs = wl.step_graphs(args.concurrent_layers)

    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.2)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    t0.record(stream)
    for it in range(args.steps):
        graphs[(args.warmup + it) % N_SETS].replay()
    t1.record(stream)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    total_ms = max_over_ranks(t0.elapsed_time(t1), dev)
    reps = max(20, min(args.steps, 50))
    per_layer = wl.per_layer(reps, peaks)
    clocks = sampler.stop() if rank == 0 else None
    wl.check_status()

    flops = [d.flops for _, d in layers]
    ms_per_step = total_ms / args.steps
    value = whole_job_tflops(world, sum(flops), ms_per_step)
    x_bytes = sum(p["x_bytes"] for p in per_layer)
    z_bytes = sum(p["z_bytes"] for p in per_layer)
    comp_us = sum(p["compress_us"] for p in per_layer)
    comp_gbs = (x_bytes + z_bytes) / comp_us / 1e3
    wg_call_tflops = sum(flops) / sum(p["wgrad_call_us"] for p in per_layer) / 1e6

    # ---- end to end: host buffers in, dW out, through the C ABI ----------------
    pinned = []
    for (name, d), (x, dy) in zip(layers, host):
        pinned.append(dict(
            x=tile_batch(x, d.N).pin_memory(), dy=tile_batch(dy, d.N).pin_memory(),
            dw=torch.empty(d.dw_shape, dtype=torch.float32).pin_memory(),
            arena=torch.empty(ac.ac_host_step_arena_bytes(d), dtype=torch.uint8, device=dev)))
    h2d = sum(p["x"].numel() * 2 + p["dy"].numel() * 2 for p in pinned)
    d2h = sum(p["dw"].numel() * 4 for p in pinned)

    def e2e_step():
        # every layer's call on a stream of its own (the layers are independent and each has its own
        # arena), so that one layer's device->host copy of dW runs while the next layer's inputs are
        # still coming in: PCIe carries both directions at once
        for s_, ((name, d), p) in zip(wl.side, zip(layers, pinned)):
            s_.wait_stream(stream)
            ac.ac_backward_step_host(d, p["x"], p["dy"], p["dw"], None, p["arena"], stream=s_)
        for s_ in wl.side:
            stream.wait_stream(s_)
    for _ in range(3):
        e2e_step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    n_e2e = max(3, min(args.steps, 10))
    t0.record(stream)
    for _ in range(n_e2e):
        e2e_step()
    t1.record(stream)
    torch.cuda.synchronize()
    e2e_ms = max_over_ranks(t0.elapsed_time(t1) / n_e2e, dev)
    e2e = {"value": whole_job_tflops(world, sum(flops), e2e_ms), "unit": UNIT,
           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms}
    del pinned
    torch.cuda.empty_cache()

    # ---- secondary block: the ResNet-18-shaped stack at batch 64 ----------------
    secondary = None
    if rank == 0 and not args.no_secondary:
        sl = descs(SECONDARY)
        shost = [host_inputs(d, seed=50 + li, n_images=SEED_IMAGES) for li, (_, d) in enumerate(sl)]
        swl = Workload(ac, sl, shost, N_SETS_SECONDARY, dev)
        # the four layers run side by side on four streams: each plans for its share of the SMs
        budget = max(1, 148 // len(sl))
        ac.ac_set_sm_budget(budget)
        for it in range(3):
            swl.step(it)
        sgraphs = swl.step_graphs(concurrent=True)
        ac.ac_set_sm_budget(0)
        n_sec = max(args.steps, 200)
        t0.record(stream)
        for it in range(n_sec):
            sgraphs[it % N_SETS_SECONDARY].replay()
        t1.record(stream)
        torch.cuda.synchronize()
        s_ms = t0.elapsed_time(t1) / n_sec
        s_layers = swl.per_layer(20, peaks, kernel_events=False)
        swl.check_status()
        s_fl = sum(d.flops for _, d in sl)
        secondary = {
            "workload": SECONDARY_WORKLOAD, "ms_per_step": s_ms, "step_tflops": s_fl / s_ms / 1e9,
            "schedule": "one CUDA graph per buffer set, every layer's chain on a stream of its own, weight gradients "
                        f"planned for {budget} SMs each (ac_set_sm_budget); per_layer: each layer alone on the whole GPU",
            "l2": f"inputs rotated over {N_SETS_SECONDARY} buffer sets ({N_SETS_SECONDARY * swl.set_bytes / 1e6:.0f} MB, L2 is 126 MB)",
            "per_layer": [{k: p[k] for k in ("layer", "compress_us", "compress_gbs", "wgrad_call_us",
                                             "wgrad_call_tflops", "splits", "ctas")} for p in s_layers]}
        del swl, sgraphs

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    top = per_layer[ROOFLINE_LAYER]
    traffic, traffic_profile = recorded_traffic(top["layer"])
    k_tflops = top["wgrad_kernel_tflops"]
    tensor_peak = peaks["bf16_tflops"]
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "impl": "ours",
        "config": {
            "workload": WORKLOAD, "layers": [n for n, _ in layers], "k": K_POOL, "layout": LAYOUT,
            "inputs": f"X = max(N(0,1),0), dY ~ N(0,1e-4): {SEED_IMAGES} seeded images per layer, repeated along the batch",
            "l2": f"inputs rotated over {N_SETS} buffer sets ({N_SETS * wl.set_bytes / 1e6:.0f} MB in total, L2 is 126 MB); "
                  "every layer's X + dY alone exceeds or nearly fills the L2",
            "multi_gpu": "independent replicas, no collective",
            "layers_in_graph": "one stream per layer" if args.concurrent_layers else "back to back on one stream",
            "timing": "value: K steps replayed as CUDA graphs (one per buffer set), compress included. "
                      "per_layer and roofline come from separate passes, each layer by itself: "
                      f"compress_us and wgrad_call_us = {reps} launches captured into one graph with nothing between "
                      "them, replayed once untimed and three times between two CUDA events each (median; *_min = the least); wgrad_kernel_ms = the smaller of that and of the interval between "
                      "events the library records around the main kernel alone (external event nodes in the "
                      "graph, which cost a few microseconds themselves): both are upper bounds of its duration. "
                      "So value (whole step) and roofline (one kernel) are different schedules."},
        "wgrad_call_tflops": wg_call_tflops,
        "compress_gbs": comp_gbs,
        "compress_frac_of_hbm_peak": comp_gbs / peaks["hbm_gbs"],
        "compress_frac_of_hbm_nominal": comp_gbs / NOMINAL_HBM_GBS,
        "peaks": {"source": peaks["source"], "bf16_tflops_burst": peaks["bf16_tflops"],
                  "bf16_tflops_sustained": peaks.get("bf16_tflops_sustained"), "hbm_gbs": peaks["hbm_gbs"],
                  "nominal_bf16_tflops": NOMINAL_TFLOPS, "nominal_hbm_gbs": NOMINAL_HBM_GBS},
        "saved_activation_bytes": {"x": x_bytes, "z": z_bytes, "saved": x_bytes - z_bytes,
                                   "reduction": 1 - z_bytes / x_bytes},
        "per_layer": per_layer,
        "roofline": {"bound": "tensor", "kernel": "wgrad_tc2_kernel", "layer": top["layer"],
                     "achieved": k_tflops, "peak": tensor_peak, "unit": "TFLOP/s",
                     "frac": k_tflops / tensor_peak, "peak_source": peaks["source"] + " burst bf16",
                     "frac_of_sustained": (k_tflops / peaks["bf16_tflops_sustained"]
                                           if peaks.get("bf16_tflops_sustained") else None),
                     "frac_of_nominal": k_tflops / NOMINAL_TFLOPS,
                     "flops_per_launch": flops[ROOFLINE_LAYER],
                     "kernel_ms": top["wgrad_kernel_ms"], "kernel_ms_source": top["wgrad_kernel_ms_source"],
                     "traffic": traffic,
                     "traffic_unit": "DRAM bytes read + written per launch (ncu), null when the kernel's "
                                     "sources differ from the ones the record was taken on",
                     "traffic_profile": traffic_profile,
                     "algorithmic_bytes": top["wgrad_bytes"],
                     "step_level": {"achieved": value / world, "frac": value / world / tensor_peak,
                                    "note": "whole step of all layers incl. compress"}},
        "secondary": secondary,
        "e2e": e2e,
        "gpu_launches": args.steps * launches_per_step(ac, layers),
        "clocks": clocks,
    }
    out["peak_memory"] = peak_memory_block(args, dev) if args.peak_memory else None
    out["cpu_baseline"] = cpu_baseline(layers, host, args.cpu_frac)
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def peak_memory_block(args, dev):
    """Peak device memory of one ResNet-50 training step with the conv inputs saved whole, saved
    compressed, and saved compressed with 1-bit ReLU masks (Section 3's points of interest), and the
    duration of two further steps per scheme (step_ms)."""
    try:
        from paper_2409_11902_b200 import train_step
    except ImportError:
        return None
    return train_step.peak_memory_report(batch=args.peak_memory_batch, k=K_POOL, device=dev, time_steps=2)


def cpu_baseline(layers, host, n_frac):
    """The CPU checker, as it stands, on the first `n_frac` of every layer's batch: pooling +
    compressed dW. Its time is linear in the number of images."""
    import oracle
    from paper_2409_11902_b200 import synth
    t_total, fl = 0.0, 0
    for (name, d), (x, dy) in zip(layers, host):
        n = max(1, int(round(d.N * n_frac)))
        x64 = synth.to_f64(synth.from_layout(tile_batch(x, n), d.layout))
        dy64 = synth.to_f64(synth.from_layout(tile_batch(dy, n), d.layout))
        t = time.perf_counter()
        z = oracle.pool(x64, d.k)
        oracle.wgrad_compressed(z, dy64, d.H, d.W, d.R, d.S, d.stride, d.pad, d.k)
        t_total += time.perf_counter() - t
        fl += d.flops * n // d.N
    return {"value": fl / t_total / 1e12, "unit": UNIT, "cores": oracle.num_threads(),
            "kind": "oracle", "seconds": t_total,
            "sample": f"first {n_frac:.4f} of each layer's batch (the checker's time is linear in the images): "
                      f"fp64 pooling + compressed dW of all {len(layers)} layers",
            "seconds_extrapolated_to_full_step": t_total / n_frac}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import __graft_entry__ as entry
    import oracle
    oracle.build()
    layers = descs(LAYERS)
    host = [host_inputs(d, seed=li, n_images=SEED_IMAGES) for li, (_, d) in enumerate(layers)]
    frac = 1.0 / 16   # of each batch per step: keeps the whole run within minutes
    for _ in range(args.warmup):
        cpu_baseline(layers, host, frac)
    t = time.perf_counter()
    res = None
    for _ in range(args.steps):
        res = cpu_baseline(layers, host, frac)
    dt = (time.perf_counter() - t) / args.steps
    fl = sum(d.flops * max(1, int(round(d.N * frac))) // d.N for _, d in layers)
    v = fl / dt / 1e12
    print(json.dumps({
        "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "impl": "reference",
        "config": {"workload": WORKLOAD, "layers": [n for n, _ in layers], "k": K_POOL,
                   "layout": "nchw", "sample": res["sample"]},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": res["cores"], "kind": "oracle",
                         "sample": res["sample"]},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--concurrent-layers", action="store_true",
                    help="capture every layer's chain on a stream of its own instead of back to back")
    ap.add_argument("--no-secondary", action="store_true", help="skip the ResNet-18-shaped stack")
    ap.add_argument("--cpu-frac", type=float, default=1.0 / 4,
                    help="share of each layer's batch the CPU checker is timed on")
    ap.add_argument("--peak-memory", action=argparse.BooleanOptionalAction, default=True,
                    help="run one ResNet-50 training step per saving scheme and report peak memory")
    ap.add_argument("--peak-memory-batch", type=int, default=256)
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        args.warmup = max(args.warmup, 3)
        run_ours(args)


if __name__ == "__main__":
    main()
