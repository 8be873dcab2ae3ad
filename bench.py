#!/usr/bin/env python
"""Benchmark of the compressed-activation backward hot path.

One step = one pass of the whole path over a stack of convolution layers:
for every layer, compress the saved input X to Z (k x k average pooling) and
compute the weight gradient dW from Z and the output gradient dY.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints one JSON line (rank 0). `--impl reference` times the CPU checker.
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
sys.path.insert(0, ROOT)

METRIC = "compressed-wgrad TFLOP/s + compress GB/s (% B200 roofline); saved-activation bytes"
UNIT = "TFLOP/s"

# ResNet-18-shaped 3x3 conv layers at batch 64, bf16, k = 2; the 7x7 map is
# padded to even (8x8).  (N, C_in, C_out, H, W, R, S, stride, pad)
WORKLOAD = "resnet18_3x3_stack_b64_bf16_k2"
LAYERS = [
    ("64ch_56x56", 64, 64, 64, 56, 56, 3, 3, 1, 1),
    ("128ch_28x28", 64, 128, 128, 28, 28, 3, 3, 1, 1),
    ("256ch_14x14", 64, 256, 256, 14, 14, 3, 3, 1, 1),
    ("512ch_8x8", 64, 512, 512, 8, 8, 3, 3, 1, 1),
]
K_POOL = 2
DTYPE = "bf16"
LAYOUT = "nhwc"
N_SETS = 4   # input buffer sets rotated between steps so that inputs are never L2-resident
# dram__bytes_read.sum + dram__bytes_write.sum of the four wgrad_tc2_kernel launches of one step, from
# one ncu capture of this command (profiles/launch_list_bench_resnet18_stack.md). Set to None whenever
# wgrad_tc2.cu changes after that capture.
WGRAD_DRAM_TRAFFIC_PER_STEP = 61_709_824


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


def descs():
    import paper_2409_11902_b200 as ac
    return [(name, ac.ConvDesc(N, ci, co, H, W, R, S, (st, st), (pd, pd), K_POOL, DTYPE, LAYOUT))
            for name, N, ci, co, H, W, R, S, st, pd in LAYERS]


def host_inputs(d, seed):
    from paper_2409_11902_b200 import synth
    x = synth.to_layout(synth.activation(seed, (d.N, d.C_in, d.H, d.W), d.dtype), d.layout)
    dy = synth.to_layout(synth.grad_output(seed, (d.N, d.C_out, d.Ho, d.Wo), d.dtype), d.layout)
    return x, dy


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
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


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
    layers = descs()

    # ---- device buffers: N_SETS rotating copies of every layer's inputs --------
    host, sets = [], []
    for li, (name, d) in enumerate(layers):
        host.append(host_inputs(d, seed=rank * 100 + li))
    for s in range(N_SETS):
        bufs = []
        for (name, d), (x, dy) in zip(layers, host):
            bufs.append(dict(
                x=x.to(dev), dy=dy.to(dev),
                z=torch.empty(d.z_shape, dtype=d.torch_dtype, device=dev),
                dw=torch.empty(d.dw_shape, dtype=torch.float32, device=dev),
                ws=torch.empty(max(ac.ac_workspace_bytes(d), 256), dtype=torch.uint8, device=dev)))
        sets.append(bufs)
    set_bytes = sum(b[k].numel() * b[k].element_size() for b in sets[0] for k in ("x", "dy", "z"))
    stream = torch.cuda.current_stream()

    def step(it, events=None):
        bufs = sets[it % N_SETS]
        for li, ((name, d), b) in enumerate(zip(layers, bufs)):
            if events is not None:
                events[li][0].record(stream)
            ac.ac_compress(d, b["x"], b["z"])
            if events is not None:
                events[li][1].record(stream)
            ac.ac_conv2d_wgrad_compressed(d, b["z"], b["dy"], b["dw"], b["ws"])
            if events is not None:
                events[li][2].record(stream)

    side = [torch.cuda.Stream(device=dev) for _ in layers]

    def step_concurrent(it):
        """The same step with every layer's chain (compress, wgrad, reduce) on a stream of its
        own: the layers of a step do not depend on one another, so their launch latencies,
        pipeline fills and drains overlap. Called under graph capture (fork / join)."""
        cur = torch.cuda.current_stream()
        bufs = sets[it % N_SETS]
        for s_, ((name, d), b) in zip(side, zip(layers, bufs)):
            s_.wait_stream(cur)
            with torch.cuda.stream(s_):
                ac.ac_compress(d, b["x"], b["z"])
                ac.ac_conv2d_wgrad_compressed(d, b["z"], b["dy"], b["dw"], b["ws"])
        for s_ in side:
            cur.wait_stream(s_)

    for it in range(args.warmup):
        step(it)
    torch.cuda.synchronize()
    for b in sets[(args.warmup - 1) % N_SETS] if args.warmup else []:
        st, detail = ac.ac_workspace_status(b["ws"])
        assert st == 0, f"device status {st} detail {detail:#x}"

    # One CUDA graph per buffer set: a step is 4 x (compress, status reset, wgrad, reduce)
    # launches of a few tens of microseconds each, so the timed loop replays graphs
    # instead of paying the Python/ctypes launch path per call.
    graphs = []
    for sidx in range(N_SETS):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            if args.serial_layers:
                step(sidx)
            else:
                step_concurrent(sidx)
        graphs.append(g)
    for sidx in range(N_SETS):
        graphs[sidx].replay()
    torch.cuda.synchronize()

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

    # Second live pass for the per-kernel figures behind the roofline: the same steps, layers
    # back to back on one stream, with a CUDA event around every C-ABI call. The calls are
    # captured into one graph per buffer set with the events as graph nodes, so that the
    # gaps between events are the kernels' and not the Python interpreter's; if this torch
    # cannot record timing events under capture, the calls are launched one by one instead.
    n_ev = min(args.steps, 200)
    comp_acc = [0.0] * len(layers)
    wgrad_acc = [0.0] * len(layers)
    kern_acc = [0.0] * len(layers)     # the main weight-gradient kernel alone
    per_kernel_mode = "graph with event nodes"
    try:
        # Two graphs per buffer set, so that the event nodes of one measurement do not sit inside the
        # other's intervals (an event-record node costs a few microseconds of its own): one with
        # events around the C-ABI calls, one with events only around the main weight-gradient
        # kernel, recorded by the library itself through its profiling hook.
        ev_sets, ev_graphs, kev_sets, kev_graphs = [], [], [], []
        for sidx in range(N_SETS):
            evs = [[torch.cuda.Event(enable_timing=True, external=True) for _ in range(3)] for _ in layers]
            kevs = [[torch.cuda.Event(enable_timing=True, external=True) for _ in range(2)] for _ in layers]
            for li in range(len(layers)):
                for e in evs[li] + kevs[li]:
                    e.record(stream)          # creates the event handles before capture
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                cur = torch.cuda.current_stream()
                for li, ((name, d), b) in enumerate(zip(layers, sets[sidx])):
                    evs[li][0].record(cur)
                    ac.ac_compress(d, b["x"], b["z"])
                    evs[li][1].record(cur)
                    ac.ac_conv2d_wgrad_compressed(d, b["z"], b["dy"], b["dw"], b["ws"])
                    evs[li][2].record(cur)
            gk = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gk):
                for li, ((name, d), b) in enumerate(zip(layers, sets[sidx])):
                    ac.ac_compress(d, b["x"], b["z"])
                    ac.ac_set_kernel_timing_events(kevs[li][0], kevs[li][1])
                    ac.ac_conv2d_wgrad_compressed(d, b["z"], b["dy"], b["dw"], b["ws"])
                    ac.ac_set_kernel_timing_events(None, None)
            ev_sets.append(evs)
            ev_graphs.append(g)
            kev_sets.append(kevs)
            kev_graphs.append(gk)
        for it in range(n_ev):
            sidx = (args.warmup + it) % N_SETS
            ev_graphs[sidx].replay()
            torch.cuda.synchronize()
            for li in range(len(layers)):
                comp_acc[li] += ev_sets[sidx][li][0].elapsed_time(ev_sets[sidx][li][1])
                wgrad_acc[li] += ev_sets[sidx][li][1].elapsed_time(ev_sets[sidx][li][2])
        for it in range(n_ev):
            sidx = (args.warmup + it) % N_SETS
            kev_graphs[sidx].replay()
            torch.cuda.synchronize()
            for li in range(len(layers)):
                kern_acc[li] += kev_sets[sidx][li][0].elapsed_time(kev_sets[sidx][li][1])
    except (RuntimeError, TypeError):
        ac.ac_set_kernel_timing_events(None, None)
        per_kernel_mode = "call by call"
        comp_acc = [0.0] * len(layers)
        wgrad_acc = [0.0] * len(layers)
        kern_acc = None
        ev = [[[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in layers] for _ in range(n_ev)]
        for it in range(n_ev):
            step(args.warmup + it, ev[it])
        torch.cuda.synchronize()
        for it in range(n_ev):
            for li in range(len(layers)):
                comp_acc[li] += ev[it][li][0].elapsed_time(ev[it][li][1])
                wgrad_acc[li] += ev[it][li][1].elapsed_time(ev[it][li][2])
    clocks = sampler.stop() if rank == 0 else None
    for b in sets[0]:
        st, detail = ac.ac_workspace_status(b["ws"])
        assert st == 0, f"device status {st} detail {detail:#x}"
    comp_ms = [v / n_ev for v in comp_acc]
    wgrad_ms = [v / n_ev for v in wgrad_acc]
    flops = [d.flops for _, d in layers]
    elt = 2
    comp_bytes = [(d.N * d.C_in * d.H * d.W + d.N * d.C_in * d.Hp * d.Wp) * elt for _, d in layers]
    x_bytes = sum(d.N * d.C_in * d.H * d.W * elt for _, d in layers)
    z_bytes = sum(d.N * d.C_in * d.Hp * d.Wp * elt for _, d in layers)
    ms_per_step = total_ms / args.steps
    value = whole_job_tflops(world, sum(flops), ms_per_step)
    wg_tflops = sum(flops) / (sum(wgrad_ms) * 1e-3) / 1e12
    # the dominant kernel by itself (events recorded by the library around that launch), else the call
    kern_ms = [v / n_ev for v in kern_acc] if kern_acc is not None else None
    kern_tflops = sum(flops) / (sum(kern_ms) * 1e-3) / 1e12 if kern_ms else wg_tflops
    comp_gbs = sum(comp_bytes) / (sum(comp_ms) * 1e-3) / 1e9
    tensor_peak = peaks["bf16_tflops"]

    # ---- end to end: host buffers in, dW out, through the C ABI ----------------
    e2e = None
    pinned = []
    for (name, d), (x, dy) in zip(layers, host):
        pinned.append(dict(
            x=x.pin_memory(), dy=dy.pin_memory(),
            dw=torch.empty(d.dw_shape, dtype=torch.float32).pin_memory(),
            arena=torch.empty(ac.ac_host_step_arena_bytes(d), dtype=torch.uint8, device=dev)))
    h2d = sum(p["x"].numel() * 2 + p["dy"].numel() * 2 for p in pinned)
    d2h = sum(p["dw"].numel() * 4 for p in pinned)

    def e2e_step():
        # every layer's call on a stream of its own (the layers are independent and each has its own
        # arena), so that one layer's device->host copy of dW runs while the next layer's inputs are
        # still coming in: PCIe carries both directions at once
        for s_, ((name, d), p) in zip(side, zip(layers, pinned)):
            s_.wait_stream(stream)
            ac.ac_backward_step_host(d, p["x"], p["dy"], p["dw"], None, p["arena"], stream=s_)
        for s_ in side:
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

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "impl": "ours",
        "config": {"workload": WORKLOAD, "layers": [n for n, _ in layers], "k": K_POOL,
                   "layout": LAYOUT, "batch": 64,
                   "l2": f"inputs rotated over {N_SETS} buffer sets "
                         f"({N_SETS * set_bytes / 1e6:.0f} MB in total, L2 is 126 MB)",
                   "multi_gpu": "independent replicas, no collective",
                   "layers_in_graph": "serial" if args.serial_layers else "one stream per layer (independent layers overlap)",
                   "timing": "value: K steps replayed as CUDA graphs (one per buffer set); "
                             "per-kernel figures: a second pass of min(K,200) steps, layers back to back, "
                             "CUDA events around each C-ABI call and, through the library's profiling hook, "
                             "around the weight-gradient kernel alone (" + per_kernel_mode + ")"},
        "wgrad_tflops": wg_tflops, "compress_gbs": comp_gbs,
        "compress_frac_of_hbm_peak": comp_gbs / peaks["hbm_gbs"],
        "saved_activation_bytes": {"x": x_bytes, "z": z_bytes, "saved": x_bytes - z_bytes,
                                   "reduction": 1 - z_bytes / x_bytes},
        "per_layer": [{"layer": n, "wgrad_ms": wgrad_ms[i], "wgrad_tflops": flops[i] / wgrad_ms[i] / 1e9,
                       "wgrad_kernel_ms": kern_ms[i] if kern_ms else None,
                       "compress_ms": comp_ms[i], "compress_gbs": comp_bytes[i] / comp_ms[i] / 1e6}
                      for i, (n, _) in enumerate(layers)],
        "roofline": {"bound": "tensor",
                     "kernel": "wgrad_tc2_kernel" if kern_ms else "ac_conv2d_wgrad_compressed (kernel + split-K reduce)",
                     "achieved": kern_tflops, "peak": tensor_peak, "unit": "TFLOP/s",
                     "frac": kern_tflops / tensor_peak, "peak_source": peaks["source"] + " burst bf16",
                     "call_level": {"achieved": wg_tflops, "frac": wg_tflops / tensor_peak,
                                    "note": "whole C-ABI call: the kernel, the split-K reduce kernel and the gap between"},
                     "traffic": WGRAD_DRAM_TRAFFIC_PER_STEP,
                     "traffic_unit": "bytes per step (4 launches), ncu",
                     "algorithmic_bytes": sum((d.N * d.C_in * d.Hp * d.Wp + d.N * d.C_out * d.Ho * d.Wo) * 2
                                              + d.C_out * d.C_in * d.R * d.S * 4 for _, d in layers),
                     "step_level": {"achieved": value / world, "frac": value / world / tensor_peak,
                                    "note": "whole step incl. compress, layers overlapped in the graph"}},
        "e2e": e2e,
        "gpu_launches": args.steps * len(layers) * 3,
        "clocks": clocks,
    }
    out["cpu_baseline"] = cpu_baseline(layers, host)
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def cpu_baseline(layers, host, n_frac=1.0):
    """The CPU checker, as it stands, on the same inputs: pooling + compressed dW
    for every layer of the step."""
    import oracle
    from paper_2409_11902_b200 import synth
    t_total, fl = 0.0, 0
    for (name, d), (x, dy) in zip(layers, host):
        n = max(1, int(round(d.N * n_frac)))
        x64 = synth.to_f64(synth.from_layout(x[:n], d.layout))
        dy64 = synth.to_f64(synth.from_layout(dy[:n], d.layout))
        t = time.perf_counter()
        z = oracle.pool(x64, d.k)
        oracle.wgrad_compressed(z, dy64, d.H, d.W, d.R, d.S, d.stride, d.pad, d.k)
        t_total += time.perf_counter() - t
        fl += d.flops * n // d.N
    return {"value": fl / t_total / 1e12, "unit": UNIT, "cores": oracle.num_threads(),
            "kind": "oracle", "seconds": t_total,
            "sample": f"{'whole step' if n_frac >= 1 else f'first {n_frac:.3f} of each batch'}: "
                      f"fp64 pooling + compressed dW of all {len(layers)} layers"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import __graft_entry__ as entry
    import oracle
    oracle.build()
    layers = descs()
    host = [host_inputs(d, seed=li) for li, (_, d) in enumerate(layers)]
    frac = 0.25   # a quarter of each batch per step keeps the whole run within minutes
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
                   "layout": "nchw", "batch": 64},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": res["cores"], "kind": "oracle",
                         "sample": res["sample"]},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--serial-layers", action="store_true",
                    help="capture the layers of a step back to back on one stream instead of one stream each")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        args.warmup = max(args.warmup, 3)
        run_ours(args)


if __name__ == "__main__":
    main()
