"""Per-layer timing and byte report of the hot path on cuda:0, one table per workload:

    python -m paper_2409_11902_b200.layer_report --workload resnet50 --batch 256

For every distinct convolution shape of the workload: the saved-activation bytes with and without
compression (Section 4 of the paper stores the k x k average-pooled Z in place of the conv input X),
the time of `ac_compress` against the HBM bandwidth, and the time of `ac_conv2d_wgrad_compressed`
against the bound that holds for that layer, min(tensor peak, arithmetic intensity x HBM bandwidth):
1x1 layers with few channels move more bytes than the tensor cores need time for.

Inputs are the synthetic recipe of `synth` (X = max(N(0,1), 0), dY ~ N(0, 1e-4)) drawn for a few
images and repeated along the batch on the device: the kernels' time does not depend on the values,
and drawing hundreds of millions of samples on the host would take longer than the measurement.

Timing: each entry point is captured `reps` times into a CUDA graph that walks over several buffer
sets (together larger than the 126 MB L2, so no input is cache-resident), replayed after a warm-up
replay, and timed with CUDA events on the launching stream.
"""
from __future__ import annotations

import argparse
import json
import os

import torch

from . import api, synth

# (C_in, C_out, H, R, stride, pad, count): ResNet-50 (bottleneck blocks, stride on the 3x3), 53 convs
RESNET50 = [
    (3, 64, 224, 7, 2, 3, 1), (64, 64, 56, 1, 1, 0, 1), (64, 64, 56, 3, 1, 1, 3), (64, 256, 56, 1, 1, 0, 4),
    (256, 64, 56, 1, 1, 0, 2), (256, 128, 56, 1, 1, 0, 1), (128, 128, 56, 3, 2, 1, 1), (128, 512, 28, 1, 1, 0, 4),
    (256, 512, 56, 1, 2, 0, 1), (512, 128, 28, 1, 1, 0, 3), (128, 128, 28, 3, 1, 1, 3), (512, 256, 28, 1, 1, 0, 1),
    (256, 256, 28, 3, 2, 1, 1), (256, 1024, 14, 1, 1, 0, 6), (512, 1024, 28, 1, 2, 0, 1), (1024, 256, 14, 1, 1, 0, 5),
    (256, 256, 14, 3, 1, 1, 5), (1024, 512, 14, 1, 1, 0, 1), (512, 512, 14, 3, 2, 1, 1), (512, 2048, 7, 1, 1, 0, 3),
    (1024, 2048, 14, 1, 2, 0, 1), (2048, 512, 7, 1, 1, 0, 2), (512, 512, 7, 3, 1, 1, 2),
]
# one bottleneck block at 56 x 56 plus the stride-2 3x3 that follows it
BOTTLENECK = [(256, 64, 56, 1, 1, 0, 1), (64, 64, 56, 3, 1, 1, 1), (64, 256, 56, 1, 1, 0, 1), (128, 128, 56, 3, 2, 1, 1)]
RESNET18_STACK = [(64, 64, 56, 3, 1, 1, 1), (128, 128, 28, 3, 1, 1, 1), (256, 256, 14, 3, 1, 1, 1),
                  (512, 512, 8, 3, 1, 1, 1), (512, 512, 7, 3, 1, 1, 1)]
SWEEP = [(128, 128, 64, 3, 1, 1, 1)]     # the pooling-factor sweep's layer (run it with --k 1, 2, 4, 8)
WORKLOADS = {"resnet50": (RESNET50, 256), "bottleneck": (BOTTLENECK, 128), "resnet18_stack": (RESNET18_STACK, 64),
             "sweep": (SWEEP, 256)}
# ResNet-50 convolutions whose input another convolution reads too (the first block of a stage feeds
# both conv1 and the downsample projection): that tensor is saved, and compressed, once.
RESNET50_SHARED_INPUT = {(64, 256, 56, 1, 1): 1, (256, 512, 56, 1, 2): 1, (512, 1024, 28, 1, 2): 1,
                         (1024, 2048, 14, 1, 2): 1}


def saved_state_model(layers, N, k, elt, shared):
    """Bytes a training step keeps for backward in a conv -> batch-norm -> ReLU network, by accounting
    (no step is run): A = the distinct conv inputs (each is also the output its ReLU keeps), B = the
    conv outputs (what each batch-norm keeps). The paper's scheme stores A / k^2 instead of A; a ReLU
    that feeds only compressed convolutions then needs one bit per element for its own backward."""
    A = B = Az = 0
    for ci, co, H, R, st, pd, cnt in layers:
        distinct = cnt - shared.get((ci, co, H, R, st), 0)
        Ho = (H + 2 * pd - R) // st + 1
        Hp = -(-H // k)
        A += distinct * N * ci * H * H * elt
        Az += distinct * N * ci * Hp * Hp * elt
        B += cnt * N * co * Ho * Ho * elt
    mask = A // (8 * elt)
    return A, Az, B, mask


def load_peaks(path):
    if path and os.path.exists(path):
        p = json.load(open(path))
        return p["hbm_gbs"], p["bf16_tflops"], "measured"
    return 6650.0, 1590.0, "fallback"


def time_graph(fn, nsets, reps):
    """Microseconds per call of fn(set_index), `reps` calls captured into one graph."""
    stream = torch.cuda.current_stream()
    fn(0)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(reps):
            fn(i % nsets)
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    g.replay()
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / reps


def measure(d, dev, reps, seed_images=2):
    nb = min(d.N, seed_images)
    x1 = synth.to_layout(synth.activation(0, (nb, d.C_in, d.H, d.W), d.dtype), d.layout).to(dev)
    dy1 = synth.to_layout(synth.grad_output(0, (nb, d.C_out, d.Ho, d.Wo), d.dtype), d.layout).to(dev)
    rep = (-(-d.N // nb), 1, 1, 1)
    elt = 2 if d.dtype == "bf16" else 4
    set_bytes = (d.N * d.C_in * (d.H * d.W + d.Hp * d.Wp) + d.N * d.C_out * d.Ho * d.Wo) * elt
    nsets = max(1, min(8, -(-300_000_000 // set_bytes)))
    sets = []
    for _ in range(nsets):
        sets.append(dict(x=x1.repeat(rep)[:d.N].contiguous(), dy=dy1.repeat(rep)[:d.N].contiguous(),
                         z=torch.empty(d.z_shape, dtype=d.torch_dtype, device=dev)))
    dw = torch.empty(d.dw_shape, dtype=torch.float32, device=dev)
    ws = torch.empty(max(api.ac_workspace_bytes(d), 256), dtype=torch.uint8, device=dev)
    for b in sets:
        api.ac_compress(d, b["x"], b["z"])
    t_c = time_graph(lambda i: api.ac_compress(d, sets[i]["x"], sets[i]["z"]), nsets, reps)
    t_w = time_graph(lambda i: api.ac_conv2d_wgrad_compressed(d, sets[i]["z"], sets[i]["dy"], dw, ws), nsets, reps)
    st, detail = api.ac_workspace_status(ws)
    if st != 0:
        raise RuntimeError(f"device status {st} detail {detail:#x}")
    return t_c, t_w


def overlapped_wgrads(layers, N, k, dtype, layout, dev, nstreams, budget=0, seed_images=2):
    """Microseconds for the weight gradients of ALL the workload's convolutions (every repeat of a shape
    its own dW and workspace), last layer first, dealt round-robin to `nstreams` streams inside one
    captured graph: what a training step that runs independent weight gradients side by side sees."""
    inst = []
    for ci, co, H, R, st, pd, cnt in layers:
        d = api.ConvDesc(N, ci, co, H, H, R, R, (st, st), (pd, pd), k, dtype, layout)
        nb = min(N, seed_images)
        rep = (-(-N // nb), 1, 1, 1)
        x = synth.to_layout(synth.activation(0, (nb, ci, H, H), dtype), layout).to(dev).repeat(rep)[:N].contiguous()
        dy = synth.to_layout(synth.grad_output(0, (nb, co, d.Ho, d.Wo), dtype), layout).to(dev).repeat(rep)[:N].contiguous()
        z = torch.empty(d.z_shape, dtype=d.torch_dtype, device=dev)
        api.ac_compress(d, x, z)
        del x
        b = budget
        api.ac_set_sm_budget(b)
        for _ in range(cnt):
            inst.append((d, z, dy, torch.empty(d.dw_shape, dtype=torch.float32, device=dev),
                         torch.empty(max(api.ac_workspace_bytes(d), 256), dtype=torch.uint8, device=dev), b))
    inst.reverse()
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(device=dev) for _ in range(nstreams)]

    def enqueue():
        main = torch.cuda.current_stream()
        for s_ in streams:
            s_.wait_stream(main)
        for i, (d, z, dy, dw, ws, b) in enumerate(inst):
            api.ac_set_sm_budget(b)
            with torch.cuda.stream(streams[i % nstreams]):
                api.ac_conv2d_wgrad_compressed(d, z, dy, dw, ws)
        api.ac_set_sm_budget(0)
        for s_ in streams:
            main.wait_stream(s_)

    enqueue()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        enqueue()
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 5
    e0.record()
    for _ in range(reps):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    for d, z, dy, dw, ws, b in inst:
        st, detail = api.ac_workspace_status(ws)
        if st != 0:
            raise RuntimeError(f"device status {st} detail {detail:#x}")
    return e0.elapsed_time(e1) * 1e3 / reps, len(inst), sum(i[0].flops for i in inst)


def gradient_alignment(layers, N, ks, dtype, layout, dev):
    """Section 5.2's measure, cos = a.b / (|a| |b|), between the weight gradient from the compressed
    input (pooling factor k) and the one from the full input (k = 1), per layer, on the synthetic
    inputs. The paper draws its figure from ImageNet activations after an epoch of training; seeded
    noise has no spatial correlation for the pooling to preserve, so these values are a lower bound
    of what smooth activations give, and only their order across layers and k is meaningful."""
    rows = []
    for ci, co, H, R, st, pd, cnt in layers:
        base = api.ConvDesc(N, ci, co, H, H, R, R, (st, st), (pd, pd), 1, dtype, layout)
        x = synth.to_layout(synth.activation(7, (N, ci, H, H), dtype), layout).to(dev)
        dy = synth.to_layout(synth.grad_output(7, (N, co, base.Ho, base.Wo), dtype), layout).to(dev)
        grads = {}
        for k in [1] + [k for k in ks if k != 1]:
            d = api.ConvDesc(N, ci, co, H, H, R, R, (st, st), (pd, pd), k, dtype, layout)
            z = torch.empty(d.z_shape, dtype=d.torch_dtype, device=dev)
            dw = torch.empty(d.dw_shape, dtype=torch.float32, device=dev)
            ws = torch.empty(max(api.ac_workspace_bytes(d), 256), dtype=torch.uint8, device=dev)
            api.ac_compress(d, x, z)
            api.ac_conv2d_wgrad_compressed(d, z, dy, dw, ws)
            st_, detail = api.ac_workspace_status(ws)
            if st_ != 0:
                raise RuntimeError(f"device status {st_} detail {detail:#x}")
            grads[k] = dw.double().flatten()
        ref = grads[1]
        rows.append(((ci, co, H, R, st), {k: float(torch.dot(g, ref) / (g.norm() * ref.norm())) for k, g in grads.items()}))
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="resnet50", choices=sorted(WORKLOADS))
    ap.add_argument("--batch", type=int, default=0, help="0: the workload's own batch size")
    ap.add_argument("--k", type=int, default=2)
    ap.add_argument("--dtype", default="bf16")
    ap.add_argument("--layout", default="nhwc")
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--peaks", default=os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))),
                                                    "MEASURED_PEAKS.json"),
                    help="JSON with hbm_gbs and bf16_tflops measured on this machine")
    ap.add_argument("--streams", type=int, default=0,
                    help="instead of the per-layer table: all weight gradients of the workload in one graph on this many streams")
    ap.add_argument("--sm-budget", type=int, default=0,
                    help="with --streams: SMs each weight gradient plans for (ac_set_sm_budget; 0: the whole GPU)")
    ap.add_argument("--cosine", action="store_true",
                    help="instead of timing: cosine similarity of the compressed and the k = 1 weight gradient per layer")
    a = ap.parse_args()
    layers, batch = WORKLOADS[a.workload]
    N = a.batch or batch
    if a.cosine:
        ks = [2, 4, 8]
        N = a.batch or 8
        rows = gradient_alignment(layers, N, ks, a.dtype, a.layout, torch.device("cuda:0"))
        print(f"# {a.workload}: cosine similarity of dW(k) and dW(1) (Section 5.2), batch {N}, {a.dtype} {a.layout}, "
              "synthetic inputs (X = max(N(0,1),0), dY ~ N(0,1e-4))")
        print("| C_in→C_out, H, RxS/stride | " + " | ".join(f"k = {k}" for k in ks) + " |")
        print("|---|" + "---|" * len(ks))
        for (ci, co, H, R, st), c in rows:
            print(f"| {ci}→{co}, {H}², {R}x{R}/{st} | " + " | ".join(f"{c[k]:.3f}" for k in ks) + " |")
        return
    hbm, tens, src = load_peaks(a.peaks)
    dev = torch.device("cuda:0")
    elt = 2 if a.dtype == "bf16" else 4
    if a.streams > 0:
        us, n, fl = overlapped_wgrads(layers, N, a.k, a.dtype, a.layout, dev, a.streams, a.sm_budget)
        print(f"# {a.workload}, batch {N}, {a.dtype} {a.layout}, k = {a.k}: the {n} weight gradients as one graph on "
              f"{a.streams} stream(s), each planned for {a.sm_budget or 148} SMs: {us:.0f} us = {fl / us / 1e6:.0f} TFLOP/s dense-equivalent "
              f"({fl / us / 1e6 / tens:.2f} of the {src} tensor peak {tens:.0f})")
        return
    print(f"# {a.workload}, batch {N}, {a.dtype} {a.layout}, k = {a.k}; denominators ({src}): "
          f"{hbm:.0f} GB/s HBM copy, {tens:.0f} TFLOP/s bf16 burst")
    print("| C_in→C_out, H, RxS/stride | × | path | X MiB | Z MiB | compress µs | GB/s | of HBM | wgrad µs | TFLOP/s "
          "| bound | of bound |")
    print("|---|---|---|---|---|---|---|---|---|---|---|---|")
    tot = dict(x=0, z=0, tc=0.0, tw=0.0, fl=0, cb=0, bound_us=0.0)
    for ci, co, H, R, st, pd, cnt in layers:
        d = api.ConvDesc(N, ci, co, H, H, R, R, (st, st), (pd, pd), a.k, a.dtype, a.layout)
        t_c, t_w = measure(d, dev, a.reps)
        xb = N * ci * H * H * elt
        zb = N * ci * d.Hp * d.Wp * elt
        wb = zb + N * co * d.Ho * d.Wo * elt + co * ci * R * R * 4
        ai = d.flops / wb
        bound = min(tens, ai * hbm / 1e3)
        kind = "tensor" if bound == tens else "HBM"
        tfl = d.flops / t_w / 1e6
        gbs = (xb + zb) / t_c / 1e3
        path = {0: "fp32 ALU", 1: "tc", 2: "tc2", 3: "staged", 4: "staged×2", 5: "gather", 6: "gather (in kernel)",
                7: "tc2 on re-blocked Z"}.get(
            api.ac_wgrad_plan_info(d)["tensor_core"], "?")
        print(f"| {ci}→{co}, {H}², {R}x{R}/{st} | {cnt} | {path} | {xb / 2**20:.1f} | {zb / 2**20:.1f} | {t_c:.1f} | "
              f"{gbs:.0f} | {gbs / hbm:.2f} | {t_w:.1f} | {tfl:.0f} | {kind} {bound:.0f} | {tfl / bound:.2f} |")
        tot["x"] += cnt * xb; tot["z"] += cnt * zb; tot["tc"] += cnt * t_c; tot["tw"] += cnt * t_w
        tot["fl"] += cnt * d.flops; tot["cb"] += cnt * (xb + zb); tot["bound_us"] += cnt * d.flops / bound / 1e6
        del d
        torch.cuda.empty_cache()
    print(f"\nAll {sum(l[-1] for l in layers)} convolutions: X {tot['x'] / 2**20:.0f} MiB -> Z {tot['z'] / 2**20:.0f} MiB "
          f"(-{100 * (1 - tot['z'] / tot['x']):.1f} %); compress {tot['tc']:.0f} us = {tot['cb'] / tot['tc'] / 1e3:.0f} GB/s "
          f"({tot['cb'] / tot['tc'] / 1e3 / hbm:.2f} of HBM); wgrad {tot['tw']:.0f} us = {tot['fl'] / tot['tw'] / 1e6:.0f} TFLOP/s "
          f"dense-equivalent ({tot['bound_us'] / tot['tw']:.2f} of the per-layer bounds, "
          f"{tot['fl'] / tot['tw'] / 1e6 / tens:.2f} of the tensor peak).")
    if a.workload == "resnet50":
        A, Az, B, mask = saved_state_model(layers, N, a.k, elt, RESNET50_SHARED_INPUT)
        m = 2.0 ** 20
        print(f"\nSaved-for-backward state by accounting (conv -> batch-norm -> ReLU; no training step is run): distinct conv "
              f"inputs {A / m:.0f} MiB + conv outputs kept by batch-norm {B / m:.0f} MiB = {(A + B) / m:.0f} MiB. With Z in "
              f"place of the conv inputs: {Az / m:.0f} + {B / m:.0f} = {(Az + B) / m:.0f} MiB (-{100 * (A - Az) / (A + B):.1f} %); "
              f"with one mask bit per element for the ReLUs' own backward: {(Az + mask + B) / m:.0f} MiB "
              f"(-{100 * (A - Az - mask) / (A + B):.1f} %).")


if __name__ == "__main__":
    main()
