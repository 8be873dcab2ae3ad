"""Runs one layer of the hot path a few times on cuda:0: the small, bounded
workload that profiler captures (ncu) are taken on.

    python -m paper_2409_11902_b200.profile_case --layer 128ch_28x28 --batch 16 --iters 3
"""
from __future__ import annotations

import argparse

import torch

from . import api, synth

LAYERS = {
    # name: (C_in, C_out, H, W, R, S, stride, pad)
    "64ch_56x56": (64, 64, 56, 56, 3, 3, 1, 1),
    "128ch_28x28": (128, 128, 28, 28, 3, 3, 1, 1),
    "256ch_14x14": (256, 256, 14, 14, 3, 3, 1, 1),
    "512ch_8x8": (512, 512, 8, 8, 3, 3, 1, 1),
    "512ch_7x7": (512, 512, 7, 7, 3, 3, 1, 1),
    "2048to512_1x1_7x7": (2048, 512, 7, 7, 1, 1, 1, 0),
    "128ch_64x64": (128, 128, 64, 64, 3, 3, 1, 1),
    "128ch_56x56_s2": (128, 128, 56, 56, 3, 3, 2, 1),
    "256to64_1x1_56x56": (256, 64, 56, 56, 1, 1, 1, 0),
    "256to1024_1x1_14x14": (256, 1024, 14, 14, 1, 1, 1, 0),
    "1024to256_1x1_14x14": (1024, 256, 14, 14, 1, 1, 1, 0),
    "1024to2048_1x1_s2_14x14": (1024, 2048, 14, 14, 1, 1, 2, 0),
    "512to2048_1x1_7x7": (512, 2048, 7, 7, 1, 1, 1, 0),
    "3to64_7x7_s2_224x224": (3, 64, 224, 224, 7, 7, 2, 3),
}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--layer", default="128ch_28x28", choices=sorted(LAYERS))
    ap.add_argument("--batch", type=int, default=16)
    ap.add_argument("--k", type=int, default=2)
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--dtype", default="bf16")
    ap.add_argument("--layout", default="nhwc")
    ap.add_argument("--relu", action="store_true", help="use the fused ReLU+compress form")
    ap.add_argument("--mask", action="store_true", help="use the fused ReLU+compress form that keeps a sign mask")
    ap.add_argument("--relu-ops", action="store_true",
                    help="instead: the masked ReLU's two passes on the layer's input tensor, forward (ReLU in place + "
                         "compress + mask, ac_compress_relu_mask_y) and backward (ac_relu_mask_backward)")
    ap.add_argument("--collapsed", action="store_true", help="time the collapsed weight-gradient entry point too")
    a = ap.parse_args()
    ci, co, H, W, R, S, st, pd = LAYERS[a.layer]
    d = api.ConvDesc(a.batch, ci, co, H, W, R, S, (st, st), (pd, pd), a.k, a.dtype, a.layout)
    dev = torch.device("cuda:0")
    x = synth.to_layout(synth.activation(0, (d.N, ci, H, W), a.dtype), a.layout).to(dev)
    dy = synth.to_layout(synth.grad_output(0, (d.N, co, d.Ho, d.Wo), a.dtype), a.layout).to(dev)
    z = torch.empty(d.z_shape, dtype=d.torch_dtype, device=dev)
    y = torch.empty_like(x) if a.relu else None
    mask = torch.empty((x.numel() + 7) // 8, dtype=torch.uint8, device=dev) if a.mask else None
    if a.relu_ops:
        acts = [synth.to_layout(synth.pre_activation(i, (d.N, ci, H, W), a.dtype), a.layout).to(dev) for i in range(2)]
        gy = synth.to_layout(synth.grad_output(1, (d.N, ci, H, W), a.dtype), a.layout).to(dev)
        gx = torch.empty_like(gy)
        m = torch.empty((x.numel() + 7) // 8, dtype=torch.uint8, device=dev)
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        nbytes = x.numel() * x.element_size()
        for it in range(a.iters):
            act = acts[it % 2].clone()
            e[0].record()
            api.ac_compress_relu_mask_y(d, act, act, z, m)
            e[1].record()
            api.ac_relu_mask_backward(d, m, gy, gx)
            e[2].record()
            torch.cuda.synchronize()
            t_f, t_b = e[0].elapsed_time(e[1]), e[1].elapsed_time(e[2])
            fb = 2 * nbytes + z.numel() * z.element_size() + m.numel()
            bb = 2 * nbytes + m.numel()
            print(f"iter {it}: relu+compress+mask {t_f * 1e3:.1f} us ({fb / t_f / 1e6:.0f} GB/s), "
                  f"relu backward from the mask {t_b * 1e3:.1f} us ({bb / t_b / 1e6:.0f} GB/s)")
        return
    dw = torch.empty(d.dw_shape, dtype=torch.float32, device=dev)
    ws = torch.empty(max(api.ac_workspace_bytes(d), 256), dtype=torch.uint8, device=dev)
    print("plan:", api.ac_wgrad_plan_info(d))
    cbytes, tiles_c, tiles_d = api.ac_collapsed_workspace_bytes(d) if a.collapsed else (0, 0, 0)
    cws = torch.empty(max(cbytes, 256), dtype=torch.uint8, device=dev)
    dwc = torch.empty_like(dw)
    e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
    for it in range(a.iters):
        e0.record()
        if a.mask:
            api.ac_compress_relu_mask(d, x, z, mask)
        else:
            api.ac_compress(d, x, z, y)
        e1.record()
        api.ac_conv2d_wgrad_compressed(d, z, dy, dw, ws)
        e2.record()
        torch.cuda.synchronize()
        st_, detail = api.ac_workspace_status(ws)
        assert st_ == 0, (st_, detail)
        if cbytes:
            e1.record()
            api.ac_conv2d_wgrad_compressed_collapsed(d, z, dy, dwc, cws)
            e2.record()
            torch.cuda.synchronize()
            ms = e1.elapsed_time(e2)
            rel = float((dwc - dw).norm() / dw.norm())
            print(f"iter {it}: collapsed {ms * 1e3:.1f} us: {d.flops / ms / 1e9:.1f} TFLOP/s dense-equivalent, "
                  f"{d.flops * tiles_c / tiles_d / ms / 1e9:.1f} performed ({tiles_c}/{tiles_d} tiles), "
                  f"vs dense entry point {rel:.1e}")
            continue
        print(f"iter {it}: compress {e0.elapsed_time(e1) * 1e3:.1f} us, wgrad {e1.elapsed_time(e2) * 1e3:.1f} us "
              f"({d.flops / e1.elapsed_time(e2) / 1e9:.1f} TFLOP/s)")


if __name__ == "__main__":
    main()
