"""One ResNet-50 training step whose convolutions keep compressed inputs for backward, and the
peak device memory of that step with and without compression.

Section 4 of the paper: a convolution computes its output from the full input X, then keeps only
the k x k average-pooled Z for the backward pass, where the weight gradient is formed from Z and
the output gradient; input and bias gradients do not need X. Section 3 reads the memory of a
training step at five points: after model initialisation (1), after the input batch is allocated
(2), at the end of the forward pass (3), after the backward pass (4) and during the optimizer step
(5). This module runs exactly that on synthetic data:

  * every convolution is an autograd function whose forward is the framework's convolution followed
    by `ac_compress`, and whose backward is the framework's input gradient plus
    `ac_conv2d_wgrad_compressed` on the stored Z (scheme "compressed");
  * a ReLU in front of a compressed convolution would still keep its output -- the very tensor the
    convolution no longer stores -- for its own backward; scheme "compressed+mask" replaces it by
    `ac_compress_relu_mask`, which leaves Z and one bit per element (all a ReLU's backward needs);
  * scheme "full" is the ordinary network: framework convolutions that keep X.

Only the two `ac_*` calls are this library's kernels; convolution forward, input gradient, batch
norm, pooling, the classifier, the loss and the optimizer are the framework's. bf16 activations in
channels-last memory, fp32 master weights, SGD with momentum. No dataset: images ~ N(0,1), labels
uniform over 1000 classes, weights randomly initialised.
"""
from __future__ import annotations

import math

import torch
import torch.nn.functional as F

from . import api

SCHEMES = ("full", "compressed", "compressed+mask")
# (blocks, bottleneck width, stride of the stage's first block)
RESNET50_STAGES = [(3, 64, 1), (4, 128, 2), (6, 256, 2), (3, 512, 2)]


class Saved:
    """What is kept of one activation tensor for the backward pass of the convolutions that read
    it: the pooled copy Z (made once, however many convolutions read the tensor)."""

    def __init__(self):
        self.z = None


def _desc(x, w, stride, pad, k):
    N, Ci, H, W = x.shape
    Co, _, R, S = w.shape
    return api.ConvDesc(N, Ci, Co, H, W, R, S, (stride, stride), (pad, pad), k, "bf16", "nhwc")


def _nhwc(t):
    """The tensor's elements as a dense [N][H][W][C] buffer (what channels-last memory is)."""
    return t if t.is_contiguous(memory_format=torch.channels_last) else t.contiguous(memory_format=torch.channels_last)


class CompressedConv(torch.autograd.Function):
    """y = conv(x, w). Keeps Z = pool_k(x) instead of x; dW comes from Z and dY."""

    @staticmethod
    def forward(ctx, x, w_master, saved, stride, pad, k, capture):
        x = _nhwc(x)
        w = w_master.to(torch.bfloat16).contiguous(memory_format=torch.channels_last)
        y = F.conv2d(x, w, None, stride, pad)
        d = _desc(x, w, stride, pad, k)
        if saved.z is None:
            saved.z = torch.empty((d.N, d.C_in, d.Hp, d.Wp), dtype=torch.bfloat16, device=x.device,
                                  memory_format=torch.channels_last)
            api.ac_compress(d, x, saved.z)
        ctx.z, ctx.d, ctx.stride, ctx.pad, ctx.capture = saved.z, d, stride, pad, capture
        ctx.x_copy = x.detach().clone() if capture is not None else None   # checks only
        ctx.x_shape = x.shape
        ctx.save_for_backward(w_master)
        return y

    @staticmethod
    def backward(ctx, dy):
        (w_master,) = ctx.saved_tensors
        d = ctx.d
        dy = _nhwc(dy)
        dx = None
        if ctx.needs_input_grad[0]:
            w = w_master.to(torch.bfloat16).contiguous(memory_format=torch.channels_last)
            # the input gradient is the transposed convolution of dY (the framework's own kernel for it; the
            # generic conv2d_input helper would first materialise a dummy input of X's size)
            H, W = ctx.x_shape[2], ctx.x_shape[3]
            R, S = w.shape[2], w.shape[3]
            op = (H - ((dy.shape[2] - 1) * ctx.stride - 2 * ctx.pad + R), W - ((dy.shape[3] - 1) * ctx.stride - 2 * ctx.pad + S))
            dx = F.conv_transpose2d(dy, w, None, ctx.stride, ctx.pad, op)
        dw = torch.empty((d.C_out, d.R, d.S, d.C_in), dtype=torch.float32, device=dy.device)
        ws = torch.empty(max(api.ac_workspace_bytes(d), 256), dtype=torch.uint8, device=dy.device)
        api.ac_conv2d_wgrad_compressed(d, ctx.z, dy, dw, ws)
        if ctx.capture is not None:
            ctx.capture.append((d, ctx.x_copy, ctx.z.detach().clone(), dy.detach().clone(), dw.clone()))
        ctx.z = None
        return dx, dw.permute(0, 3, 1, 2), None, None, None, None, None


class ReluKeepingMask(torch.autograd.Function):
    """y = max(a, 0) in place. Keeps one bit per element, and leaves Z = pool_k(y) in `saved`
    for the convolutions that read y (`ac_compress_relu_mask_y`); backward: `ac_relu_mask_backward`."""

    @staticmethod
    def forward(ctx, a, saved, k):
        a = _nhwc(a)
        N, C, H, W = a.shape
        d = api.ConvDesc(N, C, C, H, W, 1, 1, (1, 1), (0, 0), k, "bf16", "nhwc")
        saved.z = torch.empty((N, C, d.Hp, d.Wp), dtype=torch.bfloat16, device=a.device,
                              memory_format=torch.channels_last)
        mask = torch.empty((a.numel() + 7) // 8, dtype=torch.uint8, device=a.device)
        api.ac_compress_relu_mask_y(d, a, a, saved.z, mask)      # the ReLU in place, Z and the mask: one pass over A
        ctx.mask = mask
        ctx.mark_dirty(a)
        return a

    @staticmethod
    def backward(ctx, dy):
        dy = _nhwc(dy)
        N, C, H, W = dy.shape
        d = api.ConvDesc(N, C, C, H, W, 1, 1, (1, 1), (0, 0), 1, "bf16", "nhwc")
        dx = torch.empty_like(dy)      # channels-last, like dy
        api.ac_relu_mask_backward(d, ctx.mask, dy, dx)
        ctx.mask = None
        return dx, None, None


class ResNet50:
    """ResNet-50 (bottleneck blocks, stride on the 3x3) as plain parameter lists; `scheme` chooses
    what the convolutions and ReLUs keep for backward."""

    def __init__(self, scheme, k=2, device="cuda", seed=0, compress_stem=True, num_classes=1000):
        assert scheme in SCHEMES
        self.scheme, self.k, self.compress_stem = scheme, k, compress_stem
        self.capture = None
        g = torch.Generator(device="cpu").manual_seed(seed)
        self.params = []

        def conv_w(co, ci, r):
            w = torch.randn((co, ci, r, r), generator=g) * math.sqrt(2.0 / (ci * r * r))
            p = w.to(device).requires_grad_(True)
            self.params.append(p)
            return p

        def bn(c):
            wgt = torch.ones(c, device=device, requires_grad=True)
            b = torch.zeros(c, device=device, requires_grad=True)
            self.params += [wgt, b]
            return dict(w=wgt, b=b, mean=torch.zeros(c, device=device), var=torch.ones(c, device=device))

        self.stem_w, self.stem_bn = conv_w(64, 3, 7), bn(64)
        self.blocks = []
        cin = 64
        for nblocks, width, stride in RESNET50_STAGES:
            for b in range(nblocks):
                s = stride if b == 0 else 1
                blk = dict(stride=s,
                           w1=conv_w(width, cin, 1), bn1=bn(width),
                           w2=conv_w(width, width, 3), bn2=bn(width),
                           w3=conv_w(4 * width, width, 1), bn3=bn(4 * width))
                if b == 0:
                    blk["wd"], blk["bnd"] = conv_w(4 * width, cin, 1), bn(4 * width)
                self.blocks.append(blk)
                cin = 4 * width
        self.fc_w = (torch.randn((num_classes, cin), generator=g) / math.sqrt(cin)).to(device).requires_grad_(True)
        self.fc_b = torch.zeros(num_classes, device=device, requires_grad=True)
        self.params += [self.fc_w, self.fc_b]

    # -- pieces ---------------------------------------------------------------
    def conv(self, x, w, stride, pad, saved, compress=True):
        if self.scheme == "full" or not compress:
            return F.conv2d(x, w.to(torch.bfloat16), None, stride, pad)
        return CompressedConv.apply(x, w, saved, stride, pad, self.k, self.capture)

    def relu(self, a):
        """Returns (y, what the convolutions reading y keep)."""
        saved = Saved()
        if self.scheme == "compressed+mask":
            return ReluKeepingMask.apply(a, saved, self.k), saved
        return F.relu(a, inplace=True), saved

    @staticmethod
    def bn(x, p):
        return F.batch_norm(x, p["mean"], p["var"], p["w"], p["b"], True, 0.1, 1e-5)

    def forward(self, images):
        x = self.conv(images, self.stem_w, 2, 3, Saved(), compress=self.compress_stem)
        x = F.relu(self.bn(x, self.stem_bn), inplace=True)   # feeds the max pooling, which keeps it anyway
        x = F.max_pool2d(x, 3, 2, 1)
        saved = Saved()                                  # the pooled map is not a ReLU's output
        for blk in self.blocks:
            s = blk["stride"]
            a, sa = self.relu(self.bn(self.conv(x, blk["w1"], 1, 0, saved), blk["bn1"]))
            b, sb = self.relu(self.bn(self.conv(a, blk["w2"], s, 1, sa), blk["bn2"]))
            c = self.bn(self.conv(b, blk["w3"], 1, 0, sb), blk["bn3"])
            idn = x
            if "wd" in blk:   # reads the same tensor as conv1: one Z for both
                idn = self.bn(self.conv(x, blk["wd"], s, 0, saved), blk["bnd"])
            x, saved = self.relu(c + idn)
        x = F.adaptive_avg_pool2d(x, 1).flatten(1)
        return F.linear(x, self.fc_w.to(torch.bfloat16), self.fc_b.to(torch.bfloat16))


def synthetic_batch(batch, device, seed=0, num_classes=1000):
    g = torch.Generator(device="cpu").manual_seed(seed + 1)
    images = torch.randn((batch, 3, 224, 224), generator=g).to(torch.bfloat16)
    labels = torch.randint(0, num_classes, (batch,), generator=g)
    return images.to(device).contiguous(memory_format=torch.channels_last), labels.to(device)


def training_step(scheme, batch=256, k=2, device="cuda", seed=0, compress_stem=True, capture=None, time_steps=0):
    """Runs one step and reads the allocator at Section 3's five points. Returns a dict with the
    loss and the bytes; `capture`: a list that receives (desc, X, Z, dY, dW) of every compressed
    convolution's backward (for checks; X is then copied in the forward pass, so the memory figures of such
    a run mean nothing)."""
    dev = torch.device(device)
    torch.cuda.synchronize(dev)
    torch.cuda.empty_cache()
    base = torch.cuda.memory_allocated(dev)
    torch.cuda.reset_peak_memory_stats(dev)
    mib = lambda b: (b - base) / 2.0 ** 20
    model = ResNet50(scheme, k, dev, seed, compress_stem)
    model.capture = capture
    opt = torch.optim.SGD(model.params, lr=0.1, momentum=0.9)
    p1 = torch.cuda.memory_allocated(dev)
    images, labels = synthetic_batch(batch, dev, seed)
    p2 = torch.cuda.memory_allocated(dev)
    logits = model.forward(images)
    loss = F.cross_entropy(logits.float(), labels)
    torch.cuda.synchronize(dev)
    p3, p3_peak = torch.cuda.memory_allocated(dev), torch.cuda.max_memory_allocated(dev)
    torch.cuda.reset_peak_memory_stats(dev)
    loss.backward()
    torch.cuda.synchronize(dev)
    p4, p4_peak = torch.cuda.memory_allocated(dev), torch.cuda.max_memory_allocated(dev)
    torch.cuda.reset_peak_memory_stats(dev)
    opt.step()
    torch.cuda.synchronize(dev)
    p5_peak = torch.cuda.max_memory_allocated(dev)
    out = {"scheme": scheme, "loss": float(loss.detach()),
           "mib": {"1_model": mib(p1), "2_input": mib(p2), "3_forward_end": mib(p3),
                   "3_forward_peak": mib(p3_peak), "backward_peak": mib(p4_peak),
                   "4_backward_end": mib(p4), "5_optimizer_peak": mib(p5_peak)}}
    out["mib"]["step_peak"] = max(out["mib"]["3_forward_peak"], out["mib"]["backward_peak"],
                                  out["mib"]["5_optimizer_peak"])
    out["grad_norm"] = float(torch.sqrt(sum((p.grad.double() ** 2).sum() for p in model.params if p.grad is not None)))
    if time_steps > 0 and capture is None:
        # duration of further whole steps (forward, backward, optimizer), CUDA events on the current stream
        del logits, loss
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(time_steps):
            opt.zero_grad(set_to_none=True)
            lg = model.forward(images)
            ls = F.cross_entropy(lg.float(), labels)
            ls.backward()
            opt.step()
            del lg, ls
        e1.record()
        torch.cuda.synchronize(dev)
        out["step_ms"] = e0.elapsed_time(e1) / time_steps
        logits = loss = None
    del model, opt, images, labels, logits, loss
    torch.cuda.empty_cache()
    return out


def peak_memory_report(batch=256, k=2, device="cuda", compress_stem=True, time_steps=0):
    """The step under each scheme, and the reduction of the peak against scheme "full"."""
    runs = {s: training_step(s, batch, k, device, compress_stem=compress_stem, time_steps=time_steps) for s in SCHEMES}
    full = runs["full"]["mib"]
    rep = {"model": "ResNet-50 (53 convolutions), bf16 channels-last, fp32 master weights, SGD momentum",
           "batch": batch, "k": k, "compress_stem": compress_stem,
           "points": "Section 3: 1 model, 2 input, 3 forward, 4 after backward, 5 optimizer; MiB above what was "
                     "allocated before the model (torch.cuda.memory_allocated / max_memory_allocated)",
           "schemes": runs}
    for s in SCHEMES[1:]:
        m = runs[s]["mib"]
        rep[f"reduction_{s}"] = {
            "forward_end": 1.0 - m["3_forward_end"] / full["3_forward_end"],
            "step_peak": 1.0 - m["step_peak"] / full["step_peak"],
            "activation_state": 1.0 - (m["3_forward_end"] - m["2_input"]) / (full["3_forward_end"] - full["2_input"])}
    return rep


if __name__ == "__main__":
    import argparse
    import json
    ap = argparse.ArgumentParser()
    ap.add_argument("--batch", type=int, default=256)
    ap.add_argument("--k", type=int, default=2)
    ap.add_argument("--no-stem", action="store_true", help="leave the first convolution uncompressed")
    ap.add_argument("--time-steps", type=int, default=0, help="also time this many further steps per scheme (step_ms)")
    a = ap.parse_args()
    print(json.dumps(peak_memory_report(a.batch, a.k, "cuda:0", not a.no_stem, a.time_steps), indent=1))
