"""The ResNet-50 step with compressed convolution inputs (paper_2409_11902_b200.train_step), at a
reduced batch: the forward pass is untouched by the compression, the weight gradients of the step
equal the CPU checker's on the tensors the step really produced, and the memory the step holds at
the end of the forward pass (Section 3's third point) falls only when the ReLUs stop keeping their
outputs."""
import numpy as np
import pytest

import __graft_entry__ as entry
from helpers import assert_dw_close, stratified_entries

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    entry.build()


def test_weight_gradients_of_a_real_step_match_the_checker():
    import torch
    import oracle
    from paper_2409_11902_b200 import synth, train_step
    cap = []
    out = train_step.training_step("compressed+mask", batch=4, k=2, device="cuda:0", capture=cap)
    assert np.isfinite(out["loss"]) and len(cap) == 53
    # backward visits the layers last to first: the stem (3 channels, 7x7, stride 2), a 3x3 of the first
    # stage (64 channels on 56 x 56), a stride-2 3x3 and a 1x1 of the last stage (7 x 7 maps)
    picks = {}
    for d, x, z, dy, dw in cap:
        key = (d.C_in, d.C_out, d.H, d.R, d.stride[0])
        if key in ((3, 64, 224, 7, 2), (64, 64, 56, 3, 1), (512, 512, 14, 3, 2), (2048, 512, 7, 1, 1)):
            picks.setdefault(key, (d, x, z, dy, dw))
    assert len(picks) == 4
    for key, (d, x, z, dy, dw) in picks.items():
        x64 = synth.to_f64(x)                                      # logical NCHW values of the layer's input
        z_own = synth.to_storage(oracle.pool(x64, d.k), "bf16")   # the checker's own Z from the same X
        z_gpu = z.cpu()
        differ = (z_own != z_gpu)
        # one bf16 rounding of an fp32 sum against one of an fp64 sum: equal except at rounding ties
        assert int(differ.sum()) <= max(2, z_own.numel() // 1000), key
        assert float((z_own.double() - z_gpu.double()).abs().max()) <= 2.0 ** -7 * float(z_own.double().abs().max())
        idx = stratified_entries(d, 128, seed=7)
        want = oracle.wgrad_compressed_entries(synth.to_f64(z_own), synth.to_f64(dy), d.H, d.W, d.R, d.S,
                                               d.stride, d.pad, d.k, idx)
        got = dw.cpu().double().numpy().transpose(0, 3, 1, 2)
        assert_dw_close(got[idx[:, 0], idx[:, 1], idx[:, 2], idx[:, 3]], want, "bf16", key)
        # secondary cross-check (not the parity gate): the framework's own weight gradient of the
        # explicitly inflated Z, which is how the paper's experiments compute it
        xt = z.float().repeat_interleave(d.k, 2).repeat_interleave(d.k, 3)[:, :, :d.H, :d.W]
        fw = torch.nn.grad.conv2d_weight(xt, (d.C_out, d.C_in, d.R, d.S), dy.float(), d.stride, d.pad)
        g = dw.permute(0, 3, 1, 2)
        assert float((g - fw).norm() / fw.norm()) <= 1e-3, key


def test_forward_is_unchanged_and_memory_falls_only_with_the_masks():
    from paper_2409_11902_b200 import train_step
    rep = train_step.peak_memory_report(batch=8, k=2, device="cuda:0")
    runs = rep["schemes"]
    # Section 4: the forward pass uses the full input, so the loss is the same number in all schemes
    assert runs["full"]["loss"] == runs["compressed"]["loss"] == runs["compressed+mask"]["loss"]
    # ... and the gradients differ (the compressed ones are an approximation) but not wildly
    assert runs["compressed"]["grad_norm"] == pytest.approx(runs["compressed+mask"]["grad_norm"], rel=1e-3)
    assert 0.2 < runs["compressed"]["grad_norm"] / runs["full"]["grad_norm"] < 5.0
    f, c, m = (runs[s]["mib"]["3_forward_end"] for s in ("full", "compressed", "compressed+mask"))
    # a framework ReLU keeps its output, the tensor the convolution no longer stores: no saving
    assert c >= 0.93 * f
    # one bit per element instead: the conv inputs (about 45 % of what the step keeps) shrink to 1/4 + 1/16
    assert m <= 0.80 * f
    assert rep["reduction_compressed+mask"]["step_peak"] >= 0.15
    for s in runs.values():
        assert s["mib"]["1_model"] < s["mib"]["2_input"] < s["mib"]["3_forward_end"]
        assert s["mib"]["4_backward_end"] < s["mib"]["3_forward_end"]
