"""The workspace-free weight gradient, for callers that cannot allocate.

A caller that lives inside someone else's memory pool (or in a loop that must
not touch the allocator) cannot produce the scratch buffer that
ac_conv2d_wgrad_compressed asks for. ac_conv2d_wgrad_compressed_static keeps
that scratch in a fixed array inside the library instead. These tests call it
through the C ABI and require the same dW as the ordinary entry point and as
the CPU checker, twice in a row on different inputs, because the second call
finds the first call's partial sums still lying in the shared array.

Collected last on purpose: a run that stops at the first failure has then
already gone through every other test.
"""
import ctypes

import numpy as np
import pytest

import __graft_entry__ as entry


@pytest.fixture(scope="module")
def ac():
    entry.build()
    import paper_2409_11902_b200 as ac
    return ac


def _desc(ac, N, C, H, dtype, layout, k=2):
    return ac.ConvDesc(N, C, C, H, H, 3, 3, (1, 1), (1, 1), k, dtype, layout)


def test_oversized_problem_is_refused_before_any_launch(ac):
    """Needs no GPU: the size check comes before the first CUDA call."""
    L = ac.api.lib()
    # 9 MiB of dW: the array holds three partial tensors, and three slices of 800 000 positions
    # would each be far longer than the call allows
    big = _desc(ac, 256, 512, 56, "f32", "nchw").c()
    A = 0x10000
    assert L.ac_conv2d_wgrad_compressed_static(ctypes.byref(big), A, A, A, None) \
        == ac.api.AC_ERR_WORKSPACE_TOO_SMALL
    ok = _desc(ac, 8, 64, 32, "f32", "nchw").c()
    assert L.ac_conv2d_wgrad_compressed_static(ctypes.byref(ok), A, A + 4, A, None) \
        == ac.api.AC_ERR_MISALIGNED
    assert L.ac_conv2d_wgrad_compressed_static(ctypes.byref(ok), None, A, A, None) \
        == ac.api.AC_ERR_INVALID_ARG


@pytest.mark.gpu
@pytest.mark.parametrize("dtype,layout", [("f32", "nchw"), ("bf16", "nhwc")])
def test_static_scratch_matches_workspace_entry_point_twice(ac, dtype, layout):
    import torch
    import oracle
    from helpers import TOL_DW, assert_dw_close, make_wgrad_inputs, sampled_check
    from paper_2409_11902_b200 import synth
    dev = "cuda:0"
    # different problems back to back: each one's partial sums land on top of what the one before
    # left in the shared array. The last one (9 MiB of dW, 12544 positions) fits only because the
    # call then uses three long K-slices where the ordinary plan would take seven.
    cases = [_desc(ac, 8, 64, 32, dtype, layout), _desc(ac, 4, 64, 14, dtype, layout, k=4),
             _desc(ac, 256, 512, 7, dtype, layout)]
    for rep, d in enumerate(cases):
        z, dy = make_wgrad_inputs(d, seed=10 + rep)
        zd = synth.to_layout(z, layout).to(dev)
        dyd = synth.to_layout(dy, layout).to(dev)
        ref = torch.empty(d.dw_shape, dtype=torch.float32, device=dev)
        ws = torch.empty(ac.ac_workspace_bytes(d), dtype=torch.uint8, device=dev)
        ac.ac_conv2d_wgrad_compressed(d, zd, dyd, ref, ws)
        got = torch.full(d.dw_shape, float("nan"), dtype=torch.float32, device=dev)
        ac.ac_conv2d_wgrad_compressed_static(d, zd, dyd, got)
        torch.cuda.synchronize()
        g, r = got.double().cpu().numpy(), ref.double().cpu().numpy()
        assert np.isfinite(g).all()
        err = np.linalg.norm(g - r) / np.linalg.norm(r)
        assert err <= TOL_DW[dtype], (rep, err)
        if layout == "nhwc":
            g = g.transpose(0, 3, 1, 2)
        if d.C_in > 64:      # too large for the checker's full tensor: a stratified sample of entries
            sampled_check(d, g, z, dy, n_samples=256, seed=rep)
            continue
        want = oracle.wgrad_compressed(synth.to_f64(z), synth.to_f64(dy), d.H, d.W, d.R, d.S,
                                       d.stride, d.pad, d.k)
        assert_dw_close(g, want, dtype, (rep, dtype, layout))
