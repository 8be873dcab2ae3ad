"""GPU parity of ac_conv2d_wgrad_compressed against the CPU checker."""
import dataclasses

import numpy as np
import pytest

import __graft_entry__ as entry
from helpers import (TOL_DW, assert_dw_close, make_wgrad_inputs, run_wgrad, run_wgrad_collapsed,
                     sampled_check, wgrad_error_full, wgrad_error_sampled)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    entry.build()


def D(N, Ci, Co, H, W, R, S, stride, pad, k, dtype, layout):
    import paper_2409_11902_b200 as ac
    return ac.ConvDesc(N, Ci, Co, H, W, R, S, (stride, stride), (pad, pad), k, dtype, layout)


SMALL = [
    # N, Ci, Co, H, W, R, S, stride, pad, k
    (8, 64, 64, 32, 32, 3, 3, 1, 1, 2),     # config 1
    (2, 64, 64, 14, 14, 3, 3, 1, 1, 2),
    (2, 128, 64, 9, 11, 3, 3, 1, 1, 2),     # odd H, W: partial pooling blocks at the padding edge
    (2, 64, 128, 7, 7, 3, 3, 1, 1, 2),
    (2, 64, 64, 16, 16, 3, 3, 2, 1, 2),     # stride 2 (taps collapse)
    (2, 64, 64, 15, 15, 3, 3, 2, 1, 2),
    (3, 128, 64, 12, 12, 1, 1, 1, 0, 2),    # pointwise
    (3, 64, 128, 12, 12, 1, 1, 2, 0, 2),    # pointwise, stride 2
    (2, 64, 64, 16, 16, 3, 3, 1, 1, 1),     # k = 1: uncompressed
    (2, 64, 64, 16, 16, 3, 3, 1, 1, 4),
    (2, 64, 64, 16, 16, 3, 3, 1, 1, 8),
    (2, 64, 64, 13, 13, 3, 3, 1, 1, 3),     # k that divides nothing
    (1, 3, 16, 20, 20, 7, 7, 2, 3, 2),      # stem-like
    (2, 24, 40, 10, 10, 5, 3, 1, 2, 2),     # channels not multiples of 64, R != S
    (1, 8, 8, 4, 4, 3, 3, 1, 1, 2),         # tiny
    (1, 64, 64, 1, 1, 1, 1, 1, 0, 2),       # degenerate map
    # odd maps whose outputs never read the padding rows inside the partial last block (no padding):
    # served from the one full copy of the Z tile
    (3, 128, 64, 7, 9, 1, 1, 1, 0, 2),
    (2, 64, 128, 9, 7, 3, 3, 1, 0, 2),
    (2, 64, 64, 10, 10, 1, 1, 1, 0, 4),
    (2, 64, 64, 11, 11, 3, 3, 2, 0, 2),
]


@pytest.mark.parametrize("layout", ["nhwc", "nchw"])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("case", SMALL)
def test_wgrad_matches_checker(case, dtype, layout):
    err, got, want = wgrad_error_full(D(*case, dtype, layout))
    assert err <= TOL_DW[dtype], err


def _random_cases(n, seed, tensor_shapes=False, max_hw=20):
    """tensor_shapes: channel counts and stride/k pairs that the tensor-core kernels take."""
    rng = np.random.default_rng(seed)
    cases = []
    while len(cases) < n:
        chans = [64, 128, 192, 256] if tensor_shapes else [8, 24, 64, 64, 128, 192]
        Ci, Co = (int(rng.choice(chans)) for _ in range(2))
        H, W = int(rng.integers(1, max_hw + 1)), int(rng.integers(1, max_hw + 1))
        R, S = int(rng.choice([1, 3, 5])), int(rng.choice([1, 3, 5]))
        stride, pad, k = int(rng.integers(1, 4)), int(rng.integers(0, 3)), int(rng.choice([1, 2, 2, 3, 4]))
        if tensor_shapes:
            k = int(rng.choice([1, 2, 2, 4, 8]))
            stride = int(rng.choice([s for s in (1, 2, 4) if k % s == 0] + [2]))
        if H + 2 * pad < R or W + 2 * pad < S:
            continue
        cases.append((int(rng.integers(1, 6)), Ci, Co, H, W, R, S, stride, pad, k,
                      str(rng.choice(["bf16", "f32"])), str(rng.choice(["nhwc", "nchw"]))))
    return cases


@pytest.mark.parametrize("case", _random_cases(48, seed=2024) + _random_cases(64, seed=7, tensor_shapes=True) +
                         _random_cases(40, seed=11, tensor_shapes=True, max_hw=36))
def test_random_descriptors_match_checker(case):
    """Seeded random layer shapes over every dtype/layout pair: whichever kernel the planner picks
    (TMA-fed directly, on phase planes or on the inflated map, producer-fed, staged, fp32 FMA) must meet
    the bound; rectangular filters, strides that do not divide k, maps smaller than the filter's reach and
    single-pixel maps included."""
    d = D(*case)
    err, got, want = wgrad_error_full(d)     # an all-zero expected dW requires an all-zero result
    assert err <= TOL_DW[case[10]], (case, err)


def test_k1_equals_uncompressed_dw():
    """k = 1: Z is X, so the result must be the ordinary weight gradient."""
    import oracle
    from paper_2409_11902_b200 import synth
    d = D(2, 64, 64, 16, 16, 3, 3, 1, 1, 1, "bf16", "nhwc")
    z, dy = make_wgrad_inputs(d)
    got = run_wgrad(d, z, dy)
    want = oracle.wgrad_dense(synth.to_f64(z), synth.to_f64(dy), 3, 3, (1, 1), (1, 1))
    assert_dw_close(got, want, "bf16")


def test_tap_collapse_on_gpu():
    """Stride 2, k = 2, pad 1, even H: taps 1 and 2 read the same pooled value,
    so the two slices of dW must agree exactly (same products, same order)."""
    d = D(2, 64, 64, 16, 16, 3, 3, 2, 1, 2, "bf16", "nhwc")
    z, dy = make_wgrad_inputs(d)
    got = run_wgrad(d, z, dy)
    np.testing.assert_allclose(got[:, :, 1, :], got[:, :, 2, :], rtol=1e-5, atol=1e-7)
    np.testing.assert_allclose(got[:, :, :, 1], got[:, :, :, 2], rtol=1e-5, atol=1e-7)


RESNET18_STACK = [   # config 2: batch 64, bf16, k = 2 (+ the 7x7 map padded to 8x8)
    (64, 64, 64, 56, 56), (64, 128, 128, 28, 28), (64, 256, 256, 14, 14),
    (64, 512, 512, 7, 7), (64, 512, 512, 8, 8),
]


@pytest.mark.parametrize("N,Ci,Co,H,W", RESNET18_STACK)
def test_resnet18_stack_full_size_sampled(N, Ci, Co, H, W):
    err, _ = wgrad_error_sampled(D(N, Ci, Co, H, W, 3, 3, 1, 1, 2, "bf16", "nhwc"), n_samples=512)
    assert err <= TOL_DW["bf16"], err


@pytest.mark.parametrize("N,Ci,Co,H,W,k", [(64, 128, 128, 28, 28, 2), (64, 64, 64, 56, 56, 2),
                                             (32, 256, 256, 14, 14, 4), (16, 128, 128, 64, 64, 2)])
def test_fp32_inputs_on_the_tensor_cores_full_size_sampled(N, Ci, Co, H, W, k):
    """fp32 NHWC inputs run as six bf16 partial products; the fp32 bound (1e-5) still holds, with
    at least a factor of two to spare, at sizes where each entry sums 10^4 .. 10^5 products."""
    import paper_2409_11902_b200 as ac
    d = D(N, Ci, Co, H, W, 3, 3, 1, 1, k, "f32", "nhwc")
    assert ac.ac_wgrad_plan_info(d)["tensor_core"] in (3, 4)
    err, _ = wgrad_error_sampled(d, n_samples=256)
    assert err <= 0.5 * TOL_DW["f32"], err


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("N,Ci,Co,H,W,R,stride,pad,k", [(64, 128, 128, 28, 28, 3, 1, 1, 2), (32, 64, 64, 56, 56, 3, 1, 1, 2),
                                                         (16, 256, 64, 30, 30, 1, 1, 0, 2), (16, 128, 128, 27, 27, 3, 2, 1, 2),
                                                         (8, 512, 512, 7, 7, 3, 1, 1, 2), (16, 64, 128, 24, 40, 3, 1, 1, 4)])
def test_nchw_inputs_on_the_tensor_cores_full_size_sampled(N, Ci, Co, H, W, R, stride, pad, k, dtype):
    """NCHW operands are transposed (and fp32 ones split) into the workspace; dW comes back in
    NCHW order [Co][Ci][R][S]."""
    import paper_2409_11902_b200 as ac
    d = D(N, Ci, Co, H, W, R, R, stride, pad, k, dtype, "nchw")
    assert ac.ac_wgrad_plan_info(d)["tensor_core"] in (3, 4)
    err, _ = wgrad_error_sampled(d, n_samples=256)
    assert err <= (0.5 * TOL_DW["f32"] if dtype == "f32" else TOL_DW["bf16"]), err


def test_a_workspace_without_room_for_copies_takes_the_slower_path():
    """With ac_workspace_bytes_min the same call runs on the operands as they are (fp32 FMA);
    both results meet the bound, and the canary check shows neither writes past what it was given."""
    import paper_2409_11902_b200 as ac
    import oracle
    from paper_2409_11902_b200 import synth
    for dtype, layout in (("f32", "nhwc"), ("bf16", "nchw"), ("f32", "nchw")):
        d = D(4, 64, 64, 20, 20, 3, 3, 1, 1, 2, dtype, layout)
        lo, hi = ac.ac_workspace_bytes_min(d), ac.ac_workspace_bytes(d)
        assert 256 <= lo < hi
        z, dy = make_wgrad_inputs(d)
        want = oracle.wgrad_compressed(synth.to_f64(z), synth.to_f64(dy), d.H, d.W, d.R, d.S, d.stride, d.pad, d.k)
        for nbytes in (lo, hi - 256, hi):
            got = run_wgrad(d, z, dy, nbytes=nbytes)
            assert_dw_close(got, want, dtype, (dtype, layout, nbytes))
        zd = synth.to_layout(z, layout).cuda()
        dyd = synth.to_layout(dy, layout).cuda()
        import torch
        dw = torch.empty(d.dw_shape, dtype=torch.float32, device="cuda")
        ws = torch.empty(hi, dtype=torch.uint8, device="cuda")
        with pytest.raises(ac.AcError) as e:
            ac.ac_conv2d_wgrad_compressed(d, zd, dyd, dw, ws, lo - 1)
        assert e.value.status == ac.api.AC_ERR_WORKSPACE_TOO_SMALL


@pytest.mark.parametrize("dtype,layout", [("bf16", "nhwc"), ("f32", "nchw"), ("f32", "nhwc"), ("bf16", "nchw")])
def test_accumulate_adds_to_what_dw_holds(dtype, layout):
    """dW <- beta * dW + gradient: with beta = 1 on zeros it is the plain call bit for bit; with
    beta = 0.5 on a random dW it is the fused multiply-add of the two; any workspace from the
    minimum up is taken."""
    import torch
    import paper_2409_11902_b200 as ac
    from paper_2409_11902_b200 import synth
    d = D(4, 64, 64, 20, 20, 3, 3, 1, 1, 2, dtype, layout)
    z, dy = make_wgrad_inputs(d)
    zd = synth.to_layout(z, layout).cuda()
    dyd = synth.to_layout(dy, layout).cuda()
    dw_bytes = 64 * 64 * 9 * 4
    for nbytes, plain_bytes in ((ac.ac_accumulate_workspace_bytes(d), ac.ac_workspace_bytes(d)),
                                (ac.ac_workspace_bytes_min(d) + dw_bytes + 256, ac.ac_workspace_bytes_min(d))):
        plain = torch.empty(d.dw_shape, dtype=torch.float32, device="cuda")
        ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        ac.ac_conv2d_wgrad_compressed(d, zd, dyd, plain, ws, plain_bytes)
        dw = torch.zeros_like(plain)
        ac.ac_conv2d_wgrad_compressed_accumulate(d, zd, dyd, 1.0, dw, ws)
        assert ac.ac_workspace_status(ws)[0] == 0
        assert torch.equal(dw, plain)
        g = torch.Generator(device="cuda").manual_seed(5)
        old = torch.randn(d.dw_shape, generator=g, device="cuda") * plain.abs().mean()
        dw = old.clone()
        ac.ac_conv2d_wgrad_compressed_accumulate(d, zd, dyd, 0.5, dw, ws)
        want = (0.5 * old.double() + plain.double())
        assert float((dw.double() - want).abs().max()) <= 1.2e-7 * float(want.abs().max())
        with pytest.raises(ac.AcError) as e:
            ac.ac_conv2d_wgrad_compressed_accumulate(d, zd, dyd, 1.0, dw, ws, ac.ac_workspace_bytes_min(d) + dw_bytes - 1)
        assert e.value.status == ac.api.AC_ERR_WORKSPACE_TOO_SMALL


@pytest.mark.parametrize("layer", [(16, 128, 128, 28, 28), (8, 64, 64, 56, 56), (32, 512, 512, 8, 8)])
def test_back_to_back_calls_see_each_others_results(layer):
    """compress -> wgrad -> (reduce) queued without any synchronisation, inputs changing from call to
    call: each kernel may be brought onto the GPU while the one before it is still finishing, and must
    still read what that one wrote. Compared bit for bit with the same calls synchronised one by one."""
    import torch
    import paper_2409_11902_b200 as ac
    N, Ci, Co, H, W = layer
    d = D(N, Ci, Co, H, W, 3, 3, 1, 1, 2, "bf16", "nhwc")
    g = torch.Generator(device="cuda").manual_seed(11)
    xs = [torch.randn(d.x_shape, generator=g, device="cuda").relu().to(torch.bfloat16) for _ in range(4)]
    dy = (torch.randn((N, d.Ho, d.Wo, Co), generator=g, device="cuda") * 1e-2).to(torch.bfloat16)
    z = torch.empty(d.z_shape, dtype=torch.bfloat16, device="cuda")
    dw = torch.empty(d.dw_shape, dtype=torch.float32, device="cuda")
    ws = torch.empty(ac.ac_workspace_bytes(d), dtype=torch.uint8, device="cuda")
    refs = []
    for x in xs:
        ac.ac_compress(d, x, z)
        torch.cuda.synchronize()
        ac.ac_conv2d_wgrad_compressed(d, z, dy, dw, ws)
        torch.cuda.synchronize()
        refs.append(dw.clone())
    assert not torch.equal(refs[0], refs[1])
    outs = []
    for rnd in range(5):
        for x in xs:
            ac.ac_compress(d, x, z)
            ac.ac_conv2d_wgrad_compressed(d, z, dy, dw, ws)
            outs.append(dw.clone())
    torch.cuda.synchronize()
    assert ac.ac_workspace_status(ws)[0] == 0
    for i, o in enumerate(outs):
        assert torch.equal(o, refs[i % 4]), i


BOTTLENECK = [  # config 3: batch 128, bf16
    (128, 256, 64, 56, 56, 1, 1, 1, 0), (128, 64, 64, 56, 56, 3, 3, 1, 1),
    (128, 64, 256, 56, 56, 1, 1, 1, 0), (128, 128, 128, 56, 56, 3, 3, 2, 1),
]


@pytest.mark.parametrize("N,Ci,Co,H,W,R,S,stride,pad", BOTTLENECK)
def test_bottleneck_layers_full_size_sampled(N, Ci, Co, H, W, R, S, stride, pad):
    err, _ = wgrad_error_sampled(D(N, Ci, Co, H, W, R, S, stride, pad, 2, "bf16", "nhwc"),
                                 n_samples=256)
    assert err <= TOL_DW["bf16"], err


@pytest.mark.parametrize("k", [1, 2, 4, 8])
def test_pooling_sweep_full_size_sampled(k):
    """Config 4: N=256, 128 channels, 64x64, bf16 (1 Mi positions per entry)."""
    err, _ = wgrad_error_sampled(D(256, 128, 128, 64, 64, 3, 3, 1, 1, k, "bf16", "nhwc"),
                                 n_samples=96)
    assert err <= TOL_DW["bf16"], err


def test_errors_are_codes_not_faults():
    import torch
    import paper_2409_11902_b200 as ac
    d = D(2, 64, 64, 16, 16, 3, 3, 1, 1, 2, "bf16", "nhwc")
    z = torch.zeros(d.z_shape, dtype=torch.bfloat16, device="cuda")
    dy = torch.zeros(d.dy_shape, dtype=torch.bfloat16, device="cuda")
    dw = torch.zeros(d.dw_shape, device="cuda")
    n = ac.ac_workspace_bytes(d)
    ws = torch.zeros(n, dtype=torch.uint8, device="cuda")
    with pytest.raises(ac.AcError) as e:
        ac.ac_conv2d_wgrad_compressed(d, z, dy, dw, ws, n - 1)
    assert e.value.status == ac.api.AC_ERR_WORKSPACE_TOO_SMALL
    with pytest.raises(ac.AcError) as e:
        ac.ac_conv2d_wgrad_compressed(d, z, dy, dw, ws.data_ptr() + 8, n)
    assert e.value.status == ac.api.AC_ERR_MISALIGNED
    ac.ac_conv2d_wgrad_compressed(d, z, dy, dw, ws, n)
    assert ac.ac_workspace_status(ws) == (0, 0)
    assert not dw.any()


def test_host_step_matches_device_calls():
    import torch
    import paper_2409_11902_b200 as ac
    from paper_2409_11902_b200 import synth
    d = D(4, 64, 64, 16, 16, 3, 3, 1, 1, 2, "bf16", "nhwc")
    x = synth.to_layout(synth.activation(0, (d.N, d.C_in, d.H, d.W), d.dtype), d.layout).pin_memory()
    dy = synth.to_layout(synth.grad_output(0, (d.N, d.C_out, d.Ho, d.Wo), d.dtype), d.layout).pin_memory()
    dw_h = torch.empty(d.dw_shape, dtype=torch.float32).pin_memory()
    z_h = torch.empty(d.z_shape, dtype=torch.bfloat16).pin_memory()
    arena = torch.empty(ac.ac_host_step_arena_bytes(d), dtype=torch.uint8, device="cuda")
    ac.ac_backward_step_host(d, x, dy, dw_h, z_h, arena)
    torch.cuda.synchronize()
    xd, dyd = x.cuda(), dy.cuda()
    z = torch.empty(d.z_shape, dtype=torch.bfloat16, device="cuda")
    dw = torch.empty(d.dw_shape, device="cuda")
    ws = torch.empty(ac.ac_workspace_bytes(d), dtype=torch.uint8, device="cuda")
    ac.ac_compress(d, xd, z)
    ac.ac_conv2d_wgrad_compressed(d, z, dyd, dw, ws)
    torch.cuda.synchronize()
    assert torch.equal(z.cpu(), z_h) and torch.equal(dw.cpu(), dw_h)


# Config 5: every distinct conv shape of ResNet-50 (bottleneck blocks, stride on the 3x3),
# at a reduced batch; (C_in, C_out, H_in, R, stride, pad).
RESNET50_SHAPES = [
    (3, 64, 224, 7, 2, 3), (64, 64, 56, 1, 1, 0), (64, 64, 56, 3, 1, 1), (64, 256, 56, 1, 1, 0),
    (256, 64, 56, 1, 1, 0), (256, 128, 56, 1, 1, 0), (128, 128, 56, 3, 2, 1), (128, 512, 28, 1, 1, 0),
    (256, 512, 56, 1, 2, 0), (512, 128, 28, 1, 1, 0), (128, 128, 28, 3, 1, 1), (512, 256, 28, 1, 1, 0),
    (256, 256, 28, 3, 2, 1), (256, 1024, 14, 1, 1, 0), (512, 1024, 28, 1, 2, 0), (1024, 256, 14, 1, 1, 0),
    (256, 256, 14, 3, 1, 1), (1024, 512, 14, 1, 1, 0), (512, 512, 14, 3, 2, 1), (512, 2048, 7, 1, 1, 0),
    (1024, 2048, 14, 1, 2, 0), (2048, 512, 7, 1, 1, 0), (512, 512, 7, 3, 1, 1),
]


@pytest.mark.parametrize("Ci,Co,H,R,stride,pad", RESNET50_SHAPES)
def test_resnet50_layer_shapes_sampled(Ci, Co, H, R, stride, pad):
    N = 2 if H >= 56 else 8
    err, _ = wgrad_error_sampled(D(N, Ci, Co, H, H, R, R, stride, pad, 2, "bf16", "nhwc"), n_samples=192)
    assert err <= TOL_DW["bf16"], err


def test_gradient_alignment_diagnostic():
    """Section 5.2's cosine similarity between the compressed and the k = 1 weight
    gradient, on synthetic data: 1 for k = 1, below 1 and decreasing with k, and the
    GPU value equals the checker's."""
    import oracle
    from paper_2409_11902_b200 import synth
    base = D(4, 64, 64, 16, 16, 3, 3, 1, 1, 1, "bf16", "nhwc")
    x = synth.activation(3, (base.N, base.C_in, base.H, base.W), "bf16")
    dy = synth.grad_output(3, (base.N, base.C_out, base.Ho, base.Wo), "bf16")
    ref = run_wgrad(base, x, dy)
    cos = {}
    for k in (1, 2, 4):
        d = dataclasses.replace(base, k=k)
        z = synth.to_storage(oracle.pool(synth.to_f64(x), k), "bf16")
        got = run_wgrad(d, z, dy)
        cos[k] = oracle.cosine_similarity(got, ref)
        want = oracle.wgrad_compressed(synth.to_f64(z), synth.to_f64(dy), 16, 16, 3, 3, (1, 1), (1, 1), k)
        assert abs(cos[k] - oracle.cosine_similarity(want, ref)) < 1e-5
    assert cos[1] == pytest.approx(1.0, abs=1e-9)
    assert 0 < cos[4] < cos[2] < 1


def test_a_wait_that_runs_out_is_reported_not_hung():
    """Failure detection without a fault: a kernel waits, with the library's bounded wait, on
    a barrier that nothing completes; it must come back and leave AC_ERR_TIMEOUT in the status
    block, and the context must stay usable."""
    import torch
    import paper_2409_11902_b200 as ac
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    ac.ac_selftest_bounded_wait(ws, 2_000_000)      # about a millisecond
    st, detail = ac.ac_workspace_status(ws)
    assert (st, detail) == (ac.api.AC_ERR_TIMEOUT, 0x7E57)
    # the device is fine afterwards: an ordinary call still works and reports AC_OK
    d = D(2, 64, 64, 16, 16, 3, 3, 1, 1, 2, "bf16", "nhwc")
    z, dy = make_wgrad_inputs(d)
    run_wgrad(d, z, dy)


COLLAPSIBLE = [
    # N, Ci, Co, H, W, R, S, stride, pad, k
    (2, 64, 64, 16, 16, 3, 3, 1, 1, 2),
    (3, 128, 128, 12, 20, 3, 3, 1, 1, 2),
    (2, 128, 64, 16, 16, 3, 3, 2, 1, 2),     # stride 2, k = 2: one class, 4 shifts for 9 taps
    (2, 64, 128, 16, 16, 3, 3, 1, 1, 4),
    (2, 128, 128, 16, 16, 3, 3, 1, 1, 8),    # 64 classes
    (2, 256, 256, 14, 14, 3, 3, 1, 1, 2),
    (2, 64, 64, 16, 16, 5, 3, 1, 2, 2),
    (2, 128, 128, 30, 30, 7, 7, 2, 3, 2),
]


@pytest.mark.parametrize("case", COLLAPSIBLE)
def test_collapsed_form_matches_checker(case):
    """Fewer MMAs, same dW: against the fp64 checker and against the dense entry point."""
    import oracle
    from paper_2409_11902_b200 import synth
    d = D(*case, "bf16", "nhwc")
    z, dy = make_wgrad_inputs(d)
    got = run_wgrad_collapsed(d, z, dy)
    assert got is not None
    want = oracle.wgrad_compressed(synth.to_f64(z), synth.to_f64(dy), d.H, d.W, d.R, d.S, d.stride, d.pad, d.k)
    assert_dw_close(got, want, "bf16")
    dense = run_wgrad(d, z, dy)
    assert np.linalg.norm(got - dense) / np.linalg.norm(dense) <= 1e-5


def test_collapsed_form_full_size_and_refusals():
    import paper_2409_11902_b200 as ac
    import oracle
    from paper_2409_11902_b200 import synth
    d = D(64, 128, 128, 28, 28, 3, 3, 1, 1, 2, "bf16", "nhwc")
    z, dy = make_wgrad_inputs(d)
    got = run_wgrad_collapsed(d, z, dy)
    sampled_check(d, got, z, dy, n_samples=256, seed=5)
    # nothing to collapse, or not this kernel's shapes: size 0 and AC_ERR_UNSUPPORTED
    for bad in (D(2, 64, 64, 16, 16, 3, 3, 1, 1, 1, "bf16", "nhwc"), D(2, 64, 64, 16, 16, 1, 1, 1, 0, 2, "bf16", "nhwc"),
                D(2, 64, 64, 15, 15, 3, 3, 1, 1, 2, "bf16", "nhwc"), D(2, 64, 64, 16, 16, 3, 3, 1, 1, 2, "f32", "nhwc")):
        assert ac.ac_collapsed_workspace_bytes(bad)[0] == 0
        import torch
        t = torch.zeros(1024, device="cuda")
        with pytest.raises(ac.AcError) as e:
            ac.ac_conv2d_wgrad_compressed_collapsed(bad, t, t, t, t, 4096)
        assert e.value.status == ac.api.AC_ERR_UNSUPPORTED


# Few input channels (bf16 NHWC): the operand is gathered into a [positions][taps x channels] matrix
# and the tensor-core kernel runs the equivalent 1x1 problem (plan code 5).
FEW_CHANNELS = [
    # N, Ci, Co, H, W, R, S, stride, pad, k
    (2, 3, 64, 32, 32, 7, 7, 2, 3, 2),      # stem-like: stride = k, k | H: 49 taps collapse to 16 shifts
    (2, 3, 64, 31, 29, 7, 7, 2, 3, 2),      # odd map: partial last blocks, one column per tap
    (3, 3, 128, 20, 20, 3, 3, 1, 1, 2),     # stride 1 at k = 2: no collapse
    (2, 5, 128, 20, 20, 5, 5, 2, 2, 4),     # stride does not reach k
    (2, 4, 64, 24, 24, 5, 5, 4, 2, 2),      # stride = 2k: two pooled rows per output row
    (2, 3, 64, 16, 16, 7, 7, 2, 3, 1),      # k = 1
    (2, 16, 64, 12, 12, 3, 3, 1, 1, 2),     # 144 columns -> 192
    (1, 1, 64, 9, 9, 3, 3, 1, 0, 3),        # one channel, k = 3, no padding
    (2, 3, 64, 32, 32, 3, 5, 2, 1, 2),      # R != S, collapsed
    (2, 7, 192, 8, 8, 1, 1, 1, 0, 2),       # pointwise
    (3, 3, 64, 56, 64, 7, 7, 2, 3, 2),      # in-kernel form: 32 positions per row, 4 rows per K-tile
    (3, 3, 64, 56, 40, 7, 7, 2, 3, 2),      # rows of Z of 120 bytes: not for TMA, staged in the workspace
    (2, 6, 320, 24, 24, 3, 3, 2, 1, 2),     # in-kernel form, 320 output channels = 5 blocks of 64
    (2, 8, 256, 16, 48, 5, 5, 2, 2, 2),     # in-kernel form: 3 x 3 shifts x 8 channels = 72 columns -> 128, N = 256
    (5, 3, 64, 12, 12, 7, 7, 4, 3, 2),      # stride 4 = 2k: two pooled rows per output row, a 3-position row
]


@pytest.mark.parametrize("case", FEW_CHANNELS)
def test_few_input_channels_match_checker(case):
    import paper_2409_11902_b200 as ac
    d = D(*case, "bf16", "nhwc")
    N, Ci, Co, H, W, R, S, stride, pad, k = case
    # strides that are multiples of k on a map that k divides: the matrix is built inside the kernel (6);
    # otherwise it is staged in the workspace (5)
    # (and rows of Z that are a whole number of 16-byte units long, for the TMA copy of the strip)
    fused = k > 1 and stride % k == 0 and H % k == 0 and W % k == 0 and ((W // k) * Ci * 2) % 16 == 0
    assert ac.ac_wgrad_plan_info(d)["tensor_core"] == (6 if fused else 5)
    err, got, want = wgrad_error_full(d)
    assert err <= 1e-4 <= TOL_DW["bf16"], err     # bf16 products are exact in fp32: summation order only


def test_few_input_channels_small_workspace_and_full_size_stem():
    import paper_2409_11902_b200 as ac
    import oracle
    from paper_2409_11902_b200 import synth
    d = D(2, 3, 64, 32, 32, 7, 7, 2, 3, 2, "bf16", "nhwc")
    z, dy = make_wgrad_inputs(d)
    want = oracle.wgrad_compressed(synth.to_f64(z), synth.to_f64(dy), d.H, d.W, d.R, d.S, d.stride, d.pad, d.k)
    for nbytes in (ac.ac_workspace_bytes_min(d), ac.ac_workspace_bytes(d)):
        got = run_wgrad(d, z, dy, nbytes=nbytes)
        assert_dw_close(got, want, "bf16")
    # the ResNet stem at its own map size
    err, _ = wgrad_error_sampled(D(8, 3, 64, 224, 224, 7, 7, 2, 3, 2, "bf16", "nhwc"), n_samples=256)
    assert err <= 1e-4, err


# Small odd maps with padding: the TMA-fed kernel runs on an inflated copy of Z (plan code 7) where its cost
# model expects that to beat reading Z directly; the result is the same weight gradient.
ODD_MAPS_INFLATED = [
    # N, Ci, Co, H, W, R, S, stride, pad, k
    (24, 512, 512, 7, 7, 3, 3, 1, 1, 2),      # the last ResNet stage's 3x3 layers
    (64, 256, 512, 7, 9, 3, 3, 1, 1, 2),      # H != W
    (12, 512, 256, 7, 7, 3, 3, 1, 1, 4),      # k = 4: blocks of 4 and 3 rows and columns
    (16, 384, 320, 9, 9, 3, 3, 1, 1, 2),      # 320 output channels = 5 blocks of 64
    (8, 64, 64, 55, 55, 3, 3, 1, 1, 2),       # a large odd map with 64 channels
    (3, 64, 128, 28, 28, 3, 3, 1, 1, 8),      # k = 8 on a 28 x 28 map: half a block at the edge
    (5, 128, 64, 7, 7, 3, 3, 1, 1, 4),
]


@pytest.mark.parametrize("case", ODD_MAPS_INFLATED)
def test_small_odd_maps_run_on_the_inflated_copy(case):
    import paper_2409_11902_b200 as ac
    d = D(*case, "bf16", "nhwc")
    assert ac.ac_wgrad_plan_info(d)["tensor_core"] == 7
    z, dy = make_wgrad_inputs(d)
    # with the full workspace (inflated copy), and with the smallest one (the kernel reads Z itself)
    for nbytes in sorted({ac.ac_workspace_bytes_min(d), ac.ac_workspace_bytes(d)}):
        got = run_wgrad(d, z, dy, nbytes=nbytes)
        err = sampled_check(d, got, z, dy, n_samples=512)
        assert err <= 1e-4, (nbytes, err)


# A stride that is a multiple of the pooling block (k = 1 at stride 2: the uncompressed gradient of a strided
# layer): one output class whose taps read phase planes of Z, still the TMA-fed kernel.
STRIDE_ABOVE_K = [
    # N, Ci, Co, H, W, R, S, stride, pad, k, dtype, layout, plan code
    (4, 128, 128, 28, 28, 3, 3, 2, 1, 1, "bf16", "nhwc", 2),
    (4, 64, 128, 30, 30, 3, 3, 2, 1, 1, "bf16", "nhwc", 2),
    (4, 64, 64, 29, 31, 3, 3, 2, 1, 1, "bf16", "nhwc", 2),       # odd map: planes of different extents
    (4, 128, 256, 28, 28, 1, 1, 2, 0, 1, "bf16", "nhwc", 2),     # the downsample projection: one plane, one tap
    (3, 64, 64, 32, 32, 7, 7, 2, 3, 1, "bf16", "nhwc", 2),
    (4, 64, 64, 24, 24, 5, 5, 2, 2, 1, "bf16", "nhwc", 2),
    (4, 64, 64, 32, 32, 3, 3, 4, 1, 2, "bf16", "nhwc", 2),       # stride 4 at k = 2
    (3, 64, 128, 12, 20, 3, 3, (2, 1), (1, 1), 1, "bf16", "nhwc", 2),
    (4, 128, 128, 28, 28, 3, 3, 2, 1, 3, "bf16", "nhwc", 7),     # k = 3 at stride 2: inflated, then as above
    (4, 64, 64, 28, 28, 3, 3, 2, 1, 1, "f32", "nhwc", 3),        # staged operands on the same plan
    (4, 64, 128, 28, 28, 3, 3, 2, 1, 1, "bf16", "nchw", 3),
]


@pytest.mark.parametrize("case", STRIDE_ABOVE_K)
def test_stride_above_k_matches_checker(case):
    import paper_2409_11902_b200 as ac
    N, Ci, Co, H, W, R, S, stride, pad, k, dtype, layout, code = case
    pair = lambda v: v if isinstance(v, tuple) else (v, v)
    d = ac.ConvDesc(N, Ci, Co, H, W, R, S, pair(stride), pair(pad), k, dtype, layout)
    assert ac.ac_wgrad_plan_info(d)["tensor_core"] in ((code,) if code != 3 else (3, 4))
    err, got, want = wgrad_error_full(d)
    assert err <= TOL_DW[dtype], err


def test_sm_budget_layers_side_by_side_match_checker():
    """Four layers planned for a quarter of the SMs each, enqueued on four streams without synchronising in
    between: every dW against the checker, and against the same call planned for the whole GPU."""
    import torch
    import oracle
    import paper_2409_11902_b200 as ac
    from paper_2409_11902_b200 import synth
    shapes = [(6, 64, 64, 28, 28, 3, 3, 1, 1, 2), (6, 128, 128, 14, 14, 3, 3, 1, 1, 2),
              (6, 256, 128, 14, 14, 1, 1, 1, 0, 2), (6, 128, 128, 28, 28, 3, 3, 2, 1, 2)]
    work = []
    for i, sh in enumerate(shapes):
        d = D(*sh, "bf16", "nhwc")
        z, dy = make_wgrad_inputs(d, seed=20 + i)
        want = oracle.wgrad_compressed(synth.to_f64(z), synth.to_f64(dy), d.H, d.W, d.R, d.S, d.stride, d.pad, d.k)
        work.append(dict(d=d, z=synth.to_layout(z, "nhwc").cuda(), dy=synth.to_layout(dy, "nhwc").cuda(), want=want,
                         whole=run_wgrad(d, z, dy)))
    try:
        ac.ac_set_sm_budget(37)
        for w in work:
            n = ac.ac_workspace_bytes(w["d"])
            assert ac.ac_wgrad_plan_info(w["d"])["ctas"] <= 37
            w["ws"] = torch.full((n,), 0xFF, dtype=torch.uint8, device="cuda")
            w["dw"] = torch.full(w["d"].dw_shape, float("nan"), device="cuda")
            w["stream"] = torch.cuda.Stream()
        torch.cuda.synchronize()
        for rep in range(3):
            for w in work:
                with torch.cuda.stream(w["stream"]):
                    ac.ac_conv2d_wgrad_compressed(w["d"], w["z"], w["dy"], w["dw"], w["ws"])
        torch.cuda.synchronize()
    finally:
        ac.ac_set_sm_budget(0)
    for w in work:
        assert ac.ac_workspace_status(w["ws"])[0] == 0
        got = w["dw"].double().cpu().numpy().transpose(0, 3, 1, 2)
        assert_dw_close(got, w["want"], "bf16")
        assert_dw_close(got, w["whole"], "bf16")


# Few input channels with a pooling block that is a multiple of the stride (k = 4, 8 at stride 2): Z is re-blocked
# to k' = stride in the workspace (the same inflated map) and the in-kernel gather runs on that.
FEW_CHANNELS_REBLOCKED = [
    # N, Ci, Co, H, W, R, S, stride, pad, k
    (2, 3, 64, 32, 32, 7, 7, 2, 3, 4),
    (2, 3, 64, 32, 32, 7, 7, 2, 3, 8),
    (3, 3, 64, 56, 64, 7, 7, 2, 3, 4),
    (2, 6, 320, 24, 24, 3, 3, 2, 1, 4),
    (2, 3, 64, 30, 32, 7, 7, 2, 3, 4),       # k does not divide H: the partial last block is re-blocked with the rest
    (2, 8, 256, 16, 48, 5, 5, 2, 2, 8),
]


@pytest.mark.parametrize("case", FEW_CHANNELS_REBLOCKED)
def test_few_input_channels_reblocked_match_checker(case):
    import paper_2409_11902_b200 as ac
    d = D(*case, "bf16", "nhwc")
    assert ac.ac_wgrad_plan_info(d)["tensor_core"] == 6
    err, got, want = wgrad_error_full(d)
    assert err <= 1e-4 <= TOL_DW["bf16"], err


# Pooling blocks of 4 and 8: where the cost model prefers it, Z is re-blocked in the workspace to a smaller block
# k' that divides k (the same inflated map) and the TMA-fed kernel runs with k' (plan code 7, phases = its classes).
REBLOCKED = [
    # N, Ci, Co, H, W, R, S, stride, pad, k, classes of the inner plan
    (16, 64, 64, 56, 56, 3, 3, 1, 1, 4, 4),        # 64 channels: the taps pair up at k' = 2, not at k = 4
    (16, 64, 64, 56, 56, 3, 3, 1, 1, 8, 4),
    (32, 256, 256, 14, 14, 3, 3, 1, 1, 4, 4),      # 14 = 3 * 4 + 2: partial blocks at k = 4, none at k' = 2
    (8, 128, 128, 28, 28, 3, 3, 1, 1, 8, 1),       # all the way to the inflated map
]


@pytest.mark.parametrize("case", REBLOCKED)
def test_reblocked_pooling_blocks_match_checker(case):
    import paper_2409_11902_b200 as ac
    *shape, classes = case
    d = D(*shape, "bf16", "nhwc")
    info = ac.ac_wgrad_plan_info(d)
    assert (info["tensor_core"], info["phases"]) == (7, classes)
    z, dy = make_wgrad_inputs(d)
    for nbytes in sorted({ac.ac_workspace_bytes_min(d), ac.ac_workspace_bytes(d)}):
        got = run_wgrad(d, z, dy, nbytes=nbytes)
        err = sampled_check(d, got, z, dy, n_samples=512)
        assert err <= 1e-4, (nbytes, err)
