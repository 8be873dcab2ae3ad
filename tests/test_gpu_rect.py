"""Non-uniform pooling blocks (k_h x k_w) on the GPU against the CPU checker: the *_rect entry points."""
import dataclasses

import numpy as np
import pytest

import __graft_entry__ as entry
from helpers import TOL_Z, assert_dw_close, canary_intact, padded_empty

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    entry.build()


def D(N, Ci, Co, H, W, R, S, stride, pad, dtype, layout):
    import paper_2409_11902_b200 as ac
    return ac.ConvDesc(N, Ci, Co, H, W, R, S, stride, pad, 1, dtype, layout)   # desc.k is ignored by *_rect


COMPRESS = [  # N, C, H, W, (kh, kw)
    (2, 64, 16, 24, (2, 4)), (2, 64, 15, 21, (4, 2)), (3, 8, 9, 10, (1, 2)), (2, 3, 12, 12, (3, 2)),
    (1, 128, 7, 7, (2, 1)), (2, 24, 10, 18, (2, 8)),
]


@pytest.mark.parametrize("layout", ["nhwc", "nchw"])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("case", COMPRESS)
def test_rect_compress_matches_checker(case, dtype, layout):
    import torch
    import oracle
    import paper_2409_11902_b200 as ac
    from paper_2409_11902_b200 import synth
    N, C, H, W, k = case
    d = D(N, C, C, H, W, 1, 1, (1, 1), (0, 0), dtype, layout)
    Hp, Wp = oracle.pooled_hw(H, W, k)
    for fused in (False, True):
        src = synth.pre_activation(1, (N, C, H, W), dtype) if fused else synth.activation(1, (N, C, H, W), dtype)
        x64 = oracle.relu(synth.to_f64(src)) if fused else synth.to_f64(src)
        xd = synth.to_layout(src, layout).cuda()
        zshape = (N, C, Hp, Wp) if layout == "nchw" else (N, Hp, Wp, C)
        zbuf, z, zspan = padded_empty(zshape, d.torch_dtype, "cuda:0")
        y = torch.empty_like(xd) if fused else None
        ac.ac_compress_rect(d, k[0], k[1], xd, z, y)
        torch.cuda.synchronize()
        assert canary_intact(zbuf, zspan)
        z64 = synth.to_f64(synth.from_layout(z.cpu(), layout))
        z_ref, denom = oracle.pool(x64, k), oracle.pool(np.abs(x64), k)
        diff, zero = np.abs(z64 - z_ref), denom == 0
        assert not diff[zero].any()
        assert float(np.max(diff[~zero] / denom[~zero])) <= TOL_Z[dtype]
        if fused:
            assert np.array_equal(synth.to_f64(synth.from_layout(y.cpu(), layout)), x64)


WGRAD = [  # N, Ci, Co, H, W, R, S, stride, pad, (kh, kw)
    (2, 64, 64, 16, 24, 3, 3, (1, 1), (1, 1), (2, 4)),       # tensor-core class form: 2 x 4 classes
    (2, 128, 64, 16, 16, 3, 3, (1, 1), (1, 1), (4, 2)),
    (3, 64, 128, 12, 20, 3, 3, (2, 1), (1, 1), (2, 1)),      # stride (2,1) with a 2 x 1 block: one class
    (2, 64, 64, 15, 21, 3, 3, (1, 1), (1, 1), (2, 4)),       # partial last blocks in both directions
    (2, 128, 128, 14, 14, 1, 1, (1, 1), (0, 0), (1, 2)),     # pointwise
    (2, 64, 64, 16, 16, 5, 3, (1, 2), (2, 1), (2, 4)),       # rectangular filter, stride and block
    (2, 64, 64, 12, 12, 3, 3, (1, 1), (1, 1), (3, 2)),
    (2, 24, 40, 10, 12, 3, 3, (1, 1), (1, 1), (2, 3)),       # channels no tensor-core path takes
    (2, 64, 64, 12, 12, 3, 3, (2, 2), (1, 1), (3, 4)),       # strides that do not divide the block
    (1, 3, 64, 20, 20, 7, 7, (2, 2), (3, 3), (2, 4)),        # few input channels
]


@pytest.mark.parametrize("dtype,layout", [("bf16", "nhwc"), ("f32", "nhwc"), ("bf16", "nchw"), ("f32", "nchw")])
@pytest.mark.parametrize("case", WGRAD)
def test_rect_wgrad_matches_checker(case, dtype, layout):
    import torch
    import oracle
    import paper_2409_11902_b200 as ac
    from paper_2409_11902_b200 import synth
    N, Ci, Co, H, W, R, S, stride, pad, k = case
    d = D(N, Ci, Co, H, W, R, S, stride, pad, dtype, layout)
    x = synth.activation(2, (N, Ci, H, W), dtype)
    z = synth.to_storage(oracle.pool(synth.to_f64(x), k), dtype)
    dy = synth.grad_output(2, (N, Co, d.Ho, d.Wo), dtype)
    zd, dyd = synth.to_layout(z, layout).cuda(), synth.to_layout(dy, layout).cuda()
    nbytes = ac.ac_workspace_bytes_rect(d, *k)
    assert nbytes >= 256
    outs = []
    for it in range(2):
        wbuf, dw, wspan = padded_empty(d.dw_shape, torch.float32, "cuda:0")
        sbuf, ws, sspan = padded_empty((nbytes,), torch.uint8, "cuda:0")
        if it:
            ws.fill_(0xFF)
            dw.fill_(float("nan"))
        ac.ac_conv2d_wgrad_compressed_rect(d, k[0], k[1], zd, dyd, dw, ws, nbytes)
        assert ac.ac_workspace_status(ws)[0] == 0
        assert canary_intact(wbuf, wspan) and canary_intact(sbuf, sspan)
        outs.append(dw.clone())
    assert torch.equal(outs[0], outs[1])
    got = outs[0].double().cpu().numpy()
    if layout == "nhwc":
        got = got.transpose(0, 3, 1, 2)
    want = oracle.wgrad_compressed(synth.to_f64(z), synth.to_f64(dy), H, W, R, S, stride, pad, k)
    assert_dw_close(got, want, dtype, case)


def test_square_block_through_the_rect_calls_is_the_square_call():
    import torch
    import paper_2409_11902_b200 as ac
    from helpers import make_wgrad_inputs
    from paper_2409_11902_b200 import synth
    d = ac.ConvDesc(4, 64, 64, 20, 20, 3, 3, (1, 1), (1, 1), 2, "bf16", "nhwc")
    assert ac.ac_workspace_bytes_rect(d, 2, 2) == ac.ac_workspace_bytes(d) == ac.ac_workspace_bytes_rect(d, 0, 0)
    z, dy = make_wgrad_inputs(d)
    x = synth.to_layout(synth.activation(0, (4, 64, 20, 20), "bf16"), "nhwc").cuda()
    za, zb = (torch.empty(d.z_shape, dtype=torch.bfloat16, device="cuda") for _ in range(2))
    ac.ac_compress(d, x, za)
    ac.ac_compress_rect(dataclasses.replace(d, k=7), 2, 2, x, zb)
    assert torch.equal(za, zb)
    zd, dyd = synth.to_layout(z, "nhwc").cuda(), synth.to_layout(dy, "nhwc").cuda()
    ws = torch.empty(ac.ac_workspace_bytes(d), dtype=torch.uint8, device="cuda")
    a, b = (torch.empty(d.dw_shape, device="cuda") for _ in range(2))
    ac.ac_conv2d_wgrad_compressed(d, zd, dyd, a, ws)
    ac.ac_conv2d_wgrad_compressed_rect(dataclasses.replace(d, k=7), 2, 2, zd, dyd, b, ws)
    assert torch.equal(a, b)


def test_rect_full_size_sampled_on_the_tensor_cores():
    """A ResNet-sized layer with a 2 x 4 block: stratified entries against the checker."""
    import torch
    import oracle
    import paper_2409_11902_b200 as ac
    from helpers import stratified_entries
    from paper_2409_11902_b200 import synth
    N, C, H, k = 16, 128, 56, (2, 4)
    d = D(N, C, C, H, H, 3, 3, (1, 1), (1, 1), "bf16", "nhwc")
    x = synth.activation(4, (N, C, H, H), "bf16")
    z = synth.to_storage(oracle.pool(synth.to_f64(x), k), "bf16")
    dy = synth.grad_output(4, (N, C, H, H), "bf16")
    ws = torch.empty(ac.ac_workspace_bytes_rect(d, *k), dtype=torch.uint8, device="cuda")
    dw = torch.empty(d.dw_shape, device="cuda")
    ac.ac_conv2d_wgrad_compressed_rect(d, k[0], k[1], synth.to_layout(z, "nhwc").cuda(),
                                       synth.to_layout(dy, "nhwc").cuda(), dw, ws)
    assert ac.ac_workspace_status(ws)[0] == 0
    got = dw.double().cpu().numpy().transpose(0, 3, 1, 2)
    idx = stratified_entries(d, 256, seed=4)
    want = oracle.wgrad_compressed_entries(synth.to_f64(z), synth.to_f64(dy), H, H, 3, 3, (1, 1), (1, 1), k, idx)
    assert_dw_close(got[idx[:, 0], idx[:, 1], idx[:, 2], idx[:, 3]], want, "bf16")


def test_rect_block_on_the_inflated_route():
    """A small odd map with padding and a 4 x 2 block: the kernel runs on the inflated copy of Z (the
    workspace holds it beside the partial sums); stratified entries against the checker."""
    import torch
    import oracle
    import paper_2409_11902_b200 as ac
    from helpers import stratified_entries
    from paper_2409_11902_b200 import synth
    N, C, H, k = 24, 512, 7, (4, 2)
    d = D(N, C, C, H, H, 3, 3, (1, 1), (1, 1), "bf16", "nhwc")
    full = ac.ac_workspace_bytes_rect(d, *k)
    assert (full - 256) % (4 * C * C * 9) == N * H * H * C * 2      # K-slices of dW, then the inflated map
    x = synth.activation(6, (N, C, H, H), "bf16")
    z = synth.to_storage(oracle.pool(synth.to_f64(x), k), "bf16")
    dy = synth.grad_output(6, (N, C, H, H), "bf16")
    zd, dyd = synth.to_layout(z, "nhwc").cuda(), synth.to_layout(dy, "nhwc").cuda()
    idx = stratified_entries(d, 256, seed=6)
    want = oracle.wgrad_compressed_entries(synth.to_f64(z), synth.to_f64(dy), H, H, 3, 3, (1, 1), (1, 1), k, idx)
    ws = torch.empty(full, dtype=torch.uint8, device="cuda")
    dw = torch.full(d.dw_shape, float("nan"), device="cuda")
    ac.ac_conv2d_wgrad_compressed_rect(d, k[0], k[1], zd, dyd, dw, ws, full)
    assert ac.ac_workspace_status(ws)[0] == 0
    got = dw.double().cpu().numpy().transpose(0, 3, 1, 2)
    assert np.isfinite(got).all()
    assert_dw_close(got[idx[:, 0], idx[:, 1], idx[:, 2], idx[:, 3]], want, "bf16")
