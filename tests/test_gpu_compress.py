"""GPU parity of ac_compress against the CPU checker (element by element)."""
import pytest

import __graft_entry__ as entry
from helpers import TOL_Z, run_compress, run_compress_mask

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    entry.build()


def desc(N, C, H, W, k, dtype, layout):
    import paper_2409_11902_b200 as ac
    return ac.ConvDesc(N, C, 1, H, W, 1, 1, (1, 1), (0, 0), k, dtype, layout)


SHAPES = [
    # N, C, H, W -- spans several 256-thread blocks, with ragged tails
    (8, 64, 32, 32),     # config 1
    (3, 64, 56, 56),     # ResNet 56x56 map
    (2, 128, 28, 28),
    (2, 256, 14, 14),
    (2, 512, 7, 7),      # odd size: partial blocks on both edges
    (2, 24, 9, 15),      # odd H and W, C a multiple of 8
    (1, 3, 17, 23),      # stem-like: C not a multiple of the vector width
    (1, 5, 1, 1),        # degenerate map
    # NHWC with C not a multiple of the vector width but W * C one
    (2, 3, 32, 32),
    (3, 3, 15, 24),      # odd H: a partial last row of blocks
    (2, 4, 9, 14),       # partial blocks in both directions at k = 4
    (1, 12, 7, 10),
    (2, 3, 224, 224),    # the ResNet stem's input
]


@pytest.mark.parametrize("layout", ["nchw", "nhwc"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("k", [1, 2, 3, 4, 8])
@pytest.mark.parametrize("shape", SHAPES)
def test_compress_matches_checker(shape, k, dtype, layout):
    err, _, _ = run_compress(desc(*shape, k, dtype, layout))
    assert err <= TOL_Z[dtype], err


@pytest.mark.parametrize("layout", ["nchw", "nhwc"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("k", [1, 2, 4, 8])
@pytest.mark.parametrize("inplace", [False, True])
@pytest.mark.parametrize("shape", [(3, 64, 56, 56), (2, 512, 7, 7), (1, 3, 17, 23), (2, 32, 16, 64),
                                   (2, 3, 32, 32), (3, 3, 15, 24), (2, 4, 9, 14)])
def test_fused_relu_compress(shape, inplace, k, dtype, layout):
    err, _, _ = run_compress(desc(*shape, k, dtype, layout), fused_relu=True, inplace=inplace)
    assert err <= TOL_Z[dtype], err


def mask_form_exists(shape, k, layout):
    """The documented domain of ac_compress_relu_mask."""
    N, C, H, W = shape
    if k == 1:
        return (N * C * H * W) % 8 == 0
    if layout == "nhwc":
        return C % 8 == 0
    return W % 8 == 0 and W % k == 0


@pytest.mark.parametrize("layout", ["nchw", "nhwc"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("k", [1, 2, 3, 4, 8])
@pytest.mark.parametrize("shape", [(3, 64, 56, 56), (2, 512, 7, 7), (2, 24, 9, 15), (2, 32, 16, 64),
                                   (2, 16, 9, 16), (1, 3, 16, 24), (1, 3, 17, 23), (5, 8, 3, 40)])
def test_fused_relu_compress_sign_mask(shape, k, dtype, layout):
    import paper_2409_11902_b200 as ac
    d = desc(*shape, k, dtype, layout)
    if k != 3 and mask_form_exists(shape, k, layout):
        for store_y in (None, "own", "inplace"):
            err = run_compress_mask(d, store_y=store_y)
            assert err <= TOL_Z[dtype], (store_y, err)
    else:
        with pytest.raises(ac.AcError) as e:
            run_compress_mask(d)
        assert e.value.status == ac.api.AC_ERR_UNSUPPORTED


@pytest.mark.parametrize("layout", ["nchw", "nhwc"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", [(3, 64, 56, 56), (2, 512, 7, 7), (2, 32, 16, 64), (1, 8, 3, 5), (5, 8, 3, 40)])
def test_relu_backward_from_the_sign_mask(shape, dtype, layout):
    """ac_relu_mask_backward on the mask ac_compress_relu_mask wrote: bit for bit dY where A > 0, else 0 -- into a
    buffer of its own and in place."""
    import numpy as np
    import torch
    import oracle
    import paper_2409_11902_b200 as ac
    from helpers import canary_intact, padded_empty
    from paper_2409_11902_b200 import synth
    d = desc(*shape, 1, dtype, layout)
    a = synth.pre_activation(3, shape, dtype)
    dy = synth.grad_output(3, shape, dtype)
    n_el = int(np.prod(shape))
    ad, dyd = synth.to_layout(a, layout).cuda(), synth.to_layout(dy, layout).cuda()
    z = torch.empty(d.z_shape, dtype=d.torch_dtype, device="cuda")
    mask = torch.empty((n_el + 7) // 8, dtype=torch.uint8, device="cuda")
    ac.ac_compress_relu_mask(d, ad, z, mask)
    want = oracle.relu_backward(synth.to_f64(a), synth.to_f64(dy))
    xbuf, dx, xspan = padded_empty(tuple(dyd.shape), d.torch_dtype, "cuda:0")
    dx.fill_(float("nan"))
    keep = dyd.clone()
    ac.ac_relu_mask_backward(d, mask, dyd, dx)
    torch.cuda.synchronize()
    assert canary_intact(xbuf, xspan) and torch.equal(dyd.view(torch.uint8), keep.view(torch.uint8))
    assert np.array_equal(synth.to_f64(synth.from_layout(dx.cpu(), layout)), want)
    ac.ac_relu_mask_backward(d, mask, dyd, dyd)      # in place
    torch.cuda.synchronize()
    assert np.array_equal(synth.to_f64(synth.from_layout(dyd.cpu(), layout)), want)


def test_relu_mask_backward_rejects_what_it_cannot_take():
    import torch
    import paper_2409_11902_b200 as ac
    d = desc(1, 3, 5, 5, 1, "bf16", "nhwc")      # 75 elements: not a multiple of 8
    t = torch.zeros(128, dtype=torch.bfloat16, device="cuda")
    m = torch.zeros(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(ac.AcError) as e:
        ac.ac_relu_mask_backward(d, m, t, t)
    assert e.value.status == ac.api.AC_ERR_UNSUPPORTED


def test_large_map_many_blocks():
    # 64 x 128 x 64 x 64 fp32 = 128 MiB: larger than L2, > 100k thread blocks
    for layout in ("nchw", "nhwc"):
        err, _, _ = run_compress(desc(64, 128, 64, 64, 2, "f32", layout))
        assert err <= TOL_Z["f32"], err


def test_runtime_errors_are_codes():
    import torch
    import paper_2409_11902_b200 as ac
    d = desc(1, 8, 8, 8, 2, "f32", "nchw")
    x = torch.zeros(d.x_shape, device="cuda")
    z = torch.zeros(d.z_shape, device="cuda")
    with pytest.raises(ac.AcError) as e:
        ac.ac_compress(d, x.data_ptr() + 4, z)
    assert e.value.status == ac.api.AC_ERR_MISALIGNED
