"""Pins for the CPU checker: each expected value below comes from the paper,
from a closed form, from an invariant, from a library routine on a special
case, or from brute-force Python loops written here -- never from the checker
itself. A dropped term, a wrong sign or index, or a transposed operand in
oracle/ac_oracle.c fails at least one of them."""
import itertools
import os

import numpy as np
import pytest
import torch

import oracle

RNG = np.random.default_rng(1234)


# ---------------------------------------------------------------- brute force

def brute_pool(x, k):
    """Independent definition: explicit element lists per block, then mean."""
    N, C, H, W = x.shape
    Hp, Wp = -(-H // k), -(-W // k)
    z = np.zeros((N, C, Hp, Wp))
    for n, c in itertools.product(range(N), range(C)):
        for p in range(Hp):
            for q in range(Wp):
                vals = [x[n, c, h, w]
                        for w in range(W) for h in range(H)
                        if h // k == p and w // k == q]
                z[n, c, p, q] = sum(vals) / len(vals)
    return z


def brute_wgrad(x, dy, R, S, stride, pad):
    """dW by scattering every (input pixel, output pixel) pair whose offset is
    a filter tap -- a different loop nest from the checker's gather."""
    N, Ci, H, W = x.shape
    _, Co, Ho, Wo = dy.shape
    dw = np.zeros((Co, Ci, R, S))
    for n in range(N):
        for h in range(H):
            for w in range(W):
                for ho in range(Ho):
                    r = h - (ho * stride[0] - pad[0])
                    if not 0 <= r < R:
                        continue
                    for wo in range(Wo):
                        s = w - (wo * stride[1] - pad[1])
                        if not 0 <= s < S:
                            continue
                        dw[:, :, r, s] += np.outer(dy[n, :, ho, wo], x[n, :, h, w])
    return dw


def brute_inflate(z, H, W, k):
    return np.repeat(np.repeat(z, k, axis=2), k, axis=3)[:, :, :H, :W]


# ----------------------------------------------------------------------- pool

@pytest.mark.parametrize("H,W", [(4, 4), (5, 6), (7, 8), (8, 7), (1, 3)])
@pytest.mark.parametrize("k", [1, 2, 3, 4])
def test_pool_matches_brute_force(H, W, k):
    x = RNG.standard_normal((2, 3, H, W))
    np.testing.assert_allclose(oracle.pool(x, k), brute_pool(x, k), rtol=1e-14, atol=1e-15)


def test_pool_figure_structure():
    """Figure of Section 4: a 4x4 map with 2x2 pooling gives mu_pq = mean of
    the 2x2 block whose top-left element is X[2p, 2q]."""
    x = np.arange(16, dtype=np.float64).reshape(1, 1, 4, 4) ** 2
    z = oracle.pool(x, 2)
    X = x[0, 0]
    assert z.shape == (1, 1, 2, 2)
    assert z[0, 0, 0, 0] == (X[0, 0] + X[0, 1] + X[1, 0] + X[1, 1]) / 4
    assert z[0, 0, 0, 1] == (X[0, 2] + X[0, 3] + X[1, 2] + X[1, 3]) / 4
    assert z[0, 0, 1, 0] == (X[2, 0] + X[2, 1] + X[3, 0] + X[3, 1]) / 4
    assert z[0, 0, 1, 1] == (X[2, 2] + X[2, 3] + X[3, 2] + X[3, 3]) / 4


def test_pool_k1_is_identity_and_constant_is_fixed():
    x = RNG.standard_normal((2, 2, 5, 7))
    assert np.array_equal(oracle.pool(x, 1), x)
    c = np.full((1, 2, 7, 5), 0.3)
    for k in (2, 3, 4, 8):
        np.testing.assert_allclose(oracle.pool(c, k), 0.3, rtol=1e-15)


@pytest.mark.parametrize("H,W,k", [(8, 8, 2), (8, 12, 4), (7, 9, 2), (14, 14, 4)])
def test_block_means_are_preserved(H, W, k):
    """pool(inflate(pool(X))) == pool(X): bit-exact for k=2 when k divides H and
    W (z+z, 3z and 4z round back onto 4z), else to a few ulps (k*k roundings)."""
    x = RNG.standard_normal((2, 3, H, W))
    z = oracle.pool(x, k)
    z2 = oracle.pool(oracle.inflate(z, H, W, k), k)
    if H % k == 0 and W % k == 0 and k in (1, 2):
        assert np.array_equal(z2, z)
    else:
        np.testing.assert_allclose(z2, z, rtol=2e-15, atol=0)


def test_pool_is_linear():
    x1 = RNG.standard_normal((1, 2, 7, 6))
    x2 = RNG.standard_normal((1, 2, 7, 6))
    lhs = oracle.pool(2.0 * x1 - 0.5 * x2, 2)
    rhs = 2.0 * oracle.pool(x1, 2) - 0.5 * oracle.pool(x2, 2)
    np.testing.assert_allclose(lhs, rhs, rtol=1e-13, atol=1e-15)


@pytest.mark.parametrize("k", [2, 4])
def test_pool_equals_library_avgpool_when_divisible(k):
    x = RNG.standard_normal((2, 3, 8, 12))
    ref = torch.nn.functional.avg_pool2d(torch.from_numpy(x), k, k).numpy()
    np.testing.assert_allclose(oracle.pool(x, k), ref, rtol=1e-14, atol=1e-16)


@pytest.mark.parametrize("H,W,k", [(5, 7, 2), (8, 8, 4), (7, 7, 3)])
def test_inflate_matches_repeat(H, W, k):
    z = RNG.standard_normal((2, 2, -(-H // k), -(-W // k)))
    assert np.array_equal(oracle.inflate(z, H, W, k), brute_inflate(z, H, W, k))


def test_relu():
    a = RNG.standard_normal(100)
    assert np.array_equal(oracle.relu(a), np.maximum(a, 0.0))


def test_relu_backward_is_the_derivative_of_relu():
    """Central differences of L = sum(relu(A) * dY) in A (exact away from 0: L is piecewise linear), the value 0
    at A = 0, and equality with the sign mask applied to dY."""
    a = RNG.standard_normal(200)
    a[::17] = 0.0
    dy = RNG.standard_normal(200)
    got = oracle.relu_backward(a, dy)
    h = 1e-3
    away = np.abs(a) > 2 * h
    for i in np.flatnonzero(away)[:60]:
        ap, am = a.copy(), a.copy()
        ap[i] += h
        am[i] -= h
        fd = (np.sum(oracle.relu(ap) * dy) - np.sum(oracle.relu(am) * dy)) / (2 * h)
        assert abs(fd - got[i]) <= 1e-9 * max(1.0, abs(dy[i]))
    assert not got[a == 0].any() and not got[a < 0].any()
    bits = np.unpackbits(np.packbits(a > 0, bitorder="little"), bitorder="little")[:a.size].astype(bool)
    assert np.array_equal(got, np.where(bits, dy, 0.0))


# ---------------------------------------------------------------------- wgrad

CONV_CASES = [
    # H, W, R, S, stride, pad
    (6, 6, 3, 3, (1, 1), (1, 1)),
    (7, 5, 3, 3, (1, 1), (1, 1)),
    (8, 8, 3, 3, (2, 2), (1, 1)),
    (7, 7, 1, 1, (1, 1), (0, 0)),
    (8, 6, 1, 1, (2, 2), (0, 0)),
    (9, 9, 5, 3, (2, 1), (2, 0)),
    (7, 7, 3, 3, (2, 2), (1, 1)),
]


@pytest.mark.parametrize("H,W,R,S,stride,pad", CONV_CASES)
def test_dense_wgrad_matches_brute_force_and_autograd(H, W, R, S, stride, pad):
    N, Ci, Co = 2, 3, 4
    Ho, Wo = oracle.out_hw(H, W, R, S, stride, pad)
    x = RNG.standard_normal((N, Ci, H, W))
    dy = RNG.standard_normal((N, Co, Ho, Wo))
    got = oracle.wgrad_dense(x, dy, R, S, stride, pad)
    np.testing.assert_allclose(got, brute_wgrad(x, dy, R, S, stride, pad),
                               rtol=1e-12, atol=1e-13)
    # textbook identity: dW = d/dW <conv(X, W), dY> (loss linear in W)
    w = torch.zeros(Co, Ci, R, S, dtype=torch.float64, requires_grad=True)
    y = torch.nn.functional.conv2d(torch.from_numpy(x), w, None, stride, pad)
    (y * torch.from_numpy(dy)).sum().backward()
    np.testing.assert_allclose(got, w.grad.numpy(), rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("H,W,R,S,stride,pad", CONV_CASES)
def test_k1_reproduces_uncompressed_dw_exactly(H, W, R, S, stride, pad):
    N, Ci, Co = 2, 3, 2
    Ho, Wo = oracle.out_hw(H, W, R, S, stride, pad)
    x = RNG.standard_normal((N, Ci, H, W))
    dy = RNG.standard_normal((N, Co, Ho, Wo))
    z = oracle.pool(x, 1)
    assert np.array_equal(oracle.wgrad_compressed(z, dy, H, W, R, S, stride, pad, 1),
                          oracle.wgrad_dense(x, dy, R, S, stride, pad))


@pytest.mark.parametrize("H,W,R,S,stride,pad", CONV_CASES)
@pytest.mark.parametrize("k", [2, 3, 4])
def test_compressed_wgrad_matches_brute_force(H, W, R, S, stride, pad, k):
    """Independent path: numpy repeat for the inflation, scatter loop for dW."""
    N, Ci, Co = 2, 2, 3
    Ho, Wo = oracle.out_hw(H, W, R, S, stride, pad)
    z = RNG.standard_normal((N, Ci, -(-H // k), -(-W // k)))
    dy = RNG.standard_normal((N, Co, Ho, Wo))
    want = brute_wgrad(brute_inflate(z, H, W, k), dy, R, S, stride, pad)
    got = oracle.wgrad_compressed(z, dy, H, W, R, S, stride, pad, k)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("H,W,k", [(8, 8, 2), (8, 8, 4), (7, 9, 2), (6, 6, 3)])
@pytest.mark.parametrize("stride", [(1, 1), (2, 2)])
def test_block_constant_input_loses_nothing(H, W, k, stride):
    """X constant inside every k x k block => compressed dW == uncompressed dW."""
    N, Ci, Co, R, S, pad = 2, 2, 3, 3, 3, (1, 1)
    Ho, Wo = oracle.out_hw(H, W, R, S, stride, pad)
    zsrc = RNG.integers(-8, 9, size=(N, Ci, -(-H // k), -(-W // k))).astype(np.float64)
    x = brute_inflate(zsrc, H, W, k)
    dy = RNG.standard_normal((N, Co, Ho, Wo))
    z = oracle.pool(x, k)
    assert np.array_equal(z, zsrc)       # small integers: block means are exact
    assert np.array_equal(oracle.wgrad_compressed(z, dy, H, W, R, S, stride, pad, k),
                          oracle.wgrad_dense(x, dy, R, S, stride, pad))


@pytest.mark.parametrize("H,k,stride", [(8, 2, 1), (7, 2, 1), (8, 4, 1), (8, 2, 2), (7, 4, 2)])
def test_pooled_dy_identity(H, k, stride):
    """Independent algorithm: dW[co,ci,r,s] = sum_{n,p,q} Z[n,ci,p,q] * D_rs[n,co,p,q],
    D_rs = sum of dY over the outputs whose tap (r,s) lands in block (p,q)."""
    N, Ci, Co, R, S, pad = 2, 3, 2, 3, 3, 1
    W = H
    Ho, Wo = oracle.out_hw(H, W, R, S, (stride, stride), (pad, pad))
    z = RNG.standard_normal((N, Ci, -(-H // k), -(-W // k)))
    dy = RNG.standard_normal((N, Co, Ho, Wo))
    want = np.zeros((Co, Ci, R, S))
    for r in range(R):
        for s in range(S):
            D = np.zeros((N, Co) + z.shape[2:])
            for ho in range(Ho):
                h = ho * stride - pad + r
                if not 0 <= h < H:
                    continue
                for wo in range(Wo):
                    w = wo * stride - pad + s
                    if 0 <= w < W:
                        D[:, :, h // k, w // k] += dy[:, :, ho, wo]
            want[:, :, r, s] = np.einsum("nipq,nopq->oi", z, D)
    got = oracle.wgrad_compressed(z, dy, H, W, R, S, (stride, stride), (pad, pad), k)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)


def test_tap_collapse_stride2_k2():
    """3x3, stride 2, pad 1, k=2, even H: taps 1 and 2 read the same Z element."""
    N, Ci, Co, H = 2, 2, 3, 8
    z = RNG.standard_normal((N, Ci, 4, 4))
    dy = RNG.standard_normal((N, Co, 4, 4))
    dw = oracle.wgrad_compressed(z, dy, H, H, 3, 3, (2, 2), (1, 1), 2)
    assert np.array_equal(dw[:, :, 1, :], dw[:, :, 2, :])
    assert np.array_equal(dw[:, :, :, 1], dw[:, :, :, 2])
    assert not np.array_equal(dw[:, :, 0, :], dw[:, :, 1, :])


@pytest.mark.parametrize("R,stride,pad,k,H", [(7, 2, 3, 2, 12), (5, 4, 2, 2, 16), (3, 4, 1, 4, 16), (7, 2, 3, 2, 11)])
def test_strides_that_are_multiples_of_k_read_one_shift_per_tap(R, stride, pad, k, H):
    """When the stride is a multiple of k and k | H, output ho reads Z row ho*stride/k + floor((r - pad)/k)
    through tap r, for every ho: dW[..., r, s] is the plain correlation of Z, shifted by that row and
    column, with dY (written here as its own loop nest), and taps with equal shifts are equal. With a
    partial last block (k does not divide H) the equality of such taps breaks at the padding edge."""
    N, Ci, Co = 2, 2, 3
    Hp = -(-H // k)
    Ho = (H + 2 * pad - R) // stride + 1
    z = RNG.standard_normal((N, Ci, Hp, Hp))
    dy = RNG.standard_normal((N, Co, Ho, Ho))
    dw = oracle.wgrad_compressed(z, dy, H, H, R, R, (stride, stride), (pad, pad), k)
    shift = [(r - pad) // k for r in range(R)]           # Python's // floors
    if H % k:
        r0, r1 = R - 2, R - 1                             # same shift, but r1 reaches the padding row inside the block
        assert shift[r0] == shift[r1] and not np.allclose(dw[:, :, r1, :], dw[:, :, r0, :])
        return
    m = stride // k
    zpad = np.zeros((N, Ci, Hp + 2 * R + m * Ho, Hp + 2 * R + m * Ho))
    zpad[:, :, R:R + Hp, R:R + Hp] = z
    for r in range(R):
        for s_ in range(R):
            win = zpad[:, :, R + shift[r]:R + shift[r] + m * Ho:m, R + shift[s_]:R + shift[s_] + m * Ho:m]
            want = np.einsum("nipq,nopq->oi", win, dy)
            np.testing.assert_allclose(dw[:, :, r, s_], want, rtol=1e-12, atol=1e-13)
    for r in range(1, R):
        if shift[r] == shift[r - 1]:
            assert np.array_equal(dw[:, :, r, :], dw[:, :, r - 1, :])
            assert np.array_equal(dw[:, :, :, r], dw[:, :, :, r - 1])


@pytest.mark.parametrize("k", [2, 4])
def test_pointwise_conv_closed_form(k):
    """1x1, stride 1, k | H: dW[co,ci] = k^2 * sum Z * pool_k(dY)."""
    N, Ci, Co, H = 2, 3, 2, 8
    z = RNG.standard_normal((N, Ci, H // k, H // k))
    dy = RNG.standard_normal((N, Co, H, H))
    pdy = dy.reshape(N, Co, H // k, k, H // k, k).mean(axis=(3, 5))
    want = k * k * np.einsum("nipq,nopq->oi", z, pdy)
    got = oracle.wgrad_compressed(z, dy, H, H, 1, 1, (1, 1), (0, 0), k)[:, :, 0, 0]
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)


def test_bilinear_zero_and_impulse():
    N, Ci, Co, H, k = 1, 2, 2, 6, 2
    args = (H, H, 3, 3, (1, 1), (1, 1), k)
    z1, z2 = RNG.standard_normal((2, N, Ci, 3, 3))
    dy = RNG.standard_normal((N, Co, H, H))
    f = lambda z, g: oracle.wgrad_compressed(z, g, *args)
    np.testing.assert_allclose(f(2 * z1 + z2, dy), 2 * f(z1, dy) + f(z2, dy), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(f(z1, -3 * dy), -3 * f(z1, dy), rtol=1e-12, atol=1e-13)
    assert not f(z1, np.zeros_like(dy)).any()
    # one nonzero block mean and one nonzero output gradient
    z = np.zeros((N, Ci, 3, 3)); z[0, 1, 1, 2] = 5.0          # covers x rows 2..3, cols 4..5
    g = np.zeros((N, Co, H, H)); g[0, 0, 3, 4] = 7.0           # output (3,4): taps read x (2..4, 3..5)
    dw = f(z, g)
    want = np.zeros_like(dw)
    # tap (r,s) reads x (3-1+r, 4-1+s); inside the block for r in {0,1}, s in {1,2}
    for r in (0, 1):
        for s in (1, 2):
            want[0, 1, r, s] = 35.0
    assert np.array_equal(dw, want)


def test_border_only_input_exercises_every_padding_tap():
    """An inflated input that is nonzero only on the border, all-ones dY."""
    N, Ci, Co, H, k = 1, 1, 1, 4, 1
    x = np.ones((1, 1, H, H)); x[:, :, 1:-1, 1:-1] = 0.0
    dy = np.ones((1, 1, H, H))
    dw = oracle.wgrad_compressed(x, dy, H, H, 3, 3, (1, 1), (1, 1), k)[0, 0]
    # tap (r,s) sums x over the window shifted by (r-1, s-1), clipped to the map
    want = np.array([[sum(x[0, 0, h, w] for h in range(H) for w in range(H)
                          if 0 <= h - (r - 1) < H and 0 <= w - (s - 1) < H)
                      for s in range(3)] for r in range(3)])
    assert np.array_equal(dw, want)
    assert dw[1, 1] == 12 and dw[0, 0] == 5     # 12 border cells; corner tap sees 5


def test_sampled_entries_equal_full_tensor():
    N, Ci, Co, H, W, k = 2, 3, 4, 7, 9, 2
    for (R, S, stride, pad) in [(3, 3, (1, 1), (1, 1)), (3, 3, (2, 2), (1, 1)), (1, 1, (1, 1), (0, 0))]:
        Ho, Wo = oracle.out_hw(H, W, R, S, stride, pad)
        z = RNG.standard_normal((N, Ci, 4, 5))
        dy = RNG.standard_normal((N, Co, Ho, Wo))
        idx = np.array(list(itertools.product(range(Co), range(Ci), range(R), range(S))))
        got = oracle.wgrad_compressed_entries(z, dy, H, W, R, S, stride, pad, k, idx)
        want = brute_wgrad(brute_inflate(z, H, W, k), dy, R, S, stride, pad)
        np.testing.assert_allclose(got.reshape(want.shape), want, rtol=1e-12, atol=1e-13)


def test_cosine_similarity_equation():
    a = np.array([3.0, 4.0, 0.0]); b = np.array([4.0, 3.0, 0.0])
    assert oracle.cosine_similarity(a, b) == pytest.approx(24.0 / 25.0, rel=1e-15)
    assert oracle.cosine_similarity(a, -a) == pytest.approx(-1.0, rel=1e-15)


# ------------------------------------------------------- Table 1 byte counts

RESNET18_INPUT_SHAPES = {   # (C, H) of each listed conv's input at 224x224 images
    "conv1": (3, 224),
    "layer1.0.conv1": (64, 56), "layer1.0.conv2": (64, 56),
    "layer1.1.conv1": (64, 56), "layer1.1.conv2": (64, 56),
    "layer2.0.conv1": (64, 56), "layer2.0.conv2": (128, 28),
    "layer2.0.downsample.0": (64, 56),
    "layer2.1.conv1": (128, 28), "layer2.1.conv2": (128, 28),
    "layer3.0.conv1": (128, 28), "layer3.0.conv2": (256, 14),
    "layer3.0.downsample.0": (128, 28),
    "layer3.1.conv1": (256, 14), "layer3.1.conv2": (256, 14),
    "layer4.0.conv1": (256, 14), "layer4.0.conv2": (512, 7),
}


def _table1():
    path = os.path.join(os.path.dirname(__file__), "golden", "table1_resnet18_mib.txt")
    rows = []
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        name, x, z2, z4 = line.split()
        rows.append((name, float(x), float(z2), float(z4)))
    return rows


def test_table1_bytes_reproduced():
    MiB = float(1 << 20)
    sums = np.zeros(3)
    for name, x, z2, z4 in _table1():
        if name == "Sum":
            # printed per-row values are rounded; compare the sums of exact values
            assert abs(sums[0] / MiB - x) < 0.006
            assert abs(sums[1] / MiB - z2) < 0.006
            assert abs(sums[2] / MiB - z4) < 0.006
            continue
        C, H = RESNET18_INPUT_SHAPES[name]
        bx = oracle.activation_bytes(32, C, H, H, 4)
        b2 = oracle.compressed_bytes(32, C, H, H, 2, 4, "floor")
        b4 = oracle.compressed_bytes(32, C, H, H, 4, 4, "floor")
        assert abs(bx / MiB - x) < 0.006, name
        assert abs(b2 / MiB - z2) < 0.006, name
        assert abs(b4 / MiB - z4) < 0.006, name
        sums += (bx, b2, b4)
    # Section 5.3: savings of roughly 191 and 239 MiB; 29 % and 36 % of ~670 MiB
    assert round((sums[0] - sums[1]) / MiB) == 191
    assert round((sums[0] - sums[2]) / MiB) == 239
    assert round(100 * (sums[0] - sums[1]) / MiB / 670) in (28, 29)
    assert round(100 * (sums[0] - sums[2]) / MiB / 670) == 36


def test_ceil_accounting_keeps_partial_blocks():
    assert oracle.compressed_bytes(1, 1, 7, 7, 2, 4, "ceil") == 16 * 4
    assert oracle.compressed_bytes(1, 1, 7, 7, 2, 4, "floor") == 9 * 4
    assert oracle.pool(np.zeros((1, 1, 7, 7)), 2).shape == (1, 1, 4, 4)


def test_resnet50_saved_activation_bytes():
    """Byte accounting for a full ResNet-50 (bottleneck blocks, stride on the 3x3, 224x224
    images) at batch 256 in bf16, k = 2. Counted per convolution (53 convs, the way the
    paper's Table 1 lists layers) and per distinct tensor (a block input that feeds both
    conv1 and the downsample conv is stored once)."""
    per_conv, unique = [(3, 224)], [(3, 224)]                 # stem
    # (stage input channels, bottleneck width, output channels, map size at the stage input, blocks, stride)
    for cin, width, cout, H, blocks, stride in [(64, 64, 256, 56, 3, 1), (256, 128, 512, 56, 4, 2),
                                                (512, 256, 1024, 28, 6, 2), (1024, 512, 2048, 14, 3, 2)]:
        for b in range(blocks):
            h_in = H if b == 0 else H // stride
            c_in = cin if b == 0 else cout
            convs = [(c_in, h_in),                                        # conv1 (1x1)
                     (width, h_in),                                       # conv2 (3x3, carries the stride)
                     (width, h_in // (stride if b == 0 else 1))]          # conv3 (1x1)
            per_conv += convs + ([(c_in, h_in)] if b == 0 else [])        # + downsample conv of the first block
            unique += convs
    MiB = float(1 << 20)
    tot = lambda lst, f: sum(f(c, h) for c, h in lst) / MiB
    xb = lambda c, h: oracle.activation_bytes(256, c, h, h, 2)
    zb = lambda c, h: oracle.compressed_bytes(256, c, h, h, 2, 2, "ceil")
    assert len(per_conv) == 53 and len(unique) == 49
    assert round(tot(per_conv, xb)) == 5206 and round(tot(per_conv, zb)) == 1314
    assert round(tot(unique, xb)) == 4422 and round(tot(unique, zb)) == 1118
    assert 0.74 < 1 - tot(unique, zb) / tot(unique, xb) < 0.75
