"""Pins for the checker's non-uniform pooling blocks (k_h x k_w; Section 6 of the paper names
non-uniform pooling shapes as future work, Section 4's definitions carry over). As for the square
functions, no expected value below comes from the checker itself: brute-force loops, a library
routine on the divisible case, np.repeat, and the scatter-form weight gradient of test_oracle_pins.
A copy of the checker with k_h and k_w exchanged, or a partial block divided by k_h*k_w, fails."""
import ctypes
import itertools
import os
import subprocess

import numpy as np
import pytest
import torch

import oracle
import test_oracle_pins as pins

RNG = np.random.default_rng(4321)
KS = [(2, 4), (4, 2), (1, 2), (3, 2), (2, 1)]


def brute_pool_rect(x, kh, kw):
    N, C, H, W = x.shape
    Hp, Wp = -(-H // kh), -(-W // kw)
    z = np.zeros((N, C, Hp, Wp))
    for n, c, p, q in itertools.product(range(N), range(C), range(Hp), range(Wp)):
        vals = [x[n, c, h, w] for w in range(W) for h in range(H) if h // kh == p and w // kw == q]
        z[n, c, p, q] = sum(vals) / len(vals)
    return z


def repeat_inflate(z, H, W, kh, kw):
    return np.repeat(np.repeat(z, kh, axis=2), kw, axis=3)[:, :, :H, :W]


@pytest.mark.parametrize("H,W", [(4, 8), (5, 6), (7, 9), (1, 3)])
@pytest.mark.parametrize("k", KS)
def test_rect_pool_matches_brute_force(H, W, k):
    x = RNG.standard_normal((2, 2, H, W))
    z = oracle.pool(x, k)
    assert z.shape[2:] == oracle.pooled_hw(H, W, k) == (-(-H // k[0]), -(-W // k[1]))
    np.testing.assert_allclose(z, brute_pool_rect(x, *k), rtol=1e-14, atol=1e-15)


@pytest.mark.parametrize("k", [(2, 4), (4, 2), (1, 2)])
def test_rect_pool_equals_library_avgpool_when_divisible(k):
    x = RNG.standard_normal((2, 3, 8, 12))
    ref = torch.nn.functional.avg_pool2d(torch.from_numpy(x), k, k).numpy()
    np.testing.assert_allclose(oracle.pool(x, k), ref, rtol=1e-14, atol=1e-16)


@pytest.mark.parametrize("H,W,k", [(5, 7, (2, 3)), (8, 8, (4, 2)), (7, 6, (1, 4))])
def test_rect_inflate_matches_repeat(H, W, k):
    z = RNG.standard_normal((2, 2) + oracle.pooled_hw(H, W, k))
    assert np.array_equal(oracle.inflate(z, H, W, k), repeat_inflate(z, H, W, *k))


def test_square_blocks_give_the_square_functions():
    x = RNG.standard_normal((2, 3, 7, 9))
    dy = RNG.standard_normal((2, 4, 7, 9))
    for k in (1, 2, 3):
        assert np.array_equal(oracle.pool(x, (k, k)), oracle.pool(x, k))
        z = oracle.pool(x, k)
        assert np.array_equal(oracle.inflate(z, 7, 9, (k, k)), oracle.inflate(z, 7, 9, k))
        assert np.array_equal(oracle.wgrad_compressed(z, dy, 7, 9, 3, 3, (1, 1), (1, 1), (k, k)),
                              oracle.wgrad_compressed(z, dy, 7, 9, 3, 3, (1, 1), (1, 1), k))


RECT_CONV = [  # N, Ci, Co, H, W, R, S, stride, pad, (kh, kw)
    (2, 2, 3, 6, 8, 3, 3, (1, 1), (1, 1), (2, 4)),
    (1, 3, 2, 7, 7, 3, 3, (2, 2), (1, 1), (2, 1)),
    (2, 2, 2, 5, 9, 1, 1, (1, 1), (0, 0), (1, 2)),
    (1, 2, 2, 8, 6, 3, 5, (1, 2), (1, 2), (4, 2)),
]


@pytest.mark.parametrize("case", RECT_CONV)
def test_rect_compressed_wgrad_matches_brute_force(case):
    N, Ci, Co, H, W, R, S, stride, pad, k = case
    z = RNG.standard_normal((N, Ci) + oracle.pooled_hw(H, W, k))
    Ho, Wo = oracle.out_hw(H, W, R, S, stride, pad)
    dy = RNG.standard_normal((N, Co, Ho, Wo))
    want = pins.brute_wgrad(repeat_inflate(z, H, W, *k), dy, R, S, stride, pad)
    got = oracle.wgrad_compressed(z, dy, H, W, R, S, stride, pad, k)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)
    idx = np.array(list(itertools.product(range(Co), range(Ci), range(R), range(S))), dtype=np.int64)
    ent = oracle.wgrad_compressed_entries(z, dy, H, W, R, S, stride, pad, k, idx)
    np.testing.assert_allclose(ent.reshape(Co, Ci, R, S), want, rtol=1e-12, atol=1e-13)


def test_rect_block_constant_input_gives_the_uncompressed_gradient():
    """X constant on every k_h x k_w block: inflate(pool(X)) is X, so the compressed dW is the dense one."""
    k = (2, 4)
    base = RNG.standard_normal((2, 3, 3, 2))
    x = repeat_inflate(base, 6, 8, *k)
    dy = RNG.standard_normal((2, 2, 6, 8))
    z = oracle.pool(x, k)
    np.testing.assert_allclose(z, base, rtol=1e-15)
    np.testing.assert_allclose(oracle.wgrad_compressed(z, dy, 6, 8, 3, 3, (1, 1), (1, 1), k),
                               oracle.wgrad_dense(x, dy, 3, 3, (1, 1), (1, 1)), rtol=1e-12, atol=1e-13)


SRC = open(os.path.join(os.path.dirname(oracle.__file__), "ac_oracle.c")).read()
MUTANTS = {
    "partial_block_divided_by_full_size": ("zp[p * Wp + q] = sum / (double)count;\n            }\n        }\n    }\n}\n\n/* Xt[n,c,h,w] = Z[n,c,h/kh,w/kw]. */",
                                           "zp[p * Wp + q] = sum / (double)(kh * kw);\n            }\n        }\n    }\n}\n\n/* Xt[n,c,h,w] = Z[n,c,h/kh,w/kw]. */"),
    "pool_block_sizes_exchanged": ("for (int64_t h = p * kh; h < (p + 1) * kh && h < H; ++h) {\n                    for (int64_t w = q * kw; w < (q + 1) * kw && w < W; ++w) {",
                                   "for (int64_t h = p * kw; h < (p + 1) * kw && h < H; ++h) {\n                    for (int64_t w = q * kh; w < (q + 1) * kh && w < W; ++w) {"),
    "inflate_block_sizes_exchanged": ("xp[h * W + w] = zp[(h / kh) * Wp + (w / kw)];",
                                      "xp[h * W + w] = zp[(h / kw) * Wp + (w / kh)];"),
    "entries_block_sizes_exchanged": ("acc += gp[ho * Wo + wo] * zp[(h / kh) * Wp + (w / kw)];",
                                      "acc += gp[ho * Wo + wo] * zp[(h / kw) * Wp + (w / kh)];"),
}


def _calls():
    calls = [lambda H=H, W=W, k=k: test_rect_pool_matches_brute_force(H, W, k)
             for H, W in [(4, 8), (5, 6), (7, 9)] for k in KS[:3]]
    calls += [lambda c=c: test_rect_compressed_wgrad_matches_brute_force(c) for c in RECT_CONV]
    calls.append(lambda: test_rect_inflate_matches_repeat(5, 7, (2, 3)))
    return calls


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_planted_mistake_in_the_rect_functions_trips_a_pin(name, tmp_path, monkeypatch):
    old, new = MUTANTS[name]
    assert SRC.count(old) == 1, "mutation target not found: keep this test in step with ac_oracle.c"
    c = tmp_path / "mutant.c"
    c.write_text(SRC.replace(old, new, 1))
    so = tmp_path / "libmutant.so"
    subprocess.run(["gcc", "-O1", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", str(so), str(c)], check=True)
    lib = ctypes.CDLL(str(so))
    lib.oracle_num_threads.restype = ctypes.c_int
    lib.oracle_wgrad_compressed.restype = ctypes.c_int
    lib.oracle_wgrad_compressed_rect.restype = ctypes.c_int
    oracle._load()
    monkeypatch.setattr(oracle, "_lib", lib)
    tripped = 0
    for call in _calls():
        try:
            call()
        except AssertionError:
            tripped += 1
    assert tripped > 0, f"no pin noticed the planted mistake '{name}'"
