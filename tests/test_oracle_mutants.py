"""The pins must be able to fail: plausible mistakes are planted in copies of
the CPU checker (never in the CUDA path) and each one has to trip a pin."""
import ctypes
import os
import subprocess

import pytest

import oracle
import test_oracle_pins as pins

SRC = open(os.path.join(os.path.dirname(oracle.__file__), "ac_oracle.c")).read()

MUTANTS = {
    "divide_partial_blocks_by_k_squared": ("zp[p * Wp + q] = sum / (double)count;",
                                           "zp[p * Wp + q] = sum / (double)(k * k);"),
    "pool_blocks_offset_by_one": ("for (int64_t h = p * k; h < (p + 1) * k && h < H; ++h)",
                                  "for (int64_t h = p * k + 1; h < (p + 1) * k + 1 && h < H; ++h)"),
    "inflate_transposed": ("xp[h * W + w] = zp[(h / k) * Wp + (w / k)];",
                           "xp[h * W + w] = zp[(w / k) * Wp + (h / k)];"),
    "tap_rows_and_columns_swapped": ("const int64_t h = ho * sh - ph + r;\n            if (h < 0 || h >= H) continue;\n            for (int64_t wo = 0; wo < Wo; ++wo) {\n                const int64_t w = wo * sw - pw + s;\n                if (w < 0 || w >= W) continue;\n                acc += gp[ho * Wo + wo] * xp[h * W + w];",
                                     "const int64_t h = ho * sh - ph + s;\n            if (h < 0 || h >= H) continue;\n            for (int64_t wo = 0; wo < Wo; ++wo) {\n                const int64_t w = wo * sw - pw + r;\n                if (w < 0 || w >= W) continue;\n                acc += gp[ho * Wo + wo] * xp[h * W + w];"),
    "padding_sign_flipped": ("const int64_t w = wo * sw - pw + s;\n                if (w < 0 || w >= W) continue;\n                acc += gp[ho * Wo + wo] * xp[h * W + w];",
                             "const int64_t w = wo * sw + pw + s;\n                if (w < 0 || w >= W) continue;\n                acc += gp[ho * Wo + wo] * xp[h * W + w];"),
    "stride_ignored": ("const int64_t h = ho * sh - ph + r;\n            if (h < 0 || h >= H) continue;\n            for (int64_t wo = 0; wo < Wo; ++wo) {\n                const int64_t w = wo * sw - pw + s;\n                if (w < 0 || w >= W) continue;\n                acc += gp[ho * Wo + wo] * xp[h * W + w];",
                       "const int64_t h = ho - ph + r;\n            if (h < 0 || h >= H) continue;\n            for (int64_t wo = 0; wo < Wo; ++wo) {\n                const int64_t w = wo * sw - pw + s;\n                if (w < 0 || w >= W) continue;\n                acc += gp[ho * Wo + wo] * xp[h * W + w];"),
    "batch_term_dropped": ("for (int64_t n = 0; n < N; ++n) {\n        const double *xp = x + (n * Ci + ci) * H * W;",
                           "for (int64_t n = 0; n < 1; ++n) {\n        const double *xp = x + (n * Ci + ci) * H * W;"),
    "sampled_entries_forget_inflation": ("acc += gp[ho * Wo + wo] * zp[(h / k) * Wp + (w / k)];",
                                         "acc += gp[ho * Wo + wo] * zp[(h / k) * Wp + (w / k + 1) % Wp];"),
}


def _pin_calls():
    """A cross-section of the pins, with their parameters bound."""
    calls = []
    for H, W in [(4, 4), (5, 6), (7, 8)]:
        for k in (2, 3):
            calls.append(lambda H=H, W=W, k=k: pins.test_pool_matches_brute_force(H, W, k))
    calls.append(pins.test_pool_figure_structure)
    for c in pins.CONV_CASES:
        calls.append(lambda c=c: pins.test_dense_wgrad_matches_brute_force_and_autograd(*c))
        calls.append(lambda c=c: pins.test_compressed_wgrad_matches_brute_force(*c, 2))
    calls.append(lambda: pins.test_inflate_matches_repeat(5, 7, 2))
    calls.append(lambda: pins.test_pooled_dy_identity(7, 2, 1))
    calls.append(pins.test_sampled_entries_equal_full_tensor)
    calls.append(pins.test_bilinear_zero_and_impulse)
    return calls


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_planted_mistake_trips_a_pin(name, tmp_path, monkeypatch):
    old, new = MUTANTS[name]
    assert SRC.count(old) >= 1, "mutation target not found: keep this test in step with ac_oracle.c"
    c = tmp_path / "mutant.c"
    c.write_text(SRC.replace(old, new, 1))
    so = tmp_path / "libmutant.so"
    subprocess.run(["gcc", "-O1", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", str(so), str(c)], check=True)
    lib = ctypes.CDLL(str(so))
    lib.oracle_num_threads.restype = ctypes.c_int
    lib.oracle_wgrad_compressed.restype = ctypes.c_int
    oracle._load()
    monkeypatch.setattr(oracle, "_lib", lib)
    tripped = 0
    for call in _pin_calls():
        try:
            call()
        except AssertionError:
            tripped += 1
    assert tripped > 0, f"no pin noticed the planted mistake '{name}'"


def test_unmutated_checker_passes_the_same_pins():
    for call in _pin_calls():
        call()
