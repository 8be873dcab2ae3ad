"""Host-side checks of the C ABI that need no GPU: the library loads, exports
every symbol include/ac.h declares, and validates arguments before any launch."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as entry

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def ac():
    entry.build()
    import paper_2409_11902_b200 as ac
    return ac


def declared_functions():
    text = open(os.path.join(ROOT, "include", "ac.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ac_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(ac):
    names = declared_functions()
    assert {"ac_compress", "ac_conv2d_wgrad_compressed", "ac_workspace_bytes"} <= set(names)
    L = ac.api.lib()
    for n in names:
        assert hasattr(L, n), f"{n} declared in ac.h but not exported by libac.so"


def test_status_strings(ac):
    assert ac.status_string(0) == "AC_OK"
    assert ac.status_string(4) == "AC_ERR_WORKSPACE_TOO_SMALL"
    assert ac.status_string(6) == "AC_ERR_TIMEOUT"


def test_workspace_bytes_is_host_only_and_rejects_bad_descriptors(ac):
    good = ac.ConvDesc(8, 64, 64, 32, 32, 3, 3, (1, 1), (1, 1), 2, "f32", "nchw")
    assert ac.ac_workspace_bytes(good) >= 256
    import dataclasses
    for bad in (dict(N=0), dict(k=0), dict(C_out=-1), dict(R=40), dict(stride=(0, 1)),
                dict(pad=(-1, 0)), dict(H=0)):
        assert ac.ac_workspace_bytes(dataclasses.replace(good, **bad)) == 0, bad
    assert ac.api.lib().ac_workspace_bytes(None) == 0


def test_workspace_grows_with_the_problem_not_unbounded(ac):
    small = ac.ConvDesc(8, 64, 64, 32, 32, 3, 3, (1, 1), (1, 1), 2, "f32", "nchw")
    huge = ac.ConvDesc(256, 512, 512, 56, 56, 3, 3, (1, 1), (1, 1), 2, "f32", "nchw")
    assert ac.ac_workspace_bytes_min(small) < ac.ac_workspace_bytes_min(huge) < (1 << 30)
    # the fastest path for these fp32 NCHW problems stages six bf16 terms of each operand element
    # (12 bytes each) and the kernel's dW on top of its partial sums: bounded by the problem, too
    for d in (small, huge):
        staged = 12 * (d.N * d.C_in * (d.H // 2) * (d.W // 2) + d.N * d.C_out * d.H * d.W) + 4 * d.C_out * d.C_in * 9
        assert ac.ac_workspace_bytes_min(d) <= ac.ac_workspace_bytes(d) < (1 << 30) + staged + 4096
    same = ac.ConvDesc(8, 64, 64, 32, 32, 3, 3, (1, 1), (1, 1), 2, "bf16", "nhwc")
    assert ac.ac_workspace_bytes_min(same) == ac.ac_workspace_bytes(same)


def test_calls_validate_before_launching(ac):
    """No GPU here: every one of these must return before touching CUDA."""
    L = ac.api.lib()
    d = ac.ConvDesc(2, 8, 8, 8, 8, 3, 3, (1, 1), (1, 1), 2, "f32", "nchw").c()
    ref = ctypes.byref(d)
    A = 0x10000  # a 16-byte aligned, never dereferenced address
    assert L.ac_compress(ref, None, A, None, None) == ac.api.AC_ERR_INVALID_ARG
    assert L.ac_compress(ref, A + 4, A, None, None) == ac.api.AC_ERR_MISALIGNED
    assert L.ac_compress(ref, A, A, A + 8, None) == ac.api.AC_ERR_MISALIGNED
    assert L.ac_compress(None, A, A, None, None) == ac.api.AC_ERR_INVALID_ARG
    assert L.ac_compress_relu_mask(ref, A, A, None, None) == ac.api.AC_ERR_INVALID_ARG
    assert L.ac_compress_relu_mask(ref, A, A, A + 1, None) == ac.api.AC_ERR_MISALIGNED
    # the sign mask exists only where a mask byte is 8 contiguous elements of a vector kernel
    for shape in [dict(k=3, layout="nhwc"), dict(k=2, layout="nchw", W=12), dict(k=2, layout="nhwc", C=12)]:
        m = ac.ConvDesc(2, shape.get("C", 8), 8, 8, shape.get("W", 8), 3, 3, (1, 1), (1, 1), shape["k"],
                        "bf16", shape["layout"]).c()
        assert L.ac_compress_relu_mask(ctypes.byref(m), A, A, A, None) == ac.api.AC_ERR_UNSUPPORTED
    assert L.ac_conv2d_wgrad_compressed(ref, A, A, None, A, 1 << 30, None) == ac.api.AC_ERR_INVALID_ARG
    assert L.ac_conv2d_wgrad_compressed(ref, A, A + 2, A, A, 1 << 30, None) == ac.api.AC_ERR_MISALIGNED
    assert L.ac_conv2d_wgrad_compressed(ref, A, A, A, A, 16, None) == ac.api.AC_ERR_WORKSPACE_TOO_SMALL
    bad = ac.ConvDesc(2, 8, 8, 8, 8, 3, 3, (1, 1), (1, 1), 2, "f32", "nchw").c()
    bad.dtype = 7
    assert L.ac_compress(ctypes.byref(bad), A, A, None, None) == ac.api.AC_ERR_INVALID_ARG
    acc = L.ac_conv2d_wgrad_compressed_accumulate
    assert acc(ref, A, A, 1.0, None, A, 1 << 30, None) == ac.api.AC_ERR_INVALID_ARG
    assert acc(ref, A, A, 1.0, A + 4, A, 1 << 30, None) == ac.api.AC_ERR_MISALIGNED
    assert acc(ref, A, A, float("nan"), A, A, 1 << 30, None) == ac.api.AC_ERR_INVALID_ARG
    assert acc(ref, A, A, float("inf"), A, A, 1 << 30, None) == ac.api.AC_ERR_INVALID_ARG
    assert acc(ref, A, A, 1.0, A, A, 8 * 8 * 9 * 4 + 255, None) == ac.api.AC_ERR_WORKSPACE_TOO_SMALL
    assert acc(ref, A, None, 1.0, A, A, 1 << 30, None) == ac.api.AC_ERR_INVALID_ARG
    good = ac.ConvDesc(2, 8, 8, 8, 8, 3, 3, (1, 1), (1, 1), 2, "f32", "nchw")
    assert ac.ac_accumulate_workspace_bytes(good) >= ac.ac_workspace_bytes(good) + 8 * 8 * 9 * 4
    assert L.ac_backward_step_host(ref, A, A, A, None, A + 16, 1 << 30, None) == ac.api.AC_ERR_MISALIGNED
    assert L.ac_backward_step_host(ref, A, A, A, None, A, 16, None) == ac.api.AC_ERR_WORKSPACE_TOO_SMALL
    assert L.ac_workspace_status(None, None, None) == ac.api.AC_ERR_INVALID_ARG


def test_binding_fails_loudly_without_the_library(ac, monkeypatch):
    monkeypatch.setattr(ac.api, "_lib", None)
    monkeypatch.setattr(ac.api, "_LIB_PATH", "/nonexistent/libac.so")
    with pytest.raises(ImportError):
        ac.ac_workspace_bytes(ac.ConvDesc(1, 8, 8, 8, 8))


def test_plan_info_respects_hardware_limits(ac):
    """Host-side planning of the tensor-core path: shared memory, tensor memory
    and pipeline depth stay inside what one SM has, for every benchmark layer."""
    shapes = [
        (64, 64, 64, 56, 56, 3, 3, 1, 1), (64, 128, 128, 28, 28, 3, 3, 1, 1),
        (64, 256, 256, 14, 14, 3, 3, 1, 1), (64, 512, 512, 7, 7, 3, 3, 1, 1),
        (64, 512, 512, 8, 8, 3, 3, 1, 1), (128, 256, 64, 56, 56, 1, 1, 1, 0),
        (128, 64, 256, 56, 56, 1, 1, 1, 0), (128, 128, 128, 56, 56, 3, 3, 2, 1),
        (256, 128, 128, 64, 64, 3, 3, 1, 1), (256, 1024, 2048, 14, 14, 1, 1, 2, 0),
        (8, 64, 64, 30, 30, 7, 7, 2, 3), (2, 192, 320, 9, 40, 3, 3, 1, 1),
    ]
    for N, ci, co, H, W, R, S, st, pd in shapes:
        for k in (1, 2, 4, 8):
            d = ac.ConvDesc(N, ci, co, H, W, R, S, (st, st), (pd, pd), k, "bf16", "nhwc")
            i = ac.ac_wgrad_plan_info(d)
            assert i["tensor_core"] in (1, 2, 7), d
            # 7: the TMA-fed kernel on Z re-blocked to a block k2 that divides k (k2 = 1: the inflated map), kept in
            # the workspace; `phases` counts that plan's classes
            inflated = i["tensor_core"] == 7
            k2 = k
            if inflated:
                k2 = st * int(round(i["phases"] ** 0.5)) if i["phases"] > 1 else (1 if st == 1 or k % st else st)
                assert k > 1 and k % k2 == 0 and k2 < k
                assert k2 > 1 or ((H % k or W % k) and pd > 0)      # all the way to the inflated map: partial blocks only
            assert 2 <= i["stages"] <= 8
            assert i["smem_bytes"] <= 227 * 1024
            assert i["tmem_columns"] in (32, 64, 128, 256, 512)
            assert i["units_per_cta"] * i["block_n"] <= i["tmem_columns"]
            assert i["k_tile"] % 16 == 0
            if i["tensor_core"] == 1:
                assert i["k_tile"] >= i["band_rows"] * i["row_pitch"]
                assert i["row_pitch"] >= d.Wo
            else:   # per class: (band_rows / c_h) class rows of row_pitch >= Wo / c_w positions
                c_h = c_w = max(1, k2 // st)     # a stride above the block: one class, phase planes of Z
                assert i["phases"] == c_h * c_w <= 64
                assert i["k_tile"] >= (i["band_rows"] // c_h) * i["row_pitch"]
                assert i["row_pitch"] >= -(-d.Wo // c_w)
            assert 1 <= i["splits"] <= d.N * -(-d.Ho // i["band_rows"])
            assert i["ctas"] == i["splits"] * i["groups"]
            want = 256 + (i["splits"] * 4 * co * ci * R * S if i["splits"] > 1 else 0)
            if inflated:
                want = -(-want // 256) * 256 + -(-N * -(-H // k2) * -(-W // k2) * ci * 2 // 256) * 256
                assert ac.ac_workspace_bytes_min(d) <= want
            assert ac.ac_workspace_bytes(d) == want
    # 64 input channels, 3x3, k = 2: the nine taps pair up into five accumulator tiles in one CTA
    i = ac.ac_wgrad_plan_info(ac.ConvDesc(64, 64, 64, 56, 56, 3, 3, (1, 1), (1, 1), 2, "bf16", "nhwc"))
    assert (i["tensor_core"], i["units_per_cta"], i["groups"]) == (2, 5, 1)
    # k = 8 at stride 1: 64 output classes on the TMA-fed kernel when the workspace has no room for a re-blocked Z,
    # four classes on Z re-blocked to 2 x 2 when it has (k = 4: sixteen classes, read directly)
    d8 = ac.ConvDesc(256, 128, 128, 64, 64, 3, 3, (1, 1), (1, 1), 8, "bf16", "nhwc")
    i = ac.ac_wgrad_plan_info(d8)
    assert (i["tensor_core"], i["phases"]) == (7, 4)
    assert ac.ac_workspace_bytes(d8) - ac.ac_workspace_bytes_min(d8) >= 256 * 32 * 32 * 128 * 2 - 64 * 4 * 128 * 128 * 9
    i = ac.ac_wgrad_plan_info(ac.ConvDesc(256, 128, 128, 64, 64, 3, 3, (1, 1), (1, 1), 4, "bf16", "nhwc"))
    assert (i["tensor_core"], i["phases"]) == (2, 16)
    # a small map that k does not divide, with padding (partial pooling blocks that taps read past): the
    # TMA-fed kernel runs on the inflated map; without padding, or on a larger map, it reads Z itself
    i = ac.ac_wgrad_plan_info(ac.ConvDesc(64, 512, 512, 7, 7, 3, 3, (1, 1), (1, 1), 2, "bf16", "nhwc"))
    assert (i["tensor_core"], i["phases"]) == (7, 1)
    i = ac.ac_wgrad_plan_info(ac.ConvDesc(64, 128, 128, 29, 29, 3, 3, (1, 1), (1, 1), 2, "bf16", "nhwc"))
    assert (i["tensor_core"], i["phases"]) == (2, 4)
    # ... and a 1x1 layer without padding never reads the padding rows inside the partial last block,
    # so it needs no second copy of the tile: same tiles as on the 8x8 map
    i7, i8 = (ac.ac_wgrad_plan_info(ac.ConvDesc(256, 512, 2048, h, h, 1, 1, (1, 1), (0, 0), 2, "bf16", "nhwc"))
              for h in (7, 8))
    assert all(i7[f] == i8[f] for f in ("k_tile", "stages", "smem_bytes", "a_cells", "row_pitch", "ctas"))
    # a stride that is a multiple of k (k = 1 at stride 2): one class reading phase planes of Z, the TMA-fed kernel
    i = ac.ac_wgrad_plan_info(ac.ConvDesc(8, 128, 128, 28, 28, 3, 3, (2, 2), (1, 1), 1, "bf16", "nhwc"))
    assert (i["tensor_core"], i["phases"]) == (2, 1)
    i = ac.ac_wgrad_plan_info(ac.ConvDesc(8, 128, 128, 28, 28, 3, 3, (2, 2), (1, 1), 3, "bf16", "nhwc"))
    assert i["tensor_core"] == 7      # k = 3 at stride 2: the same kernel on the inflated map (k = 1 at stride 2)
    # what is left to the producer-fed tensor-core kernel: phase planes whose tiles do not fit the shared memory
    i = ac.ac_wgrad_plan_info(ac.ConvDesc(8, 128, 128, 64, 64, 5, 5, (2, 2), (0, 0), 1, "bf16", "nhwc"))
    assert i["tensor_core"] == 1
    # shapes the tensor-core kernel does not take go to the fp32-ALU kernel
    for d in (ac.ConvDesc(8, 24, 64, 32, 32, 3, 3, (1, 1), (1, 1), 2, "f32", "nchw"),
              ac.ConvDesc(8, 64, 40, 32, 32, 3, 3, (1, 1), (1, 1), 2, "bf16", "nchw"),
              ac.ConvDesc(8, 3, 64, 32, 32, 7, 7, (2, 2), (3, 3), 2, "f32", "nhwc"),
              ac.ConvDesc(8, 64, 64, 32, 32, 3, 3, (3, 3), (1, 1), 2, "bf16", "nhwc")):
        assert ac.ac_wgrad_plan_info(d)["tensor_core"] == 0
    # fp32 NHWC goes to the tensor cores as six bf16 products: the same kernel on six times the
    # images, with room for the split operands in the workspace
    d32 = ac.ConvDesc(8, 64, 64, 32, 32, 3, 3, (1, 1), (1, 1), 2, "f32", "nhwc")
    d16 = ac.ConvDesc(48, 64, 64, 32, 32, 3, 3, (1, 1), (1, 1), 2, "bf16", "nhwc")
    i32, i16 = ac.ac_wgrad_plan_info(d32), ac.ac_wgrad_plan_info(d16)
    assert i32["tensor_core"] == 3 and i16["tensor_core"] == 2
    # ... except that the K-slices are shorter (bounded accumulation chains), hence more of them
    varies = ("tensor_core", "splits", "ctas")
    assert {k: v for k, v in i32.items() if k not in varies} == {k: v for k, v in i16.items() if k not in varies}
    assert i32["splits"] >= i16["splits"] and i32["ctas"] == i32["splits"] * i32["groups"]
    z6 = 48 * 64 * 16 * 16 * 2
    g6 = 48 * 64 * 32 * 32 * 2
    dw_bytes = 64 * 64 * 9 * 4
    assert ac.ac_workspace_bytes(d32) == 256 + i32["splits"] * dw_bytes + z6 + g6
    # NCHW inputs are transposed on the way: same kernel, plus room for its NHWC-ordered dW
    for dt, mult in (("bf16", 1), ("f32", 6)):
        dn = ac.ConvDesc(8, 64, 64, 32, 32, 3, 3, (1, 1), (1, 1), 2, dt, "nchw")
        info = ac.ac_wgrad_plan_info(dn)
        assert info["tensor_core"] == 3
        assert ac.ac_workspace_bytes(dn) == (256 + info["splits"] * dw_bytes + (z6 + g6) * mult // 6 + dw_bytes)


def test_few_input_channels_are_gathered_for_the_tensor_cores(ac):
    """bf16 NHWC layers with fewer than 64 input channels (the 3-channel stem): the operand is
    gathered into a [positions][taps x channels] matrix in the workspace and the tensor-core kernel
    runs the equivalent 1x1 problem on the output map."""
    def inner(N, cols, co, Ho, Wo):
        return ac.ConvDesc(N, cols, co, Ho, Wo, 1, 1, (1, 1), (0, 0), 1, "bf16", "nhwc")
    # 7x7, stride 2, pad 3, k = 2, k | H: taps collapse to 4 x 4 shifts -> 48 columns, padded to 64; such layers
    # have the matrix built inside the kernel (plan code 6): K-tiles of 16 whole output rows of 16 positions, and no
    # staged copy in the workspace, only the K-slices of the [C_out][64] result
    d = ac.ConvDesc(8, 3, 64, 32, 32, 7, 7, (2, 2), (3, 3), 2, "bf16", "nhwc")
    i = ac.ac_wgrad_plan_info(d)
    assert i["tensor_core"] == 6 and i["k_tile"] == 256 and i["band_rows"] == 16 and i["block_n"] == 64
    assert i["splits"] == 8 * 16 // 16 and i["smem_bytes"] <= 227 * 1024 and i["tmem_columns"] == 64
    assert ac.ac_workspace_bytes(d) == 256 + i["splits"] * 64 * 64 * 4
    assert ac.ac_workspace_bytes_min(d) <= ac.ac_workspace_bytes(d)
    # an odd map cannot collapse (the partial last block): one column per tap, 147 -> 192
    d = ac.ConvDesc(8, 3, 64, 31, 31, 7, 7, (2, 2), (3, 3), 2, "bf16", "nhwc")
    assert ac.ac_wgrad_plan_info(d)["tensor_core"] == 5
    assert ac.ac_workspace_bytes(d) == ac.ac_workspace_bytes(inner(8, 192, 64, 16, 16)) + 8 * 16 * 16 * 192 * 2 + 64 * 192 * 4
    # stride 1 at k = 2: no collapse either; 3x3x3 = 27 columns -> 64
    d = ac.ConvDesc(4, 3, 128, 20, 20, 3, 3, (1, 1), (1, 1), 2, "bf16", "nhwc")
    assert ac.ac_wgrad_plan_info(d)["tensor_core"] == 5
    assert ac.ac_workspace_bytes(d) == ac.ac_workspace_bytes(inner(4, 64, 128, 20, 20)) + 4 * 20 * 20 * 64 * 2 + 128 * 64 * 4
    # the least workspace the call accepts is the fp32-ALU kernel's
    assert 256 <= ac.ac_workspace_bytes_min(d) < ac.ac_workspace_bytes(d)
    # more than 256 columns, other dtypes or layouts, C_out not a multiple of 64: not taken
    for d in (ac.ConvDesc(4, 32, 64, 20, 20, 3, 3, (1, 1), (1, 1), 2, "bf16", "nhwc"),
              ac.ConvDesc(4, 3, 64, 20, 20, 3, 3, (1, 1), (1, 1), 2, "f32", "nhwc"),
              ac.ConvDesc(4, 3, 64, 20, 20, 3, 3, (1, 1), (1, 1), 2, "bf16", "nchw"),
              ac.ConvDesc(4, 3, 40, 20, 20, 3, 3, (1, 1), (1, 1), 2, "bf16", "nhwc")):
        assert ac.ac_wgrad_plan_info(d)["tensor_core"] != 5


def test_layer_report_tables_match_the_network():
    """The report tool's ResNet-50 layer table and saved-state accounting against an independent
    walk over the network (bottleneck blocks, stride on the 3x3, 224 x 224 images, batch 256, bf16)."""
    from paper_2409_11902_b200 import layer_report as lr
    assert sum(l[-1] for l in lr.RESNET50) == 53 and len(lr.RESNET50) == 23
    inputs, outputs, flops = [(3, 224)], [(64, 112)], 2 * 112 * 112 * 64 * 3 * 49
    for cin, width, cout, H, blocks, stride in [(64, 64, 256, 56, 3, 1), (256, 128, 512, 56, 4, 2),
                                                (512, 256, 1024, 28, 6, 2), (1024, 512, 2048, 14, 3, 2)]:
        for b in range(blocks):
            h_in = H if b == 0 else H // stride
            h_out = H // stride
            c_in = cin if b == 0 else cout
            inputs += [(c_in, h_in), (width, h_in), (width, h_out)]
            outputs += [(width, h_in), (width, h_out), (cout, h_out)] + ([(cout, h_out)] if b == 0 else [])
            flops += 2 * (h_in * h_in * width * c_in + h_out * h_out * width * width * 9 + h_out * h_out * cout * width
                          + (h_out * h_out * cout * c_in if b == 0 else 0))
    A, Az, B, mask = lr.saved_state_model(lr.RESNET50, 256, 2, 2, lr.RESNET50_SHARED_INPUT)
    assert A == sum(256 * c * h * h * 2 for c, h in inputs)
    assert Az == sum(256 * c * (-(-h // 2)) ** 2 * 2 for c, h in inputs)
    assert B == sum(256 * c * h * h * 2 for c, h in outputs)
    assert mask == A // 16
    table_flops = sum(cnt * 2 * ((H + 2 * pd - R) // st + 1) ** 2 * co * ci * R * R
                      for ci, co, H, R, st, pd, cnt in lr.RESNET50)
    assert table_flops == flops


def test_rect_entry_points_validate_the_block(ac):
    """Needs no GPU: sizes and argument checks of the k_h x k_w calls are host code."""
    L = ac.api.lib()
    d = ac.ConvDesc(4, 64, 64, 20, 20, 3, 3, (1, 1), (1, 1), 2, "bf16", "nhwc")
    assert ac.ac_workspace_bytes_rect(d, 2, 2) == ac.ac_workspace_bytes(d)
    assert ac.ac_workspace_bytes_rect(d, 0, 0) == ac.ac_workspace_bytes(d)
    assert ac.ac_workspace_bytes_rect(d, 2, 4) >= 256
    for bad in ((0, 2), (2, 0), (-1, 2), (2, -3)):
        assert ac.ac_workspace_bytes_rect(d, *bad) == 0
        c = d.c()
        A = 0x10000
        assert L.ac_compress_rect(ctypes.byref(c), bad[0], bad[1], A, A, None, None) == ac.api.AC_ERR_INVALID_ARG
        assert L.ac_conv2d_wgrad_compressed_rect(ctypes.byref(c), bad[0], bad[1], A, A, A, A, 1 << 30, None) \
            == ac.api.AC_ERR_INVALID_ARG
    c = d.c()
    assert L.ac_conv2d_wgrad_compressed_rect(ctypes.byref(c), 2, 4, 0x10000, 0x10000, 0x10000, 0x10000, 16, None) \
        == ac.api.AC_ERR_WORKSPACE_TOO_SMALL


def test_sm_budget_is_a_per_thread_planning_hint(ac):
    """Fewer SMs to count on: fewer K-slices, fewer CTAs, a smaller workspace; 0 restores the default; another
    host thread is not affected."""
    import threading
    d = ac.ConvDesc(64, 256, 256, 14, 14, 3, 3, (1, 1), (1, 1), 2, "bf16", "nhwc")
    assert ac.ac_get_sm_budget() == 148
    full, full_ws = ac.ac_wgrad_plan_info(d), ac.ac_workspace_bytes(d)
    try:
        ac.ac_set_sm_budget(37)
        assert ac.ac_get_sm_budget() == 37
        part, part_ws = ac.ac_wgrad_plan_info(d), ac.ac_workspace_bytes(d)
        assert part["groups"] == full["groups"] and part["ctas"] <= 37 < full["ctas"]
        assert part["splits"] < full["splits"] and part_ws < full_ws
        assert part_ws == 256 + part["splits"] * 4 * 256 * 256 * 9
        seen = []
        t = threading.Thread(target=lambda: seen.append((ac.ac_get_sm_budget(), ac.ac_workspace_bytes(d))))
        t.start(); t.join()
        assert seen == [(148, full_ws)]
        with pytest.raises(ac.AcError):
            ac.ac_set_sm_budget(-1)
        assert ac.ac_get_sm_budget() == 37
        ac.ac_set_sm_budget(10 ** 6)
        assert ac.ac_get_sm_budget() == 148
    finally:
        ac.ac_set_sm_budget(0)
    assert ac.ac_workspace_bytes(d) == full_ws
