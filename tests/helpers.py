"""Shared machinery of the GPU parity tests: run the CUDA library through its
C ABI on seeded inputs and compare with the CPU checker (oracle/)."""
import numpy as np
import torch

import oracle
import paper_2409_11902_b200 as ac
from paper_2409_11902_b200 import synth

CANARY = 0x5A

# Tolerances of this path:
#   fp32 compress: max relative error <= 1e-6 (relative to the block's mean |x|)
#   bf16 compress: one rounding to bf16 (half an ulp = 2^-9 .. 2^-8 relative) on top
#   dW: relative Frobenius error <= 1e-5 (fp32 inputs), <= 1e-2 (bf16 inputs, fp32 accumulate)
TOL_Z = {"f32": 1e-6, "bf16": 2.0 ** -8 * 1.001 + 1e-6}
TOL_DW = {"f32": 1e-5, "bf16": 1e-2}
# Beside the stated bounds, what the arithmetic itself allows. bf16 x bf16 products are exact in
# fp32, so a bf16 result differs from the checker by fp32 accumulation only (1e-7 .. 1e-6 measured):
# a kernel that rounded partial sums to bf16 (~2e-3) or dropped a few positions of a map would pass
# the 1e-2 bound but not this one.
TOL_DW_ARITH = {"f32": 1e-5, "bf16": 1e-4}
# Per entry: |got - want| <= TOL_ENTRY * (root mean square of the expected entries). One position
# dropped from a sum of K products moves an entry by about 1/sqrt(K) of that (1e-3 at K = 2^20).
TOL_ENTRY = 1e-4


def assert_dw_close(got, want, dtype, what=""):
    """The three bounds on a weight gradient (or a sample of its entries): relative Frobenius error
    within the stated tolerance and within what fp32 accumulation allows, and every single entry
    close. Returns the relative Frobenius error."""
    got, want = np.asarray(got, dtype=np.float64), np.asarray(want, dtype=np.float64)
    assert np.isfinite(got).all(), what
    nrm = float(np.linalg.norm(want))
    if nrm == 0.0:
        assert not got.any(), what
        return 0.0
    err = float(np.linalg.norm(got - want)) / nrm
    assert err <= TOL_DW[dtype], (what, err)
    assert err <= TOL_DW_ARITH[dtype], (what, err)
    worst = float(np.max(np.abs(got - want)))
    assert worst <= TOL_ENTRY * nrm / np.sqrt(want.size), (what, worst, nrm / np.sqrt(want.size))
    return err


def stratified_entries(d, n_min, seed):
    """Entries (co, ci, r, s) of dW that leave no part of any kernel's output unexamined: one entry,
    at a random place inside, for every (32 output channels) x (32 input channels) x (filter tap)
    cell -- the tensor-core kernels write dW in pieces of 32 accumulator columns (output channels)
    by 32 accumulator rows (input channels of one tap), and every CTA owns whole pieces -- plus the
    four corners, topped up with uniformly random entries to at least n_min."""
    rng = np.random.default_rng(seed + 99)
    idx = [[0, 0, 0, 0], [d.C_out - 1, d.C_in - 1, d.R - 1, d.S - 1],
           [0, d.C_in - 1, 0, d.S - 1], [d.C_out - 1, 0, d.R - 1, 0]]
    for co0 in range(0, d.C_out, 32):
        for ci0 in range(0, d.C_in, 32):
            for r in range(d.R):
                for s in range(d.S):
                    idx.append([int(rng.integers(co0, min(co0 + 32, d.C_out))),
                                int(rng.integers(ci0, min(ci0 + 32, d.C_in))), r, s])
    idx = np.asarray(idx, dtype=np.int64)
    if len(idx) < n_min:
        m = n_min - len(idx)
        extra = np.stack([rng.integers(0, d.C_out, m), rng.integers(0, d.C_in, m),
                          rng.integers(0, d.R, m), rng.integers(0, d.S, m)], axis=1)
        idx = np.concatenate([idx, extra])
    return idx


def padded_empty(shape, dtype, dev, pad_bytes=512):
    """A device tensor of `shape` carved from a larger byte buffer filled with a
    canary, so that writes outside the tensor can be detected afterwards."""
    n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
    n_al = (n + 255) // 256 * 256
    buf = torch.full((pad_bytes + n_al + pad_bytes,), CANARY, dtype=torch.uint8, device=dev)
    view = buf[pad_bytes:pad_bytes + n].view(dtype).view(shape)
    return buf, view, (pad_bytes, n)


def canary_intact(buf, span):
    lo, n = span
    b = buf.cpu()
    return bool((b[:lo] == CANARY).all()) and bool((b[lo + n:] == CANARY).all())


def compress_error(z_got_nchw: np.ndarray, x_nchw: np.ndarray, k: int):
    """max_i |z_i - zhat_i| / mean_{block i} |x|; blocks whose inputs are all
    zero must give exactly 0."""
    z_ref = oracle.pool(x_nchw, k)
    denom = oracle.pool(np.abs(x_nchw), k)
    diff = np.abs(z_got_nchw - z_ref)
    zero = denom == 0
    assert not diff[zero].any(), "all-zero block must pool to exactly 0"
    return float(np.max(diff[~zero] / denom[~zero])) if (~zero).any() else 0.0


def run_compress(d: ac.ConvDesc, seed=0, fused_relu=False, inplace=False, dev="cuda:0"):
    """Returns (error, z as NCHW float64, x as NCHW float64 (post-ReLU))."""
    shape = (d.N, d.C_in, d.H, d.W)
    if fused_relu:
        a = synth.pre_activation(seed, shape, d.dtype)
        x64 = oracle.relu(synth.to_f64(a))
        src = a
    else:
        src = synth.activation(seed, shape, d.dtype)
        x64 = synth.to_f64(src)
    xd = synth.to_layout(src, d.layout).to(dev)
    zbuf, z, zspan = padded_empty(d.z_shape, d.torch_dtype, dev)
    ybuf = y = None
    if fused_relu:
        if inplace:
            y = xd
        else:
            ybuf, y, yspan = padded_empty(d.x_shape, d.torch_dtype, dev)
    ac.ac_compress(d, xd, z, y)
    torch.cuda.synchronize()
    assert canary_intact(zbuf, zspan), "ac_compress wrote outside Z"
    if ybuf is not None:
        assert canary_intact(ybuf, yspan), "ac_compress wrote outside Y"
    if fused_relu:
        y64 = synth.to_f64(synth.from_layout(y.cpu(), d.layout))
        assert np.array_equal(y64, x64), "fused ReLU output differs from max(A, 0)"
    z64 = synth.to_f64(synth.from_layout(z.cpu(), d.layout))
    return compress_error(z64, x64, d.k), z64, x64


def run_compress_mask(d: ac.ConvDesc, seed=0, dev="cuda:0", store_y=None):
    """The mask form of the fused call. Returns the pooling error; the mask is compared bit for
    bit with (A > 0) in memory order. `store_y`: "own" or "inplace" runs the variant that also writes
    Y = max(A, 0), into a buffer of its own or over A."""
    shape = (d.N, d.C_in, d.H, d.W)
    a = synth.pre_activation(seed, shape, d.dtype)
    x64 = oracle.relu(synth.to_f64(a))
    ad = synth.to_layout(a, d.layout).to(dev)
    n_el = int(np.prod(shape))
    zbuf, z, zspan = padded_empty(d.z_shape, d.torch_dtype, dev)
    mbuf, m, mspan = padded_empty(((n_el + 7) // 8,), torch.uint8, dev)
    before = ad.clone()
    if store_y is None:
        ac.ac_compress_relu_mask(d, ad, z, m)
    else:
        ybuf, y, yspan = padded_empty(tuple(ad.shape), d.torch_dtype, dev)
        y.fill_(float("nan"))
        out = ad if store_y == "inplace" else y
        ac.ac_compress_relu_mask_y(d, ad, out, z, m)
        torch.cuda.synchronize()
        assert canary_intact(ybuf, yspan), "wrote outside Y"
        y64 = synth.to_f64(synth.from_layout(out.cpu(), d.layout))
        assert np.array_equal(y64, x64), "fused ReLU output differs from max(A, 0)"
    torch.cuda.synchronize()
    assert canary_intact(zbuf, zspan), "wrote outside Z"
    assert canary_intact(mbuf, mspan), "wrote outside the mask"
    if store_y != "inplace":
        assert torch.equal(ad.view(torch.uint8), before.view(torch.uint8)), "the input must not be modified"
    a_mem = synth.to_f64(synth.to_layout(a, d.layout)).reshape(-1)   # memory order of the layout
    want = np.packbits(a_mem > 0, bitorder="little")
    assert np.array_equal(m.cpu().numpy(), want), "sign mask differs from (A > 0)"
    z64 = synth.to_f64(synth.from_layout(z.cpu(), d.layout))
    return compress_error(z64, x64, d.k)


def make_wgrad_inputs(d: ac.ConvDesc, seed=0):
    """X -> Z by the checker's pooling, rounded once to the storage dtype, so
    that the checker and the GPU read identical bits of Z and dY."""
    x = synth.activation(seed, (d.N, d.C_in, d.H, d.W), d.dtype)
    z = synth.to_storage(oracle.pool(synth.to_f64(x), d.k), d.dtype)
    dy = synth.grad_output(seed, (d.N, d.C_out, d.Ho, d.Wo), d.dtype)
    return z, dy


def dw_to_oihw(dw: torch.Tensor, layout: str) -> np.ndarray:
    a = dw.detach().cpu().double().numpy()
    return a.transpose(0, 3, 1, 2) if layout == "nhwc" else a


def run_wgrad(d: ac.ConvDesc, z, dy, dev="cuda:0", repeat=2, nbytes=None):
    """Runs the library `repeat` times (bitwise-equal results required) and
    returns dW as float64 [Co,Ci,R,S]. `nbytes`: workspace size to hand over
    (default: what the fastest path asks for)."""
    zd = synth.to_layout(z, d.layout).to(dev)
    dyd = synth.to_layout(dy, d.layout).to(dev)
    if nbytes is None:
        nbytes = ac.ac_workspace_bytes(d)
    assert nbytes > 0
    outs = []
    for it in range(repeat):
        wbuf, dw, wspan = padded_empty(d.dw_shape, torch.float32, dev)
        sbuf, ws, sspan = padded_empty((nbytes,), torch.uint8, dev)
        if it == 1:
            ws.fill_(0xFF)          # workspace contents on entry must not matter
            dw.fill_(float("nan"))  # dW is overwritten, not accumulated into
        ac.ac_conv2d_wgrad_compressed(d, zd, dyd, dw, ws, nbytes)
        st, detail = ac.ac_workspace_status(ws)
        assert st == 0, f"device status {st} detail {detail:#x}"
        assert canary_intact(wbuf, wspan), "wgrad wrote outside dW"
        assert canary_intact(sbuf, sspan), "wgrad wrote outside the workspace"
        outs.append(dw.clone())
    for o in outs[1:]:
        assert torch.equal(o, outs[0]), "results differ between identical calls"
    return dw_to_oihw(outs[0], d.layout)


def wgrad_error_full(d: ac.ConvDesc, seed=0, dev="cuda:0"):
    z, dy = make_wgrad_inputs(d, seed)
    got = run_wgrad(d, z, dy, dev)
    want = oracle.wgrad_compressed(synth.to_f64(z), synth.to_f64(dy), d.H, d.W, d.R, d.S,
                                   d.stride, d.pad, d.k)
    return assert_dw_close(got, want, d.dtype, repr(d)), got, want


def sampled_check(d: ac.ConvDesc, got, z, dy, n_samples=256, seed=0):
    """The checker evaluates a stratified sample of dW's entries one by one (see
    stratified_entries); `got` must meet all bounds on it. Returns the relative l2 error."""
    idx = stratified_entries(d, n_samples, seed)
    want = oracle.wgrad_compressed_entries(synth.to_f64(z), synth.to_f64(dy), d.H, d.W, d.R, d.S,
                                           d.stride, d.pad, d.k, idx)
    g = got[idx[:, 0], idx[:, 1], idx[:, 2], idx[:, 3]]
    assert np.isfinite(got).all()
    return assert_dw_close(g, want, d.dtype, repr(d))


def wgrad_error_sampled(d: ac.ConvDesc, n_samples=512, seed=0, dev="cuda:0"):
    """Full-size case: the error is the relative l2 error over a stratified sample of entries."""
    z, dy = make_wgrad_inputs(d, seed)
    got = run_wgrad(d, z, dy, dev)
    return sampled_check(d, got, z, dy, n_samples, seed), got


def run_wgrad_collapsed(d: ac.ConvDesc, z, dy, dev="cuda:0", repeat=2):
    """The collapsed entry point, same protocol as run_wgrad. Returns None if the library does
    not take the problem in that form."""
    nbytes, tiles_c, tiles_d = ac.ac_collapsed_workspace_bytes(d)
    if nbytes == 0:
        return None
    assert 0 < tiles_c < tiles_d
    zd = synth.to_layout(z, d.layout).to(dev)
    dyd = synth.to_layout(dy, d.layout).to(dev)
    outs = []
    for it in range(repeat):
        wbuf, dw, wspan = padded_empty(d.dw_shape, torch.float32, dev)
        sbuf, ws, sspan = padded_empty((nbytes,), torch.uint8, dev)
        if it == 1:
            ws.fill_(0xFF)
            dw.fill_(float("nan"))
        ac.ac_conv2d_wgrad_compressed_collapsed(d, zd, dyd, dw, ws, nbytes)
        st, detail = ac.ac_workspace_status(ws)
        assert st == 0, f"device status {st} detail {detail:#x}"
        assert canary_intact(wbuf, wspan), "collapsed wgrad wrote outside dW"
        assert canary_intact(sbuf, sspan), "collapsed wgrad wrote outside the workspace"
        outs.append(dw.clone())
    for o in outs[1:]:
        assert torch.equal(o, outs[0]), "results differ between identical calls"
    return dw_to_oihw(outs[0], d.layout)
