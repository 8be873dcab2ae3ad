"""CPU checker (fp64) for backpropagation with pooling-compressed activations.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg. The CUDA library never imports, links or calls
anything here, and nothing here imports the CUDA package.

The arithmetic lives in ``ac_oracle.c`` (plain nested loops, one function per
passage of the paper's Section 4); this file only marshals NumPy float64
arrays (logical NCHW) into it, plus the byte accounting of the paper's
Table 1, which is integer arithmetic written out below.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ac_oracle.c")
_LIB = os.path.join(_HERE, "libac_oracle.so")
_lib = None

_i64 = ctypes.c_int64
_dp = ctypes.POINTER(ctypes.c_double)
_ip = ctypes.POINTER(ctypes.c_int64)


def build(force: bool = False) -> str:
    """Compile ac_oracle.c with gcc (OpenMP) next to this file."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fPIC",
           "-shared", "-o", _LIB, _SRC]
    subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.oracle_num_threads.restype = ctypes.c_int
        _lib.oracle_wgrad_compressed.restype = ctypes.c_int
        _lib.oracle_wgrad_compressed_rect.restype = ctypes.c_int
    return _lib


def _c(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float64)
    return a


def _p(a: np.ndarray):
    return a.ctypes.data_as(_dp)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def out_hw(H, W, R, S, stride, pad):
    """Convolution output size, dilation 1."""
    sh, sw = stride
    ph, pw = pad
    return (H + 2 * ph - R) // sh + 1, (W + 2 * pw - S) // sw + 1


def _khw(k):
    """k as (k_h, k_w); an int means a square block."""
    return (int(k), int(k)) if np.isscalar(k) else (int(k[0]), int(k[1]))


def pooled_hw(H, W, k):
    """Size of Z: partial edge blocks are kept (ceil). k: int, or (k_h, k_w)."""
    kh, kw = _khw(k)
    return -(-H // kh), -(-W // kw)


def pool(x: np.ndarray, k: int) -> np.ndarray:
    """Z = k x k average pooling of X [N,C,H,W] (Section 4, figure)."""
    x = _c(x)
    N, C, H, W = x.shape
    Hp, Wp = pooled_hw(H, W, k)
    z = np.empty((N, C, Hp, Wp), dtype=np.float64)
    if not np.isscalar(k):      # non-uniform block (k_h, k_w)
        _load().oracle_pool_rect(_p(x), _i64(N), _i64(C), _i64(H), _i64(W), _i64(k[0]), _i64(k[1]), _p(z))
        return z
    _load().oracle_pool(_p(x), _i64(N), _i64(C), _i64(H), _i64(W), _i64(k), _p(z))
    return z


def inflate(z: np.ndarray, H: int, W: int, k: int) -> np.ndarray:
    """Expand Z back to [N,C,H,W]: each block mean fills its block (Section 4)."""
    z = _c(z)
    N, C, Hp, Wp = z.shape
    assert (Hp, Wp) == pooled_hw(H, W, k)
    xt = np.empty((N, C, H, W), dtype=np.float64)
    if not np.isscalar(k):
        _load().oracle_inflate_rect(_p(z), _i64(N), _i64(C), _i64(H), _i64(W), _i64(k[0]), _i64(k[1]), _p(xt))
        return xt
    _load().oracle_inflate(_p(z), _i64(N), _i64(C), _i64(H), _i64(W), _i64(k), _p(xt))
    return xt


def relu(a: np.ndarray) -> np.ndarray:
    a = _c(a)
    y = np.empty_like(a)
    _load().oracle_relu(_p(a), _i64(a.size), _p(y))
    return y


def relu_backward(a: np.ndarray, dy: np.ndarray) -> np.ndarray:
    """Gradient of Y = max(A, 0) with respect to A: dY where A > 0, else 0 (the value 0 at A = 0 is
    the one a sign mask `A > 0` stands for)."""
    a, dy = _c(a), _c(dy)
    assert a.shape == dy.shape
    return np.where(a > 0, dy, 0.0)


def wgrad_dense(x, dy, R, S, stride=(1, 1), pad=(0, 0)) -> np.ndarray:
    """Ordinary convolution weight gradient, dW [Co,Ci,R,S]."""
    x, dy = _c(x), _c(dy)
    N, Ci, H, W = x.shape
    Co = dy.shape[1]
    assert dy.shape == (N, Co) + out_hw(H, W, R, S, stride, pad)
    dw = np.empty((Co, Ci, R, S), dtype=np.float64)
    _load().oracle_wgrad_dense(_p(x), _p(dy), _i64(N), _i64(Ci), _i64(Co), _i64(H),
                               _i64(W), _i64(R), _i64(S), _i64(stride[0]),
                               _i64(stride[1]), _i64(pad[0]), _i64(pad[1]), _p(dw))
    return dw


def wgrad_compressed(z, dy, H, W, R, S, stride=(1, 1), pad=(0, 0), k=2) -> np.ndarray:
    """dW from the stored Z: inflate, then the ordinary weight gradient
    (Section 4; figure: dL/dW ~ Z (*) dL/dY)."""
    z, dy = _c(z), _c(dy)
    N, Ci = z.shape[:2]
    Co = dy.shape[1]
    assert z.shape[2:] == pooled_hw(H, W, k)
    assert dy.shape == (N, Co) + out_hw(H, W, R, S, stride, pad)
    dw = np.empty((Co, Ci, R, S), dtype=np.float64)
    if not np.isscalar(k):
        rc = _load().oracle_wgrad_compressed_rect(
            _p(z), _p(dy), _i64(N), _i64(Ci), _i64(Co), _i64(H), _i64(W), _i64(R),
            _i64(S), _i64(stride[0]), _i64(stride[1]), _i64(pad[0]), _i64(pad[1]),
            _i64(k[0]), _i64(k[1]), _p(dw))
        if rc != 0:
            raise MemoryError("oracle_wgrad_compressed_rect: temporary allocation failed")
        return dw
    rc = _load().oracle_wgrad_compressed(
        _p(z), _p(dy), _i64(N), _i64(Ci), _i64(Co), _i64(H), _i64(W), _i64(R),
        _i64(S), _i64(stride[0]), _i64(stride[1]), _i64(pad[0]), _i64(pad[1]),
        _i64(k), _p(dw))
    if rc != 0:
        raise MemoryError("oracle_wgrad_compressed: temporary allocation failed")
    return dw


def wgrad_compressed_entries(z, dy, H, W, R, S, stride, pad, k, idx) -> np.ndarray:
    """The same definition at chosen entries idx[i] = (co, ci, r, s)."""
    z, dy = _c(z), _c(dy)
    idx = np.ascontiguousarray(idx, dtype=np.int64).reshape(-1, 4)
    N, Ci = z.shape[:2]
    Co = dy.shape[1]
    assert z.shape[2:] == pooled_hw(H, W, k)
    assert dy.shape == (N, Co) + out_hw(H, W, R, S, stride, pad)
    out = np.empty(idx.shape[0], dtype=np.float64)
    if not np.isscalar(k):
        _load().oracle_wgrad_compressed_rect_entries(
            _p(z), _p(dy), _i64(N), _i64(Ci), _i64(Co), _i64(H), _i64(W), _i64(R),
            _i64(S), _i64(stride[0]), _i64(stride[1]), _i64(pad[0]), _i64(pad[1]),
            _i64(k[0]), _i64(k[1]), idx.ctypes.data_as(_ip), _i64(idx.shape[0]), _p(out))
        return out
    _load().oracle_wgrad_compressed_entries(
        _p(z), _p(dy), _i64(N), _i64(Ci), _i64(Co), _i64(H), _i64(W), _i64(R),
        _i64(S), _i64(stride[0]), _i64(stride[1]), _i64(pad[0]), _i64(pad[1]),
        _i64(k), idx.ctypes.data_as(_ip), _i64(idx.shape[0]), _p(out))
    return out


def cosine_similarity(a: np.ndarray, b: np.ndarray) -> float:
    """cos(a,b) = a.b / (|a| |b|) (Section 5.2, the layer-sensitivity equation)."""
    a = np.asarray(a, dtype=np.float64).ravel()
    b = np.asarray(b, dtype=np.float64).ravel()
    return float(np.dot(a, b) / (np.sqrt(np.dot(a, a)) * np.sqrt(np.dot(b, b))))


# ---- byte accounting (Section 5.3, Table 1) --------------------------------

def activation_bytes(N, C, H, W, elt=4) -> int:
    """Bytes of a saved conv input X."""
    return N * C * H * W * elt


def compressed_bytes(N, C, H, W, k, elt=4, accounting="ceil") -> int:
    """Bytes of the stored Z. ``accounting="ceil"`` is what this library stores
    (partial edge blocks kept); ``"floor"`` reproduces the paper's Table 1,
    whose odd sizes (14 -> 3, 7 -> 3, 7 -> 1) drop the trailing rows/columns."""
    if accounting == "ceil":
        hp, wp = -(-H // k), -(-W // k)
    elif accounting == "floor":
        hp, wp = H // k, W // k
    else:
        raise ValueError(accounting)
    return N * C * hp * wp * elt
