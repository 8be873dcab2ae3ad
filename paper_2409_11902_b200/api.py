"""Thin ctypes binding of libac.so: the same names and arguments as include/ac.h.

Argument marshalling only. Tensors are torch tensors used as plain device (or
pinned host) buffers; every step of the path runs inside the CUDA library.
There is no fallback: if the library is missing or cannot be loaded, importing
a function from here raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

AC_OK = 0
AC_ERR_INVALID_ARG = 1
AC_ERR_UNSUPPORTED = 2
AC_ERR_MISALIGNED = 3
AC_ERR_WORKSPACE_TOO_SMALL = 4
AC_ERR_CUDA = 5
AC_ERR_TIMEOUT = 6
AC_F32, AC_BF16 = 0, 1
AC_NCHW, AC_NHWC = 0, 1

_DTYPES = {"f32": AC_F32, "bf16": AC_BF16}
_LAYOUTS = {"nchw": AC_NCHW, "nhwc": AC_NHWC}
_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libac.so")


class ac_conv_desc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "N", "C_in", "C_out", "H", "W", "R", "S", "stride_h", "stride_w",
        "pad_h", "pad_w", "k", "dtype", "layout")]


class ac_plan_info(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "tensor_core", "splits", "ctas", "groups", "band_rows", "k_tile", "row_pitch", "stages",
        "smem_bytes", "tmem_columns", "units_per_cta", "block_n", "a_cells", "phases")]


class AcError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)}")


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(
                f"{_LIB_PATH} not found: build it with __graft_entry__.build() "
                "or `python -m paper_2409_11902_b200.build`")
        L = ctypes.CDLL(_LIB_PATH)
        vp, sz = ctypes.c_void_p, ctypes.c_size_t
        dp = ctypes.POINTER(ac_conv_desc)
        L.ac_workspace_bytes.restype = sz
        L.ac_workspace_bytes.argtypes = [dp]
        L.ac_workspace_bytes_min.restype = sz
        L.ac_workspace_bytes_min.argtypes = [dp]
        L.ac_compress.restype = ctypes.c_int
        L.ac_compress.argtypes = [dp, vp, vp, vp, vp]
        L.ac_compress_relu_mask.restype = ctypes.c_int
        L.ac_compress_relu_mask.argtypes = [dp, vp, vp, vp, vp]
        L.ac_compress_relu_mask_y.restype = ctypes.c_int
        L.ac_compress_relu_mask_y.argtypes = [dp, vp, vp, vp, vp, vp]
        L.ac_relu_mask_backward.restype = ctypes.c_int
        L.ac_relu_mask_backward.argtypes = [dp, vp, vp, vp, vp]
        L.ac_conv2d_wgrad_compressed.restype = ctypes.c_int
        L.ac_conv2d_wgrad_compressed.argtypes = [dp, vp, vp, vp, vp, sz, vp]
        L.ac_accumulate_workspace_bytes.restype = sz
        L.ac_accumulate_workspace_bytes.argtypes = [dp]
        L.ac_conv2d_wgrad_compressed_accumulate.restype = ctypes.c_int
        L.ac_conv2d_wgrad_compressed_accumulate.argtypes = [dp, vp, vp, ctypes.c_float, vp, vp, sz, vp]
        L.ac_set_kernel_timing_events.restype = ctypes.c_int
        L.ac_set_kernel_timing_events.argtypes = [vp, vp]
        L.ac_set_sm_budget.restype = ctypes.c_int
        L.ac_set_sm_budget.argtypes = [ctypes.c_int32]
        L.ac_get_sm_budget.restype = ctypes.c_int32
        L.ac_get_sm_budget.argtypes = []
        L.ac_workspace_status.restype = ctypes.c_int
        L.ac_workspace_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_uint32)]
        L.ac_host_step_arena_bytes.restype = sz
        L.ac_host_step_arena_bytes.argtypes = [dp]
        L.ac_backward_step_host.restype = ctypes.c_int
        L.ac_backward_step_host.argtypes = [dp, vp, vp, vp, vp, vp, sz, vp]
        L.ac_conv2d_wgrad_compressed_static.restype = ctypes.c_int
        L.ac_conv2d_wgrad_compressed_static.argtypes = [dp, vp, vp, vp, vp]
        L.ac_wgrad_plan_info.restype = ctypes.c_int
        L.ac_wgrad_plan_info.argtypes = [dp, ctypes.POINTER(ac_plan_info)]
        L.ac_selftest_bounded_wait.restype = ctypes.c_int
        L.ac_selftest_bounded_wait.argtypes = [vp, ctypes.c_uint64, vp]
        L.ac_collapsed_workspace_bytes.restype = sz
        L.ac_collapsed_workspace_bytes.argtypes = [dp, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32)]
        L.ac_conv2d_wgrad_compressed_collapsed.restype = ctypes.c_int
        L.ac_conv2d_wgrad_compressed_collapsed.argtypes = [dp, vp, vp, vp, vp, sz, vp]
        i32 = ctypes.c_int32
        L.ac_workspace_bytes_rect.restype = sz
        L.ac_workspace_bytes_rect.argtypes = [dp, i32, i32]
        L.ac_compress_rect.restype = ctypes.c_int
        L.ac_compress_rect.argtypes = [dp, i32, i32, vp, vp, vp, vp]
        L.ac_conv2d_wgrad_compressed_rect.restype = ctypes.c_int
        L.ac_conv2d_wgrad_compressed_rect.argtypes = [dp, i32, i32, vp, vp, vp, vp, sz, vp]
        L.ac_status_string.restype = ctypes.c_char_p
        L.ac_status_string.argtypes = [ctypes.c_int]
        _lib = L
    return _lib


@dataclass(frozen=True)
class ConvDesc:
    """Python mirror of ac_conv_desc (see include/ac.h)."""
    N: int
    C_in: int
    C_out: int
    H: int
    W: int
    R: int = 1
    S: int = 1
    stride: tuple = (1, 1)
    pad: tuple = (0, 0)
    k: int = 2
    dtype: str = "bf16"
    layout: str = "nhwc"

    def c(self) -> ac_conv_desc:
        return ac_conv_desc(self.N, self.C_in, self.C_out, self.H, self.W, self.R, self.S,
                            self.stride[0], self.stride[1], self.pad[0], self.pad[1], self.k,
                            _DTYPES[self.dtype], _LAYOUTS[self.layout])

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def Hp(self): return -(-self.H // self.k)
    @property
    def Wp(self): return -(-self.W // self.k)
    @property
    def Ho(self): return (self.H + 2 * self.pad[0] - self.R) // self.stride[0] + 1
    @property
    def Wo(self): return (self.W + 2 * self.pad[1] - self.S) // self.stride[1] + 1

    def shape(self, C, H, W):
        return (self.N, C, H, W) if self.layout == "nchw" else (self.N, H, W, C)

    @property
    def x_shape(self): return self.shape(self.C_in, self.H, self.W)
    @property
    def z_shape(self): return self.shape(self.C_in, self.Hp, self.Wp)
    @property
    def dy_shape(self): return self.shape(self.C_out, self.Ho, self.Wo)
    @property
    def dw_shape(self):
        return ((self.C_out, self.C_in, self.R, self.S) if self.layout == "nchw"
                else (self.C_out, self.R, self.S, self.C_in))
    @property
    def flops(self):
        """Dense-equivalent FLOPs of the weight gradient (padding taps counted)."""
        return 2 * self.N * self.Ho * self.Wo * self.C_out * self.C_in * self.R * self.S


def status_string(status: int) -> str:
    return lib().ac_status_string(int(status)).decode()


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def ac_workspace_bytes(desc: ConvDesc) -> int:
    c = desc.c()
    return int(lib().ac_workspace_bytes(ctypes.byref(c)))


def ac_workspace_bytes_min(desc: ConvDesc) -> int:
    c = desc.c()
    return int(lib().ac_workspace_bytes_min(ctypes.byref(c)))


def ac_compress(desc: ConvDesc, x, z, y_out=None, stream=None) -> None:
    c = desc.c()
    st = lib().ac_compress(ctypes.byref(c), _ptr(x), _ptr(z), _ptr(y_out), _stream(stream))
    if st != AC_OK:
        raise AcError(st, "ac_compress")


def ac_compress_relu_mask(desc: ConvDesc, a, z, mask, stream=None) -> None:
    c = desc.c()
    st = lib().ac_compress_relu_mask(ctypes.byref(c), _ptr(a), _ptr(z), _ptr(mask), _stream(stream))
    if st != AC_OK:
        raise AcError(st, "ac_compress_relu_mask")


def ac_compress_relu_mask_y(desc: ConvDesc, a, y_out, z, mask, stream=None) -> None:
    """Y = max(A, 0) (y_out may be a), Z = pool(Y) and the sign mask in one pass."""
    c = desc.c()
    st = lib().ac_compress_relu_mask_y(ctypes.byref(c), _ptr(a), _ptr(y_out), _ptr(z), _ptr(mask), _stream(stream))
    if st != AC_OK:
        raise AcError(st, "ac_compress_relu_mask_y")


def ac_relu_mask_backward(desc: ConvDesc, mask, dy, dx, stream=None) -> None:
    """dx = dy where the mask's bit is set, else 0 (elements in memory order); dx may be dy."""
    c = desc.c()
    st = lib().ac_relu_mask_backward(ctypes.byref(c), _ptr(mask), _ptr(dy), _ptr(dx), _stream(stream))
    if st != AC_OK:
        raise AcError(st, "ac_relu_mask_backward")


def ac_conv2d_wgrad_compressed(desc: ConvDesc, z, dy, dw, workspace, workspace_bytes=None,
                               stream=None) -> None:
    c = desc.c()
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    st = lib().ac_conv2d_wgrad_compressed(ctypes.byref(c), _ptr(z), _ptr(dy), _ptr(dw),
                                          _ptr(workspace), workspace_bytes, _stream(stream))
    if st != AC_OK:
        raise AcError(st, "ac_conv2d_wgrad_compressed")


def ac_accumulate_workspace_bytes(desc: ConvDesc) -> int:
    c = desc.c()
    return int(lib().ac_accumulate_workspace_bytes(ctypes.byref(c)))


def ac_conv2d_wgrad_compressed_accumulate(desc: ConvDesc, z, dy, beta, dw, workspace, workspace_bytes=None,
                                          stream=None) -> None:
    c = desc.c()
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    st = lib().ac_conv2d_wgrad_compressed_accumulate(ctypes.byref(c), _ptr(z), _ptr(dy), float(beta), _ptr(dw),
                                                     _ptr(workspace), workspace_bytes, _stream(stream))
    if st != AC_OK:
        raise AcError(st, "ac_conv2d_wgrad_compressed_accumulate")


def ac_set_kernel_timing_events(before=None, after=None) -> None:
    """`before`, `after`: torch.cuda.Event objects (already recorded once or created eagerly, so that
    their handles exist) or raw cudaEvent_t integers; None clears."""
    def raw(e):
        if e is None:
            return None
        return int(getattr(e, "cuda_event", e))
    st = lib().ac_set_kernel_timing_events(raw(before), raw(after))
    if st != AC_OK:
        raise AcError(st, "ac_set_kernel_timing_events")


def ac_set_sm_budget(sms: int) -> None:
    """SMs the calling thread's weight-gradient plans may count on (0: the whole GPU); see ac.h."""
    st = lib().ac_set_sm_budget(int(sms))
    if st != AC_OK:
        raise AcError(st, "ac_set_sm_budget")


def ac_get_sm_budget() -> int:
    return int(lib().ac_get_sm_budget())


def ac_workspace_status(workspace, stream=None):
    detail = ctypes.c_uint32(0)
    st = lib().ac_workspace_status(_ptr(workspace), _stream(stream), ctypes.byref(detail))
    return int(st), int(detail.value)


def ac_host_step_arena_bytes(desc: ConvDesc) -> int:
    c = desc.c()
    return int(lib().ac_host_step_arena_bytes(ctypes.byref(c)))


def ac_backward_step_host(desc: ConvDesc, x_host, dy_host, dw_host, z_host, arena,
                          arena_bytes=None, stream=None) -> None:
    c = desc.c()
    if arena_bytes is None:
        arena_bytes = arena.numel() * arena.element_size()
    st = lib().ac_backward_step_host(ctypes.byref(c), _ptr(x_host), _ptr(dy_host), _ptr(dw_host),
                                     _ptr(z_host), _ptr(arena), arena_bytes, _stream(stream))
    if st != AC_OK:
        raise AcError(st, "ac_backward_step_host")


def ac_conv2d_wgrad_compressed_static(desc: ConvDesc, z, dy, dw, stream=None) -> None:
    """dW without a workspace argument: the scratch is a fixed array inside the
    library (see include/ac.h). For callers that cannot allocate device memory."""
    c = desc.c()
    st = lib().ac_conv2d_wgrad_compressed_static(ctypes.byref(c), _ptr(z), _ptr(dy), _ptr(dw),
                                                 _stream(stream))
    if st != AC_OK:
        raise AcError(st, "ac_conv2d_wgrad_compressed_static")


def ac_workspace_bytes_rect(desc: ConvDesc, k_h: int, k_w: int) -> int:
    c = desc.c()
    return int(lib().ac_workspace_bytes_rect(ctypes.byref(c), k_h, k_w))


def ac_compress_rect(desc: ConvDesc, k_h: int, k_w: int, x, z, y_out=None, stream=None) -> None:
    c = desc.c()
    st = lib().ac_compress_rect(ctypes.byref(c), k_h, k_w, _ptr(x), _ptr(z), _ptr(y_out), _stream(stream))
    if st != AC_OK:
        raise AcError(st, "ac_compress_rect")


def ac_conv2d_wgrad_compressed_rect(desc: ConvDesc, k_h: int, k_w: int, z, dy, dw, workspace,
                                    workspace_bytes=None, stream=None) -> None:
    c = desc.c()
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    st = lib().ac_conv2d_wgrad_compressed_rect(ctypes.byref(c), k_h, k_w, _ptr(z), _ptr(dy), _ptr(dw),
                                               _ptr(workspace), workspace_bytes, _stream(stream))
    if st != AC_OK:
        raise AcError(st, "ac_conv2d_wgrad_compressed_rect")


def ac_wgrad_plan_info(desc: ConvDesc) -> dict:
    """How the library will run this problem (host arithmetic only)."""
    c = desc.c()
    info = ac_plan_info()
    st = lib().ac_wgrad_plan_info(ctypes.byref(c), ctypes.byref(info))
    if st != AC_OK:
        raise AcError(st, "ac_wgrad_plan_info")
    return {n: getattr(info, n) for n, _ in ac_plan_info._fields_}


def ac_selftest_bounded_wait(workspace, limit_cycles: int, stream=None) -> None:
    st = lib().ac_selftest_bounded_wait(_ptr(workspace), int(limit_cycles), _stream(stream))
    if st != AC_OK:
        raise AcError(st, "ac_selftest_bounded_wait")


def ac_collapsed_workspace_bytes(desc: ConvDesc):
    """(bytes, tiles accumulated in the collapsed form, tiles in the dense form); bytes == 0 if
    the problem is not taken in the collapsed form."""
    c = desc.c()
    a, b = ctypes.c_int32(0), ctypes.c_int32(0)
    n = int(lib().ac_collapsed_workspace_bytes(ctypes.byref(c), ctypes.byref(a), ctypes.byref(b)))
    return n, int(a.value), int(b.value)


def ac_conv2d_wgrad_compressed_collapsed(desc: ConvDesc, z, dy, dw, workspace, workspace_bytes=None,
                                         stream=None) -> None:
    c = desc.c()
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    st = lib().ac_conv2d_wgrad_compressed_collapsed(ctypes.byref(c), _ptr(z), _ptr(dy), _ptr(dw),
                                                    _ptr(workspace), workspace_bytes, _stream(stream))
    if st != AC_OK:
        raise AcError(st, "ac_conv2d_wgrad_compressed_collapsed")
