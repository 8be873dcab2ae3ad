"""Seeded synthetic inputs for the compressed-activation backward path.

This module holds no arithmetic of the method itself (no pooling, no
convolution): it only draws random tensors of the shapes and value
distributions that convolution layers see during training, and converts
between storage formats. Both the CPU checker and the CUDA library are fed
from here so that they see identical bits.

Generator (version independent, counter based):
  u64 stream  = splitmix64 finaliser applied to (seed, stream_id, counter)
  uniforms    = top 53 bits / 2^53, shifted into (0, 1]
  normals     = Box-Muller on consecutive uniform pairs

Workload recipe (stands in for post-ReLU ResNet activations and their output
gradients, which need a dataset and trained weights):
  X  = max(g, 0), g ~ N(0, 1)      -> about half the entries are exact zeros
  dY ~ N(0, (1e-2)^2)
"""
from __future__ import annotations

import numpy as np
import torch

_MASK = np.uint64(0xFFFFFFFFFFFFFFFF)


def _splitmix64(x: np.ndarray) -> np.ndarray:
    """splitmix64 output function on an array of uint64 counters."""
    with np.errstate(over="ignore"):
        x = (x + np.uint64(0x9E3779B97F4A7C15)) & _MASK
        z = x
        z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _MASK
        z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _MASK
        z = z ^ (z >> np.uint64(31))
    return z


def uniform01(seed: int, stream: int, n: int) -> np.ndarray:
    """n doubles in (0, 1], a pure function of (seed, stream, index)."""
    with np.errstate(over="ignore"):
        base = _splitmix64(np.array([seed], dtype=np.uint64))[0]
        base = _splitmix64(np.array([base ^ np.uint64(stream)], dtype=np.uint64))[0]
        ctr = np.arange(n, dtype=np.uint64) + base
    bits = _splitmix64(ctr) >> np.uint64(11)
    return (bits.astype(np.float64) + 1.0) * (1.0 / 9007199254740992.0)


def normal(seed: int, stream: int, shape, std: float = 1.0) -> np.ndarray:
    """float64 N(0, std^2) samples of the given shape (Box-Muller)."""
    n = int(np.prod(shape))
    m = (n + 1) // 2
    u = uniform01(seed, stream, 2 * m)
    r = np.sqrt(-2.0 * np.log(u[:m]))
    t = (2.0 * np.pi) * u[m:]
    out = np.concatenate([r * np.cos(t), r * np.sin(t)])[:n]
    return (out * std).reshape(shape)


def to_storage(a: np.ndarray, dtype: str) -> torch.Tensor:
    """Round a float64 array once (nearest-even) to the storage dtype."""
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype == "f32":
        return t.to(torch.float32)
    if dtype == "bf16":
        return t.to(torch.float32).to(torch.bfloat16)
    raise ValueError(dtype)


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Exact widening of a stored tensor to float64 (NumPy)."""
    return t.detach().cpu().to(torch.float64).numpy()


def activation(seed: int, shape_nchw, dtype: str, stream: int = 1) -> torch.Tensor:
    """Post-ReLU activation X = max(N(0,1), 0), logical NCHW, stored dtype."""
    g = normal(seed, stream, shape_nchw)
    return to_storage(np.maximum(g, 0.0), dtype)


def pre_activation(seed: int, shape_nchw, dtype: str, stream: int = 3) -> torch.Tensor:
    """Pre-ReLU tensor A ~ N(0,1) (input of the fused ReLU+compress path)."""
    return to_storage(normal(seed, stream, shape_nchw), dtype)


def grad_output(seed: int, shape_nchw, dtype: str, stream: int = 2) -> torch.Tensor:
    """Output gradient dY ~ N(0, 1e-2^2), logical NCHW, stored dtype."""
    return to_storage(normal(seed, stream, shape_nchw, std=1e-2), dtype)


def to_layout(t_nchw: torch.Tensor, layout: str) -> torch.Tensor:
    """Return a dense buffer holding the logical NCHW tensor in `layout`
    ("nchw": [N,C,H,W] contiguous; "nhwc": [N,H,W,C] contiguous)."""
    if layout == "nchw":
        return t_nchw.contiguous()
    if layout == "nhwc":
        return t_nchw.permute(0, 2, 3, 1).contiguous()
    raise ValueError(layout)


def from_layout(buf: torch.Tensor, layout: str) -> torch.Tensor:
    """Inverse of to_layout: a logical NCHW view of a dense buffer."""
    if layout == "nchw":
        return buf
    if layout == "nhwc":
        return buf.permute(0, 3, 1, 2)
    raise ValueError(layout)
