"""Seeded, counter-keyed generators for parameters and gradients.

Every array is a pure function of (seed, tensor index, step): the oracle's
tests and the CUDA path's tests call the same functions and therefore see the
same bits.  Gradients that a workload stores as bf16 are rounded here (round to
nearest even) and handed out both as the rounded fp32 values and as the raw
16-bit patterns, so neither consumer has to round anything itself.
"""
from __future__ import annotations

import numpy as np

from .shapes import Tensor, Workload, ROLE_VECTOR

_SIGMA = 1e-3          # "N(0, 1e-3)" is read as standard deviation 1e-3
_STREAM_PARAM = 0x5eed0001
_STREAM_GRAD = 0x5eed0002
_STREAM_ROWS = 0x5eed0003


def _rng(stream: int, seed: int, a: int, b: int = 0) -> np.random.Generator:
    # Philox is counter based: the 128-bit key selects an independent stream.
    key = (int(stream) << 32 | (int(seed) & 0xFFFFFFFF), (int(a) & 0xFFFFFFFF) << 32 | (int(b) & 0xFFFFFFFF))
    return np.random.Generator(np.random.Philox(key=np.array(key, dtype=np.uint64)))


def init_params(t: Tensor, tensor_index: int, seed: int = 1) -> np.ndarray:
    """Initial fp32 parameters of one tensor: N(0, 0.02^2), ones or zeros."""
    if t.init == "ones":
        return np.ones((t.rows, t.cols), dtype=np.float32)
    if t.init == "zeros":
        return np.zeros((t.rows, t.cols), dtype=np.float32)
    r = _rng(_STREAM_PARAM, seed, tensor_index)
    x = r.standard_normal((t.rows, t.cols), dtype=np.float32)
    x *= np.float32(0.02)
    return x


def row_scales(w: Workload, t: Tensor, tensor_index: int, seed: int = 0) -> np.ndarray | None:
    """Per-row multipliers of a tensor's gradient; fixed over steps."""
    if w.grad_recipe == "rowscale":
        r = _rng(_STREAM_ROWS, seed, tensor_index)
        # log-uniform on [0.1, 10]
        return np.exp(r.uniform(np.log(0.1), np.log(10.0), size=(t.rows, 1))).astype(np.float32)
    if w.grad_recipe == "heavyrows":
        r = _rng(_STREAM_ROWS, seed, tensor_index)
        heavy = r.random(size=(t.rows, 1)) < 0.05
        return np.where(heavy, np.float32(100.0), np.float32(1.0)).astype(np.float32)
    return None


def grad_for_tensor(w: Workload, tensor_index: int, step: int, seed: int = 0) -> np.ndarray:
    """fp32 gradient of tensor `tensor_index` at 1-based `step`, before dtype rounding."""
    t = w.tensors[tensor_index]
    r = _rng(_STREAM_GRAD, seed, tensor_index, step)
    shape = (t.rows, t.cols)
    if w.grad_recipe == "student_t3":
        x = r.standard_t(3.0, size=shape).astype(np.float32)
    else:
        x = r.standard_normal(shape, dtype=np.float32)
    x *= np.float32(_SIGMA)
    s = row_scales(w, t, tensor_index, seed)
    if s is not None and t.role != ROLE_VECTOR:
        x *= s
    return x


def round_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to bf16 (nearest even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    rounded = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def to_grad_dtype(x: np.ndarray, dtype: str):
    """Return (values, raw): the fp32 values the device will see, and the raw storage.

    dtype "f32": both are x itself.  dtype "bf16": raw is a uint16 array of bit
    patterns and values is raw widened back to fp32 (exact).
    """
    if dtype == "f32":
        x = np.ascontiguousarray(x, dtype=np.float32)
        return x, x
    if dtype == "bf16":
        bits = round_to_bf16_bits(x)
        return bf16_bits_to_f32(bits).reshape(x.shape), bits.reshape(x.shape)
    raise ValueError(dtype)


class GradPool:
    """Cheap stand-in gradients for tensors no oracle looks at.

    A full-size run needs 1.5e9 fresh values per step although the oracle
    follows only a sample of the blocks.  Tensors outside the sample take a
    window of one pre-drawn pool (same distribution and dtype) at an offset
    that depends on (tensor, step); tensors inside the sample always use
    grad_for_tensor.
    """

    def __init__(self, w: Workload, pool_elems: int = 1 << 25, seed: int = 0):
        self.w = w
        r = _rng(_STREAM_GRAD, seed, 0xFFFFFF, 0)
        if w.grad_recipe == "student_t3":
            x = r.standard_t(3.0, size=pool_elems).astype(np.float32)
        else:
            x = r.standard_normal(pool_elems, dtype=np.float32)
        x *= np.float32(_SIGMA)
        self.values, self.raw = to_grad_dtype(x, w.grad_dtype)
        self.n = pool_elems

    def window(self, tensor_index: int, step: int, numel: int) -> np.ndarray:
        """Raw-storage window of `numel` elements (wraps around the pool)."""
        start = ((tensor_index * 0x9E3779B1 + step * 0x85EBCA77) & 0x7FFFFFFF) % self.n
        start -= start % 8
        if start + numel <= self.n:
            return self.raw[start:start + numel]
        reps = -(-(start + numel) // self.n)
        return np.tile(self.raw, reps)[start:start + numel]
