"""Seeded synthetic inputs with the shapes of ViT activations.

This module is the only code shared by the CUDA path's tests/benchmark and the CPU
oracle's tests.  It holds no arithmetic of the method itself: it draws random
tensors, rounds them to the I/O type, and names the workload shapes.  Every stream is
a counter-based Philox generator keyed by (seed, stream name), so any tensor can be
regenerated on its own, in any order.

Workloads (stand-ins for the image-classification fine-tuning runs the paper
measures; the shapes are those of ViT-B/16, ViT-L/16 and ViT-H/14 at 224 px):

* GELU pre-activations: ``0.9 z + 0.1 (2 t3)`` with ``z ~ N(0,1)`` and ``t3`` a
  Student-t variate with 3 degrees of freedom built from four normals -- a Gaussian
  bulk with a heavy tail, so a few percent of the values fall outside [-2, 2].
* Attention logits: ``2 z + u_row`` with one offset ``u_row ~ U(-5, 5)`` per row.
* Upstream gradients: ``scale * z``.
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass

import numpy as np

F32 = 0
BF16 = 1

_CHUNK = 1 << 22  # elements drawn per internal step (bounds temporary memory)


def generator(seed: int, *stream) -> np.random.Generator:
    """Philox generator keyed by the seed and a hash of the stream name."""
    h = hashlib.blake2b(repr(stream).encode(), digest_size=8).digest()
    key = np.array([np.uint64(seed), np.uint64(int.from_bytes(h, "little"))], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """binary32 -> bfloat16 bit patterns, round-to-nearest-even (finite inputs)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def to_io(a: np.ndarray, dt: int) -> np.ndarray:
    """float32 array -> the I/O representation (float32, or uint16 bfloat16 bits)."""
    return np.ascontiguousarray(a, dtype=np.float32) if dt == F32 else f32_to_bf16_bits(a)


def io_to_f32(a: np.ndarray, dt: int) -> np.ndarray:
    return np.asarray(a, dtype=np.float32) if dt == F32 else bf16_bits_to_f32(a)


def io_numpy_dtype(dt: int):
    return np.float32 if dt == F32 else np.uint16


def io_itemsize(dt: int) -> int:
    return 4 if dt == F32 else 2


def _fill(out: np.ndarray, draw) -> np.ndarray:
    flat = out.reshape(-1)
    for lo in range(0, flat.size, _CHUNK):
        hi = min(flat.size, lo + _CHUNK)
        flat[lo:hi] = draw(hi - lo)
    return out


def normal(seed: int, stream, n: int, scale: float = 1.0) -> np.ndarray:
    g = generator(seed, *stream)
    out = np.empty(n, dtype=np.float32)
    return _fill(out, lambda m: g.standard_normal(m, dtype=np.float32) * np.float32(scale))


def gelu_preact(seed: int, stream, n: int) -> np.ndarray:
    """Gaussian bulk plus a Student-t(3) tail (a sum, not a mixture)."""
    g = generator(seed, *stream)

    def draw(m):
        z = g.standard_normal((5, m), dtype=np.float32)
        t3 = z[1] / np.sqrt((z[2] * z[2] + z[3] * z[3] + z[4] * z[4]) / np.float32(3.0))
        return np.float32(0.9) * z[0] + np.float32(0.2) * t3

    return _fill(np.empty(n, dtype=np.float32), draw)


def softmax_logits(seed: int, stream, rows: int, row_len: int) -> np.ndarray:
    g = generator(seed, *stream)
    out = np.empty((rows, row_len), dtype=np.float32)
    step = max(1, _CHUNK // row_len)
    for lo in range(0, rows, step):
        hi = min(rows, lo + step)
        z = g.standard_normal((hi - lo, row_len), dtype=np.float32)
        u = g.uniform(-5.0, 5.0, size=(hi - lo, 1)).astype(np.float32)
        out[lo:hi] = np.float32(2.0) * z + u
    return out.reshape(-1)


# ------------------------------------------------------------------ workload shapes
@dataclass(frozen=True)
class VitShape:
    name: str
    batch: int
    tokens: int
    hidden: int   # MLP hidden width = GELU row length
    heads: int
    blocks: int
    dtype: int

    @property
    def gelu_rows(self) -> int:
        return self.batch * self.tokens

    @property
    def gelu_elems(self) -> int:
        return self.gelu_rows * self.hidden

    @property
    def softmax_rows(self) -> int:
        return self.batch * self.heads * self.tokens

    @property
    def softmax_elems(self) -> int:
        return self.softmax_rows * self.tokens


VIT_B16_B8_F32 = VitShape("vit_b16_b8_f32_gelu", 8, 197, 3072, 12, 1, F32)
VIT_B16_B64 = VitShape("vit_b16_b64_bf16", 64, 197, 3072, 12, 12, BF16)
VIT_L16_B64 = VitShape("vit_l16_b64_bf16", 64, 197, 4096, 16, 24, BF16)
VIT_H14_B32 = VitShape("vit_h14_b32_bf16", 32, 257, 5120, 16, 32, BF16)

SHAPES = {s.name: s for s in (VIT_B16_B8_F32, VIT_B16_B64, VIT_L16_B64, VIT_H14_B32)}

GRAD_SCALE = 0.01


def vit_gelu_inputs(shape: VitShape, seed: int, block: int, rows: int | None = None):
    """(x, grad_out) in I/O representation for one block's GELU, optionally the first rows."""
    rows = shape.gelu_rows if rows is None else rows
    n = rows * shape.hidden
    if shape.name == VIT_B16_B8_F32.name:  # the single-layer case: plain N(0,1) for both
        x = normal(seed, (shape.name, block, "gelu_x"), n)
        g = normal(seed, (shape.name, block, "gelu_g"), n)
    else:
        x = gelu_preact(seed, (shape.name, block, "gelu_x"), n)
        g = normal(seed, (shape.name, block, "gelu_g"), n, GRAD_SCALE)
    return to_io(x, shape.dtype), to_io(g, shape.dtype)


def vit_softmax_inputs(shape: VitShape, seed: int, block: int, rows: int | None = None):
    rows = shape.softmax_rows if rows is None else rows
    x = softmax_logits(seed, (shape.name, block, "softmax_x"), rows, shape.tokens)
    g = normal(seed, (shape.name, block, "softmax_g"), rows * shape.tokens, GRAD_SCALE)
    return to_io(x, shape.dtype), to_io(g, shape.dtype)

