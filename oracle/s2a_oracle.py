"""ctypes front end of the CPU oracle (``s2a_oracle.cpp``).  TEST INFRASTRUCTURE.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
module.  It compiles the oracle with g++ on first use and exposes its functions on
numpy arrays.  bfloat16 tensors travel as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "s2a_oracle.cpp")
_OUT_DIR = os.path.join(_HERE, "_build")
_OUT = os.path.join(_OUT_DIR, "libs2a_oracle.so")

F32 = 0
BF16 = 1

_lock = threading.Lock()
_lib = None

# The flags are part of the oracle's definition: no FMA contraction, no fast-math.
CXXFLAGS = ["-O2", "-std=c++17", "-ffp-contract=off", "-fPIC", "-shared", "-pthread"]


def build(force: bool = False) -> str:
    """Compile the oracle shared object if it is missing or older than its source."""
    with _lock:
        stale = (not os.path.exists(_OUT)) or os.path.getmtime(_OUT) < os.path.getmtime(_SRC)
        if force or stale:
            os.makedirs(_OUT_DIR, exist_ok=True)
            tmp = _OUT + ".tmp.%d" % os.getpid()
            subprocess.run(["g++", *CXXFLAGS, _SRC, "-o", tmp], check=True)
            os.replace(tmp, _OUT)
    return _OUT


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        c = ctypes
        sz, vp, dbl, flt, i32 = c.c_size_t, c.c_void_p, c.c_double, c.c_float, c.c_int
        for name in ("s2a_oracle_gelu", "s2a_oracle_gelu_grad_exact", "s2a_oracle_gelu_grad_sine",
                     "s2a_oracle_silu", "s2a_oracle_silu_grad"):
            getattr(L, name).argtypes = [dbl]
            getattr(L, name).restype = dbl
        L.s2a_oracle_softmax_row.argtypes = [vp, vp, sz]
        L.s2a_oracle_softmax_row.restype = None
        L.s2a_oracle_softmax_vjp_row.argtypes = [vp, vp, vp, sz]
        L.s2a_oracle_softmax_vjp_row.restype = None
        L.s2a_oracle_quantize_row.argtypes = [vp, sz, vp, vp, vp]
        L.s2a_oracle_quantize_row.restype = None
        L.s2a_oracle_quantize_row_definition.argtypes = [vp, sz, vp]
        L.s2a_oracle_quantize_row_definition.restype = None
        L.s2a_oracle_pack.argtypes = [vp, sz, vp]
        L.s2a_oracle_pack.restype = None
        L.s2a_oracle_unpack.argtypes = [vp, sz, vp]
        L.s2a_oracle_unpack.restype = None
        L.s2a_oracle_dequantize.argtypes = [c.c_uint8, flt, flt]
        L.s2a_oracle_dequantize.restype = dbl
        L.s2a_oracle_round_bf16.argtypes = [dbl]
        L.s2a_oracle_round_bf16.restype = c.c_uint16
        L.s2a_oracle_bf16_to_float.argtypes = [c.c_uint16]
        L.s2a_oracle_bf16_to_float.restype = flt
        for name in ("s2a_oracle_gelu_fwd", "s2a_oracle_softmax_fwd", "s2a_oracle_silu_fwd"):
            getattr(L, name).argtypes = [vp, vp, vp, vp, sz, sz, i32, i32]
            getattr(L, name).restype = i32
        for name in ("s2a_oracle_gelu_bwd", "s2a_oracle_softmax_bwd", "s2a_oracle_silu_bwd"):
            getattr(L, name).argtypes = [vp, vp, vp, vp, sz, sz, i32, i32]
            getattr(L, name).restype = i32
        L.s2a_oracle_gelu_fwd_tensor_range.argtypes = [vp, vp, vp, vp, sz, sz, i32]
        L.s2a_oracle_gelu_fwd_tensor_range.restype = i32
        L.s2a_oracle_fwd_bits.argtypes = [i32, vp, vp, vp, vp, sz, sz, i32, i32]
        L.s2a_oracle_fwd_bits.restype = i32
        L.s2a_oracle_bwd_bits.argtypes = [i32, vp, vp, vp, vp, sz, sz, i32, i32]
        L.s2a_oracle_bwd_bits.restype = i32
        L.s2a_oracle_quantize_row_levels.argtypes = [vp, sz, i32, vp, vp, vp]
        L.s2a_oracle_quantize_row_levels.restype = None
        L.s2a_oracle_pack_bits.argtypes = [vp, sz, i32, vp]
        L.s2a_oracle_pack_bits.restype = None
        L.s2a_oracle_unpack_bits.argtypes = [vp, sz, i32, vp]
        L.s2a_oracle_unpack_bits.restype = None
        L.s2a_oracle_quantize_tensor.argtypes = [vp, vp, vp, sz, sz, i32, i32]
        L.s2a_oracle_quantize_tensor.restype = i32
        L.s2a_oracle_relu_fwd.argtypes = [vp, vp, vp, sz, i32]
        L.s2a_oracle_relu_fwd.restype = i32
        L.s2a_oracle_relu_bwd.argtypes = [vp, vp, vp, sz, i32]
        L.s2a_oracle_relu_bwd.restype = i32
        L.s2a_oracle_cap_fwd.argtypes = [vp, vp, sz, sz, sz, i32]
        L.s2a_oracle_cap_fwd.restype = i32
        L.s2a_oracle_cap_bwd.argtypes = [vp, vp, sz, sz, sz, i32]
        L.s2a_oracle_cap_bwd.restype = i32
        L.s2a_oracle_lrp_fwd.argtypes = [vp, vp, vp, vp, sz, sz, sz, sz, i32]
        L.s2a_oracle_lrp_fwd.restype = i32
        L.s2a_oracle_hardware_threads.argtypes = []
        L.s2a_oracle_hardware_threads.restype = i32
        _lib = L
    return _lib


def _ptr(a: np.ndarray):
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(ctypes.c_void_p)


def _io_dtype(dt: int):
    return np.float32 if dt == F32 else np.uint16


def _check_io(a: np.ndarray, dt: int) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != _io_dtype(dt):
        raise TypeError("expected %s for dtype code %d, got %s" % (_io_dtype(dt), dt, a.dtype))
    return a


def codes_bytes(n: int) -> int:
    return (n + 1) // 2


# ------------------------------------------------------------------ scalar blocks
def gelu(x: float) -> float:
    return lib().s2a_oracle_gelu(float(x))


def gelu_grad_exact(x: float) -> float:
    return lib().s2a_oracle_gelu_grad_exact(float(x))


def gelu_grad_sine(x: float) -> float:
    return lib().s2a_oracle_gelu_grad_sine(float(x))


def softmax_row(x) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float64)
    y = np.empty_like(x)
    lib().s2a_oracle_softmax_row(_ptr(x), _ptr(y), x.size)
    return y


def softmax_vjp_row(y, g) -> np.ndarray:
    y = np.ascontiguousarray(y, dtype=np.float64)
    g = np.ascontiguousarray(g, dtype=np.float64)
    out = np.empty_like(y)
    lib().s2a_oracle_softmax_vjp_row(_ptr(y), _ptr(g), _ptr(out), y.size)
    return out


def quantize_row(v):
    """Eq. 8 in its binary32 specification.  Returns (codes uint8[n], min, s)."""
    v = np.ascontiguousarray(v, dtype=np.float32)
    q = np.empty(v.size, dtype=np.uint8)
    mn = np.empty(1, dtype=np.float32)
    s = np.empty(1, dtype=np.float32)
    lib().s2a_oracle_quantize_row(_ptr(v), v.size, _ptr(q), _ptr(mn), _ptr(s))
    return q, np.float32(mn[0]), np.float32(s[0])


def quantize_row_definition(v) -> np.ndarray:
    v = np.ascontiguousarray(v, dtype=np.float32)
    q = np.empty(v.size, dtype=np.uint8)
    lib().s2a_oracle_quantize_row_definition(_ptr(v), v.size, _ptr(q))
    return q


def pack(q) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.uint8)
    out = np.empty(codes_bytes(q.size), dtype=np.uint8)
    lib().s2a_oracle_pack(_ptr(q), q.size, _ptr(out))
    return out


def unpack(b, n: int) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint8)
    assert b.size >= codes_bytes(n)
    out = np.empty(n, dtype=np.uint8)
    lib().s2a_oracle_unpack(_ptr(b), n, _ptr(out))
    return out


def dequantize(q: int, mn, s) -> float:
    return lib().s2a_oracle_dequantize(int(q), float(mn), float(s))


def round_bf16(d: float) -> int:
    return int(lib().s2a_oracle_round_bf16(float(d)))


def bf16_to_float(b: int) -> float:
    return float(lib().s2a_oracle_bf16_to_float(int(b)))


def hardware_threads() -> int:
    return int(lib().s2a_oracle_hardware_threads())


# ------------------------------------------------------------------ tensor entry points
def _fwd(fn, x, L, dt, threads):
    x = _check_io(x, dt).reshape(-1)
    n = x.size
    y = np.empty_like(x)
    codes = np.zeros(codes_bytes(n), dtype=np.uint8)
    meta = np.zeros(2 * (n // L if L else 0), dtype=np.float32)
    rc = fn(_ptr(x), _ptr(y), _ptr(codes), _ptr(meta), n, L, dt, threads)
    if rc != 0:
        raise ValueError("oracle rejected the shape (n=%d, row_len=%d)" % (n, L))
    return y, codes, meta


def _bwd(fn, g, codes, meta, L, dt, threads):
    g = _check_io(g, dt).reshape(-1)
    n = g.size
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    meta = np.ascontiguousarray(meta, dtype=np.float32)
    assert codes.size >= codes_bytes(n) and meta.size >= 2 * (n // L)
    gin = np.empty_like(g)
    rc = fn(_ptr(g), _ptr(codes), _ptr(meta), _ptr(gin), n, L, dt, threads)
    if rc != 0:
        raise ValueError("oracle rejected the shape (n=%d, row_len=%d)" % (n, L))
    return gin


def gelu_fwd(x, row_len: int, dt: int, threads: int = 1):
    """Returns (y, packed codes, meta) for the GELU forward with the 4-bit stash."""
    return _fwd(lib().s2a_oracle_gelu_fwd, x, row_len, dt, threads)


def gelu_fwd_tensor_range(x, row_len: int, dt: int):
    """GELU forward whose 4-bit stash uses ONE (min, s) for the whole tensor."""
    fn = lib().s2a_oracle_gelu_fwd_tensor_range
    return _fwd(lambda a, b, c, d, n, L, t, _threads: fn(a, b, c, d, n, L, t), x, row_len, dt, 1)


def gelu_bwd(g, codes, meta, row_len: int, dt: int, threads: int = 1):
    return _bwd(lib().s2a_oracle_gelu_bwd, g, codes, meta, row_len, dt, threads)


def silu(x: float) -> float:
    return lib().s2a_oracle_silu(float(x))


def silu_grad(x: float) -> float:
    return lib().s2a_oracle_silu_grad(float(x))


def silu_fwd(x, row_len: int, dt: int, threads: int = 1):
    """Returns (y, packed codes, meta) for the SiLU forward with the 4-bit stash."""
    return _fwd(lib().s2a_oracle_silu_fwd, x, row_len, dt, threads)


def silu_bwd(g, codes, meta, row_len: int, dt: int, threads: int = 1):
    return _bwd(lib().s2a_oracle_silu_bwd, g, codes, meta, row_len, dt, threads)


def softmax_fwd(x, row_len: int, dt: int, threads: int = 1):
    return _fwd(lib().s2a_oracle_softmax_fwd, x, row_len, dt, threads)


def softmax_bwd(g, codes, meta, row_len: int, dt: int, threads: int = 1):
    return _bwd(lib().s2a_oracle_softmax_bwd, g, codes, meta, row_len, dt, threads)


def mask_bytes(n: int) -> int:
    return (n + 7) // 8


def relu_fwd(x, dt: int):
    """Returns (y, bit mask) for the ReLU forward with the 1-bit stash."""
    x = _check_io(x, dt).reshape(-1)
    y = np.empty_like(x)
    mask = np.zeros(mask_bytes(x.size), dtype=np.uint8)
    lib().s2a_oracle_relu_fwd(_ptr(x), _ptr(y), _ptr(mask), x.size, dt)
    return y, mask


def relu_bwd(g, mask, dt: int):
    g = _check_io(g, dt).reshape(-1)
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    assert mask.size >= mask_bytes(g.size)
    gin = np.empty_like(g)
    lib().s2a_oracle_relu_bwd(_ptr(g), _ptr(mask), _ptr(gin), g.size, dt)
    return gin


def cap_fwd(x, n_rows: int, channels: int, r: int, dt: int):
    """Channel Average Pooling (Eq. 5): [n_rows, channels] -> [n_rows, channels / r]."""
    x = _check_io(x, dt).reshape(-1)
    assert x.size == n_rows * channels
    y = np.empty(n_rows * (channels // r if r else 0), dtype=x.dtype)
    if lib().s2a_oracle_cap_fwd(_ptr(x), _ptr(y), n_rows, channels, r, dt) != 0:
        raise ValueError("oracle rejected the shape")
    return y


def cap_bwd(g, n_rows: int, channels: int, r: int, dt: int):
    g = _check_io(g, dt).reshape(-1)
    assert g.size == n_rows * (channels // r)
    gin = np.empty(n_rows * channels, dtype=g.dtype)
    if lib().s2a_oracle_cap_bwd(_ptr(g), _ptr(gin), n_rows, channels, r, dt) != 0:
        raise ValueError("oracle rejected the shape")
    return gin


def lrp_fwd(x, A, B, batch: int, tokens: int, channels: int, rank: int, dt: int):
    """Low-Rank Prompt (Eq. 3): y[b] = x[b] + A @ B for every sample b."""
    x = _check_io(x, dt).reshape(-1)
    A = np.ascontiguousarray(A, dtype=np.float32)
    B = np.ascontiguousarray(B, dtype=np.float32)
    assert x.size == batch * tokens * channels and A.size == tokens * rank and B.size == rank * channels
    y = np.empty_like(x)
    lib().s2a_oracle_lrp_fwd(_ptr(x), _ptr(A), _ptr(B), _ptr(y), batch, tokens, channels, rank, dt)
    return y


def codes_bytes_bits(n: int, bits: int) -> int:
    return (n * bits + 7) // 8


def quantize_row_levels(v, levels: int):
    v = np.ascontiguousarray(v, dtype=np.float32)
    q = np.empty(v.size, dtype=np.uint8)
    mn = np.empty(1, dtype=np.float32)
    s = np.empty(1, dtype=np.float32)
    lib().s2a_oracle_quantize_row_levels(_ptr(v), v.size, levels, _ptr(q), _ptr(mn), _ptr(s))
    return q, np.float32(mn[0]), np.float32(s[0])


def pack_bits(q, bits: int) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.uint8)
    out = np.empty(codes_bytes_bits(q.size, bits), dtype=np.uint8)
    lib().s2a_oracle_pack_bits(_ptr(q), q.size, bits, _ptr(out))
    return out


def unpack_bits(b, n: int, bits: int) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint8)
    out = np.empty(n, dtype=np.uint8)
    lib().s2a_oracle_unpack_bits(_ptr(b), n, bits, _ptr(out))
    return out


def fwd_bits(kind: str, x, row_len: int, bits: int, dt: int):
    """GELU ('gelu') or softmax ('softmax') forward with an N-bit stash; returns (y, codes, meta)."""
    x = _check_io(x, dt).reshape(-1)
    n = x.size
    y = np.empty_like(x)
    codes = np.zeros(codes_bytes_bits(n, bits), dtype=np.uint8)
    meta = np.zeros(2 * (n // row_len if row_len else 0), dtype=np.float32)
    rc = lib().s2a_oracle_fwd_bits(0 if kind == "gelu" else 1, _ptr(x), _ptr(y), _ptr(codes), _ptr(meta), n,
                                   row_len, bits, dt)
    if rc != 0:
        raise ValueError("oracle rejected the shape or the bit width")
    return y, codes, meta


def bwd_bits(kind: str, g, codes, meta, row_len: int, bits: int, dt: int):
    g = _check_io(g, dt).reshape(-1)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    meta = np.ascontiguousarray(meta, dtype=np.float32)
    gin = np.empty_like(g)
    rc = lib().s2a_oracle_bwd_bits(0 if kind == "gelu" else 1, _ptr(g), _ptr(codes), _ptr(meta), _ptr(gin), g.size,
                                   row_len, bits, dt)
    if rc != 0:
        raise ValueError("oracle rejected the shape or the bit width")
    return gin


def quantize_tensor(v, row_len: int, dt: int, threads: int = 1):
    """Eq. 8 + packing over an existing tensor.  Returns (packed codes, meta)."""
    v = _check_io(v, dt).reshape(-1)
    n = v.size
    codes = np.zeros(codes_bytes(n), dtype=np.uint8)
    meta = np.zeros(2 * (n // row_len), dtype=np.float32)
    rc = lib().s2a_oracle_quantize_tensor(_ptr(v), _ptr(codes), _ptr(meta), n, row_len, dt, threads)
    if rc != 0:
        raise ValueError("oracle rejected the shape")
    return codes, meta


def widen(a: np.ndarray, dt: int) -> np.ndarray:
    """I/O array -> float64 values (bfloat16 bit patterns are widened exactly)."""
    if dt == F32:
        return np.asarray(a, dtype=np.float32).astype(np.float64)
    u = np.asarray(a, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)
