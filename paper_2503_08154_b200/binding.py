"""Thin ctypes binding of libs2a.so: argument marshalling only.

Each function takes torch CUDA tensors (PyTorch is used for device memory and streams,
nothing else), passes their raw pointers, the element count, the row length and the
current stream to the C-ABI call of the same name, and raises on a non-zero status.
There is no CPU path: a missing or unloadable library is an error.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libs2a.so")

F32 = 0
BF16 = 1
GELU_FWD, GELU_BWD, SOFTMAX_FWD, SOFTMAX_BWD, SILU_FWD, SILU_BWD = 0, 1, 2, 3, 4, 5

EXPORTS = (
    "s2a_codes_bytes", "s2a_meta_bytes", "s2a_status_string", "s2a_gelu_fwd", "s2a_gelu_bwd",
    "s2a_softmax_fwd", "s2a_softmax_bwd", "s2a_device_error", "s2a_describe_plan",
    "s2a_mask_bytes", "s2a_relu_fwd", "s2a_relu_bwd",
    "s2a_tensor_range_scratch_bytes", "s2a_gelu_fwd_tensor_range",
    "s2a_tensor_range_static_max_elems", "s2a_gelu_fwd_tensor_range_static",
    "s2a_silu_fwd", "s2a_silu_bwd", "s2a_cap_fwd", "s2a_cap_bwd", "s2a_lrp_fwd",
    "s2a_selftest_wait_expiry",
    "s2a_selftest_exp2_monotone",
    "s2a_codes_bytes_bits", "s2a_gelu_fwd_bits", "s2a_gelu_bwd_bits", "s2a_softmax_fwd_bits", "s2a_softmax_bwd_bits",
)

_lib = None


class S2AError(RuntimeError):
    pass


def use_library(path: str) -> None:
    """Loads another build of the library (e.g. libs2a_tuning.so) instead of libs2a.so.
    Must be called before the first call into the library."""
    global LIB_PATH
    if _lib is not None:
        raise S2AError("the library is already loaded")
    LIB_PATH = os.path.abspath(path)


def lib() -> ctypes.CDLL:
    """Loads libs2a.so (built in-tree by ``build.py``); raises if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise S2AError("libs2a.so is not built: run `python -m paper_2503_08154_b200.build` "
                           "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        c = ctypes
        L.s2a_codes_bytes.argtypes = [c.c_size_t]
        L.s2a_codes_bytes.restype = c.c_size_t
        L.s2a_meta_bytes.argtypes = [c.c_size_t, c.c_size_t]
        L.s2a_meta_bytes.restype = c.c_size_t
        L.s2a_status_string.argtypes = [c.c_int]
        L.s2a_status_string.restype = c.c_char_p
        L.s2a_selftest_wait_expiry.argtypes = [c.c_void_p]
        L.s2a_selftest_wait_expiry.restype = c.c_int
        L.s2a_selftest_exp2_monotone.argtypes = [c.POINTER(c.c_ulonglong), c.c_void_p]
        L.s2a_selftest_exp2_monotone.restype = c.c_int
        for name in ("s2a_gelu_fwd", "s2a_softmax_fwd", "s2a_gelu_bwd", "s2a_softmax_bwd", "s2a_silu_fwd",
                     "s2a_silu_bwd"):
            f = getattr(L, name)
            f.argtypes = [c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_size_t, c.c_size_t,
                          c.c_int, c.c_void_p]
            f.restype = c.c_int
        L.s2a_tensor_range_scratch_bytes.argtypes = [c.c_size_t]
        L.s2a_tensor_range_scratch_bytes.restype = c.c_size_t
        L.s2a_gelu_fwd_tensor_range.argtypes = [c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p,
                                                c.c_size_t, c.c_size_t, c.c_int, c.c_void_p]
        L.s2a_gelu_fwd_tensor_range.restype = c.c_int
        L.s2a_tensor_range_static_max_elems.argtypes = []
        L.s2a_tensor_range_static_max_elems.restype = c.c_size_t
        L.s2a_gelu_fwd_tensor_range_static.argtypes = [c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_size_t,
                                                       c.c_size_t, c.c_int, c.c_void_p]
        L.s2a_gelu_fwd_tensor_range_static.restype = c.c_int
        for name in ("s2a_cap_fwd", "s2a_cap_bwd"):
            f = getattr(L, name)
            f.argtypes = [c.c_void_p, c.c_void_p, c.c_size_t, c.c_size_t, c.c_size_t, c.c_int, c.c_void_p]
            f.restype = c.c_int
        L.s2a_lrp_fwd.argtypes = [c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_size_t, c.c_size_t, c.c_size_t,
                                  c.c_size_t, c.c_int, c.c_void_p]
        L.s2a_lrp_fwd.restype = c.c_int
        L.s2a_codes_bytes_bits.argtypes = [c.c_size_t, c.c_int]
        L.s2a_codes_bytes_bits.restype = c.c_size_t
        for name in ("s2a_gelu_fwd_bits", "s2a_gelu_bwd_bits", "s2a_softmax_fwd_bits", "s2a_softmax_bwd_bits"):
            f = getattr(L, name)
            f.argtypes = [c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p, c.c_size_t, c.c_size_t, c.c_int, c.c_int,
                          c.c_void_p]
            f.restype = c.c_int
        L.s2a_mask_bytes.argtypes = [c.c_size_t]
        L.s2a_mask_bytes.restype = c.c_size_t
        for name in ("s2a_relu_fwd", "s2a_relu_bwd"):
            f = getattr(L, name)
            f.argtypes = [c.c_void_p, c.c_void_p, c.c_void_p, c.c_size_t, c.c_int, c.c_void_p]
            f.restype = c.c_int
        L.s2a_device_error.argtypes = [c.POINTER(c.c_uint), c.c_int]
        L.s2a_device_error.restype = c.c_int
        L.s2a_describe_plan.argtypes = [c.c_int, c.c_size_t, c.c_size_t, c.c_int, c.c_char_p, c.c_size_t]
        L.s2a_describe_plan.restype = c.c_int
        _lib = L
    return _lib


def dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise S2AError("unsupported dtype %s (float32 or bfloat16)" % t.dtype)


def codes_bytes(n_elems: int) -> int:
    return int(lib().s2a_codes_bytes(n_elems))


def meta_bytes(n_elems: int, row_len: int) -> int:
    return int(lib().s2a_meta_bytes(n_elems, row_len))


def status_string(status: int) -> str:
    return lib().s2a_status_string(int(status)).decode()


def check(status: int) -> None:
    if status != 0:
        raise S2AError(status_string(status))


_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream_ptr(t: torch.Tensor = None) -> int:
    """The current CUDA stream of the tensor's device (of the current device without one) as
    a raw handle.  torch's raw-stream query is several times cheaper than building a Stream
    object on every call; the slower public route is the fallback."""
    if _raw_stream is not None:
        idx = t.device.index if t is not None and t.device.index is not None else torch.cuda.current_device()
        return _raw_stream(idx)
    return torch.cuda.current_stream(t.device if t is not None else None).cuda_stream


def _dev(t: torch.Tensor, what: str) -> torch.Tensor:
    if not t.is_cuda:
        raise S2AError("%s must be a CUDA tensor" % what)
    if not t.is_contiguous():
        raise S2AError("%s must be contiguous" % what)
    return t


def alloc_stash(n_elems: int, row_len: int, device) -> tuple[torch.Tensor, torch.Tensor]:
    """Device buffers for the packed codes (uint8) and the per-row (min, s) metadata."""
    codes = torch.empty(codes_bytes(n_elems), dtype=torch.uint8, device=device)
    meta = torch.empty(meta_bytes(n_elems, row_len) // 4, dtype=torch.float32, device=device)
    return codes, meta


def _fwd(fn, x, y, codes, meta, row_len):
    _dev(x, "x"), _dev(y, "y"), _dev(codes, "codes"), _dev(meta, "meta")
    n = x.numel()
    if y.numel() != n or y.dtype != x.dtype:
        raise S2AError("y must match x in size and dtype")
    if codes.dtype != torch.uint8 or meta.dtype != torch.float32:
        raise S2AError("codes must be uint8 and meta float32")
    if row_len > 0 and (codes.numel() < codes_bytes(n) or meta.numel() * 4 < meta_bytes(n, row_len)):
        raise S2AError("codes/meta buffers are too small")
    check(fn(x.data_ptr(), y.data_ptr(), codes.data_ptr(), meta.data_ptr(), n, row_len,
             dtype_code(x), _stream_ptr(x)))


def _bwd(fn, grad_out, codes, meta, grad_in, row_len):
    _dev(grad_out, "grad_out"), _dev(grad_in, "grad_in"), _dev(codes, "codes"), _dev(meta, "meta")
    n = grad_out.numel()
    if grad_in.numel() != n or grad_in.dtype != grad_out.dtype:
        raise S2AError("grad_in must match grad_out in size and dtype")
    if codes.dtype != torch.uint8 or meta.dtype != torch.float32:
        raise S2AError("codes must be uint8 and meta float32")
    if row_len > 0 and (codes.numel() < codes_bytes(n) or meta.numel() * 4 < meta_bytes(n, row_len)):
        raise S2AError("codes/meta buffers are too small")
    check(fn(grad_out.data_ptr(), codes.data_ptr(), meta.data_ptr(), grad_in.data_ptr(), n,
             row_len, dtype_code(grad_out), _stream_ptr(grad_out)))


def s2a_gelu_fwd(x, y, codes, meta, row_len: int) -> None:
    _fwd(lib().s2a_gelu_fwd, x, y, codes, meta, row_len)


def s2a_gelu_bwd(grad_out, codes, meta, grad_in, row_len: int) -> None:
    _bwd(lib().s2a_gelu_bwd, grad_out, codes, meta, grad_in, row_len)


def s2a_silu_fwd(x, y, codes, meta, row_len: int) -> None:
    _fwd(lib().s2a_silu_fwd, x, y, codes, meta, row_len)


def s2a_silu_bwd(grad_out, codes, meta, grad_in, row_len: int) -> None:
    _bwd(lib().s2a_silu_bwd, grad_out, codes, meta, grad_in, row_len)


def s2a_softmax_fwd(x, y, codes, meta, row_len: int) -> None:
    _fwd(lib().s2a_softmax_fwd, x, y, codes, meta, row_len)


def s2a_softmax_bwd(grad_out, codes, meta, grad_in, row_len: int) -> None:
    _bwd(lib().s2a_softmax_bwd, grad_out, codes, meta, grad_in, row_len)


def tensor_range_scratch_bytes(n_elems: int) -> int:
    return int(lib().s2a_tensor_range_scratch_bytes(n_elems))


def s2a_gelu_fwd_tensor_range(x, y, codes, meta, scratch, row_len: int) -> None:
    """GELU forward with one quantiser range for the whole tensor; `scratch` is a uint8 CUDA
    tensor of at least tensor_range_scratch_bytes(x.numel()) bytes."""
    _dev(x, "x"), _dev(y, "y"), _dev(codes, "codes"), _dev(meta, "meta"), _dev(scratch, "scratch")
    n = x.numel()
    if y.numel() != n or y.dtype != x.dtype:
        raise S2AError("y must match x in size and dtype")
    if codes.dtype != torch.uint8 or meta.dtype != torch.float32:
        raise S2AError("codes must be uint8 and meta float32")
    if row_len > 0 and (codes.numel() < codes_bytes(n) or meta.numel() * 4 < meta_bytes(n, row_len)):
        raise S2AError("codes/meta buffers are too small")
    if scratch.numel() * scratch.element_size() < tensor_range_scratch_bytes(n):
        raise S2AError("scratch is too small")
    check(lib().s2a_gelu_fwd_tensor_range(x.data_ptr(), y.data_ptr(), codes.data_ptr(), meta.data_ptr(),
                                          scratch.data_ptr(), n, row_len, dtype_code(x), _stream_ptr(x)))


def tensor_range_static_max_elems() -> int:
    return int(lib().s2a_tensor_range_static_max_elems())


def s2a_gelu_fwd_tensor_range_static(x, y, codes, meta, row_len: int) -> None:
    """s2a_gelu_fwd_tensor_range without a scratch argument, for callers that may not
    allocate device memory: the range partials live in a fixed array inside the library
    (shared by all calls on a GPU -- do not overlap them), and tensors beyond
    tensor_range_static_max_elems() elements are refused."""
    _dev(x, "x"), _dev(y, "y"), _dev(codes, "codes"), _dev(meta, "meta")
    n = x.numel()
    if y.numel() != n or y.dtype != x.dtype:
        raise S2AError("y must match x in size and dtype")
    if codes.dtype != torch.uint8 or meta.dtype != torch.float32:
        raise S2AError("codes must be uint8 and meta float32")
    if row_len > 0 and (codes.numel() < codes_bytes(n) or meta.numel() * 4 < meta_bytes(n, row_len)):
        raise S2AError("codes/meta buffers are too small")
    check(lib().s2a_gelu_fwd_tensor_range_static(x.data_ptr(), y.data_ptr(), codes.data_ptr(), meta.data_ptr(),
                                                 n, row_len, dtype_code(x), _stream_ptr(x)))


def s2a_cap_fwd(x, y, n_rows: int, channels: int, r: int) -> None:
    _dev(x, "x"), _dev(y, "y")
    if x.numel() != n_rows * channels or r <= 0 or y.numel() * r != x.numel() or y.dtype != x.dtype:
        raise S2AError("x must be [n_rows, channels] and y [n_rows, channels / r] of the same dtype")
    check(lib().s2a_cap_fwd(x.data_ptr(), y.data_ptr(), n_rows, channels, r, dtype_code(x), _stream_ptr(x)))


def s2a_cap_bwd(grad_out, grad_in, n_rows: int, channels: int, r: int) -> None:
    _dev(grad_out, "grad_out"), _dev(grad_in, "grad_in")
    if grad_in.numel() != n_rows * channels or r <= 0 or grad_out.numel() * r != grad_in.numel() \
            or grad_in.dtype != grad_out.dtype:
        raise S2AError("grad_out must be [n_rows, channels / r] and grad_in [n_rows, channels]")
    check(lib().s2a_cap_bwd(grad_out.data_ptr(), grad_in.data_ptr(), n_rows, channels, r, dtype_code(grad_out),
                            _stream_ptr()))


def s2a_lrp_fwd(x, A, B, y, batch: int, tokens: int, channels: int, rank: int) -> None:
    _dev(x, "x"), _dev(y, "y"), _dev(A, "A"), _dev(B, "B")
    if x.numel() != batch * tokens * channels or y.numel() != x.numel() or y.dtype != x.dtype:
        raise S2AError("x and y must be [batch, tokens, channels] of the same dtype")
    if A.dtype != torch.float32 or B.dtype != torch.float32 or A.numel() != tokens * rank or B.numel() != rank * channels:
        raise S2AError("A must be float32 [tokens, rank] and B float32 [rank, channels]")
    check(lib().s2a_lrp_fwd(x.data_ptr(), A.data_ptr(), B.data_ptr(), y.data_ptr(), batch, tokens, channels, rank,
                            dtype_code(x), _stream_ptr(x)))


def codes_bytes_bits(n_elems: int, bits: int) -> int:
    return int(lib().s2a_codes_bytes_bits(n_elems, bits))


def _call_bits(name, a, b, c_, d, n, row_len, bits, dt_code):
    check(getattr(lib(), name)(a.data_ptr(), b.data_ptr(), c_.data_ptr(), d.data_ptr(), n, row_len, bits, dt_code,
                               _stream_ptr()))


def s2a_fwd_bits(kind: str, x, y, codes, meta, row_len: int, bits: int) -> None:
    """s2a_gelu_fwd_bits / s2a_softmax_fwd_bits (kind = 'gelu' or 'softmax')."""
    _dev(x, "x"), _dev(y, "y"), _dev(codes, "codes"), _dev(meta, "meta")
    n = x.numel()
    if y.numel() != n or y.dtype != x.dtype or codes.dtype != torch.uint8 or meta.dtype != torch.float32:
        raise S2AError("y must match x; codes must be uint8 and meta float32")
    if codes.numel() < codes_bytes_bits(n, bits) or (row_len > 0 and meta.numel() * 4 < meta_bytes(n, row_len)):
        raise S2AError("codes/meta buffers are too small")
    _call_bits("s2a_%s_fwd_bits" % kind, x, y, codes, meta, n, row_len, bits, dtype_code(x))


def s2a_bwd_bits(kind: str, grad_out, codes, meta, grad_in, row_len: int, bits: int) -> None:
    _dev(grad_out, "grad_out"), _dev(grad_in, "grad_in"), _dev(codes, "codes"), _dev(meta, "meta")
    n = grad_out.numel()
    if grad_in.numel() != n or grad_in.dtype != grad_out.dtype:
        raise S2AError("grad_in must match grad_out in size and dtype")
    _call_bits("s2a_%s_bwd_bits" % kind, grad_out, codes, meta, grad_in, n, row_len, bits, dtype_code(grad_out))


def mask_bytes(n_elems: int) -> int:
    return int(lib().s2a_mask_bytes(n_elems))


def s2a_relu_fwd(x, y, mask) -> None:
    _dev(x, "x"), _dev(y, "y"), _dev(mask, "mask")
    n = x.numel()
    if y.numel() != n or y.dtype != x.dtype:
        raise S2AError("y must match x in size and dtype")
    if mask.dtype != torch.uint8 or mask.numel() < mask_bytes(n):
        raise S2AError("mask must be uint8 with at least mask_bytes(n) elements")
    check(lib().s2a_relu_fwd(x.data_ptr(), y.data_ptr(), mask.data_ptr(), n, dtype_code(x), _stream_ptr(x)))


def s2a_relu_bwd(grad_out, mask, grad_in) -> None:
    _dev(grad_out, "grad_out"), _dev(grad_in, "grad_in"), _dev(mask, "mask")
    n = grad_out.numel()
    if grad_in.numel() != n or grad_in.dtype != grad_out.dtype:
        raise S2AError("grad_in must match grad_out in size and dtype")
    if mask.dtype != torch.uint8 or mask.numel() < mask_bytes(n):
        raise S2AError("mask must be uint8 with at least mask_bytes(n) elements")
    check(lib().s2a_relu_bwd(grad_out.data_ptr(), mask.data_ptr(), grad_in.data_ptr(), n,
                             dtype_code(grad_out), _stream_ptr()))


def s2a_device_error(clear: bool = False) -> int:
    flags = ctypes.c_uint(0)
    check(lib().s2a_device_error(ctypes.byref(flags), int(clear)))
    return int(flags.value)


def s2a_describe_plan(kernel: int, n_elems: int, row_len: int, dt: int) -> str:
    buf = ctypes.create_string_buffer(256)
    check(lib().s2a_describe_plan(kernel, n_elems, row_len, dt, buf, 256))
    return buf.value.decode()
