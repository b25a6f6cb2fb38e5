"""Helpers of the GPU parity tests: moving seeded host arrays through the C-ABI calls
(with guard bands around every output), and the tolerance checks.

Tolerances (all written out here, used by every parity test):

* 4-bit codes and (min, s) metadata: bit-exact.  GELU codes depend on x only, so they
  must equal the oracle's everywhere.  Softmax codes are Q(y as written): they must
  equal an independent numpy binary32 evaluation of Eq. 8 on the GPU's own y with zero
  tolerance, and may differ from the oracle's codes only where the GPU's y (or the
  row's min/max) differs from the oracle's by its allowed rounding -- such elements sit
  within one ulp of a bin edge; they are counted and the count is bounded.
* binary32 outputs: |a - b| <= rtol * (|b| + M) + 2^-126 with rtol = 1e-6 (results below
  the normal range, 2^-126, may be flushed to zero).  M is 0
  except for the softmax VJP, where it is y_hat_i * sum_j |g_j| y_hat_j (the size of the
  terms that cancel in g_i - dot), and for softmax y, where rtol is widened by
  2^-24 * |x_i - max_j x_j| (the rounding of the exponent's argument).
* bfloat16 outputs: within 1 bfloat16 ulp of max(|b|, M), plus the same 2^-126 floor.
* softmax codes against the ORACLE's codes: an element's code may differ only if the oracle's
  scaled value t = (y - min) * 15 / (max - min), evaluated in binary64 from the oracle's own
  y, lies within B of a bin edge k + 1/2, where B is what the tolerances above allow y, min
  and max to move t by: B = inv * (tol(y_i) + (1 - t/15) tol(min) + (t/15) tol(max)) plus
  1e-5 for the binary32 evaluation of t.  Every such element is counted; the count, the worst
  distance as a fraction of B, and the worst distance in units of ulp(y_i) * inv are reported.
"""
from __future__ import annotations

import numpy as np
import torch

from paper_2503_08154_b200 import binding, synth

F32, BF16 = 0, 1
FLOOR = 2.0 ** -126  # the smallest normal binary32 / bfloat16 magnitude: results below it may flush
GUARD = 512  # bytes of canary on each side of every output buffer
CANARY = 0xA5


def torch_dtype(dt):
    return torch.float32 if dt == F32 else torch.bfloat16


def to_device(a: np.ndarray, dt: int) -> torch.Tensor:
    if dt == F32:
        return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.uint16).view(np.int16)).cuda().view(torch.bfloat16)


def to_host(t: torch.Tensor, dt: int) -> np.ndarray:
    if dt == F32:
        return t.detach().cpu().numpy()
    return t.detach().view(torch.int16).cpu().numpy().view(np.uint16)


class Guarded:
    """A device buffer of `nbytes` with canary bytes on both sides."""

    def __init__(self, nbytes: int):
        self.nbytes = nbytes
        self.raw = torch.full((nbytes + 2 * GUARD,), CANARY, dtype=torch.uint8, device="cuda")
        self.body = self.raw[GUARD:GUARD + nbytes]

    def view(self, dtype):
        return self.body.view(dtype) if self.nbytes else torch.empty(0, dtype=dtype, device="cuda")

    def check(self, what: str):
        raw = self.raw.cpu().numpy()
        assert (raw[:GUARD] == CANARY).all(), "%s: bytes before the buffer were overwritten" % what
        assert (raw[GUARD + self.nbytes:] == CANARY).all(), "%s: bytes after the buffer were overwritten" % what


def _round16(n):
    return (n + 15) // 16 * 16


def gpu_fwd(kind: str, x: np.ndarray, L: int, dt: int, inplace: bool = False):
    """Runs s2a_{gelu,softmax}_fwd on a host array; returns (y, codes, meta) as numpy."""
    n = x.size
    item = synth.io_itemsize(dt)
    xd = to_device(x, dt)
    yg = Guarded(n * item)
    cg = Guarded(binding.codes_bytes(n))
    mg = Guarded(binding.meta_bytes(n, L))
    if inplace:
        yg.view(torch_dtype(dt)).copy_(xd)
        xin = yg.view(torch_dtype(dt))
    else:
        xin = xd
    fn = {"gelu": binding.s2a_gelu_fwd, "softmax": binding.s2a_softmax_fwd, "silu": binding.s2a_silu_fwd}[kind]
    fn(xin, yg.view(torch_dtype(dt)), cg.view(torch.uint8), mg.view(torch.float32), L)
    torch.cuda.synchronize()
    assert binding.s2a_device_error() == 0
    for g, w in ((yg, "y"), (cg, "codes"), (mg, "meta")):
        g.check(kind + "_fwd " + w)
    if not inplace:
        assert np.array_equal(to_host(xd, dt), x), "the input tensor was modified"
    return to_host(yg.view(torch_dtype(dt)), dt), cg.view(torch.uint8).cpu().numpy(), mg.view(torch.float32).cpu().numpy()


def gpu_bwd(kind: str, g: np.ndarray, codes: np.ndarray, meta: np.ndarray, L: int, dt: int,
            inplace: bool = False):
    n = g.size
    item = synth.io_itemsize(dt)
    gd = to_device(g, dt)
    cd = torch.from_numpy(np.ascontiguousarray(codes)).cuda()
    md = torch.from_numpy(np.ascontiguousarray(meta)).cuda()
    og = Guarded(n * item)
    if inplace:
        og.view(torch_dtype(dt)).copy_(gd)
        gin = og.view(torch_dtype(dt))
    else:
        gin = gd
    fn = {"gelu": binding.s2a_gelu_bwd, "softmax": binding.s2a_softmax_bwd, "silu": binding.s2a_silu_bwd}[kind]
    fn(gin, cd, md, og.view(torch_dtype(dt)), L)
    torch.cuda.synchronize()
    assert binding.s2a_device_error() == 0
    og.check(kind + "_bwd grad_in")
    assert np.array_equal(cd.cpu().numpy(), codes) and np.array_equal(md.cpu().numpy(), meta)
    return to_host(og.view(torch_dtype(dt)), dt)


# ------------------------------------------------------------------ host-side checks
def widen(a: np.ndarray, dt: int) -> np.ndarray:
    return synth.io_to_f32(a, dt).astype(np.float64)


def numpy_quantize(v32: np.ndarray, L: int):
    """Eq. 8 as the header specifies it, in numpy binary32 (independent of the oracle and
    of the kernels).  Returns (unpacked codes uint8 [rows, L], meta float32 [2*rows])."""
    v = np.ascontiguousarray(v32, dtype=np.float32).reshape(-1, L)
    mn = v.min(axis=1, keepdims=True)
    mx = v.max(axis=1, keepdims=True)
    d = (mx - mn).astype(np.float32)
    with np.errstate(divide="ignore", invalid="ignore"):
        inv = np.where(d == 0, np.float32(0), np.float32(15) / d).astype(np.float32)
        s = np.where(d == 0, np.float32(0), d / np.float32(15)).astype(np.float32)
    t = ((v - mn).astype(np.float32) * inv).astype(np.float32)
    q = np.clip(np.rint(t), 0, 15).astype(np.uint8)
    meta = np.empty(2 * v.shape[0], dtype=np.float32)
    meta[0::2] = mn[:, 0]
    meta[1::2] = s[:, 0]
    return q, meta


def unpack_np(codes: np.ndarray, n: int) -> np.ndarray:
    out = np.empty(2 * codes.size, dtype=np.uint8)
    out[0::2] = codes & 0xF
    out[1::2] = codes >> 4
    return out[:n]


def bf16_ulp(mag: np.ndarray) -> np.ndarray:
    """Spacing of bfloat16 numbers at magnitude `mag` (>= the subnormal spacing)."""
    mag = np.maximum(np.abs(mag), 2.0 ** -126)
    return np.exp2(np.floor(np.log2(mag)) - 7)


def tolerance(want, dt, extra_mag=None, extra_rtol=None):
    """The allowed |got - want| per element (see the module docstring); want is float64."""
    want = np.asarray(want, dtype=np.float64).reshape(-1)
    mag = np.abs(want) if extra_mag is None else np.abs(want) + np.asarray(extra_mag).reshape(-1)
    if dt == F32:
        rtol = 1e-6 if extra_rtol is None else 1e-6 + np.asarray(extra_rtol).reshape(-1)
        tol = rtol * mag + FLOOR
    else:
        ref = np.abs(want) if extra_mag is None else np.maximum(np.abs(want), np.asarray(extra_mag).reshape(-1))
        tol = bf16_ulp(ref) + FLOOR
        if extra_rtol is not None:
            tol = tol + np.asarray(extra_rtol).reshape(-1) * mag
    return tol, mag


def assert_close(got, want, dt, what, extra_mag=None, extra_rtol=None):
    """got/want: float64 arrays of widened outputs.  See the module docstring."""
    got = np.asarray(got, dtype=np.float64).reshape(-1)
    want = np.asarray(want, dtype=np.float64).reshape(-1)
    tol, mag = tolerance(want, dt, extra_mag, extra_rtol)
    err = np.abs(got - want)
    bad = err > tol
    if bad.any():
        i = int(np.argmax(err / tol))
        raise AssertionError("%s: %d of %d outside tolerance; worst at %d: got %r want %r tol %r"
                             % (what, int(bad.sum()), got.size, i, got[i], want[i], tol[i]))
    return float(np.max(err / np.maximum(mag, 1e-300)))


def ulp_of(v, dt):
    """Spacing of the I/O type at |v| (float64 in, float64 out)."""
    if dt == BF16:
        return bf16_ulp(v)
    a = np.maximum(np.abs(np.asarray(v, dtype=np.float64)), 2.0 ** -126)
    return np.exp2(np.floor(np.log2(a)) - 23)


def check_edge_flips(q_got, q_want, y_want, meta_want, tol_y, dt, levels=15, what="softmax"):
    """Code differences against the oracle (see the module docstring).  q_*: unpacked codes
    [rows, L]; y_want: the oracle's y widened to float64 [rows, L]; meta_want: the oracle's
    (min, s) float32 [2 * rows]; tol_y: allowed |y_got - y_want| per element [rows, L].
    Returns {"flips", "elements", "worst_frac_of_bound", "worst_ulps"}."""
    rows, L = q_want.shape
    diff = q_got != q_want
    out = {"flips": int(diff.sum()), "elements": int(q_want.size), "worst_frac_of_bound": 0.0, "worst_ulps": 0.0}
    if not diff.any():
        return out
    assert np.abs(q_got.astype(int) - q_want.astype(int)).max() <= 1, "%s: a code differs by more than one level" % what
    r, c = np.nonzero(diff)
    yw = np.asarray(y_want, dtype=np.float64).reshape(rows, L)
    tol_y = np.asarray(tol_y, dtype=np.float64).reshape(rows, L)
    mn = meta_want[0::2].astype(np.float64)
    # the row maximum as the oracle saw it (s is rounded, so take max from y itself)
    amin, amax = yw.argmin(axis=1), yw.argmax(axis=1)
    mx = yw[np.arange(rows), amax]
    assert np.array_equal(yw[np.arange(rows), amin], mn), "oracle metadata is not the row minimum"
    d = (mx - mn)[r]
    assert (d > 0).all(), "%s: a constant row has differing codes" % what
    inv = levels / d
    t = (yw[r, c] - mn[r]) * inv
    dist = np.abs((t - np.floor(t)) - 0.5)
    w = t / levels
    bound = inv * (tol_y[r, c] + (1.0 - w) * tol_y[r, amin[r]] + w * tol_y[r, amax[r]]) + 1e-5
    frac = dist / bound
    if (frac > 1.0).any():
        i = int(np.argmax(frac))
        raise AssertionError("%s: code differs at row %d col %d although the oracle's t = %.9g is %.3g from a bin "
                             "edge (allowed %.3g): codes %d vs %d" % (what, r[i], c[i], t[i], dist[i], bound[i],
                                                                      q_got[r[i], c[i]], q_want[r[i], c[i]]))
    out["worst_frac_of_bound"] = float(frac.max())
    out["worst_ulps"] = float((dist / (inv * ulp_of(yw[r, c], dt))).max())
    return out
