"""Pins for the CPU oracle: every check here gets its expected value from somewhere
other than the oracle -- numbers the paper prints, closed forms, exact rational
arithmetic, library routines (scipy / numpy / torch), finite differences, or brute
force on tiny rows.  A dropped term, a flipped sign, a transposed index or a wrong
nibble order in the oracle fails at least one of them.
"""
import json
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import scipy.special as sp
import torch

from oracle import s2a_oracle as o
from paper_2503_08154_b200 import synth

F32, BF16 = o.F32, o.BF16
GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_values.json")))
A = float(np.float32(GOLD["gelu_sigmoid_slope"]["value"]))     # Eq. 10 slope as binary32
B = float(np.float32(GOLD["gelu_sine_amplitude"]["value"]))    # Eq. 12 amplitude
W = float(np.float32(GOLD["gelu_sine_frequency"]["value"]))    # Eq. 12 frequency
LEVELS = GOLD["code_set_max"]["value"]


# ------------------------------------------------------------------ number formats
def test_bf16_rounding_matches_torch_on_binary32_inputs():
    g = np.random.default_rng(1)
    vals = np.concatenate([g.standard_normal(4000) * 10.0 ** g.uniform(-30, 30, 4000),
                           [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895313892515355e38, 1e-40, -1e-45]])
    vals = vals.astype(np.float32)
    want = torch.from_numpy(vals).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([o.round_bf16(float(v)) for v in vals], dtype=np.uint16)
    assert np.array_equal(got, want)
    # the shared input helper rounds the same way
    assert np.array_equal(synth.f32_to_bf16_bits(vals), want)


def test_bf16_rounding_is_single_step_from_binary64():
    one, one_up = 0x3F80, 0x3F81                      # 1.0 and 1 + 2^-7
    assert o.round_bf16(1.0 + 2.0 ** -8) == one       # exact tie -> even
    assert o.round_bf16(1.0 + 2.0 ** -8 + 2.0 ** -40) == one_up
    # via binary32 this value would first collapse onto the tie and then round down
    assert o.round_bf16(1.0 + 2.0 ** -8 + 2.0 ** -30) == one_up
    assert o.round_bf16(1.0 + 3 * 2.0 ** -8) == 0x3F82  # tie between odd and even -> even
    assert o.bf16_to_float(one_up) == 1.0 + 2.0 ** -7
    assert o.round_bf16(-2.5) == 0xC020 and o.bf16_to_float(0xC020) == -2.5


# ------------------------------------------------------------------ Eq. 10 / 11 / 12
def test_gelu_forward_closed_forms_and_library():
    assert o.gelu(0.0) == 0.0
    xs = np.linspace(-12, 12, 1201)
    for x in xs:
        y = o.gelu(x)
        assert y == pytest.approx(x * sp.expit(A * x), rel=1e-14, abs=1e-300)   # library sigmoid
        assert y == pytest.approx(0.5 * x * (1 + math.tanh(0.5 * A * x)), rel=1e-12, abs=1e-15)
        # sigma(z) + sigma(-z) = 1  =>  y(x) - y(-x) = x
        assert y - o.gelu(-x) == pytest.approx(x, abs=1e-14)
    assert o.gelu(40.0) == pytest.approx(40.0, rel=1e-15)
    assert -1e-25 < o.gelu(-40.0) < 0.0


def test_exact_derivative_is_derivative_of_forward_and_has_the_printed_range():
    xs = np.linspace(-8, 8, 3201)
    h = 1e-5
    d = np.array([o.gelu_grad_exact(x) for x in xs])
    fd = np.array([(o.gelu(x + h) - o.gelu(x - h)) / (2 * h) for x in xs])
    assert np.max(np.abs(d - fd)) < 1e-8
    lo, hi = GOLD["gelu_derivative_range"]["value"]
    fine = np.array([o.gelu_grad_exact(x) for x in np.linspace(-6, 6, 120001)])
    assert lo < fine.min() < lo + 5e-4 and hi - 5e-4 < fine.max() < hi
    # "the second term is odd and vanishes at both infinities"
    second = lambda x: o.gelu_grad_exact(x) - sp.expit(A * x)
    for x in (0.3, 0.9, 1.7, 4.0):
        assert second(x) == pytest.approx(-second(-x), abs=1e-14)
    assert abs(second(30.0)) < 1e-12 and abs(second(-30.0)) < 1e-12


def test_sine_fitted_derivative():
    assert o.gelu_grad_sine(0.0) == 0.5
    for x in np.linspace(-2, 2, 401):
        d = o.gelu_grad_sine(x)
        assert d == pytest.approx(sp.expit(A * x) + B * math.sin(W * x), rel=1e-14, abs=1e-16)
        assert d + o.gelu_grad_sine(-x) == pytest.approx(1.0, abs=1e-15)   # sigma + odd term
    # amplitude and frequency: the sine term peaks at x = pi/3 with height 0.22
    peak = o.gelu_grad_sine(math.pi / 3) - sp.expit(A * math.pi / 3)
    assert peak == pytest.approx(0.22, abs=1e-7)
    assert o.gelu_grad_sine(2 * math.pi / 3) - sp.expit(A * 2 * math.pi / 3) == pytest.approx(0.0, abs=1e-12)
    # it is a fit of Eq. 11 on the clipped input: worst gap is at |x| = 2, about 0.075
    xs = np.linspace(-6, 6, 24001)
    gap = np.array([abs(o.gelu_grad_sine(float(np.clip(x, -2, 2))) - o.gelu_grad_exact(x)) for x in xs])
    assert 0.070 < gap.max() < 0.0750
    assert abs(abs(xs[gap.argmax()]) - 2.0) < 1e-3
    # and both stay within 0.09 of the erf-based GELU derivative Phi(x) + x phi(x)
    erf_d = lambda x: 0.5 * (1 + math.erf(x / math.sqrt(2))) + x * math.exp(-x * x / 2) / math.sqrt(2 * math.pi)
    assert max(abs(o.gelu_grad_exact(x) - erf_d(x)) for x in xs) < 0.030
    assert max(abs(o.gelu_grad_sine(float(np.clip(x, -2, 2))) - erf_d(x)) for x in xs) < 0.087


# ------------------------------------------------------------------ Eq. 8 / Eq. 9
def _exact_codes(v):
    """Eq. 8 in exact rational arithmetic; also returns which elements sit on a tie."""
    fr = [Fraction(float(x)) for x in v]
    mn, mx = min(fr), max(fr)
    if mx == mn:
        return [0] * len(fr), [False] * len(fr)
    codes, ties = [], []
    for x in fr:
        t = (x - mn) * LEVELS / (mx - mn)
        fl = t.numerator // t.denominator
        rem = t - fl
        if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
            fl += 1
        codes.append(int(fl))
        ties.append(abs(rem - Fraction(1, 2)) < Fraction(1, 10 ** 6))
    return codes, ties


def test_quantiser_against_exact_rational_arithmetic():
    g = np.random.default_rng(7)
    checked = 0
    for trial in range(200):
        n = int(g.integers(2, 40))
        v = (g.standard_normal(n) * 10.0 ** g.uniform(-3, 2)).astype(np.float32)
        if trial % 3 == 0:
            v = sp.softmax(v.astype(np.float64)).astype(np.float32)
        q, mn, s = o.quantize_row(v)
        want, near_tie = _exact_codes(v)
        qd = o.quantize_row_definition(v)
        for i in range(n):
            if not near_tie[i]:
                assert q[i] == want[i] and qd[i] == want[i]
                checked += 1
        assert mn == v.min()
        assert float(s) == float(np.float32(np.float32(v.max() - v.min()) / np.float32(LEVELS)))
        assert q[np.argmin(v)] == 0 and q[np.argmax(v)] == LEVELS
        order = np.argsort(v, kind="stable")
        assert np.all(np.diff(q[order].astype(int)) >= 0)          # monotone
        vh = np.array([o.dequantize(int(q[i]), mn, s) for i in range(n)])
        assert np.all(np.abs(vh - v) <= 0.5 * float(s) * (1 + 1e-5) + 1e-30)
    assert checked > 3000


def test_quantiser_hand_codes_on_a_saturated_gelu_row():
    # bin edges of a [-2, 2] row sit at -2 + (k + 1/2) * 4/15; 0 is the exact tie 7.5 -> 8
    row = np.array([-3, -2, -1, -0.1333333, 0, 0.1333334, 0.5, 1, 2, 2.5], dtype=np.float32)
    c = np.clip(row, *GOLD["gelu_clip"]["value"]).astype(np.float32)
    q, mn, s = o.quantize_row(c)
    assert q.tolist() == [0, 0, 4, 7, 8, 8, 9, 11, 15, 15]
    assert mn == np.float32(-2.0) and s == np.float32(np.float32(4.0) / np.float32(15.0))
    want, _ = _exact_codes(c)
    assert q.tolist() == want
    # the exact tie at 0 is where dividing by the rounded s would go wrong
    assert float(np.float32(2.0) / s) < 7.5


def test_quantiser_degenerate_rows():
    q, mn, s = o.quantize_row(np.full(9, 0.37, dtype=np.float32))
    assert q.tolist() == [0] * 9 and mn == np.float32(0.37) and s == 0.0
    assert o.dequantize(0, mn, s) == float(np.float32(0.37))
    q, mn, s = o.quantize_row(np.array([5.0], dtype=np.float32))
    assert q.tolist() == [0] and s == 0.0
    q, mn, s = o.quantize_row(np.array([1.0, -1.0], dtype=np.float32))
    assert q.tolist() == [15, 0]


def test_dequantiser_is_q_times_s_plus_min():
    for qv, mn, s in [(0, -2.0, 4 / 15), (7, -2.0, 4 / 15), (15, 0.03, 0.04), (3, 1e-5, 2e-6)]:
        mn32, s32 = float(np.float32(mn)), float(np.float32(s))
        assert o.dequantize(qv, mn32, s32) == float(Fraction(qv) * Fraction(s32) + Fraction(mn32))


def test_packing_low_nibble_first_flat_index():
    q = np.array([0, 1, 5, 15], dtype=np.uint8)
    assert o.pack(q).tolist() == [0x10, 0xF5]
    q = np.array([3, 9, 12], dtype=np.uint8)
    assert o.pack(q).tolist() == [0x93, 0x0C]           # unpaired last nibble: high half zero
    g = np.random.default_rng(3)
    q = g.integers(0, 16, 1001).astype(np.uint8)
    b = o.pack(q)
    assert b.size == 501
    assert np.array_equal(b[:500], q[0:1000:2] | (q[1:1000:2] << 4))
    assert np.array_equal(o.unpack(b, 1001), q)


def test_flat_packing_crosses_row_boundaries_when_row_len_is_odd():
    # 2 rows of 3: element 3 (row 1, col 0) shares byte 1 with element 2 (row 0, col 2)
    x = np.array([0.0, 1.0, 2.0, 5.0, 3.0, 4.0], dtype=np.float32)
    codes, meta = o.quantize_tensor(x, 3, F32)
    # row 0: (0, 7.5->8, 15), row 1: (15, 0, 7.5->8)
    assert o.unpack(codes, 6).tolist() == [0, 8, 15, 15, 0, 8]
    assert codes.tolist() == [0x80, 0xFF, 0x80]
    assert meta.tolist() == [0.0, float(np.float32(2 / 15)), 3.0, float(np.float32(2 / 15))]


# ------------------------------------------------------------------ Eq. 7
def test_softmax_forward_against_library_and_closed_forms():
    g = np.random.default_rng(11)
    for n in (1, 2, 3, 17, 197):
        x = g.standard_normal(n) * 3 + g.uniform(-5, 5)
        y = o.softmax_row(x)
        assert np.allclose(y, sp.softmax(x), rtol=1e-13, atol=0)
        assert abs(y.sum() - 1.0) < 1e-14
        assert np.allclose(o.softmax_row(x + 123.25), y, rtol=1e-12)
    y = o.softmax_row([0.7, -1.9])
    assert y[0] == pytest.approx(sp.expit(0.7 + 1.9), rel=1e-15)
    e = [math.exp(i) for i in range(4)]
    assert np.allclose(o.softmax_row([0, 1, 2, 3]), np.array(e) / sum(e), rtol=1e-15)
    assert np.allclose(o.softmax_row([700.0, 710.0]), [sp.expit(-10.0), sp.expit(10.0)], rtol=1e-14)


def test_softmax_vjp_against_explicit_jacobian_and_finite_differences():
    g = np.random.default_rng(13)
    n = 7
    x = g.standard_normal(n)
    gout = g.standard_normal(n)
    y = o.softmax_row(x)
    J = np.empty((n, n))                      # J[i, j] = dy_i / dx_j, the two cases of Eq. 7
    for i in range(n):
        for j in range(n):
            J[i, j] = y[i] * (1 - y[j]) if i == j else -y[i] * y[j]
    want = J.T @ gout
    got = o.softmax_vjp_row(y, gout)
    assert np.allclose(got, want, rtol=1e-12, atol=1e-15)
    h = 1e-6
    fd = np.empty(n)
    for j in range(n):
        e = np.zeros(n)
        e[j] = h
        fd[j] = gout @ (o.softmax_row(x + e) - o.softmax_row(x - e)) / (2 * h)
    assert np.allclose(got, fd, rtol=1e-6, atol=1e-9)
    assert abs(got.sum()) < 1e-15             # exact y: rows of the VJP sum to zero


def test_softmax_worked_row_end_to_end():
    x = np.array([0, 1, 2, 3], dtype=np.float32)
    y, codes, meta = o.softmax_fwd(x, 4, F32)
    e = np.array([math.exp(i) for i in range(4)])
    y_true = e / e.sum()
    assert np.array_equal(y, y_true.astype(np.float32))
    # t = 15 (y - y0) / (y3 - y0) = (0, 1.350.., 5.021.., 15) -> codes 0 1 5 15
    t = 15 * (y_true - y_true[0]) / (y_true[3] - y_true[0])
    assert np.round(t).tolist() == [0, 1, 5, 15]
    assert codes.tolist() == [0x10, 0xF5]
    assert meta[0] == y[0] and meta[1] == np.float32(np.float32(y[3] - y[0]) / np.float32(15))
    gout = np.array([1, -1, 0.5, 2], dtype=np.float32)
    gin = o.softmax_bwd(gout, codes, meta, 4, F32)
    yh = np.array([0, 1, 5, 15]) * float(meta[1]) + float(meta[0])
    dot = float(gout.astype(np.float64) @ yh)
    want = yh * (gout - dot)
    assert np.allclose(gin, want, rtol=2e-7)
    # closed-form invariant of the quantised VJP: sum_i grad_in_i = dot * (1 - sum_i y_hat_i)
    assert gin.astype(np.float64).sum() == pytest.approx(dot * (1 - yh.sum()), rel=1e-5)


# ------------------------------------------------------------------ tensor entry points
@pytest.mark.parametrize("dt", [F32, BF16])
@pytest.mark.parametrize("rows,L", [(6, 64), (5, 197), (4, 257), (3, 1), (2, 3072)])
def test_gelu_tensor_path(dt, rows, L):
    n = rows * L
    x = synth.to_io(synth.gelu_preact(5, ("t", rows, L), n) * 1.3, dt)
    gout = synth.to_io(synth.normal(5, ("g", rows, L), n), dt)
    y, codes, meta = o.gelu_fwd(x, L, dt)
    xw = o.widen(x, dt)
    y_lib = xw * sp.expit(A * xw)
    if dt == F32:
        assert np.array_equal(y, y_lib.astype(np.float32))
    else:
        want = torch.from_numpy(y_lib).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        assert np.mean(y != want) < 1e-3       # torch goes through its own rounding; ties aside
        assert np.max(np.abs(o.widen(y, dt) - y_lib) / np.maximum(np.abs(y_lib), 1e-30)) <= 2.0 ** -8
    assert codes.size == (n + 1) // 2 and meta.size == 2 * rows
    q = o.unpack(codes, n).reshape(rows, L)
    c = np.clip(xw, -2, 2).reshape(rows, L)
    for r in range(rows):
        want, tie = _exact_codes(c[r].astype(np.float32))
        ok = ~np.array(tie)
        assert np.array_equal(q[r][ok], np.array(want)[ok])
        assert meta[2 * r] == np.float32(c[r].min())
        xh = q[r].astype(np.float64) * float(meta[2 * r + 1]) + float(meta[2 * r])
        assert np.all(np.abs(xh - c[r]) <= 0.5 * float(meta[2 * r + 1]) * (1 + 1e-5))
    gin = o.gelu_bwd(gout, codes, meta, L, dt)
    xh = q.astype(np.float64) * meta[1::2, None].astype(np.float64) + meta[0::2, None].astype(np.float64)
    want = o.widen(gout, dt).reshape(rows, L) * (sp.expit(A * xh) + B * np.sin(W * xh))
    got = o.widen(gin, dt).reshape(rows, L)
    tol = 2.0 ** -24 if dt == F32 else 2.0 ** -8
    assert np.all(np.abs(got - want) <= tol * np.abs(want) + 1e-40)


@pytest.mark.parametrize("dt", [F32, BF16])
@pytest.mark.parametrize("rows,L", [(8, 64), (6, 197), (3, 257), (4, 1), (5, 2), (2, 1024)])
def test_softmax_tensor_path(dt, rows, L):
    n = rows * L
    x = synth.to_io(synth.softmax_logits(9, ("t", rows, L), rows, L), dt)
    gout = synth.to_io(synth.normal(9, ("g", rows, L), n), dt)
    y, codes, meta = o.softmax_fwd(x, L, dt)
    xw = o.widen(x, dt).reshape(rows, L)
    y_lib = sp.softmax(xw, axis=1)
    yw = o.widen(y, dt).reshape(rows, L)
    tol = 2.0 ** -23 if dt == F32 else 2.0 ** -8
    assert np.all(np.abs(yw - y_lib) <= tol * y_lib + 1e-45)
    q = o.unpack(codes, n).reshape(rows, L)
    for r in range(rows):
        want, tie = _exact_codes(yw[r].astype(np.float32))     # codes are Q(y as written)
        ok = ~np.array(tie)
        assert np.array_equal(q[r][ok], np.array(want)[ok])
        assert meta[2 * r] == np.float32(yw[r].min())
        if L > 1 and yw[r].max() > yw[r].min():
            assert q[r].min() == 0 and q[r].max() == LEVELS
        else:
            assert meta[2 * r + 1] == 0.0 and not q[r].any()
    codes2, meta2 = o.quantize_tensor(y, L, dt)
    assert np.array_equal(codes2, codes) and np.array_equal(meta2, meta)
    gin = o.widen(o.softmax_bwd(gout, codes, meta, L, dt), dt).reshape(rows, L)
    yh = q.astype(np.float64) * meta[1::2, None].astype(np.float64) + meta[0::2, None].astype(np.float64)
    gw = o.widen(gout, dt).reshape(rows, L)
    dot = (gw * yh).sum(axis=1, keepdims=True)
    want = yh * (gw - dot)
    scale = yh * (np.abs(gw) * yh).sum(axis=1, keepdims=True)      # size of the cancelling terms
    assert np.all(np.abs(gin - want) <= tol * (np.abs(want) + scale) + 1e-40)


def test_row_parallel_driver_gives_identical_results():
    L, rows = 197, 37
    x = synth.to_io(synth.softmax_logits(2, "p", rows, L), BF16)
    a = o.softmax_fwd(x, L, BF16, threads=1)
    b = o.softmax_fwd(x, L, BF16, threads=5)
    for u, v in zip(a, b):
        assert np.array_equal(u, v)
    gx = synth.to_io(synth.gelu_preact(2, "q", rows * L), F32)
    a = o.gelu_fwd(gx, L, F32, threads=1)
    b = o.gelu_fwd(gx, L, F32, threads=8)
    for u, v in zip(a, b):
        assert np.array_equal(u, v)


def test_bad_shapes_are_rejected_and_empty_is_fine():
    with pytest.raises(ValueError):
        o.gelu_fwd(np.zeros(10, dtype=np.float32), 3, F32)
    with pytest.raises(ValueError):
        o.softmax_fwd(np.zeros(10, dtype=np.float32), 0, F32)
    y, c, m = o.gelu_fwd(np.zeros(0, dtype=np.float32), 4, F32)
    assert y.size == 0 and c.size == 0 and m.size == 0


# ------------------------------------------------------------------ per-tensor range reading
@pytest.mark.parametrize("dt", [F32, BF16])
def test_gelu_tensor_range_reading(dt):
    rows, L = 6, 40
    # small-variance rows: no row reaches the clip, rows have different ranges
    x32 = synth.normal(8, ("tr", dt), rows * L) * 0.3
    x32[5] = 1.9
    x = synth.to_io(x32, dt)
    y, codes, meta = o.gelu_fwd_tensor_range(x, L, dt)
    y_row, codes_row, meta_row = o.gelu_fwd(x, L, dt)
    assert np.array_equal(y, y_row)                        # only the stash differs
    c = np.clip(o.widen(x, dt), -2, 2).astype(np.float32)
    want, tie = _exact_codes(c)                            # Eq. 8 over the whole tensor, exactly
    q = o.unpack(codes, rows * L)
    ok = ~np.array(tie)
    assert np.array_equal(q[ok], np.array(want)[ok])
    assert np.all(meta[0::2] == np.float32(c.min()))
    assert np.all(meta[1::2] == np.float32(np.float32(c.max() - c.min()) / np.float32(15)))
    assert not np.array_equal(codes, codes_row)            # and it IS a different stash here
    # on a tensor whose every row saturates the clip the two readings coincide
    xs = synth.to_io(synth.gelu_preact(8, ("trs", dt), 4 * 3072), dt)
    a = o.gelu_fwd_tensor_range(xs, 3072, dt)
    b = o.gelu_fwd(xs, 3072, dt)
    for u, v in zip(a, b):
        assert np.array_equal(u, v)
    # the backward pass takes this stash as it is
    g = synth.to_io(synth.normal(8, ("trg", dt), rows * L), dt)
    gin = o.widen(o.gelu_bwd(g, codes, meta, L, dt), dt)
    xh = q.astype(np.float64) * float(meta[1]) + float(meta[0])
    wantg = o.widen(g, dt) * (sp.expit(A * xh) + B * np.sin(W * xh))
    tol = 2.0 ** -24 if dt == F32 else 2.0 ** -8
    assert np.all(np.abs(gin - wantg) <= tol * np.abs(wantg) + 1e-40)


# ------------------------------------------------------------------ general bit width (Eq. 8)
def _exact_codes_levels(v, levels):
    fr = [Fraction(float(x)) for x in v]
    mn, mx = min(fr), max(fr)
    if mx == mn:
        return [0] * len(fr), [False] * len(fr)
    codes, ties = [], []
    for x in fr:
        t = (x - mn) * levels / (mx - mn)
        fl = t.numerator // t.denominator
        rem = t - fl
        if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
            fl += 1
        codes.append(int(fl))
        ties.append(abs(rem - Fraction(1, 2)) < Fraction(1, 10 ** 5))
    return codes, ties


@pytest.mark.parametrize("bits", [1, 2, 4, 8])
def test_general_bit_width_quantiser_and_packing(bits):
    levels = 2 ** bits - 1
    g = np.random.default_rng(bits)
    for _ in range(40):
        v = (g.standard_normal(int(g.integers(2, 50))) * 10.0 ** g.uniform(-2, 1)).astype(np.float32)
        q, mn, s = o.quantize_row_levels(v, levels)
        want, tie = _exact_codes_levels(v, levels)
        ok = ~np.array(tie)
        assert np.array_equal(q[ok], np.array(want)[ok])
        assert q.max() == levels and q.min() == 0 and mn == v.min()
        assert float(s) == float(np.float32(np.float32(v.max() - v.min()) / np.float32(levels)))
    q = g.integers(0, levels + 1, 1003).astype(np.uint8)
    packed = o.pack_bits(q, bits)
    assert packed.size == (1003 * bits + 7) // 8
    # little-endian bit order: numpy's unpackbits recovers the codes
    bitsarr = np.unpackbits(packed, bitorder="little")[:1003 * bits].reshape(1003, bits)
    assert np.array_equal((bitsarr * (1 << np.arange(bits))).sum(axis=1), q)
    assert np.array_equal(o.unpack_bits(packed, 1003, bits), q)
    if bits == 4:
        assert np.array_equal(packed, o.pack(q))          # the 4-bit layout is the nibble layout


@pytest.mark.parametrize("dt", [F32, BF16])
@pytest.mark.parametrize("kind,rows,L", [("gelu", 5, 197), ("softmax", 6, 65), ("gelu", 3, 64), ("softmax", 2, 1024)])
def test_tensor_path_at_other_bit_widths(kind, rows, L, dt):
    n = rows * L
    if kind == "gelu":
        x = synth.to_io(synth.gelu_preact(31, (kind, rows, L), n), dt)
    else:
        x = synth.to_io(synth.softmax_logits(31, (kind, rows, L), rows, L), dt)
    gout = synth.to_io(synth.normal(31, ("g", kind, rows, L), n), dt)
    # N = 4 is the existing path, bit for bit
    four = o.fwd_bits(kind, x, L, 4, dt)
    ref = o.gelu_fwd(x, L, dt) if kind == "gelu" else o.softmax_fwd(x, L, dt)
    for a, b in zip(four, ref):
        assert np.array_equal(a, b)
    ref_b = (o.gelu_bwd if kind == "gelu" else o.softmax_bwd)(gout, ref[1], ref[2], L, dt)
    assert np.array_equal(o.bwd_bits(kind, gout, four[1], four[2], L, 4, dt), ref_b)
    prev_err = None
    for bits in (2, 4, 8):
        y, codes, meta = o.fwd_bits(kind, x, L, bits, dt)
        assert np.array_equal(y, ref[0]) and codes.size == (n * bits + 7) // 8
        q = o.unpack_bits(codes, n, bits).reshape(rows, L)
        v = (np.clip(o.widen(x, dt), -2, 2) if kind == "gelu" else o.widen(y, dt)).reshape(rows, L)
        for r in range(rows):
            want, tie = _exact_codes_levels(v[r].astype(np.float32), 2 ** bits - 1)
            ok = ~np.array(tie)
            assert np.array_equal(q[r][ok], np.array(want)[ok])
        vh = q.astype(np.float64) * meta[1::2, None].astype(np.float64) + meta[0::2, None].astype(np.float64)
        err = np.abs(vh - v).max()
        assert err <= 0.5 * float(meta[1::2].max()) * (1 + 1e-5)
        if prev_err is not None:
            assert err < prev_err                          # more bits, smaller reconstruction error
        prev_err = err
        gin = o.widen(o.bwd_bits(kind, gout, codes, meta, L, bits, dt), dt).reshape(rows, L)
        gw = o.widen(gout, dt).reshape(rows, L)
        if kind == "gelu":
            want_g = gw * (sp.expit(A * vh) + B * np.sin(W * vh))
            scale = 0.0
        else:
            dot = (gw * vh).sum(axis=1, keepdims=True)
            want_g = vh * (gw - dot)
            scale = vh * (np.abs(gw) * vh).sum(axis=1, keepdims=True)
        tol = 2.0 ** -23 if dt == F32 else 2.0 ** -8
        assert np.all(np.abs(gin - want_g) <= tol * (np.abs(want_g) + scale) + 1e-40)
    with pytest.raises(ValueError):
        o.fwd_bits(kind, x, L, 3, dt)


# ------------------------------------------------------------------ SiLU / Swish
def test_silu_closed_forms_and_derivative():
    assert o.silu(0.0) == 0.0 and o.silu_grad(0.0) == 0.5
    h = 1e-5
    for x in np.linspace(-9, 9, 721):
        assert o.silu(x) == pytest.approx(x * sp.expit(x), rel=1e-14, abs=1e-300)
        assert o.silu(x) - o.silu(-x) == pytest.approx(x, abs=1e-14)          # sigma(x) + sigma(-x) = 1
        fd = (o.silu(x + h) - o.silu(x - h)) / (2 * h)
        assert o.silu_grad(x) == pytest.approx(fd, abs=1e-8)
        assert o.silu_grad(x) + o.silu_grad(-x) == pytest.approx(1.0, abs=1e-14)
    fine = np.array([o.silu_grad(x) for x in np.linspace(-8, 8, 16001)])
    assert -0.1 < fine.min() < -0.09 and 1.09 < fine.max() < 1.1              # the same band as GELU's
    # SiLU is the sigmoid-GELU with its argument stretched by 1.702
    for x in (-3.0, -0.7, 0.4, 2.5):
        assert o.silu(A * x) == pytest.approx(A * o.gelu(x), rel=1e-13)
        assert o.silu_grad(A * x) == pytest.approx(o.gelu_grad_exact(x), rel=1e-12)


@pytest.mark.parametrize("dt", [F32, BF16])
@pytest.mark.parametrize("rows,L", [(6, 64), (5, 197), (3, 1), (2, 3072)])
def test_silu_tensor_path(dt, rows, L):
    n = rows * L
    clip = float(np.float32(2.0) * np.float32(1.702))
    x = synth.to_io(synth.gelu_preact(15, ("silu", rows, L), n) * 2.2, dt)
    gout = synth.to_io(synth.normal(15, ("silug", rows, L), n), dt)
    y, codes, meta = o.silu_fwd(x, L, dt)
    xw = o.widen(x, dt)
    y_lib = xw * sp.expit(xw)
    tol = 2.0 ** -24 if dt == F32 else 2.0 ** -8
    assert np.all(np.abs(o.widen(y, dt) - y_lib) <= tol * np.abs(y_lib) + 1e-40)
    q = o.unpack(codes, n).reshape(rows, L)
    c = np.clip(xw, -clip, clip).reshape(rows, L)
    for r in range(rows):
        want, tie = _exact_codes(c[r].astype(np.float32))
        ok = ~np.array(tie)
        assert np.array_equal(q[r][ok], np.array(want)[ok])
        assert meta[2 * r] == np.float32(c[r].min())
    if L >= 64:
        assert np.abs(xw).max() > clip and meta[0] == np.float32(-clip)       # the clip is exercised
    gin = o.widen(o.silu_bwd(gout, codes, meta, L, dt), dt).reshape(rows, L)
    xh = q.astype(np.float64) * meta[1::2, None].astype(np.float64) + meta[0::2, None].astype(np.float64)
    sg = sp.expit(xh)
    want = o.widen(gout, dt).reshape(rows, L) * (sg * (1 + xh * (1 - sg)))
    assert np.all(np.abs(gin - want) <= tol * np.abs(want) + 1e-40)


# ------------------------------------------------------------------ ReLU 1-bit stash
@pytest.mark.parametrize("dt", [F32, BF16])
@pytest.mark.parametrize("n", [1, 7, 8, 9, 1000, 4099])
def test_relu_mask_against_numpy(dt, n):
    x32 = synth.normal(4, ("relu", n, dt), n)
    x32[::5] = 0.0
    if n > 3:
        x32[3] = -0.0
    x = synth.to_io(x32, dt)
    g = synth.to_io(synth.normal(4, ("relug", n, dt), n), dt)
    xw = o.widen(x, dt)
    y, mask = o.relu_fwd(x, dt)
    assert np.array_equal(o.widen(y, dt), np.maximum(xw, 0.0))
    assert not np.signbit(o.widen(y, dt)).any()                       # -0 and negatives become +0
    assert np.array_equal(mask, np.packbits(xw > 0, bitorder="little"))
    assert mask.size == (n + 7) // 8                                   # one bit per element
    gin = o.relu_bwd(g, mask, dt)
    assert np.array_equal(o.widen(gin, dt), np.where(xw > 0, o.widen(g, dt), 0.0))
    # the derivative takes the two values 0 and 1 only: finite differences of the forward
    h = 1e-3
    far = np.abs(xw) > 2 * h
    fd = (np.maximum(xw + h, 0) - np.maximum(xw - h, 0)) / (2 * h)
    bits = np.unpackbits(mask, bitorder="little")[:n]
    assert np.allclose(fd[far], bits[far])


# ------------------------------------------------------------------ CAP (Eq. 5) and LRP (Eq. 3)
@pytest.mark.parametrize("dt", [F32, BF16])
@pytest.mark.parametrize("rows,ch,r", [(3, 8, 8), (5, 24, 3), (4, 768, 8), (2, 10, 1)])
def test_cap_against_numpy_mean_and_finite_differences(dt, rows, ch, r):
    x = synth.to_io(synth.normal(21, ("cap", rows, ch, r), rows * ch), dt)
    xw = o.widen(x, dt).reshape(rows, ch // r, r)
    y = o.widen(o.cap_fwd(x, rows, ch, r, dt), dt).reshape(rows, ch // r)
    tol = 2.0 ** -24 if dt == F32 else 2.0 ** -8
    assert np.all(np.abs(y - xw.mean(axis=2)) <= tol * np.abs(xw.mean(axis=2)) + 1e-40)
    g = synth.to_io(synth.normal(21, ("capg", rows, ch, r), rows * ch // r), dt)
    gw = o.widen(g, dt).reshape(rows, ch // r)
    gin = o.widen(o.cap_bwd(g, rows, ch, r, dt), dt).reshape(rows, ch // r, r)
    want = np.repeat((gw / r)[:, :, None], r, axis=2)          # the gradient of a mean: g / r to every input
    assert np.all(np.abs(gin - want) <= tol * np.abs(want) + 1e-40)
    # vector-Jacobian identity: <g, CAP(x)> = <CAP^T(g), x>
    assert float((gw * xw.mean(axis=2)).sum()) == pytest.approx(float((want * xw).sum()), rel=1e-9, abs=1e-12)
    with pytest.raises(ValueError):
        o.cap_fwd(x, rows, ch, ch + 1, dt)


@pytest.mark.parametrize("dt", [F32, BF16])
def test_lrp_against_numpy_matmul(dt):
    batch, tokens, ch, rank = 3, 7, 16, 5
    x = synth.to_io(synth.normal(22, "lrpx", batch * tokens * ch), dt)
    A = synth.normal(22, "lrpa", tokens * rank).reshape(tokens, rank)
    B = synth.normal(22, "lrpb", rank * ch).reshape(rank, ch)
    y = o.widen(o.lrp_fwd(x, A, B, batch, tokens, ch, rank, dt), dt).reshape(batch, tokens, ch)
    want = o.widen(x, dt).reshape(batch, tokens, ch) + (A.astype(np.float64) @ B.astype(np.float64))[None]
    tol = 2.0 ** -24 if dt == F32 else 2.0 ** -8
    assert np.all(np.abs(y - want) <= tol * np.abs(want) + 1e-40)
    # A = 0 (the paper's initialisation) leaves the activation unchanged
    y0 = o.lrp_fwd(x, np.zeros_like(A), B, batch, tokens, ch, rank, dt)
    assert np.array_equal(y0, x)


# ------------------------------------------------------------------ memory accounting
def test_stash_size_and_the_papers_memory_delta():
    # 0.5 B per element, against the 4 B of the 32-bit activation the paper replaces
    n = 32 * 197 * 3072
    assert (n + 1) // 2 * GOLD["nonparametric_memory_ratio"]["value"] == 4 * n
    # Table 2, ViT-B/16, batch 32: moving the 12 GELU inputs and the 12 softmax outputs
    # from 4 B to 0.5 B per element accounts for the printed 2097 -> 640 MB
    t = GOLD["table2_vit_b16_memory_mb"]
    elems = t["batch"] * 197 * 3072 + t["batch"] * 12 * 197 * 197
    saved_mb = elems * (4 - 0.5) * 12 / 1e6
    assert abs(saved_mb - (t["unquantised"] - t["quantised"])) / (t["unquantised"] - t["quantised"]) < 0.02
    # the synthetic bulk+tail input saturates every row at [-2, 2]
    x = synth.gelu_preact(0, "sat", 64 * 3072).reshape(64, 3072)
    assert (x.max(axis=1) >= 2).all() and (x.min(axis=1) <= -2).all()
    assert 0.02 < np.mean(np.abs(x) > 2) < 0.06
