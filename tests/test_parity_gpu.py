"""GPU parity: the CUDA kernels, called through the C ABI, against the CPU oracle on the
same seeded inputs, element by element.  Tolerances are in parity_util's docstring."""
import os

import numpy as np
import pytest
import torch

from oracle import s2a_oracle as o
from paper_2503_08154_b200 import binding, synth
import parity_util as pu

pytestmark = pytest.mark.gpu
F32, BF16 = 0, 1
THREADS = max(1, os.cpu_count() or 1)


# ------------------------------------------------------------------ the two checks
def check_gelu(x, g, L, dt, inplace=False):
    n = x.size
    y_o, codes_o, meta_o = o.gelu_fwd(x, L, dt, threads=THREADS)
    y_g, codes_g, meta_g = pu.gpu_fwd("gelu", x, L, dt, inplace=inplace)
    assert np.array_equal(codes_g, codes_o), "GELU codes differ from the oracle's"
    assert np.array_equal(meta_g.view(np.uint32), meta_o.view(np.uint32)), "GELU (min, s) differ"
    pu.assert_close(pu.widen(y_g, dt), pu.widen(y_o, dt), dt, "gelu y")
    gin_o = o.gelu_bwd(g, codes_o, meta_o, L, dt, threads=THREADS)
    gin_g = pu.gpu_bwd("gelu", g, codes_o, meta_o, L, dt, inplace=inplace)
    pu.assert_close(pu.widen(gin_g, dt), pu.widen(gin_o, dt), dt, "gelu grad_in")
    return n


def check_softmax(x, g, L, dt, inplace=False, max_flip_frac=2e-3, report=None):
    """Returns the edge-flip statistics of parity_util.check_edge_flips plus "y_worst_rel", the
    largest |y - y_oracle| / y_oracle seen (for binary32: to be read against the 1e-6 line)."""
    n = x.size
    rows = n // L
    y_o, codes_o, meta_o = o.softmax_fwd(x, L, dt, threads=THREADS)
    y_g, codes_g, meta_g = pu.gpu_fwd("softmax", x, L, dt, inplace=inplace)
    xw = pu.widen(x, dt).reshape(rows, L)
    arg_gap = (xw.max(axis=1, keepdims=True) - xw) * 2.0 ** -24
    yw_o = pu.widen(y_o, dt)
    worst_rel = pu.assert_close(pu.widen(y_g, dt), yw_o, dt, "softmax y", extra_rtol=arg_gap)
    # the stash is exactly Q(y as written), checked without the oracle and without tolerance
    q_np, meta_np = pu.numpy_quantize(synth.io_to_f32(y_g, dt), L)
    q_g = pu.unpack_np(codes_g, n).reshape(rows, L)
    assert np.array_equal(q_g, q_np), "softmax codes are not Q(y as written)"
    assert np.array_equal(meta_g.view(np.uint32), meta_np.view(np.uint32))
    if n % 2 == 1:
        assert codes_g[-1] >> 4 == 0, "unpaired last nibble must be zero"
    # against the oracle's codes: a code may differ only where the oracle's scaled value sits
    # within the tolerance's reach of a bin edge; such elements are counted
    q_o = pu.unpack_np(codes_o, n).reshape(rows, L)
    tol_y, _ = pu.tolerance(yw_o, dt, extra_rtol=arg_gap)
    stats = pu.check_edge_flips(q_g, q_o, yw_o, meta_o, tol_y, dt)
    assert stats["flips"] <= max_flip_frac * n, "too many edge flips: %d of %d" % (stats["flips"], n)
    stats["y_worst_rel"] = worst_rel
    # backward from the ORACLE's stash, so that both sides see identical inputs
    gin_o = o.softmax_bwd(g, codes_o, meta_o, L, dt, threads=THREADS)
    gin_g = pu.gpu_bwd("softmax", g, codes_o, meta_o, L, dt, inplace=inplace)
    yh = q_o.astype(np.float64) * meta_o[1::2, None].astype(np.float64) + meta_o[0::2, None].astype(np.float64)
    gw = pu.widen(g, dt).reshape(rows, L)
    M = yh * (np.abs(gw) * yh).sum(axis=1, keepdims=True)
    pu.assert_close(pu.widen(gin_g, dt), pu.widen(gin_o, dt), dt, "softmax grad_in", extra_mag=M)
    if report is not None:
        print("%s: softmax code flips vs oracle: %d of %d (worst %.2f of the allowed edge distance, %.2f ulp(y)*inv); "
              "worst relative error of y %.3g%s" % (report, stats["flips"], n, stats["worst_frac_of_bound"], stats["worst_ulps"],
                                                   worst_rel, " (binary32 line: 1e-6)" if dt == F32 else ""))
    return stats


def _gelu_inputs(rows, L, dt, seed=0, scale=1.3):
    n = rows * L
    x = synth.to_io(synth.gelu_preact(seed, ("pg", rows, L, dt), n) * np.float32(scale), dt)
    g = synth.to_io(synth.normal(seed, ("pgg", rows, L, dt), n), dt)
    return x, g


def _softmax_inputs(rows, L, dt, seed=0):
    x = synth.to_io(synth.softmax_logits(seed, ("ps", rows, L, dt), rows, L), dt)
    g = synth.to_io(synth.normal(seed, ("psg", rows, L, dt), rows * L), dt)
    return x, g


# ------------------------------------------------------------------ small shapes, tails
# Row counts are chosen so that the pipelined path runs several tiles AND leaves a ragged
# remainder for the row-at-a-time path; the very long and the tiny cases take the latter only.
GELU_SHAPES = [(5, 1), (3, 2), (7, 3), (9, 63), (701, 63), (64, 64), (1001, 64), (33, 65), (531, 65),
               (41, 197), (451, 197), (301, 257), (137, 1024), (300, 66), (203, 1000),
               (40, 3072), (13, 3072), (11, 4096), (9, 5120), (3, 8191), (5, 8192), (1, 16384), (2, 40000)]
SOFTMAX_SHAPES = [(7, 1), (4, 2), (5, 3), (33, 63), (701, 63), (77, 64), (1001, 64), (531, 65), (300, 197),
                  (1, 197), (1283, 197), (130, 257), (257, 257), (323, 257), (137, 1024), (300, 66),
                  (203, 1000), (9, 4096), (21, 3072), (7, 5120), (5, 8191), (5, 8192), (2, 40000),
                  # widths that are not whole 16-byte vectors (masked vector ends), tiles + ragged tails
                  (90, 17), (2049, 49), (1500, 50), (999, 145), (641, 198), (333, 577), (163, 1025),
                  (1100, 196), (37, 16384), (300, 40), (513, 56), (2000, 48),
                  (700, 401), (300, 785), (200, 1370), (1500, 100), (901, 33), (350, 255),
                  (170, 2049),                 # tiles too large to double-buffer: a single stage
                  # 577 / 1025: tiles of 8 or 16 rows whose code bytes start off the 16-byte grid; with
                  # these row counts the last tile ends off it too and is left to the row path
                  (9000, 1025), (40, 1025), (48, 1025), (72, 577), (2000, 577)]


@pytest.mark.parametrize("dt", [F32, BF16])
@pytest.mark.parametrize("rows,L", GELU_SHAPES)
def test_gelu_small(rows, L, dt):
    check_gelu(*_gelu_inputs(rows, L, dt), L, dt)


@pytest.mark.parametrize("dt", [F32, BF16])
@pytest.mark.parametrize("rows,L", SOFTMAX_SHAPES)
def test_softmax_small(rows, L, dt):
    check_softmax(*_softmax_inputs(rows, L, dt), L, dt)


@pytest.mark.parametrize("dt", [F32, BF16])
def test_in_place(dt):
    check_gelu(*_gelu_inputs(70, 3072, dt, seed=3), 3072, dt, inplace=True)
    check_gelu(*_gelu_inputs(70, 197, dt, seed=3), 197, dt, inplace=True)
    check_softmax(*_softmax_inputs(700, 197, dt, seed=3), 197, dt, inplace=True)
    check_softmax(*_softmax_inputs(20, 4096, dt, seed=3), 4096, dt, inplace=True)
    check_softmax(*_softmax_inputs(515, 145, dt, seed=3), 145, dt, inplace=True)


def test_benchmark_shapes_take_the_pipelined_path():
    for sh in (synth.VIT_B16_B8_F32, synth.VIT_B16_B64, synth.VIT_L16_B64, synth.VIT_H14_B32):
        for kernel in range(4):
            if kernel >= 2 and sh is synth.VIT_B16_B8_F32:
                continue  # the single-layer workload is GELU only
            n, L = (sh.gelu_elems, sh.hidden) if kernel < 2 else (sh.softmax_elems, sh.tokens)
            plan = binding.s2a_describe_plan(kernel, n, L, sh.dtype)
            assert plan.startswith("tile") and plan.endswith("tail_rows=0"), plan


# ------------------------------------------------------------------ degenerate inputs
@pytest.mark.parametrize("L", [197, 145, 200])
@pytest.mark.parametrize("dt", [F32, BF16])
def test_degenerate_rows(dt, L):
    rows = 66
    x = np.zeros((rows, L), dtype=np.float32)
    x[1] = 0.37          # constant rows: max == min
    x[2] = -5.0
    x[3] = 7.0           # constant beyond the clip
    x[4, ::2] = 1e4      # extreme magnitudes
    x[4, 1::2] = -1e4
    x[5] = np.linspace(-3, 3, L)
    x[6, 0] = 2.0        # exactly on the clip
    x[6, 1] = -2.0
    x[7:] = synth.normal(1, "deg", (rows - 7) * L).reshape(rows - 7, L) * 0.05  # unsaturated rows
    g = synth.normal(1, "degg", rows * L)
    check_gelu(synth.to_io(x.reshape(-1), dt), synth.to_io(g, dt), L, dt)
    xs = x.copy()
    xs[4, ::2] = 80.0    # softmax: differences of 160 underflow to zero
    xs[4, 1::2] = -80.0
    xs[8] = 0.0
    xs[8, 5] = 30.0      # one-hot row
    check_softmax(synth.to_io(xs.reshape(-1), dt), synth.to_io(g, dt), L, dt)


@pytest.mark.parametrize("L", [49, 50, 64, 197, 257])
@pytest.mark.parametrize("dt", [F32, BF16])
def test_softmax_extremes_at_every_position(dt, L):
    # The fixed-width bfloat16 kernels find the range of y from the row's smallest and largest
    # input.  Every position of a row takes a turn at holding the maximum and the minimum (the
    # first and last elements share a 4-byte word with the neighbouring row when L is odd), some
    # rows hold several equal extremes, some a masked (hugely negative) entry: check_softmax
    # compares (min, s) and every code with Q(y as written), without tolerance.
    rows = 3 * L + 5
    x = synth.normal(9, ("ext", L, dt), rows * L).reshape(rows, L) * np.float32(1.5)
    r = np.arange(rows)
    hi_at, lo_at = r % L, (3 * r + 1) % L
    x[r, lo_at] = -9.0
    x[r, hi_at] = 6.0                       # where both fall on one element the maximum wins
    x[5, :] = np.where(np.arange(L) % 2 == 0, 1.25, -1.25)   # many equal extremes
    x[6, 0], x[6, L - 1] = 6.5, -9.5        # extremes in the two halves shared with neighbours
    x[7, 0], x[7, L - 1] = -9.5, 6.5
    x[8, L // 2] = -1.0e4                   # a masked entry: y underflows to exactly 0
    x[9, 0] = -1.0e4
    x[10, L - 1] = -1.0e4
    g = synth.normal(9, ("extg", L, dt), rows * L)
    check_softmax(synth.to_io(x.reshape(-1).astype(np.float32), dt), synth.to_io(g, dt), L, dt, max_flip_frac=5e-3)


def _random_shapes(seed, count):
    """Seeded (rows, L) pairs: lengths near the widths that have kernels of their own, powers of
    two and their neighbours, and arbitrary ones; row counts that leave ragged tails or none."""
    rng = np.random.RandomState(seed)
    special = [49, 50, 64, 145, 196, 197, 198, 257, 577, 1025, 3072, 4096]
    out = []
    for i in range(count):
        kind = i % 3
        if kind == 0:
            L = int(special[rng.randint(len(special))] + rng.randint(-1, 2))
        elif kind == 1:
            L = int(2 ** rng.randint(3, 12) + rng.randint(-1, 2))
        else:
            L = int(rng.randint(1, 2200))
        rows = int(rng.randint(1, max(2, min(3000, 600000 // max(L, 1)))))
        if rng.randint(2):
            rows = max(32, rows // 32 * 32)      # whole tiles, no tail
        out.append((rows, max(L, 1)))
    return out


@pytest.mark.parametrize("dt", [F32, BF16])
def test_seeded_random_shapes(dt):
    # the planner picks a kernel form and a tile per (kernel, length, type): a seeded walk over
    # shapes nobody chose by hand, every one compared with the oracle like the listed shapes
    for rows, L in _random_shapes(20250308, 36):
        check_gelu(*_gelu_inputs(rows, L, dt, seed=rows + L), L, dt)
        check_softmax(*_softmax_inputs(rows, L, dt, seed=rows + L), L, dt, max_flip_frac=8e-3)


@pytest.mark.parametrize("rows,L,dt", [(97536, 1025, F32), (173280, 577, BF16)])
def test_sweep_size_tensors_of_the_wide_odd_widths(rows, L, dt):
    # the bandwidth sweep's tensors at 577 / 1025 (1e8 elements): thousands of tiles whose code
    # bytes start at every offset of the 16-byte grid, all ranks of the persistent grid busy
    check_softmax(*_softmax_inputs(rows, L, dt, seed=3), L, dt, report="[%d, %d]" % (rows, L))


def test_hardware_exp2_never_decreases_over_the_arguments_softmax_uses():
    # exhaustive: every binary32 argument in [-150, 1], neighbours compared on the device
    import ctypes
    lib = binding.lib()
    bad = ctypes.c_ulonglong(12345)
    assert lib.s2a_selftest_exp2_monotone(ctypes.byref(bad), ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)) == 0
    assert bad.value == 0, "2^x approximate decreases at %d neighbouring arguments" % bad.value
    assert lib.s2a_selftest_exp2_monotone(None, None) == 1   # S2A_ERR_NULL


@pytest.mark.parametrize("L", [197, 64, 145, 1024])
@pytest.mark.parametrize("dt", [F32, BF16])
def test_softmax_large_common_offset(dt, L):
    # softmax is invariant to a per-row shift: rows riding on offsets of thousands (where the
    # spacing of the I/O type is far coarser than near zero) must still match the oracle.  The
    # offsets are exactly representable, so the shifted logits are too where they fit the type.
    rows = 320
    z = synth.normal(5, ("off", L, dt), rows * L).reshape(rows, L)
    step = np.float32(32.0 if dt == BF16 else 0.25)       # a multiple of the spacing at the offsets used
    offs = np.array([0, 1024, -2048, 4096, -4096, 3072, 512, -1536], dtype=np.float32)
    x = np.round(z * np.float32(2.0)) * step + offs[np.arange(rows) % offs.size, None]
    g = synth.normal(5, ("offg", L, dt), rows * L)
    check_softmax(synth.to_io(x.reshape(-1).astype(np.float32), dt), synth.to_io(g, dt), L, dt, max_flip_frac=5e-3)


@pytest.mark.parametrize("dt", [F32, BF16])
@pytest.mark.parametrize("rows,L", [(70, 3072), (41, 197), (300, 64), (9, 5)])
def test_gelu_far_negative_inputs_keep_their_tiny_outputs(rows, L, dt):
    # y = x * sigmoid(1.702 x) at x in [-56, -48] runs from 2^-110 down through the smallest
    # normal number (2^-126 at x = -53.7): still representable results that must come out
    # within tolerance, not flushed; every third row carries such inputs, the others none
    n = rows * L
    x = synth.gelu_preact(13, ("far", rows, L, dt), n).reshape(rows, L)
    deep = np.linspace(-56.0, -48.0, 4 * L, dtype=np.float32).reshape(4, L)
    for r in range(0, rows, 3):
        x[r, ::2] = deep[(r // 3) % 4, ::2]
    g = synth.normal(13, ("farg", rows, L, dt), n)
    check_gelu(synth.to_io(x.reshape(-1), dt), synth.to_io(g, dt), L, dt)


@pytest.mark.parametrize("L", [64, 128, 256, 1024, 3072])
def test_gelu_rows_whose_maximum_hides_at_the_end(L):
    # The bfloat16 forward takes a row's maximum from the first 16-byte vector of every lane and
    # searches the whole row only when that sample stays below the clip.  Neighbouring rows here
    # take different turns: saturated within the sample, saturated only by the row's last
    # element, not saturated at all, constant -- in one warp where several rows share a warp.
    rows = 96
    x = synth.normal(11, ("hide", L), rows * L).reshape(rows, L) * np.float32(0.3)
    x = np.clip(x, -1.5, 1.5)
    kind = np.arange(rows) % 6
    x[kind == 0, 0] = 5.0
    x[kind == 0, 1] = -5.0
    x[kind == 1, L - 1] = 2.5           # only the last element reaches the clip
    x[kind == 2, L - 1] = 1.75          # the maximum sits at the end and stays below the clip
    x[kind == 3, L - 1] = -7.0          # the minimum sits at the end
    x[kind == 4, :] = 0.625             # constant
    g = synth.normal(11, ("hideg", L), rows * L)
    check_gelu(synth.to_io(x.reshape(-1).astype(np.float32), BF16), synth.to_io(g, BF16), L, BF16)


def _double_rounding_tie_rows(L, n_rows, seed):
    """binary32 rows whose elements sit where Eq. 8's pinned sequence needs BOTH of its roundings:
    the exact product (x - min) * inv is not a half-integer, but its binary32 rounding is exactly
    k + 1/2, which the second rounding (to the nearest even code) then resolves.  An evaluation
    that fuses the multiplication into the rounding step gets the neighbouring code."""
    rng = np.random.default_rng(seed)
    rows = []
    f = np.float32
    while len(rows) < n_rows:
        mn, mx = f(-rng.uniform(0.3, 1.9)), f(rng.uniform(0.3, 1.9))
        inv = f(f(15) / f(mx - mn))
        found = []
        for k in range(15):
            x0 = f(mn + f((k + 0.5) / float(inv)))
            cand = x0.view(np.uint32).astype(np.int64) + np.arange(-300, 301)
            x = cand.astype(np.uint32).view(np.float32)
            t = ((x - mn).astype(np.float32) * inv).astype(np.float32)
            exact = (x.astype(np.float64) - float(mn))            # exact: few bits, close exponents
            hit = (t == f(k + 0.5)) & (exact * float(inv) != k + 0.5) & (x > mn) & (x < mx)
            found.extend(x[hit].tolist())
        if len(found) < 4:
            continue
        row = rng.choice(np.array(found, dtype=np.float32), size=L)
        row[0], row[1] = mn, mx
        rows.append(row)
    return np.stack(rows)


@pytest.mark.parametrize("L", [3072, 197, 64])
def test_gelu_codes_where_the_quantiser_needs_both_of_its_roundings(L):
    x = _double_rounding_tie_rows(L, 70, seed=L)
    g = synth.normal(21, ("tie", L), x.size)
    check_gelu(x.reshape(-1), g, L, F32)


def test_gelu_saturated_row_hand_codes():
    # bin edges of a [-2, 2] row; 0 is the exact tie 7.5 and must round to 8
    row = np.array([-3, -2, -1, -0.1333333, 0, 0.1333334, 0.5, 1, 2, 2.5], dtype=np.float32)
    y, codes, meta = pu.gpu_fwd("gelu", row, 10, F32)
    assert pu.unpack_np(codes, 10).tolist() == [0, 0, 4, 7, 8, 8, 9, 11, 15, 15]
    assert meta[0] == -2.0 and meta[1] == np.float32(np.float32(4) / np.float32(15))


def test_softmax_worked_row():
    x = np.array([0, 1, 2, 3], dtype=np.float32)
    y, codes, meta = pu.gpu_fwd("softmax", x, 4, F32)
    e = np.exp(np.arange(4.0))
    assert np.allclose(y, e / e.sum(), rtol=1e-6)
    assert codes.tolist() == [0x10, 0xF5]
    gin = pu.gpu_bwd("softmax", np.array([1, -1, 0.5, 2], dtype=np.float32), codes, meta, 4, F32)
    yh = np.array([0, 1, 5, 15]) * float(meta[1]) + float(meta[0])
    dot = float(np.array([1, -1, 0.5, 2]) @ yh)
    assert np.allclose(gin, yh * (np.array([1, -1, 0.5, 2]) - dot), rtol=2e-6)


def test_empty_and_argument_errors():
    L = binding.lib()
    dev = torch.device("cuda")
    x = torch.zeros(64, device=dev)
    codes, meta = binding.alloc_stash(64, 8, dev)
    s = torch.cuda.current_stream().cuda_stream
    before = (x.clone(), codes.clone().fill_(7), meta.clone().fill_(3))
    codes.fill_(7), meta.fill_(3)
    args = lambda xp, yp, cp, mp, n, rl, dt: L.s2a_gelu_fwd(xp, yp, cp, mp, n, rl, dt, s)
    assert args(x.data_ptr(), x.data_ptr(), codes.data_ptr(), meta.data_ptr(), 0, 8, 0) == 0      # empty
    assert args(None, x.data_ptr(), codes.data_ptr(), meta.data_ptr(), 64, 8, 0) == 1               # NULL
    assert args(x.data_ptr(), x.data_ptr(), codes.data_ptr(), meta.data_ptr(), 64, 0, 0) == 2       # row_len 0
    assert args(x.data_ptr(), x.data_ptr(), codes.data_ptr(), meta.data_ptr(), 63, 8, 0) == 2       # ragged
    assert args(x.data_ptr() + 4, x.data_ptr(), codes.data_ptr(), meta.data_ptr(), 32, 8, 0) == 3   # alignment
    assert args(x.data_ptr(), x.data_ptr(), codes.data_ptr(), meta.data_ptr() + 4, 32, 8, 0) == 3
    assert args(x.data_ptr(), x.data_ptr(), codes.data_ptr(), meta.data_ptr(), 64, 8, 7) == 4       # dtype
    for f in (L.s2a_gelu_bwd, L.s2a_softmax_fwd, L.s2a_softmax_bwd):
        assert f(x.data_ptr(), None, meta.data_ptr(), x.data_ptr(), 64, 8, 0, s) == 1
    torch.cuda.synchronize()
    assert torch.equal(x, before[0]) and torch.equal(codes, before[1]) and torch.equal(meta, before[2])
    with pytest.raises(binding.S2AError):
        binding.s2a_gelu_fwd(x.cpu(), x, codes, meta, 8)


# ------------------------------------------------------------------ the named workloads
def test_config1_single_gelu_layer_f32_full():
    sh = synth.VIT_B16_B8_F32
    x, g = synth.vit_gelu_inputs(sh, 0, 0)
    assert x.size == 8 * 197 * 3072
    check_gelu(x, g, sh.hidden, sh.dtype)


# Every block of the benchmark workload (ViT-B/16), the first and the last block of the two
# larger ones: each block has its own seeded tensors.
FULL_SIZE_BLOCKS = ([(synth.VIT_B16_B64, b) for b in range(synth.VIT_B16_B64.blocks)] +
                    [(sh, b) for sh in (synth.VIT_L16_B64, synth.VIT_H14_B32) for b in (0, sh.blocks - 1)])


@pytest.mark.parametrize("shape,block", FULL_SIZE_BLOCKS, ids=lambda v: v.name if hasattr(v, "name") else "block%d" % v)
def test_vit_block_full_size(shape, block):
    """One block of a ViT workload at its full size, every element compared."""
    x, g = synth.vit_gelu_inputs(shape, 0, block)
    assert x.size == shape.gelu_elems
    check_gelu(x, g, shape.hidden, shape.dtype)
    # every row of the bulk+tail input saturates the clip: per-row == per-tensor range
    del x, g
    x, g = synth.vit_softmax_inputs(shape, 0, block)
    assert x.size == shape.softmax_elems
    check_softmax(x, g, shape.tokens, shape.dtype, report="%s block %d" % (shape.name, block))


@pytest.mark.parametrize("shape", [synth.VIT_B16_B64, synth.VIT_L16_B64, synth.VIT_H14_B32], ids=lambda s: s.name)
def test_vit_softmax_binary32_error_against_the_1e6_line(shape):
    """The attention shapes of the three workloads in binary32 (a slice of a block): the largest
    relative error of y is printed next to the 1e-6 line, so that the allowance for the rounding
    of the exponent's argument (2^-24 |x_i - max x|) is visible as a number."""
    rows = 20000
    x, g = synth.vit_softmax_inputs(shape, 0, 0, rows)
    x, g = synth.io_to_f32(x, shape.dtype), synth.io_to_f32(g, shape.dtype)   # the same logits, held in binary32
    st = check_softmax(x, g, shape.tokens, F32, report="%s block 0, %d rows in binary32" % (shape.name, rows))
    assert st["y_worst_rel"] < 4e-6


def test_tensor_beyond_2_to_31_elements_uses_64_bit_indexing():
    """2.2e9 bfloat16 elements (the largest size of the bandwidth sweep): a seeded block of
    rows is repeated down the tensor, every repeat must come out identical, and the first
    and the last repeat are compared with the oracle element by element."""
    L, block_rows, repeats = 4096, 1024, 525          # 2,202,009,600 elements
    free, _ = torch.cuda.mem_get_info()
    n = L * block_rows * repeats
    if free < 2.6 * 2 * n:
        pytest.skip("not enough free device memory for a 2.2e9-element tensor")
    x, g = _gelu_inputs(block_rows, L, BF16, seed=5)
    xb = pu.to_device(x, BF16)
    xd = xb.repeat(repeats)
    assert xd.numel() == n and n > 2 ** 31
    yd = torch.empty_like(xd)
    codes, meta = binding.alloc_stash(n, L, xd.device)
    binding.s2a_gelu_fwd(xd, yd, codes, meta, L)
    torch.cuda.synchronize()
    assert binding.s2a_device_error() == 0
    y_o, codes_o, meta_o = o.gelu_fwd(x, L, BF16, threads=THREADS)
    yv = yd.view(repeats, -1)
    cv = codes.view(repeats, -1)
    mv = meta.view(repeats, -1)
    assert bool((yv == yv[0]).all()) and bool((cv == cv[0]).all()) and bool((mv == mv[0]).all())
    for rep in (0, repeats - 1):
        assert np.array_equal(cv[rep].cpu().numpy(), codes_o)
        assert np.array_equal(mv[rep].cpu().numpy(), meta_o)
        pu.assert_close(pu.widen(pu.to_host(yv[rep], BF16), BF16), pu.widen(y_o, BF16), BF16, "gelu y (large)")
    del yd, yv
    gd = pu.to_device(g, BF16).repeat(repeats)
    gin = torch.empty_like(gd)
    binding.s2a_gelu_bwd(gd, codes, meta, gin, L)
    torch.cuda.synchronize()
    assert binding.s2a_device_error() == 0
    gin_o = o.gelu_bwd(g, codes_o, meta_o, L, BF16, threads=THREADS)
    gv = gin.view(repeats, -1)
    assert bool((gv == gv[0]).all())
    pu.assert_close(pu.widen(pu.to_host(gv[repeats - 1], BF16), BF16), pu.widen(gin_o, BF16), BF16, "gelu grad_in (large)")


# ------------------------------------------------------------------ SiLU with the 4-bit stash
@pytest.mark.parametrize("dt", [F32, BF16])
@pytest.mark.parametrize("rows,L", [(5, 1), (7, 3), (33, 65), (451, 197), (1001, 64), (137, 1024), (41, 3072),
                                    (11, 4096), (9, 5120), (3, 8191), (2, 40000)])
def test_silu(rows, L, dt):
    n = rows * L
    x = synth.to_io(synth.gelu_preact(9, ("silu", rows, L, dt), n) * np.float32(2.2), dt)
    g = synth.to_io(synth.normal(9, ("silug", rows, L, dt), n), dt)
    for inplace in (False, True):
        y_o, codes_o, meta_o = o.silu_fwd(x, L, dt, threads=THREADS)
        y_g, codes_g, meta_g = pu.gpu_fwd("silu", x, L, dt, inplace=inplace)
        assert np.array_equal(codes_g, codes_o), "SiLU codes differ from the oracle's"
        assert np.array_equal(meta_g.view(np.uint32), meta_o.view(np.uint32))
        pu.assert_close(pu.widen(y_g, dt), pu.widen(y_o, dt), dt, "silu y")
        gin_o = o.silu_bwd(g, codes_o, meta_o, L, dt, threads=THREADS)
        gin_g = pu.gpu_bwd("silu", g, codes_o, meta_o, L, dt, inplace=inplace)
        pu.assert_close(pu.widen(gin_g, dt), pu.widen(gin_o, dt), dt, "silu grad_in")
    plan = binding.s2a_describe_plan(binding.SILU_FWD, n, L, dt)
    # pipelined whenever rows are whole 16-byte vectors and two of them fit a shared-memory stage
    fits = 2 * L * synth.io_itemsize(dt) <= 176 * 1024
    assert plan.startswith("tile") == (L % (4 if dt == F32 else 8) == 0 and rows >= 2 and fits), plan


# ------------------------------------------------------------------ other bit widths (Eq. 8, general N)
@pytest.mark.parametrize("dt", [F32, BF16])
@pytest.mark.parametrize("bits", [2, 4, 8])
@pytest.mark.parametrize("kind,rows,L", [("gelu", 7, 3), ("gelu", 41, 197), ("gelu", 24, 3072), ("gelu", 5, 1),
                                         ("gelu", 1237, 4096), ("gelu", 77, 1024), ("gelu", 311, 5120),
                                         ("gelu", 13, 8192), ("gelu_narrow", 2001, 3072), ("gelu_narrow", 90, 2048),
                                         ("softmax", 9, 65), ("softmax", 300, 197), ("softmax", 12, 1024),
                                         ("softmax", 3, 2), ("softmax", 131, 257), ("softmax", 1283, 198),
                                         ("softmax", 700, 49), ("softmax", 401, 50), ("softmax", 150, 577),
                                         ("softmax", 90, 4096), ("softmax", 517, 64), ("softmax", 1000, 197)])
def test_other_bit_widths(kind, rows, L, bits, dt):
    # "gelu_narrow": rows that do not reach the clip, so that every row has its own (min, s)
    # and the backward's derivative table is rebuilt row after row
    n = rows * L
    if kind.startswith("gelu"):
        x, g = _gelu_inputs(rows, L, dt, seed=20 + bits, scale=0.3 if kind == "gelu_narrow" else 1.3)
        kind = "gelu"
    else:
        x, g = _softmax_inputs(rows, L, dt, seed=20 + bits)
    y_o, codes_o, meta_o = o.fwd_bits(kind, x, L, bits, dt)
    item = synth.io_itemsize(dt)
    tdt = pu.torch_dtype(dt)
    yg, cg, mg = pu.Guarded(n * item), pu.Guarded(binding.codes_bytes_bits(n, bits)), pu.Guarded(binding.meta_bytes(n, L))
    binding.s2a_fwd_bits(kind, pu.to_device(x, dt), yg.view(tdt), cg.view(torch.uint8), mg.view(torch.float32), L, bits)
    og = pu.Guarded(n * item)
    binding.s2a_bwd_bits(kind, pu.to_device(g, dt), torch.from_numpy(codes_o).cuda(), torch.from_numpy(meta_o).cuda(),
                         og.view(tdt), L, bits)
    torch.cuda.synchronize()
    for buf, what in ((yg, "y"), (cg, "codes"), (mg, "meta"), (og, "grad_in")):
        buf.check("%s bits=%d %s" % (kind, bits, what))
    assert binding.codes_bytes_bits(n, bits) == (n * bits + 7) // 8
    y_g = pu.to_host(yg.view(tdt), dt)
    codes_g = cg.view(torch.uint8).cpu().numpy()
    meta_g = mg.view(torch.float32).cpu().numpy()
    q_g = o.unpack_bits(codes_g, n, bits).reshape(rows, L)
    q_o = o.unpack_bits(codes_o, n, bits).reshape(rows, L)
    xw = pu.widen(x, dt).reshape(rows, L)
    if kind == "gelu":
        assert np.array_equal(codes_g, codes_o) and np.array_equal(meta_g.view(np.uint32), meta_o.view(np.uint32))
        pu.assert_close(pu.widen(y_g, dt), pu.widen(y_o, dt), dt, "gelu y")
        mag = None
    else:
        gap = (xw.max(axis=1, keepdims=True) - xw) * 2.0 ** -24
        pu.assert_close(pu.widen(y_g, dt), pu.widen(y_o, dt), dt, "softmax y", extra_rtol=gap)
        # codes are Q_N(y as written): an independent numpy evaluation, zero tolerance
        v = synth.io_to_f32(y_g, dt).reshape(rows, L)
        mn, mx = v.min(axis=1, keepdims=True), v.max(axis=1, keepdims=True)
        d = (mx - mn).astype(np.float32)
        levels = np.float32(2 ** bits - 1)
        with np.errstate(divide="ignore", invalid="ignore"):
            inv = np.where(d == 0, np.float32(0), levels / d).astype(np.float32)
        q_np = np.rint(((v - mn).astype(np.float32) * inv).astype(np.float32)).astype(np.uint8)
        assert np.array_equal(q_g, q_np)
        tol_y, _ = pu.tolerance(pu.widen(y_o, dt), dt, extra_rtol=gap)
        st = pu.check_edge_flips(q_g, q_o, pu.widen(y_o, dt), meta_o, tol_y, dt, levels=2 ** bits - 1,
                                 what="softmax bits=%d" % bits)
        assert st["flips"] <= max(2, 0.02 * n)
        yh = q_o.astype(np.float64) * meta_o[1::2, None].astype(np.float64) + meta_o[0::2, None].astype(np.float64)
        mag = yh * (np.abs(pu.widen(g, dt).reshape(rows, L)) * yh).sum(axis=1, keepdims=True)
    gin_o = o.bwd_bits(kind, g, codes_o, meta_o, L, bits, dt)
    pu.assert_close(pu.widen(pu.to_host(og.view(tdt), dt), dt), pu.widen(gin_o, dt), dt, "grad_in", extra_mag=mag)
    if bits == 4:   # the same bytes as the 4-bit entry points
        y4, c4, m4 = pu.gpu_fwd(kind, x, L, dt)
        assert np.array_equal(c4, codes_g) and np.array_equal(m4, meta_g) and np.array_equal(y4, y_g)


@pytest.mark.parametrize("dt", [F32, BF16])
@pytest.mark.parametrize("bits", [2, 8])
@pytest.mark.parametrize("kind,L", [("gelu", 3072), ("softmax", 197), ("softmax", 1024)])
def test_other_bit_widths_degenerate_rows(kind, L, bits, dt):
    # constant rows (max == min: codes 0, s = 0), rows beyond the clip, one-hot rows
    rows = 130
    x = synth.normal(9, ("bdeg", kind, L), rows * L).reshape(rows, L).astype(np.float32)
    x[1] = 0.37
    x[2] = -5.0
    x[3] = 7.0
    x[4] = 0.0
    x[4, 5] = 30.0
    x[5, ::2] = 80.0
    x[5, 1::2] = -80.0
    n = rows * L
    xi = synth.to_io(x.reshape(-1), dt)
    y_o, codes_o, meta_o = o.fwd_bits(kind, xi, L, bits, dt)
    tdt = pu.torch_dtype(dt)
    yg, cg, mg = pu.Guarded(n * synth.io_itemsize(dt)), pu.Guarded(binding.codes_bytes_bits(n, bits)), pu.Guarded(binding.meta_bytes(n, L))
    binding.s2a_fwd_bits(kind, pu.to_device(xi, dt), yg.view(tdt), cg.view(torch.uint8), mg.view(torch.float32), L, bits)
    torch.cuda.synchronize()
    for buf, what in ((yg, "y"), (cg, "codes"), (mg, "meta")):
        buf.check("%s bits=%d %s" % (kind, bits, what))
    meta_g = mg.view(torch.float32).cpu().numpy()
    q_g = o.unpack_bits(cg.view(torch.uint8).cpu().numpy(), n, bits).reshape(rows, L)
    q_o = o.unpack_bits(codes_o, n, bits).reshape(rows, L)
    for r in (1, 2, 3):  # constant rows
        assert meta_g[2 * r + 1] == 0.0 and not q_g[r].any()
    if kind == "gelu":
        assert np.array_equal(q_g, q_o) and np.array_equal(meta_g.view(np.uint32), meta_o.view(np.uint32))
    else:
        assert q_g[4].max() == 2 ** bits - 1 and int((q_g[4] != 0).sum()) == 1   # one-hot row
        assert np.abs(q_g.astype(int) - q_o.astype(int)).max() <= 1


def test_other_bit_widths_reject_unsupported_values():
    L = binding.lib()
    x = torch.zeros(64, device="cuda")
    codes, meta = binding.alloc_stash(64 * 2, 8, "cuda")
    s = torch.cuda.current_stream().cuda_stream
    for bits in (0, 1, 3, 16):
        assert L.s2a_gelu_fwd_bits(x.data_ptr(), x.data_ptr(), codes.data_ptr(), meta.data_ptr(), 64, 8, bits, 0, s) == 2
        assert binding.codes_bytes_bits(64, bits) == 0


# ------------------------------------------------------------------ CAP (Eq. 5) and LRP add (Eq. 3)
@pytest.mark.parametrize("dt", [F32, BF16])
@pytest.mark.parametrize("rows,ch,r", [(3, 8, 8), (5, 24, 3), (12608, 768, 8), (1000, 96, 4), (7, 10, 1), (64, 1024, 16)])
def test_cap(rows, ch, r, dt):
    x = synth.to_io(synth.normal(3, ("cap", rows, ch, r, dt), rows * ch), dt)
    g = synth.to_io(synth.normal(3, ("capg", rows, ch, r, dt), rows * ch // r), dt)
    y_o = o.cap_fwd(x, rows, ch, r, dt)
    gin_o = o.cap_bwd(g, rows, ch, r, dt)
    item = synth.io_itemsize(dt)
    tdt = pu.torch_dtype(dt)
    yg, og = pu.Guarded(rows * ch // r * item), pu.Guarded(rows * ch * item)
    binding.s2a_cap_fwd(pu.to_device(x, dt), yg.view(tdt), rows, ch, r)
    binding.s2a_cap_bwd(pu.to_device(g, dt), og.view(tdt), rows, ch, r)
    torch.cuda.synchronize()
    yg.check("cap y"), og.check("cap grad_in")
    mean_abs = np.abs(pu.widen(x, dt)).reshape(-1, r).mean(axis=1)        # size of the summed terms
    pu.assert_close(pu.widen(pu.to_host(yg.view(tdt), dt), dt), pu.widen(y_o, dt), dt, "cap y",
                    extra_mag=mean_abs * (1.0 if dt == F32 else 2.0 ** -12))
    pu.assert_close(pu.widen(pu.to_host(og.view(tdt), dt), dt), pu.widen(gin_o, dt), dt, "cap grad_in")


@pytest.mark.parametrize("dt", [F32, BF16])
@pytest.mark.parametrize("batch,tokens,ch,rank", [(3, 7, 16, 5), (64, 197, 768, 30), (2, 5, 12, 3), (9, 50, 1024, 30)])
def test_lrp_add(batch, tokens, ch, rank, dt):
    n = batch * tokens * ch
    x = synth.to_io(synth.normal(4, ("lrp", batch, tokens, ch, dt), n), dt)
    A = synth.normal(4, ("lrpA", tokens, rank), tokens * rank)
    B = synth.normal(4, ("lrpB", rank, ch), rank * ch)
    y_o = o.lrp_fwd(x, A, B, batch, tokens, ch, rank, dt)
    tdt = pu.torch_dtype(dt)
    yg = pu.Guarded(n * synth.io_itemsize(dt))
    binding.s2a_lrp_fwd(pu.to_device(x, dt), torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), yg.view(tdt),
                        batch, tokens, ch, rank)
    torch.cuda.synchronize()
    yg.check("lrp y")
    terms = np.abs(A.reshape(tokens, rank).astype(np.float64)) @ np.abs(B.reshape(rank, ch).astype(np.float64))
    mag = np.broadcast_to(terms[None], (batch, tokens, ch)).reshape(-1) + np.abs(pu.widen(x, dt))
    pu.assert_close(pu.widen(pu.to_host(yg.view(tdt), dt), dt), pu.widen(y_o, dt), dt, "lrp y",
                    extra_mag=mag * (4.0 if dt == F32 else 2.0 ** -12))


# ------------------------------------------------------------------ per-tensor range variant
@pytest.mark.parametrize("dt", [F32, BF16])
@pytest.mark.parametrize("rows,L,scale", [(3, 5, 0.3), (1, 1, 1.0), (7, 197, 0.2), (300, 66, 0.4), (64, 3072, 0.25),
                                          (1576, 3072, 1.3), (40, 65536, 0.5), (3, 100003, 0.3)])
def test_gelu_tensor_range(rows, L, scale, dt):
    n = rows * L
    x = synth.to_io(synth.gelu_preact(7, ("gtr", rows, L, dt), n) * np.float32(scale), dt)
    g = synth.to_io(synth.normal(7, ("gtrg", rows, L, dt), n), dt)
    y_o, codes_o, meta_o = o.gelu_fwd_tensor_range(x, L, dt)
    item = synth.io_itemsize(dt)
    tdt = pu.torch_dtype(dt)
    xd = pu.to_device(x, dt)
    yg, cg, mg = pu.Guarded(n * item), pu.Guarded(binding.codes_bytes(n)), pu.Guarded(binding.meta_bytes(n, L))
    sg = pu.Guarded(binding.tensor_range_scratch_bytes(n))
    binding.s2a_gelu_fwd_tensor_range(xd, yg.view(tdt), cg.view(torch.uint8), mg.view(torch.float32),
                                      sg.view(torch.uint8), L)
    torch.cuda.synchronize()
    for buf, what in ((yg, "y"), (cg, "codes"), (mg, "meta"), (sg, "scratch")):
        buf.check("gelu_fwd_tensor_range " + what)
    assert np.array_equal(pu.to_host(xd, dt), x)
    assert np.array_equal(cg.view(torch.uint8).cpu().numpy(), codes_o)
    assert np.array_equal(mg.view(torch.float32).cpu().numpy().view(np.uint32), meta_o.view(np.uint32))
    pu.assert_close(pu.widen(pu.to_host(yg.view(tdt), dt), dt), pu.widen(y_o, dt), dt, "gelu y (tensor range)")
    # the ordinary backward consumes this stash
    gin_o = o.gelu_bwd(g, codes_o, meta_o, L, dt, threads=THREADS)
    gin_g = pu.gpu_bwd("gelu", g, codes_o, meta_o, L, dt)
    pu.assert_close(pu.widen(gin_g, dt), pu.widen(gin_o, dt), dt, "gelu grad_in (tensor range)")


def test_gelu_tensor_range_in_place_and_argument_errors():
    L = binding.lib()
    x = torch.zeros(64, device="cuda")
    y = torch.zeros(64, device="cuda")
    codes, meta = binding.alloc_stash(64, 8, "cuda")
    scratch = torch.zeros(64, dtype=torch.uint8, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    f = L.s2a_gelu_fwd_tensor_range
    assert f(x.data_ptr(), x.data_ptr() + 64, codes.data_ptr(), meta.data_ptr(), scratch.data_ptr(), 32, 8, 0, s) == 8
    assert f(x.data_ptr(), y.data_ptr(), codes.data_ptr(), meta.data_ptr(), None, 64, 8, 0, s) == 1
    assert f(x.data_ptr(), y.data_ptr(), codes.data_ptr(), meta.data_ptr(), scratch.data_ptr(), 63, 8, 0, s) == 2
    assert binding.tensor_range_scratch_bytes(1) == 16 and binding.tensor_range_scratch_bytes(65537) == 24
    # in place (y is x itself): the same results as out of place
    for dt in (F32, BF16):
        rows, Lr = 300, 3072
        xh = synth.to_io(synth.gelu_preact(17, ("gtr_inplace", dt), rows * Lr) * np.float32(0.4), dt)
        y_o, codes_o, meta_o = o.gelu_fwd_tensor_range(xh, Lr, dt)
        xd = pu.to_device(xh, dt)
        cg, mg = binding.alloc_stash(rows * Lr, Lr, "cuda")
        sc = torch.empty(binding.tensor_range_scratch_bytes(rows * Lr), dtype=torch.uint8, device="cuda")
        binding.s2a_gelu_fwd_tensor_range(xd, xd, cg, mg, sc, Lr)
        torch.cuda.synchronize()
        assert np.array_equal(cg.cpu().numpy(), codes_o) and np.array_equal(mg.cpu().numpy(), meta_o)
        pu.assert_close(pu.widen(pu.to_host(xd, dt), dt), pu.widen(y_o, dt), dt, "gelu y (tensor range, in place)")


def test_a_wait_that_runs_out_sets_the_error_word_and_leaves_the_context_usable():
    # the self-test's wait has nothing to wait for: it must give up after its 2 ms, record its
    # bit, and return; the word reads 4 until cleared, and ordinary calls work afterwards
    import ctypes
    lib = binding.lib()
    lib.s2a_selftest_wait_expiry.argtypes = [ctypes.c_void_p]
    lib.s2a_selftest_wait_expiry.restype = ctypes.c_int
    flags = ctypes.c_uint(0)
    assert lib.s2a_device_error(ctypes.byref(flags), 1) == 0
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    assert lib.s2a_selftest_wait_expiry(ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)) == 0
    t1.record()
    torch.cuda.synchronize()
    assert 1.5 < t0.elapsed_time(t1) < 500.0, "the wait should give up after about 2 ms"
    assert lib.s2a_device_error(ctypes.byref(flags), 0) == 0 and flags.value == 4
    assert lib.s2a_device_error(ctypes.byref(flags), 1) == 0 and flags.value == 4
    assert lib.s2a_device_error(ctypes.byref(flags), 0) == 0 and flags.value == 0
    check_gelu(*_gelu_inputs(70, 3072, BF16, seed=4), 3072, BF16)       # the context is as usable as before


def test_device_error_word_reads_zero_and_clears():
    # no kernel of this suite gives up on a wait: the word stays 0, and reading it with
    # clear = 1 leaves it 0 (the expiry path itself is not provoked on a shared GPU)
    lib = binding.lib()
    import ctypes
    flags = ctypes.c_uint(0xFFFFFFFF)
    assert lib.s2a_device_error(ctypes.byref(flags), 1) == 0 and flags.value == 0
    flags = ctypes.c_uint(0xFFFFFFFF)
    assert lib.s2a_device_error(ctypes.byref(flags), 0) == 0 and flags.value == 0
    assert lib.s2a_device_error(None, 0) == 1


# ------------------------------------------------------------------ ReLU with a 1-bit stash
@pytest.mark.parametrize("dt", [F32, BF16])
@pytest.mark.parametrize("n", [1, 7, 8, 9, 1023, 1024 * 8, 100003, 5_000_001, 40_000_008])
def test_relu_mask(n, dt):
    x32 = synth.normal(6, ("relu", n, dt), n)
    x32[::7] = 0.0
    x32[3::11] = -0.0
    x = synth.to_io(x32, dt)
    g = synth.to_io(synth.normal(6, ("relug", n, dt), n), dt)
    y_o, mask_o = o.relu_fwd(x, dt)
    gin_o = o.relu_bwd(g, mask_o, dt)
    item = synth.io_itemsize(dt)
    tdt = pu.torch_dtype(dt)
    for inplace in (False, True):
        xd, gd = pu.to_device(x, dt), pu.to_device(g, dt)
        yg, mg, og = pu.Guarded(n * item), pu.Guarded(binding.mask_bytes(n)), pu.Guarded(n * item)
        if inplace:
            yg.view(tdt).copy_(xd)
            og.view(tdt).copy_(gd)
        binding.s2a_relu_fwd(yg.view(tdt) if inplace else xd, yg.view(tdt), mg.view(torch.uint8))
        md = torch.from_numpy(mask_o).cuda()
        binding.s2a_relu_bwd(og.view(tdt) if inplace else gd, md, og.view(tdt))
        torch.cuda.synchronize()
        for buf, what in ((yg, "y"), (mg, "mask"), (og, "grad_in")):
            buf.check("relu " + what)
        # exact: the ReLU stash is lossless
        assert np.array_equal(pu.to_host(yg.view(tdt), dt).view(np.uint8), y_o.view(np.uint8))
        assert np.array_equal(mg.view(torch.uint8).cpu().numpy(), mask_o)
        assert np.array_equal(pu.to_host(og.view(tdt), dt).view(np.uint8), gin_o.view(np.uint8))
    assert binding.mask_bytes(n) == (n + 7) // 8


def test_softmax_ten_million_rows_of_197():
    """The largest softmax case of the bandwidth sweep (1e7 rows of 197, 1.97e9 bfloat16
    elements, beyond 2^32 bytes per tensor): a seeded block of rows repeated down the tensor;
    every repeat must be identical and the first and last are compared with the oracle."""
    L, block_rows, repeats = 197, 4000, 2500
    n = L * block_rows * repeats
    free, _ = torch.cuda.mem_get_info()
    if free < 2.7 * 2 * n:
        pytest.skip("not enough free device memory")
    x, g = _softmax_inputs(block_rows, L, BF16, seed=8)
    y_o, codes_o, meta_o = o.softmax_fwd(x, L, BF16, threads=THREADS)
    xd = pu.to_device(x, BF16).repeat(repeats)
    yd = torch.empty_like(xd)
    codes, meta = binding.alloc_stash(n, L, xd.device)
    binding.s2a_softmax_fwd(xd, yd, codes, meta, L)
    torch.cuda.synchronize()
    assert binding.s2a_device_error() == 0
    yv, cv, mv = yd.view(repeats, -1), codes.view(repeats, -1), meta.view(repeats, -1)
    assert bool((yv == yv[0]).all()) and bool((cv == cv[0]).all()) and bool((mv == mv[0]).all())
    for rep in (0, repeats - 1):
        y_g = pu.to_host(yv[rep], BF16)
        pu.assert_close(pu.widen(y_g, BF16), pu.widen(y_o, BF16), BF16, "softmax y (large)")
        q_np, meta_np = pu.numpy_quantize(synth.io_to_f32(y_g, BF16), L)
        assert np.array_equal(pu.unpack_np(cv[rep].cpu().numpy(), block_rows * L).reshape(block_rows, L), q_np)
        assert np.array_equal(mv[rep].cpu().numpy().view(np.uint32), meta_np.view(np.uint32))
    del yd, yv, xd
    # backward from the oracle's stash, repeated the same way
    cd = torch.from_numpy(codes_o).cuda().repeat(repeats)
    md = torch.from_numpy(meta_o).cuda().repeat(repeats)
    gd = pu.to_device(g, BF16).repeat(repeats)
    gin = torch.empty_like(gd)
    binding.s2a_softmax_bwd(gd, cd, md, gin, L)
    torch.cuda.synchronize()
    assert binding.s2a_device_error() == 0
    gv = gin.view(repeats, -1)
    assert bool((gv == gv[0]).all())
    gin_o = o.softmax_bwd(g, codes_o, meta_o, L, BF16, threads=THREADS)
    q_o = pu.unpack_np(codes_o, block_rows * L).reshape(block_rows, L)
    yh = q_o.astype(np.float64) * meta_o[1::2, None].astype(np.float64) + meta_o[0::2, None].astype(np.float64)
    M = yh * (np.abs(pu.widen(g, BF16).reshape(block_rows, L)) * yh).sum(axis=1, keepdims=True)
    pu.assert_close(pu.widen(pu.to_host(gv[repeats - 1], BF16), BF16), pu.widen(gin_o, BF16), BF16,
                    "softmax grad_in (large)", extra_mag=M)


def test_metadata_that_is_only_8_byte_aligned_takes_the_row_path_and_matches():
    """The pipelined path moves metadata with 16-byte bulk copies; a metadata pointer that is
    only 8-byte aligned (allowed by the ABI) must be served by the row-at-a-time path with
    the same results."""
    rows, L, dt = 256, 3072, BF16
    x, g = _gelu_inputs(rows, L, dt, seed=12)
    y_o, codes_o, meta_o = o.gelu_fwd(x, L, dt, threads=THREADS)
    xd = pu.to_device(x, dt)
    yd = torch.empty_like(xd)
    codes = torch.empty(binding.codes_bytes(rows * L), dtype=torch.uint8, device="cuda")
    meta_big = torch.full((2 * rows + 4,), -7.0, dtype=torch.float32, device="cuda")
    meta = meta_big[2:2 + 2 * rows]                       # 8 bytes past a 16-byte boundary
    assert meta.data_ptr() % 16 == 8
    binding.s2a_gelu_fwd(xd, yd, codes, meta, L)
    gin = torch.empty_like(xd)
    binding.s2a_gelu_bwd(pu.to_device(g, dt), codes, meta, gin, L)
    torch.cuda.synchronize()
    assert np.array_equal(codes.cpu().numpy(), codes_o) and np.array_equal(meta.cpu().numpy(), meta_o)
    assert meta_big[:2].tolist() == [-7.0, -7.0] and meta_big[-2:].tolist() == [-7.0, -7.0]
    pu.assert_close(pu.widen(pu.to_host(yd, dt), dt), pu.widen(y_o, dt), dt, "gelu y (row path)")
    gin_o = o.gelu_bwd(g, codes_o, meta_o, L, dt, threads=THREADS)
    pu.assert_close(pu.widen(pu.to_host(gin, dt), dt), pu.widen(gin_o, dt), dt, "gelu grad_in (row path)")


def test_stash_bytes_are_half_a_byte_per_element_plus_row_metadata():
    for sh in (synth.VIT_B16_B64, synth.VIT_L16_B64, synth.VIT_H14_B32):
        total = 0
        for n, L in ((sh.gelu_elems, sh.hidden), (sh.softmax_elems, sh.tokens)):
            assert binding.codes_bytes(n) == (n + 1) // 2
            assert binding.meta_bytes(n, L) == 8 * (n // L)
            total += sh.blocks * (binding.codes_bytes(n) + binding.meta_bytes(n, L))
        bf16_stash = sh.blocks * 2 * (sh.gelu_elems + sh.softmax_elems)
        assert 3.8 < bf16_stash / total < 4.0
        free, _ = torch.cuda.mem_get_info()
        assert total < 0.02 * 180e9 and total < free
