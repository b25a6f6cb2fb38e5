"""Host-side checks of bench.py's helpers (no GPU): the byte accounting and the code-flip count
that goes into the benchmark line."""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402
from oracle import s2a_oracle as o  # noqa: E402
from paper_2503_08154_b200 import synth  # noqa: E402


def test_algorithmic_bytes_are_two_tensors_plus_half_a_byte_per_element_plus_row_metadata():
    assert bench.algorithmic_bytes(197 * 10, 197, 2) == 2 * 1970 * 2 + 985 + 80
    assert bench.algorithmic_bytes(64 * 197 * 3072, 3072, 2) == 174393856        # one ViT-B/16 GELU launch
    assert bench.algorithmic_bytes(64 * 12 * 197 * 197, 197, 2) == 135334272      # one ViT-B/16 softmax launch


def test_code_flip_count_accepts_flips_at_a_bin_edge_only():
    rows, L, dt = 64, 197, synth.BF16
    x = synth.to_io(synth.softmax_logits(3, ("flips", rows, L), rows, L), dt)
    y, codes, meta = o.softmax_fwd(x, L, dt)
    assert bench.softmax_code_flips(codes, y, codes, x, L, dt) == (0, 0)
    q = bench._unpack4(codes, rows * L).astype(np.int64)
    yw = synth.io_to_f32(y, dt).astype(np.float64).reshape(rows, L)
    mn, mx = yw.min(axis=1, keepdims=True), yw.max(axis=1, keepdims=True)
    t = ((yw - mn) * 15.0 / (mx - mn)).reshape(-1)
    dist = np.abs(t - np.floor(t) - 0.5)

    def repack(qq):
        out = np.zeros((qq.size + 1) // 2, dtype=np.uint8)
        out[: (qq.size + 1) // 2] = qq[0::2]
        out[: qq.size // 2] |= (qq[1::2] << 4).astype(np.uint8)
        return out

    # a code moved to its neighbour where the scaled value sits far from every edge: counted as not at an edge
    far = int(np.argmax(np.where((q > 0) & (q < 15), dist, -1.0)))
    planted = q.copy()
    planted[far] += 1
    assert bench.softmax_code_flips(repack(planted.astype(np.uint8)), y, codes, x, L, dt) == (1, 1)
    # a code off by two levels is never explained by rounding
    planted = q.copy()
    planted[far] += 2 if q[far] <= 13 else -2
    assert bench.softmax_code_flips(repack(planted.astype(np.uint8)), y, codes, x, L, dt) == (1, 1)
    # the element nearest to an edge, moved across it: a flip within reach (if it is within one ulp's reach at all)
    near = int(np.argmin(np.where((q > 0) & (q < 15), dist, 1.0)))
    planted = q.copy()
    planted[near] += 1 if t[near] - np.floor(t[near]) < 0.5 else -1
    flips, outside = bench.softmax_code_flips(repack(planted.astype(np.uint8)), y, codes, x, L, dt)
    assert flips == 1
    if dist[near] <= 1e-5:       # within the slack every flip is granted, whatever the row's scale
        assert outside == 0
