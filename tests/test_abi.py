"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol
the header declares, and its size helpers and status strings behave."""
import ctypes
import os
import re

import pytest

from paper_2503_08154_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "s2a.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(s2a_[a-z0-9_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_size_helpers(lib):
    assert binding.codes_bytes(0) == 0
    assert binding.codes_bytes(1) == 1
    assert binding.codes_bytes(197 * 3) == 296
    assert binding.meta_bytes(197 * 3, 197) == 24
    assert binding.meta_bytes(10, 0) == 0
    n = 64 * 197 * 3072
    assert binding.codes_bytes(n) * 2 == n          # 0.5 byte per element
    assert binding.meta_bytes(n, 3072) == 8 * 64 * 197


def test_relu_argument_checks(lib):
    a = ctypes.c_void_p(0x1000)
    assert binding.mask_bytes(0) == 0 and binding.mask_bytes(1) == 1 and binding.mask_bytes(8) == 1
    assert binding.mask_bytes(9) == 2
    assert lib.s2a_relu_fwd(None, a, a, 8, 0, None) == 1
    assert lib.s2a_relu_fwd(ctypes.c_void_p(0x1008), a, a, 8, 0, None) == 3
    assert lib.s2a_relu_bwd(a, a, a, 8, 9, None) == 4
    assert lib.s2a_relu_bwd(a, a, a, 0, 1, None) == 0


def test_status_strings(lib):
    assert binding.status_string(0) == "S2A_OK"
    for code, word in ((1, "NULL"), (2, "SHAPE"), (3, "ALIGN"), (4, "DTYPE"), (5, "CUDA"), (6, "DEVICE"),
                       (7, "TOO_LARGE"), (8, "OVERLAP")):
        assert word in binding.status_string(code)
    assert "unknown" in binding.status_string(99)


def test_argument_checks_run_before_any_launch(lib):
    # all of these fail on the host, so they are safe without a device
    s2a = lib
    a = ctypes.c_void_p(0x1000)
    assert s2a.s2a_gelu_fwd(None, a, a, a, 8, 4, 0, None) == 1
    assert s2a.s2a_gelu_fwd(a, a, a, a, 8, 0, 0, None) == 2
    assert s2a.s2a_gelu_fwd(a, a, a, a, 9, 4, 0, None) == 2
    assert s2a.s2a_softmax_fwd(ctypes.c_void_p(0x1004), a, a, a, 8, 4, 0, None) == 3
    assert s2a.s2a_softmax_bwd(a, a, a, a, 8, 4, 5, None) == 4
    assert s2a.s2a_gelu_bwd(a, a, a, a, 0, 4, 1, None) == 0


def test_plan_description_is_host_only(lib):
    for kernel in range(4):
        for dt in (0, 1):
            text = binding.s2a_describe_plan(kernel, 64 * 197 * 3072, 3072, dt)
            assert text.startswith("tile") or text.startswith("rowwise")
    with pytest.raises(binding.S2AError):
        binding.s2a_describe_plan(0, 10, 3, 0)


def test_partial_overlap_of_input_and_output_is_rejected(lib):
    # 64 binary32 elements = 256 bytes: an output 128 bytes into the input overlaps it; the
    # same pointer (in place) and a disjoint output pass the argument checks.  n_elems = 0
    # keeps the accepted cases from reaching a launch.
    a, c, m = 0x10000, 0x40000, 0x50000
    for f in (lib.s2a_gelu_fwd, lib.s2a_softmax_fwd, lib.s2a_silu_fwd):
        assert f(a, a + 128, c, m, 64, 8, 0, None) == 8
        assert f(a + 128, a, c, m, 64, 8, 0, None) == 8
    for f in (lib.s2a_gelu_bwd, lib.s2a_softmax_bwd):
        assert f(a, c, m, a + 64, 64, 8, 0, None) == 8
    # bfloat16: 64 elements = 128 bytes, so an output 128 bytes on is disjoint -- checked via the
    # scratch variant, whose missing scratch is reported only after the overlap test passed
    assert lib.s2a_gelu_fwd_tensor_range(a, a + 128, c, m, None, 64, 8, 1, None) == 1
    assert lib.s2a_gelu_fwd_tensor_range(a, a + 64, c, m, None, 64, 8, 1, None) == 8
    assert lib.s2a_gelu_fwd_tensor_range(a, a, c, m, None, 64, 8, 1, None) == 1      # in place is allowed


def _plan_fields(text):
    return dict(kv.split("=") for kv in text.split()[1:])


def test_plans_ignore_the_environment(lib, monkeypatch):
    cases = [(k, rows * L, L, dt) for k in range(6) for dt in (0, 1)
             for rows, L in ((12608, 3072), (151296, 197), (4000, 64), (900, 1025), (131584, 257))]
    before = [binding.s2a_describe_plan(*c) for c in cases]
    for name, value in (("S2A_PATH", "rowwise"), ("S2A_UNIT", "32"), ("S2A_TILE_ROWS", "64"), ("S2A_WARPS", "2"),
                        ("S2A_STAGES", "2"), ("S2A_CTAS_PER_SM", "1"), ("S2A_VARIANT", "generic"), ("S2A_FIXED", "0"),
                        ("S2A_PDL", "0"), ("S2A_SPREAD", "0"), ("S2A_SINGLE_STAGE", "0")):
        monkeypatch.setenv(name, value)
    assert [binding.s2a_describe_plan(*c) for c in cases] == before
    src = open(os.path.join(ROOT, "paper_2503_08154_b200", "csrc", "s2a_tile.cu")).read()
    default_build = re.sub(r"#ifdef S2A_TUNING.*?#else", "", src, flags=re.S)
    assert "getenv" not in default_build


def test_every_plan_gives_each_unit_whole_row_groups(lib):
    """Host-side sweep of the planner: a tile holds a whole number of row groups, and where
    the units of a warp take groups a stride apart, the groups divide evenly among them."""
    lengths = [16, 17, 33, 40, 48, 49, 50, 56, 63, 64, 65, 100, 128, 145, 196, 197, 198, 255, 256, 257, 401, 512,
               577, 785, 1000, 1024, 1025, 1370, 2048, 2049, 3072, 4096, 5120, 8192]
    seen_spread = 0
    for kernel in range(6):
        for dt in (0, 1):
            for L in lengths:
                text = binding.s2a_describe_plan(kernel, 100000 * L, L, dt)
                if not text.startswith("tile"):
                    continue
                f = {k: int(v) for k, v in _plan_fields(text).items() if v.isdigit()}
                G, unit, rows = f["group"], f["unit"], f["rows/tile"]
                assert G >= 1 and rows % G == 0, text
                upw = 32 // unit if unit < 32 else 1
                if f["spread"]:
                    seen_spread += 1
                    assert upw > 1 and (rows // G) % upw == 0, text
                # every unit of the CTA finds a group in every round, or the rounds cover the tile
                n_units = f["warps"] * 32 // unit
                assert n_units >= 1 and (f["warps"] * 32) % unit == 0, text
    assert seen_spread > 0


def test_tiles_whose_codes_start_off_the_16_byte_grid_stay_inside_the_code_tensor(lib):
    """Widths 577 / 1025 may take tiles of 8 or 16 rows, whose code bytes begin anywhere.  The
    data of such a tile must still be whole 16-byte pieces, its rows even (no byte shared with
    another tile), and the aligned span the backward loads for the LAST tile must end inside the
    code tensor: either rows are left for the row path, or the tiles end on the grid."""
    seen = 0
    for L in (577, 1025):
        for dt, esize in ((0, 4), (1, 2)):
            for kernel in (2, 3):
                for n_rows in (16, 40, 48, 72, 163, 1000, 2000, 9000, 97536, 173280):
                    text = binding.s2a_describe_plan(kernel, n_rows * L, L, dt)
                    if not text.startswith("tile"):
                        continue
                    f = {k: int(v) for k, v in _plan_fields(text).items() if v.isdigit()}
                    rows, tiles, tail = f["rows/tile"], f["tiles"], f["tail_rows"]
                    assert tiles * rows + tail == n_rows, text
                    assert rows % 2 == 0 and (rows * L * esize) % 16 == 0, text
                    if f["ragged_codes"]:
                        seen += 1
                        code_bytes = rows * L // 2
                        assert (rows * L) % 2 == 0 and code_bytes >= 32, text
                        end = tiles * code_bytes
                        total = (n_rows * L + 1) // 2
                        assert (end + 15) // 16 * 16 <= total or end % 16 == 0, text
                    else:
                        assert (rows * L // 2) % 16 == 0, text
    assert seen > 0
