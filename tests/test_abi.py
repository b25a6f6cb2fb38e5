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
    for code, word in ((1, "NULL"), (2, "SHAPE"), (3, "ALIGN"), (4, "DTYPE"), (5, "CUDA"), (6, "DEVICE")):
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
