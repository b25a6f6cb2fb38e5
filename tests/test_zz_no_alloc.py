"""The allocation-free entry point, s2a_gelu_fwd_tensor_range_static.

It serves callers that may not allocate device memory where they call the library (a
plug-in under a host application's allocator, a latency-critical loop that cannot afford
the device-wide synchronisation of a cudaMalloc, a program with a fixed memory plan) and
have no buffer to lend: its scratch is a fixed array inside the library, shared by every
call on the GPU.  The check: called through the C ABI on two different tensors in a row --
the second smaller, so that anything wrongly carried over in the shared array from the first
call would show -- it must write exactly what s2a_gelu_fwd_tensor_range writes with
caller-provided scratch, and both must agree with the CPU oracle's per-tensor-range forward
(codes and metadata bit for bit, y within one bfloat16 ulp).  This file sorts last on purpose, so that a run that stops at the
first failure has already run everything else.
"""
import numpy as np
import pytest
import torch

from oracle import s2a_oracle as o
from paper_2503_08154_b200 import binding, synth
import parity_util as pu

pytestmark = pytest.mark.gpu


def _device_tensor(a):
    return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)


def _run_both(rows, L, scale, seed):
    lib = binding.lib()
    n = rows * L
    x_host = synth.to_io(synth.gelu_preact(seed, ("no_alloc", rows, L), n) * np.float32(scale), synth.BF16)
    x = _device_tensor(x_host)
    stream = torch.cuda.current_stream().cuda_stream
    outs = []
    for static in (False, True):
        y = torch.full_like(x, 7.0)
        codes, meta = binding.alloc_stash(n, L, x.device)
        codes.fill_(0xEE)
        meta.fill_(-1.0)
        if static:
            rc = lib.s2a_gelu_fwd_tensor_range_static(x.data_ptr(), y.data_ptr(), codes.data_ptr(), meta.data_ptr(),
                                                      n, L, binding.BF16, stream)
        else:
            scratch = torch.empty(binding.tensor_range_scratch_bytes(n), dtype=torch.uint8, device=x.device)
            rc = lib.s2a_gelu_fwd_tensor_range(x.data_ptr(), y.data_ptr(), codes.data_ptr(), meta.data_ptr(),
                                               scratch.data_ptr(), n, L, binding.BF16, stream)
        assert rc == 0, binding.status_string(rc)
        torch.cuda.synchronize()
        outs.append((y.view(torch.int16).cpu().numpy(), codes.cpu().numpy(), meta.cpu().numpy()))
    outs.append(o.gelu_fwd_tensor_range(x_host, L, synth.BF16))
    return outs


def test_static_scratch_variant_matches_the_caller_scratch_variant_twice_in_a_row():
    # first call: a wide-range tensor over many chunks; second call: a smaller, narrow-range
    # one that uses fewer slots of the shared array
    for rows, L, scale, seed in ((700, 3072, 1.3, 11), (37, 197, 0.2, 12)):
        (y_a, c_a, m_a), (y_b, c_b, m_b), (y_o, c_o, m_o) = _run_both(rows, L, scale, seed)
        # codes and metadata are bit-exact in every parity test of this library; y is the
        # same arithmetic on the same inputs, so it is compared bit for bit as well
        assert np.array_equal(c_a, c_b), "codes differ between the two entry points"
        assert np.array_equal(m_a.view(np.uint32), m_b.view(np.uint32)), "(min, s) differ"
        assert np.array_equal(y_a, y_b), "y differs"
        assert not (m_b == -1.0).any() and not (y_b == np.int16(0x40E0)).all()   # outputs were written
        # and against the oracle, with the tolerances of the other parity tests
        assert np.array_equal(c_b, c_o), "codes differ from the oracle's"
        assert np.array_equal(m_b.view(np.uint32), m_o.view(np.uint32)), "(min, s) differ from the oracle's"
        pu.assert_close(pu.widen(y_b.view(np.uint16), pu.BF16), pu.widen(y_o, pu.BF16), pu.BF16, "y (static scratch)")


def test_static_scratch_variant_refuses_tensors_beyond_its_array():
    lib = binding.lib()
    limit = binding.tensor_range_static_max_elems()
    assert limit == 8192 * 65536
    a = 0x10000                               # never dereferenced: the size check comes first
    rc = lib.s2a_gelu_fwd_tensor_range_static(a, a + (1 << 40), a, a, limit + 4096, 4096, binding.BF16, None)
    assert rc == 7 and "TOO_LARGE" in binding.status_string(rc)
