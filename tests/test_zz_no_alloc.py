"""fastsgd_abs_sum_noalloc: the sum for callers that cannot provide scratch memory.

Some users of the library only ever receive an input and an output pointer: they may not call
cudaMalloc (device-wide synchronisation, failure under memory pressure) and own no allocator,
so they cannot register a workspace either.  For them the entry point keeps its scratch in a
fixed array inside the library.  This test calls it through the C ABI, twice in a row with
different inputs, and checks each result against the regular entry point (which uses the
caller's workspace) and against the CPU oracle's tree sum: the sums must be the same fp64 bits,
as everywhere else in this suite.  The largest accepted size (every partial of the built-in
array in use) and a single-chunk input are covered too.

Collected last (file name) so that a run that stops at the first failure has run everything else.
It does not depend on any other test: it passes alone in a fresh process too.
"""
import ctypes as C

import numpy as np
import pytest

import oracle
from paper_2112_04291_b200 import binding

pytestmark = pytest.mark.gpu


def _sum_both_ways(v):
    import torch
    from paper_2112_04291_b200 import binding
    g = torch.from_numpy(v).cuda()
    n = g.numel()
    lib = binding.lib()
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    # the new entry point first: it must work before any workspace was ever registered
    out_new = torch.full((1,), -1.0, dtype=torch.float64, device="cuda")
    rc = lib.fastsgd_abs_sum_noalloc(C.c_void_p(g.data_ptr()), C.c_uint64(n), C.c_void_p(out_new.data_ptr()), stream)
    assert rc == 0, binding.strerror(rc)
    # the existing entry point, with a caller-provided workspace
    binding.ensure_workspace(n, binding.params(1.1))
    out_old = torch.full((1,), -2.0, dtype=torch.float64, device="cuda")
    rc = lib.fastsgd_abs_sum(C.c_void_p(g.data_ptr()), C.c_uint64(n), C.c_void_p(out_old.data_ptr()), stream)
    assert rc == 0, binding.strerror(rc)
    torch.cuda.synchronize()
    return out_new.item(), out_old.item()


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    rng = np.random.default_rng(2024)
    # second call: smaller and different, so anything left over from the first would show
    for n in (3_000_017, 70_001):
        v = (rng.standard_normal(n) * 10.0 ** rng.integers(-6, 3, n)).astype(np.float32)
        new, old = _sum_both_ways(v)
        assert new == old                       # same fp64 value, bit for bit
        assert new == oracle.abs_sum(v)         # ... and the oracle's tree sum, directly
        assert abs(new - float(np.abs(v).astype(np.float64).sum())) <= 1e-9 * new


def test_largest_accepted_size_and_a_single_chunk():
    # n = 2^28 uses all 16384 partials of the built-in array; n <= 2^14 is one chunk (a grid of one block)
    rng = np.random.default_rng(77)
    for n in (binding.NOALLOC_MAX_N, 16_384, 9_001):
        v = rng.standard_normal(n, dtype=np.float32)
        v[::7] *= np.float32(1e-4)
        new, old = _sum_both_ways(v)
        assert new == old == oracle.abs_sum(v)
        del v


def test_sizes_beyond_the_built_in_scratch_are_refused():
    import torch
    from paper_2112_04291_b200 import binding
    lib = binding.lib()
    g = torch.zeros(16, dtype=torch.float32, device="cuda")
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    too_many = binding.NOALLOC_MAX_N + 1        # checked before anything is read or launched
    rc = lib.fastsgd_abs_sum_noalloc(C.c_void_p(g.data_ptr()), C.c_uint64(too_many), C.c_void_p(out.data_ptr()), stream)
    assert rc == binding.E_TOO_LARGE
    assert "2^28" in binding.strerror(rc)
    assert lib.fastsgd_abs_sum_noalloc(None, C.c_uint64(16), C.c_void_p(out.data_ptr()), stream) == binding.E_NULL
    assert lib.fastsgd_abs_sum_noalloc(C.c_void_p(g.data_ptr() + 4), C.c_uint64(8), C.c_void_p(out.data_ptr()), stream) == binding.E_ALIGN
    # a refused call leaves nothing behind: the next accepted call on the same stream is exact
    v = np.linspace(-3.0, 5.0, 40_003, dtype=np.float32)
    gv = torch.from_numpy(v).cuda()
    rc = lib.fastsgd_abs_sum_noalloc(C.c_void_p(gv.data_ptr()), C.c_uint64(v.size), C.c_void_p(out.data_ptr()), stream)
    assert rc == 0
    torch.cuda.synchronize()
    assert out.item() == oracle.abs_sum(v)
