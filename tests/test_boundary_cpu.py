"""The C-ABI library loads without a GPU, exports every symbol the header declares, and its
host-side argument checks work (no kernel is launched here)."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import oracle
from paper_2112_04291_b200 import binding, build, workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def test_every_declared_symbol_is_exported(lib):
    declared = set()
    inc = os.path.join(ROOT, "include")
    for name in sorted(os.listdir(inc)):
        if name.endswith(".h"):
            hdr = re.sub(r"/\*.*?\*/", "", open(os.path.join(inc, name)).read(), flags=re.S)
            declared |= set(re.findall(r"\b(fastsgd_[a-z_]+)\s*\(", hdr))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_version_and_messages(lib):
    assert lib.fastsgd_version() == 1
    for code in (0, -1, -2, -3, -4, -5, -6, -7, -8, -9, 1, 2, 3, 16, 17, 18, 19, 20, 21, 22, 23, 24):
        assert binding.strerror(code) != "unknown code"
    assert binding.strerror(12345) == "unknown code"


def test_bounds_and_workspace_sizes(lib):
    for n in (1, 5, 16384, 16385, 25_557_032, 335_141_888):
        for l in (1, 2, 5):
            p = binding.params(1.1, 128, l, 14)
            G = (n + 16383) // 16384
            b = binding.compress_bound(n, p)
            assert b == 64 + 8 * G + 4 * G * ((16384 * (8 + l + 14) + 31) // 32)
            # the oracle's writer states the same worst case independently
            assert b == oracle.compress_bound(n, oracle.params(1.1, 128, l, 14))
            assert binding.workspace_bytes(n, p) >= 1024 + 16 * G
            assert binding.host_scratch_bytes(n, p) >= 4 * n + b
    assert binding.compress_bound(0, binding.params(1.1)) == 0
    assert binding.compress_bound(10, binding.params(0.9)) == 0


def test_host_side_argument_checks(lib):
    p = binding.params(1.1)
    fake = 1 << 20    # never dereferenced: the checks below fail before any launch
    assert lib.fastsgd_compress(None, 10, C.byref(p), fake, 1 << 20, None) == binding.E_NULL
    assert lib.fastsgd_compress(fake, 10, None, fake, 1 << 20, None) == binding.E_NULL
    assert lib.fastsgd_compress(fake + 4, 10, C.byref(p), fake, 1 << 20, None) == binding.E_ALIGN
    assert lib.fastsgd_compress(fake, 0, C.byref(p), fake, 1 << 20, None) == binding.E_BAD_N
    assert lib.fastsgd_compress(fake, 1 << 31, C.byref(p), fake, 1 << 40, None) == binding.E_BAD_N
    assert lib.fastsgd_compress(fake, 100000, C.byref(p), fake, 64, None) == binding.E_CAPACITY
    assert lib.fastsgd_compress(fake, 10, C.byref(p), fake, 1 << 20, None) == binding.E_NO_WORKSPACE
    for bad in (binding.params(1.0), binding.params(float("nan")), binding.params(1.1, 0), binding.params(1.1, 129),
                binding.params(1.1, 128, 0), binding.params(1.1, 128, 6), binding.params(1.1, 128, 2, 21),
                binding.params(1e10, 128), binding.Params(1.1, 128, 2, 14, 1)):
        assert lib.fastsgd_compress(fake, 10, C.byref(bad), fake, 1 << 20, None) == binding.E_BAD_PARAM
        assert lib.fastsgd_decompress_accumulate(fake, 100, 10, C.byref(bad), fake, None) == binding.E_BAD_PARAM
    # (group sizes below 2^8 have no kernel; the check comes after the workspace check, which fails first without a GPU)
    assert lib.fastsgd_compress(fake, 10, C.byref(binding.params(1.1, 128, 2, 12)), fake, 1 << 20, None) == binding.E_NO_WORKSPACE
    assert lib.fastsgd_decompress_accumulate(fake, 10, 10, C.byref(p), fake, None) == binding.E_TRUNCATED
    assert lib.fastsgd_decompress_accumulate(fake + 8, 100, 10, C.byref(p), fake, None) == binding.E_ALIGN
    assert lib.fastsgd_set_workspace(None, 4096, None) == binding.E_NULL
    assert lib.fastsgd_set_workspace(fake + 16, 4096, None) == binding.E_ALIGN


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libfastsgd_b200.so")
    with pytest.raises(ImportError):
        binding.lib()


def test_workload_generators_are_seeded_and_shaped():
    a = workloads.make("c1", n=50_000)
    b = workloads.make("c1", n=50_000)
    assert np.array_equal(a.grads[0], b.grads[0]) and a.base == b.base
    rc, keys, codes, S = oracle.value_encode(a.grads[0], a.base, a.tau)
    assert rc == 0 and abs(keys.size / 50_000 - 0.01) < 0.002
    w2 = workloads.make("c2", n=200_000, workers=2)
    assert len(w2.grads) == 2 and not np.array_equal(w2.grads[0], w2.grads[1])
    rc, keys, codes, S = oracle.value_encode(w2.grads[0], w2.base, w2.tau)
    assert abs(keys.size / 200_000 - 0.005) < 0.001
    w3 = workloads.make("c3", n=2_000_000)
    nnz = np.count_nonzero(w3.grads[0])
    assert 0.0005 < nnz / 2_000_000 < 0.0015
    rc, keys, codes, S = oracle.value_encode(w3.grads[0], w3.base, w3.tau)
    assert abs(keys.size / nnz - 0.8) < 0.05
    w4 = workloads.make("c4", n=300_000, workers=1, keep=0.001)
    rc, keys, codes, S = oracle.value_encode(w4.grads[0], w4.base, w4.tau)
    assert abs(keys.size / 300_000 - 0.001) < 0.0005
    w5 = workloads.make("c5", n=1 << 16, keep=0.1)
    rc, keys, codes, S = oracle.value_encode(w5.grads[0], w5.base, w5.tau)
    assert abs(keys.size / (1 << 16) - 0.1) < 0.01
