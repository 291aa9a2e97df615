"""Parity on the five benchmark configurations at their full sizes, in the launch configuration
the benchmark times (same entry points, same capacity rule): streams byte-equal to the oracle's,
accumulated dense vector within 1e-6 relative / 1e-12 absolute (and bit-equal)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2112_04291_b200 import binding, workloads

pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-6, 1e-12


def _run(wl, check_workers=None):
    n, W = wl.n, wl.workers
    pg = binding.params(wl.base, wl.tau, wl.flag_bits, wl.group_log2)
    po = oracle.params(wl.base, wl.tau, wl.flag_bits, wl.group_log2)
    binding.ensure_workspace(n, pg)
    cap = (min(binding.compress_bound(n, pg), max(4 * n, 1 << 20)) + 255) & ~255
    dense = torch.zeros(n, dtype=torch.float32, device="cuda")
    odense = np.zeros(n, np.float32)
    out = torch.empty(cap, dtype=torch.uint8, device="cuda")
    kept_total = 0
    for w in range(W):
        g = torch.from_numpy(wl.grads[w]).cuda()
        assert binding.compress(g, pg, out) == 0
        total, d, status = binding.stream_info(out)
        assert status == 0
        assert binding.decompress_accumulate(out, cap, n, pg, dense) == 0
        if check_workers is None or w in check_workers:
            orc, ostream = oracle.compress(wl.grads[w], po)
            assert orc == 0 and total == ostream.size
            assert np.array_equal(out[:total].cpu().numpy(), ostream), f"worker {w}: stream differs"
            assert d == int(np.frombuffer(ostream[24:32].tobytes(), np.uint64)[0])
            assert oracle.decompress_accumulate(ostream, n, po, odense) == 0
            kept_total += d
        del g
    assert binding.decode_status() == 0
    if check_workers is None or len(check_workers) == W:
        got = dense.cpu().numpy()
        assert np.allclose(got, odense, rtol=RTOL, atol=ATOL)
        assert np.array_equal(got, odense)
    return kept_total


def _run_batched(wl):
    """The launch configuration bench.py times: all workers' gradients through one
    fastsgd_compress_batch call, all streams through one fastsgd_decompress_accumulate_batch call."""
    n, W = wl.n, wl.workers
    pg = binding.params(wl.base, wl.tau, wl.flag_bits, wl.group_log2)
    po = oracle.params(wl.base, wl.tau, wl.flag_bits, wl.group_log2)
    binding.ensure_workspace(n, pg)
    cap = (min(binding.compress_bound(n, pg), max(4 * n, 1 << 20)) + 255) & ~255
    grads = [torch.from_numpy(g).cuda() for g in wl.grads]
    outs = [torch.empty(cap, dtype=torch.uint8, device="cuda") for _ in range(W)]
    dense = torch.zeros(n, dtype=torch.float32, device="cuda")
    odense = np.zeros(n, np.float32)
    for rep in range(2):                       # the second launch reuses the workspace as the first left it
        for o in outs:
            o.fill_(0xA5)
        assert binding.compress_batch(grads, pg, outs) == 0
        for w in range(W):
            total, d, status = binding.stream_info(outs[w])
            orc, ostream = oracle.compress(wl.grads[w], po)
            assert status == orc == 0 and total == ostream.size, f"worker {w}"
            assert np.array_equal(outs[w][:total].cpu().numpy(), ostream), f"worker {w}: stream differs (launch {rep})"
            if rep == 0:
                assert oracle.decompress_accumulate(ostream, n, po, odense) == 0
    assert binding.decompress_accumulate_batch(outs, [cap] * W, n, pg, dense) == 0
    assert binding.decode_status() == 0
    got = dense.cpu().numpy()
    assert np.allclose(got, odense, rtol=RTOL, atol=ATOL)
    assert np.array_equal(got, odense)


def _run_batched_checked(wl, check_workers):
    """All W gradients in ONE fastsgd_compress_batch launch and all W streams in ONE
    fastsgd_decompress_accumulate_batch launch (what bench.py times); the streams of `check_workers` are
    compared byte for byte with the oracle's, the dense sum with the oracle's over all W workers."""
    n, W = wl.n, wl.workers
    pg = binding.params(wl.base, wl.tau, wl.flag_bits, wl.group_log2)
    po = oracle.params(wl.base, wl.tau, wl.flag_bits, wl.group_log2)
    binding.ensure_workspace(n, pg)
    cap = (min(binding.compress_bound(n, pg), max(4 * n, 1 << 20)) + 255) & ~255
    grads = [torch.from_numpy(g).cuda() for g in wl.grads]
    outs = [torch.empty(cap, dtype=torch.uint8, device="cuda") for _ in range(W)]
    for o in outs:
        o.fill_(0x3C)
    assert binding.compress_batch(grads, pg, outs) == 0
    dense = torch.zeros(n, dtype=torch.float32, device="cuda")
    assert binding.decompress_accumulate_batch(outs, [cap] * W, n, pg, dense) == 0
    assert binding.decode_status() == 0
    del grads
    odense = np.zeros(n, np.float32)
    for w in range(W):
        total, d, status = binding.stream_info(outs[w])
        orc, ostream = oracle.compress(wl.grads[w], po)
        assert status == orc == 0 and total == ostream.size, f"worker {w}"
        assert d == int(np.frombuffer(ostream[24:32].tobytes(), np.uint64)[0])
        if w in check_workers:
            assert np.array_equal(outs[w][:total].cpu().numpy(), ostream), f"worker {w}: stream differs"
        assert oracle.decompress_accumulate(ostream, n, po, odense) == 0
    got = dense.cpu().numpy()
    assert np.allclose(got, odense, rtol=RTOL, atol=ATOL)
    assert np.array_equal(got, odense)


_C4_GRADS = {}


def _config4_eight_workers(keep):
    """Config 4 with its 8 workers; the gradients are drawn once per test session and shared by the keep ratios."""
    if "grads" not in _C4_GRADS:
        _C4_GRADS["grads"] = workloads.make("c4", workers=8, keep=1e-3).grads
    grads = _C4_GRADS["grads"]
    n = grads[0].size
    base = workloads.base_for_keep(grads[0], int(round(keep * n)))
    return workloads.Workload("c4", n, 8, float(keep), grads, base)


@pytest.mark.parametrize("keep", [1e-4, 1e-2])
def test_config4_eight_workers_one_launch_as_benchmarked(keep):
    # the launch bench.py times for config 4: 8 gradients of 335 M entries in one k_compress launch, 8 streams in one
    # decoder launch; three streams compared byte for byte, the dense sum over all eight
    wl = _config4_eight_workers(keep)
    assert wl.n == 335_141_888 and wl.workers == 8
    _run_batched_checked(wl, check_workers=(0, 3, 7))
    if keep == 1e-2:
        _C4_GRADS.clear()


def test_config1_full():
    wl = workloads.make("c1")
    kept = _run(wl)
    assert abs(kept / wl.n - 0.01) < 0.002


def test_config2_full_four_workers():
    wl = workloads.make("c2")
    assert wl.n == 25_557_032 and wl.workers == 4
    kept = _run(wl)
    assert abs(kept / (4 * wl.n) - 0.005) < 0.002


def test_config2_batched_as_benchmarked():
    _run_batched(workloads.make("c2"))


@pytest.mark.parametrize("keep", [1e-3, 1e-2])
def test_config4_batched_as_benchmarked(keep):
    # three of the eight workers in one launch (an odd count: the two teams of blocks get unequal shares)
    _run_batched(workloads.make("c4", workers=3, keep=keep))


def test_config3_full_clustered_sparse():
    wl = workloads.make("c3")
    assert wl.n == 50_000_000
    kept = _run(wl)
    assert 0.6 < kept / np.count_nonzero(wl.grads[0]) < 0.95


@pytest.mark.parametrize("keep", [1e-4, 1e-3, 1e-2])
def test_config4_full(keep):
    # two of the eight workers at each keep ratio (generation and the oracle dominate the run time)
    wl = workloads.make("c4", workers=2, keep=keep)
    assert wl.n == 335_141_888
    kept = _run(wl)
    assert 0.3 * keep < kept / (2 * wl.n) < 3 * keep


@pytest.mark.parametrize("log2n", [10, 12, 14, 16, 18, 20, 22, 24, 26])
@pytest.mark.parametrize("keep", [1e-4, 1e-3, 1e-2, 1e-1])
def test_config5_sweep(log2n, keep):
    wl = workloads.make("c5", n=1 << log2n, keep=keep)
    _run(wl)


@pytest.mark.parametrize("keep", [1e-4, 1e-3, 1e-2, 1e-1])
def test_config5_sweep_2_28(keep):
    # n = 2^28: the kernel variant for gradients with more than 8192 tiles, at all four keep ratios
    # (10 %: every tile of the launch goes through the dense-tile packer)
    _run(workloads.make("c5", n=1 << 28, keep=keep))


@pytest.mark.parametrize("keep", [1e-3, 1e-1])
def test_config5_sweep_largest(keep):
    wl = workloads.make("c5", n=1 << 30, keep=keep)
    _run(wl)


def test_config2_sparse_adam_update_as_benchmarked():
    # config 2's four streams, the model update bench.py times: theta, m, v bit-equal to the oracle's
    wl = workloads.make("c2")
    n, W = wl.n, wl.workers
    pg = binding.params(wl.base, wl.tau, wl.flag_bits, wl.group_log2)
    po = oracle.params(wl.base, wl.tau, wl.flag_bits, wl.group_log2)
    binding.ensure_workspace(n, pg)
    cap = (min(binding.compress_bound(n, pg), max(4 * n, 1 << 20)) + 255) & ~255
    outs = [torch.empty(cap, dtype=torch.uint8, device="cuda") for _ in range(W)]
    assert binding.compress_batch([torch.from_numpy(g).cuda() for g in wl.grads], pg, outs) == 0
    streams = []
    for o in outs:
        total, d, status = binding.stream_info(o)
        assert status == 0
        streams.append(o[:total].cpu().numpy())
    rng = np.random.default_rng(9)
    theta0 = rng.standard_normal(n).astype(np.float32)
    ot, om, ov = theta0.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32)
    lr, b1, b2, eps = 1e-3, 0.9, 0.999, 1e-8
    assert oracle.sparse_adam_update(streams, n, po, lr, b1, b2, eps, ot, om, ov) == 0
    theta = torch.from_numpy(theta0).cuda()
    m = torch.zeros(n, dtype=torch.float32, device="cuda"); v = torch.zeros_like(m); scratch = torch.zeros_like(m)
    assert binding.sparse_adam_update_batch(outs, [cap] * W, n, pg, binding.Adam(lr, b1, b2, eps), scratch, theta, m, v) == 0
    assert binding.decode_status() == 0 and not bool(scratch.any().item())
    assert np.array_equal(theta.cpu().numpy(), ot) and np.array_equal(m.cpu().numpy(), om) and np.array_equal(v.cpu().numpy(), ov)
    assert 0 < int((ot != theta0).sum()) <= 4 * n // 100
    # the same step on the packed state (theta, m, v, g per coordinate), as bench.py's packed_state_ms times it
    host = np.zeros((n, 4), np.float32)
    host[:, 0] = theta0
    state = torch.from_numpy(host.reshape(-1)).cuda()
    assert binding.sparse_adam_update_packed_batch(outs, [cap] * W, n, pg, binding.Adam(lr, b1, b2, eps), state) == 0
    got = state.cpu().numpy().reshape(n, 4)
    assert binding.decode_status() == 0 and not got[:, 3].any()
    assert np.array_equal(got[:, 0], ot) and np.array_equal(got[:, 1], om) and np.array_equal(got[:, 2], ov)


def test_config3_key_value_input_as_benchmarked():
    # config 3 is sparse before it is compressed: its non-zero entries as key-value pairs give the dense call's stream
    wl = workloads.make("c3")
    n = wl.n
    v = wl.grads[0]
    pg = binding.params(wl.base, wl.tau, wl.flag_bits, wl.group_log2)
    po = oracle.params(wl.base, wl.tau, wl.flag_bits, wl.group_log2)
    binding.ensure_workspace(n, pg)
    keys = np.flatnonzero(v)
    assert 0 < keys.size < n // 500
    cap = (min(binding.compress_bound(n, pg), max(4 * n, 1 << 20)) + 255) & ~255
    out = torch.full((cap,), 0x5A, dtype=torch.uint8, device="cuda")
    dk = torch.from_numpy(keys.astype(np.uint32).view(np.int32)).cuda()
    dv = torch.from_numpy(v[keys]).cuda()
    orc, ostream = oracle.compress(v, po)
    for rep in range(2):
        assert binding.compress_kv(dk, dv, n, pg, out) == 0
        total, d, status = binding.stream_info(out)
        assert status == orc == 0 and total == ostream.size
        assert np.array_equal(out[:total].cpu().numpy(), ostream)


def test_key_value_input_scattered_pairs_bert_size():
    # pairs scattered uniformly over n = 335 M (about 16 per chunk, every chunk touched): the stream of the dense call
    n = 335_141_888
    rng = np.random.default_rng(31)
    keys = np.unique(rng.integers(0, n, 340_000)).astype(np.uint64)
    vals = rng.laplace(0.0, 1e-2, keys.size).astype(np.float32)
    v = np.zeros(n, np.float32)
    v[keys.astype(np.int64)] = vals
    b = workloads.base_for_keep(v, int(0.8 * keys.size))
    pg, po = binding.params(b), oracle.params(b)
    binding.ensure_workspace(n, pg)
    cap = (min(binding.compress_bound(n, pg), max(4 * n, 1 << 20)) + 255) & ~255
    out = torch.full((cap,), 0x5A, dtype=torch.uint8, device="cuda")
    dk = torch.from_numpy(keys.astype(np.uint32).view(np.int32)).cuda()
    dv = torch.from_numpy(vals).cuda()
    orc, ostream = oracle.compress(v, po)
    for rep in range(2):
        assert binding.compress_kv(dk, dv, n, pg, out) == 0
        total, d, status = binding.stream_info(out)
        assert status == orc == 0 and total == ostream.size
        assert np.array_equal(out[:total].cpu().numpy(), ostream)
