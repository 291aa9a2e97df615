"""GPU-vs-oracle parity through the C-ABI: sum bit-equal, stream byte-equal, kept keys and
codes equal, decoded and accumulated values within 1e-6 relative / 1e-12 absolute (they are
expected to be bit-equal, which is asserted too).  Sizes span several tiles and ragged tails."""
import numpy as np
import pytest

import oracle
from paper_2112_04291_b200 import binding, workloads

pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-6, 1e-12


def _params(b, tau=128, l=2):
    return binding.params(b, tau, l, 14), oracle.params(b, tau, l, 14)


def _check_roundtrip(v, b, tau=128, l=2, workers_dense0=None):
    import gpu_util as G
    v = np.ascontiguousarray(v, np.float32)
    n = v.size
    pg, po = _params(b, tau, l)
    orc, ostream = oracle.compress(v, po)
    rc, status, gstream, intact = G.gpu_compress(v, pg, fill=0xEE)
    assert rc == 0 and intact
    assert status == orc
    # header (incl. the fp64 sum) and every byte of the stream
    assert gstream.size == ostream.size, (gstream.size, ostream.size)
    assert np.array_equal(gstream[:64], ostream[:64]), "header differs"
    assert np.array_equal(gstream, ostream), "stream differs"
    if orc != 0:
        return ostream
    # kept keys and integer codes
    rc1, keys, codes, S = oracle.parse(gstream, n, po)
    rc2, okeys, ocodes, oS = oracle.value_encode(v, b, tau)
    assert rc1 == 0 and np.array_equal(keys, okeys) and np.array_equal(codes, ocodes) and S == oS
    assert np.all((np.abs(codes) >= 1) & (np.abs(codes) <= tau))
    # decode + accumulate
    dense0 = workers_dense0 if workers_dense0 is not None else np.zeros(n, np.float32)
    odense = dense0.copy()
    assert oracle.decompress_accumulate(ostream, n, po, odense) == 0
    rc, st, gdense, intact = G.gpu_decompress(gstream, n, pg, dense0)
    assert rc == 0 and st == 0 and intact
    assert np.allclose(gdense, odense, rtol=RTOL, atol=ATOL)
    assert np.array_equal(gdense, odense)
    return ostream


@pytest.mark.parametrize("n", [1, 2, 3, 4, 5, 15, 16, 17, 127, 128, 129, 1023, 1024, 1025, 4097,
                               16383, 16384, 16385, 32768 + 5, 49152, 100_003, 1_000_000])
def test_sizes_and_ragged_tails(n):
    rng = np.random.default_rng(n)
    v = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    b = workloads.base_for_keep(v, max(1, n // 20))
    _check_roundtrip(v, b)


@pytest.mark.parametrize("l", [1, 2, 3, 4, 5])
@pytest.mark.parametrize("keep", [0.001, 0.05, 0.5])
def test_flag_sizes_and_keep_ratios(l, keep):
    n = 70_000
    rng = np.random.default_rng(l * 100 + int(keep * 1000))
    v = (rng.standard_t(3, n) * 1e-3).astype(np.float32)
    b = workloads.base_for_keep(v, int(keep * n))
    _check_roundtrip(v, b, l=l)


@pytest.mark.parametrize("tau", [1, 7, 64, 100, 128])
def test_thresholds(tau):
    n = 40_000
    rng = np.random.default_rng(tau)
    v = rng.standard_normal(n).astype(np.float32)
    b = workloads.base_for_keep(v, n // 50, tau=tau)
    _check_roundtrip(v, b, tau=tau)


def test_all_kept_dense_tiles():
    # b^tau huge: every nonzero entry survives; blobs reach their widest form
    n = 3 * 16384 + 77
    rng = np.random.default_rng(5)
    v = rng.standard_normal(n).astype(np.float32)
    _check_roundtrip(v, 2.0, tau=128, l=2)
    _check_roundtrip(v, 2.0, tau=128, l=5)


def test_degenerate_inputs():
    n = 40_000
    z = np.zeros(n, np.float32)
    _check_roundtrip(z, 1.1)                                   # all zero: d = 0
    one = z.copy(); one[12345] = -3.0
    _check_roundtrip(one, 1.1)                                 # single nonzero: L = 0 raised to 1
    ends = z.copy(); ends[0] = 1.0; ends[n - 1] = -1.0
    _check_roundtrip(ends, 1.1)                                # keys 0 and n-1
    neg0 = z.copy(); neg0[::7] = -0.0; neg0[5] = 1e-3
    _check_roundtrip(neg0, 1.1)
    rng = np.random.default_rng(8)
    den = (rng.standard_normal(n) * 1e-41).astype(np.float32)  # denormals, no flush to zero
    assert np.any(den != 0) and np.all(np.abs(den) < 1.2e-38)
    _check_roundtrip(den, 1.05)
    mixed = den.copy(); mixed[::3] *= np.float32(1e20)
    _check_roundtrip(mixed, 1.3)
    # none kept: tau = 1 and b barely above 1 put the threshold above every entry
    flat = np.ones(n, np.float32)
    s = _check_roundtrip(flat, 1.0001, tau=1)
    assert int(np.frombuffer(s[24:32].tobytes(), np.uint64)[0]) == 0
    # values exactly on boundaries: powers of two with b = 2
    pw = (2.0 ** -rng.integers(0, 30, n)).astype(np.float32)
    _check_roundtrip(pw, 2.0, tau=40)


def test_nonfinite_and_capacity():
    import gpu_util as G
    n = 50_000
    rng = np.random.default_rng(9)
    v = rng.standard_normal(n).astype(np.float32)
    for bad in (np.inf, -np.inf, np.nan):
        w = v.copy(); w[31337] = bad
        s = _check_roundtrip(w, 1.1)
        assert s.size == 64
    pg, po = _params(1.2)
    orc, full = oracle.compress(v, po)
    assert orc == 0
    for cap in (full.size - 4, 64 + 8 * 4 + 16, full.size):
        orc, ostream = oracle.compress(v, po, cap=cap)
        rc, status, gstream, intact = G.gpu_compress(v, pg, cap=cap, fill=0x11)
        assert rc == 0 and intact and status == orc
        assert np.array_equal(gstream, ostream)
    rc, status, gstream, intact = G.gpu_compress(v, pg, cap=64)
    assert rc == binding.E_CAPACITY and intact


def test_sum_entry_point_bit_equal():
    import torch
    import gpu_util as G
    for n in (1, 5, 1000, 16384, 16385, 123_457, 3_000_001):
        rng = np.random.default_rng(n)
        v = (rng.standard_normal(n) * 10.0 ** rng.integers(-6, 3, n)).astype(np.float32)
        g = G.to_dev(v)
        binding.ensure_workspace(n, binding.params(1.1))
        out = torch.zeros(1, dtype=torch.float64, device=g.device)
        assert binding.abs_sum(g, out) == 0
        torch.cuda.synchronize()
        assert out.item() == oracle.abs_sum(v)


def test_workers_accumulate_in_call_order():
    import gpu_util as G
    n = 200_000
    W = 4
    pg = po = None
    rng = np.random.default_rng(3)
    dense_o = rng.standard_normal(n).astype(np.float32)
    dense_g = dense_o.copy()
    for w in range(W):
        v = workloads.student_t_layers(n, seed=w, blocks=9)
        b = workloads.base_for_keep(v, n // 100)
        pg, po = _params(b)
        orc, ostream = oracle.compress(v, po)
        rc, status, gstream, intact = G.gpu_compress(v, pg)
        assert np.array_equal(gstream, ostream)
        assert oracle.decompress_accumulate(ostream, n, po, dense_o) == 0
        rc, st, dense_g, intact = G.gpu_decompress(gstream, n, pg, dense_g)
        assert rc == 0 and st == 0 and intact
    assert np.allclose(dense_g, dense_o, rtol=RTOL, atol=ATOL)
    assert np.array_equal(dense_g, dense_o)


def test_repeatable():
    import gpu_util as G
    n = 300_000
    v = workloads.normal_outliers(n, seed=4)
    pg, po = _params(workloads.base_for_keep(v, n // 10))
    first = None
    for _ in range(10):
        rc, status, s, intact = G.gpu_compress(v, pg)
        assert rc == 0 and status == 0 and intact
        first = s if first is None else first
        assert np.array_equal(s, first)


def _damage(stream, pos, value, width=4):
    s = stream.copy()
    s[pos:pos + width] = np.frombuffer(int(value).to_bytes(width, "little"), np.uint8)
    return s


@pytest.mark.parametrize("blocks", [1, 7, 37, 148, 211])
def test_same_bytes_whatever_the_grid(blocks):
    # the fixed sum tree and the order-preserving offsets make the stream a function of the input alone: one gradient,
    # three gradients in one launch and key-value input, each with the launch capped at `blocks` thread blocks
    import torch
    import gpu_util as G
    n = 2_000_003
    host = [workloads.student_t_layers(n, seed=70 + w, blocks=5) for w in range(3)]
    b = workloads.base_for_keep(host[0], n // 150)
    pg, po = _params(b)
    binding.ensure_workspace(n, pg)
    want = [oracle.compress(v, po)[1] for v in host]
    grads = [torch.from_numpy(v).cuda() for v in host]
    cap = binding.compress_bound(n, pg)
    outs = [torch.zeros(cap, dtype=torch.uint8, device="cuda") for _ in range(3)]
    keys = np.flatnonzero(np.abs(host[0]) > 1e-3)
    dk = torch.from_numpy(keys.astype(np.uint32).view(np.int32)).cuda()
    dv = torch.from_numpy(host[0][keys]).cuda()
    sparse = np.zeros(n, np.float32); sparse[keys] = host[0][keys]
    want_kv = oracle.compress(sparse, po)[1]
    try:
        binding.debug_set_grid(blocks)
        assert binding.compress(grads[0], pg, outs[0]) == 0
        total, d, status = binding.stream_info(outs[0])
        assert status == 0 and np.array_equal(outs[0][:total].cpu().numpy(), want[0])
        assert binding.compress_batch(grads, pg, outs) == 0
        for w in range(3):
            total, d, status = binding.stream_info(outs[w])
            assert status == 0 and np.array_equal(outs[w][:total].cpu().numpy(), want[w]), w
        assert binding.compress_kv(dk, dv, n, pg, outs[1]) == 0
        total, d, status = binding.stream_info(outs[1])
        assert status == 0 and np.array_equal(outs[1][:total].cpu().numpy(), want_kv)
    finally:
        binding.debug_set_grid(0)


def test_damaged_streams_report_the_oracles_status_and_stay_in_bounds():
    import gpu_util as G
    n = 5 * 16384 + 100
    rng = np.random.default_rng(21)
    v = rng.standard_normal(n).astype(np.float32)
    b = 1.1            # threshold ~0.4: most entries survive, every group is non-empty
    pg, po = _params(b)
    orc, st0 = oracle.compress(v, po)
    assert orc == 0
    G_ = (n + 16383) // 16384
    cases = [
        _damage(st0, 0, 0x12345678), _damage(st0, 4, 7), _damage(st0, 8, 2), _damage(st0, 16, n + 1, 8),
        _damage(st0, 12, 127), _damage(st0, 56, 3, 1), _damage(st0, 60, G_ + 1), _damage(st0, 32, st0.size + 4, 8),
        _damage(st0, 32, 60, 8),
    ]
    a0 = int.from_bytes(st0[64:68].tobytes(), "little")
    cases.append(_damage(st0, 64, (a0 & 0xFF000000) | 16385))            # count > T
    cases.append(_damage(st0, 64, (a0 & 0xFFFFFF) | (15 << 24)))          # M > group_log2
    cases.append(_damage(st0, 64, (a0 & 0xFFFFFF)))                       # M = 0
    off1 = int.from_bytes(st0[76:80].tobytes(), "little")
    cases.append(_damage(st0, 76, off1 + 1))
    cases.append(_damage(st0, 76, off1 - 1))
    cases.append(_damage(st0, 68, 5))                                     # first offset inside the header
    cases.append(_damage(st0, 64 + 8 * 3, 0))                             # non-empty group marked empty
    last = G_ - 1
    offl = int.from_bytes(st0[64 + 8 * last + 4:64 + 8 * last + 8].tobytes(), "little")
    cnt = int.from_bytes(st0[64 + 8 * last:64 + 8 * last + 4].tobytes(), "little") & 0xFFFFFF
    s2 = st0.copy(); s2[4 * offl + cnt:] = 0xFF                           # last group: widest flags, max deltas
    cases.append(s2)
    s3 = st0.copy(); s3[4 * off1] = 0x7F | 0x80                           # code byte L = 128 is fine for tau = 128
    cases.append(s3)
    for i, s in enumerate(cases):
        expect = oracle.decompress_accumulate(s, n, po, np.zeros(n, np.float32))
        rc, st, dense, intact = G.gpu_decompress(s, n, pg)
        assert rc == 0 and intact, i
        assert st == expect, (i, st, expect)
    # BAD_CODE needs tau < 128
    pg2, po2 = _params(2.0, tau=20)
    orc, st1 = oracle.compress(v, po2)
    o1 = int.from_bytes(st1[68:72].tobytes(), "little")
    s4 = st1.copy(); s4[4 * o1 + 2] = 90
    expect = oracle.decompress_accumulate(s4, n, po2, np.zeros(n, np.float32))
    rc, st, dense, intact = G.gpu_decompress(s4, n, pg2)
    assert expect == oracle.DEC_BAD_CODE and st == expect and intact
    # truncated buffer
    expect = oracle.decompress_accumulate(st0, n, po, np.zeros(n, np.float32), nbytes=st0.size - 8)
    rc, st, dense, intact = G.gpu_decompress(st0, n, pg, nbytes=st0.size - 8)
    assert st == expect == oracle.DEC_TRUNCATED and intact and not dense.any()
    # and a clean stream still decodes after all that (the status word was cleared)
    rc, st, dense, intact = G.gpu_decompress(st0, n, pg)
    assert rc == 0 and st == 0


def test_host_buffer_calls():
    import torch
    n = 150_000
    v = workloads.normal(n, seed=2)
    b = workloads.base_for_keep(v, n // 100)
    pg, po = _params(b)
    binding.ensure_workspace(n, pg)
    scratch = torch.empty(binding.host_scratch_bytes(n, pg), dtype=torch.uint8, device="cuda")
    out = torch.zeros(binding.compress_bound(n, pg), dtype=torch.uint8).pin_memory()
    gh = torch.from_numpy(v).pin_memory()
    rc, produced, status = binding.compress_host(gh, pg, out, scratch)
    orc, ostream = oracle.compress(v, po)
    assert rc == 0 and status == 0 and produced == ostream.size
    assert np.array_equal(out[:produced].numpy(), ostream)
    dense = torch.zeros(n, dtype=torch.float32).pin_memory()
    rc, st = binding.decompress_accumulate_host([out, out], [produced, produced], n, pg, dense, scratch)
    odense = np.zeros(n, np.float32)
    oracle.decompress_accumulate(ostream, n, po, odense)
    oracle.decompress_accumulate(ostream, n, po, odense)
    assert rc == 0 and st == 0 and np.array_equal(dense.numpy(), odense)


@pytest.mark.parametrize("nstreams", [1, 3, 8, 10])
def test_batched_decode_equals_one_call_per_stream(nstreams):
    # several workers' streams in one launch: same result, bit for bit, as sequential calls and as
    # the oracle applied in the same order; the streams share many keys (same layer layout) and two
    # of them are identical, so the per-group ordering matters
    import torch
    import gpu_util as G
    n = 6 * 16384 + 321
    rng = np.random.default_rng(nstreams)
    dense0 = rng.standard_normal(n).astype(np.float32)
    odense = dense0.copy()
    streams, sizes, pg, po = [], [], None, None
    base = None
    for w in range(nstreams):
        v = workloads.student_t_layers(n, seed=min(w, nstreams - 2) if nstreams > 1 else 0, blocks=5, lo=1e-3, hi=1e-1)
        if base is None:
            base = workloads.base_for_keep(v, n // 30)
            pg, po = _params(base)
        orc, ostream = oracle.compress(v, po)
        rc, status, gstream, intact = G.gpu_compress(v, pg)
        assert rc == 0 and status == 0 and np.array_equal(gstream, ostream)
        assert oracle.decompress_accumulate(ostream, n, po, odense) == 0
        pad = (-gstream.size) % 16
        streams.append(G.to_dev(np.concatenate([gstream, np.zeros(pad + 16, np.uint8)])))
        sizes.append(gstream.size)
    binding.ensure_workspace(n, pg)
    buf = G.Guarded(4 * n)
    dense = buf.view.view(torch.float32)
    dense.copy_(torch.from_numpy(dense0))
    assert binding.decompress_accumulate_batch(streams, sizes, n, pg, dense) == 0
    assert binding.decode_status() == 0 and buf.intact()
    got = dense.cpu().numpy()
    assert np.allclose(got, odense, rtol=RTOL, atol=ATOL) and np.array_equal(got, odense)
    seq = torch.from_numpy(dense0).cuda()
    for s, b in zip(streams, sizes):
        assert binding.decompress_accumulate(s, b, n, pg, seq) == 0
    assert np.array_equal(seq.cpu().numpy(), got)


@pytest.mark.parametrize("ngrads", [2, 4, 9])
def test_batched_compress_equals_one_call_per_gradient(ngrads):
    # several workers' gradients in one launch: every stream byte-equal to the oracle's (hence to
    # what one call per gradient gives), including a tile-ragged length and an all-zero gradient
    import torch
    import gpu_util as G
    n = 7 * 16384 + 4097
    grads = [workloads.student_t_layers(n, seed=w, blocks=6, lo=1e-3, hi=1e-1) for w in range(ngrads)]
    grads[1] = np.zeros(n, np.float32)
    base = workloads.base_for_keep(grads[0], n // 40)
    pg, po = _params(base)
    binding.ensure_workspace(n, pg)
    cap = binding.compress_bound(n, pg)
    dg = [G.to_dev(v) for v in grads]
    bufs = [G.Guarded(cap, fill=0x5A) for _ in range(ngrads)]
    assert binding.compress_batch(dg, pg, [b.view for b in bufs]) == 0
    for w in range(ngrads):
        total, d, status = binding.stream_info(bufs[w].view)
        orc, ostream = oracle.compress(grads[w], po)
        assert status == orc == 0 and total == ostream.size and bufs[w].intact()
        assert np.array_equal(bufs[w].view[:total].cpu().numpy(), ostream), f"gradient {w}"
    # and a second launch right after reuses the workspace cleanly
    assert binding.compress_batch(dg[::-1], pg, [b.view for b in bufs]) == 0
    for w in range(ngrads):
        total, d, status = binding.stream_info(bufs[w].view)
        orc, ostream = oracle.compress(grads[ngrads - 1 - w], po)
        assert status == 0 and np.array_equal(bufs[w].view[:total].cpu().numpy(), ostream)


@pytest.mark.parametrize("ngrads", [2, 3, 5, 8])
def test_batched_compress_with_two_teams_of_blocks(ngrads):
    # enough tiles (>= two per SM) for the launch to split its blocks into two teams that work on
    # different gradients; gradients with tiles too dense for the per-warp lists, an all-zero one,
    # a ragged last tile; every stream byte-equal to the oracle's, twice in a row
    import torch
    import gpu_util as G
    n = 330 * 16384 + 777
    grads = []
    for w in range(ngrads):
        g = workloads.student_t_layers(n, seed=10 + w, blocks=12, lo=1e-4, hi=1e-1)
        grads.append(g)
    if ngrads > 2:
        grads[2] = np.zeros(n, np.float32)
    base = workloads.base_for_keep(grads[0], n // 20)
    pg, po = _params(base)
    binding.ensure_workspace(n, pg)
    cap = binding.compress_bound(n, pg)
    dg = [G.to_dev(v) for v in grads]
    bufs = [G.Guarded(cap, fill=0x3C) for _ in range(ngrads)]
    expect = [oracle.compress(g, po) for g in grads]
    dense_tiles = 0
    for rep in range(2):
        assert binding.compress_batch(dg, pg, [b.view for b in bufs]) == 0
        for w in range(ngrads):
            total, d, status = binding.stream_info(bufs[w].view)
            orc, ostream = expect[w]
            assert status == orc == 0 and total == ostream.size and bufs[w].intact()
            assert np.array_equal(bufs[w].view[:total].cpu().numpy(), ostream), f"gradient {w}, launch {rep}"
    # the case is only worth its name if some tile took the dense path (a 1024-entry slab with more than 192 kept)
    for g in grads[:2]:
        S = np.abs(g.astype(np.float64)).sum()
        thr = S / base ** 128
        k = np.abs(np.concatenate([g, np.zeros((-n) % 1024, np.float32)])) >= thr
        dense_tiles += int((k.reshape(-1, 1024).sum(1) > 192).sum())
    assert dense_tiles > 0


@pytest.mark.parametrize("keep_div", [400, 30])
def test_damaged_stream_among_sound_ones_in_one_launch(keep_div):
    # three streams decoded by one launch, the middle one damaged inside a group's blob: the status is
    # the oracle's for that stream, nothing outside dense_out is touched, and the groups the damage
    # does not reach hold exactly what the oracle holds.  keep_div = 400 keeps the groups small
    # (decoded by warps, streams parsed side by side), 30 makes them large enough for whole blocks.
    import torch
    import gpu_util as G
    n = 6 * 16384 + 77
    grads = [workloads.student_t_layers(n, seed=70 + w, blocks=1, lo=1e-2, hi=1e-2) for w in range(3)]
    base = workloads.base_for_keep(grads[0], n // keep_div)
    pg, po = _params(base)
    streams = []
    for v in grads:
        orc, st = oracle.compress(v, po)
        assert orc == 0
        streams.append(st)
    G_ = (n + 16383) // 16384
    bad_group = 3
    off = int.from_bytes(streams[1][64 + 8 * bad_group + 4:64 + 8 * bad_group + 8].tobytes(), "little")
    cnt = int.from_bytes(streams[1][64 + 8 * bad_group:64 + 8 * bad_group + 4].tobytes(), "little") & 0xFFFFFF
    assert cnt > 8
    for kind in ("flags", "deltas"):
        dmg = streams[1].copy()
        if kind == "flags":
            dmg[4 * off + cnt:4 * off + cnt + 2] ^= 0xFF           # first flag bytes: widths change, blob length no longer fits
        else:
            nxt = int.from_bytes(dmg[64 + 8 * (bad_group + 1) + 4:64 + 8 * (bad_group + 1) + 8].tobytes(), "little")
            dmg[4 * nxt - 6:4 * nxt - 2] = 0                       # last deltas zero: a repeated key
        expect = oracle.decompress_accumulate(dmg, n, po, np.zeros(n, np.float32))
        assert expect != 0
        odense = np.zeros(n, np.float32)
        assert oracle.decompress_accumulate(streams[0], n, po, odense) == 0
        good_only = odense.copy()
        assert oracle.decompress_accumulate(streams[2], n, po, good_only) == 0
        full = odense.copy()
        assert oracle.decompress_accumulate(streams[1], n, po, full) == 0
        assert oracle.decompress_accumulate(streams[2], n, po, full) == 0
        binding.ensure_workspace(n, pg)
        devs, sizes = [], []
        for st in (streams[0], dmg, streams[2]):
            pad = (-st.size) % 16
            devs.append(G.to_dev(np.concatenate([st, np.zeros(pad + 16, np.uint8)])))
            sizes.append(st.size)
        buf = G.Guarded(4 * n)
        dense = buf.view.view(torch.float32)
        dense.zero_()
        assert binding.decompress_accumulate_batch(devs, sizes, n, pg, dense) == 0
        st = binding.decode_status()
        assert st == expect and buf.intact(), (kind, st, expect)
        got = dense.cpu().numpy()
        lo, hi = bad_group * 16384, (bad_group + 1) * 16384
        # the damaged group of the damaged stream is dropped as a whole; every other (group, stream) is applied
        assert np.array_equal(got[:lo], full[:lo]) and np.array_equal(got[hi:], full[hi:]), kind
        assert np.array_equal(got[lo:hi], good_only[lo:hi]), kind


def _random_gradient(rng, n, kind):
    if kind == 0:
        return (rng.standard_normal(n) * 1e-3).astype(np.float32)
    if kind == 1:
        return workloads.student_t_layers(n, seed=int(rng.integers(1 << 30)), blocks=int(rng.integers(1, 9)), lo=1e-4, hi=1e-1)
    if kind == 2:          # mostly zeros with runs of non-zeros
        v = np.zeros(n, np.float32)
        for _ in range(int(rng.integers(1, 40))):
            a = int(rng.integers(0, n))
            b = min(n, a + int(rng.integers(1, 400)))
            v[a:b] = rng.laplace(0.0, 1e-2, b - a).astype(np.float32)
        return v
    v = (rng.standard_normal(n) * 1e-3).astype(np.float32)          # a few huge entries, denormals and exact ties
    idx = rng.integers(0, n, max(1, n // 50))
    v[idx] *= np.float32(1e4)
    v[rng.integers(0, n, max(1, n // 100))] = np.float32(1e-42)
    v[rng.integers(0, n, max(1, n // 100))] = v[0]
    return v


@pytest.mark.parametrize("case", range(24))
def test_random_configurations_through_the_batched_calls(case):
    # seeded random draws of size, parameters, value distribution, keep ratio and worker count; the
    # batched calls must give the oracle's streams byte for byte and the oracle's accumulated vector
    import torch
    import gpu_util as G
    rng = np.random.default_rng(1000 + case)
    tiles = int(rng.choice([1, 2, 3, 7, 20, 41, 310, 345]))
    n = max(1, tiles * 16384 - int(rng.integers(0, 16384)))
    workers = int(rng.integers(1, 6))
    l = int(rng.integers(1, 6))
    tau = int(rng.choice([1, 2, 5, 17, 64, 127, 128]))
    kind = int(rng.integers(0, 4))
    grads = [_random_gradient(rng, n, kind) for _ in range(workers)]
    if workers > 2 and case % 3 == 0:
        grads[1] = np.zeros(n, np.float32)
    keep = float(rng.choice([0.0005, 0.005, 0.03, 0.2, 0.7]))
    ref = grads[0] if np.count_nonzero(grads[0]) else grads[-1]
    kth = max(1, min(int(np.count_nonzero(ref)), int(keep * n)))
    base = workloads.base_for_keep(ref, kth, tau)
    pg, po = binding.params(base, tau, l, 14), oracle.params(base, tau, l, 14)
    binding.ensure_workspace(n, pg)
    cap = binding.compress_bound(n, pg)
    dg = [G.to_dev(v) for v in grads]
    bufs = [G.Guarded(cap, fill=0x77) for _ in range(workers)]
    assert binding.compress_batch(dg, pg, [b.view for b in bufs]) == 0
    dense0 = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    odense = dense0.copy()
    sizes = []
    for w in range(workers):
        total, d, status = binding.stream_info(bufs[w].view)
        orc, ostream = oracle.compress(grads[w], po)
        assert status == orc and bufs[w].intact(), (case, w, status, orc)
        assert total == ostream.size and np.array_equal(bufs[w].view[:total].cpu().numpy(), ostream), (case, w)
        sizes.append(total)
        if orc == 0:
            assert oracle.decompress_accumulate(ostream, n, po, odense) == 0
    if all(binding.stream_info(b.view)[2] == 0 for b in bufs):
        buf = G.Guarded(4 * n)
        dense = buf.view.view(torch.float32)
        dense.copy_(torch.from_numpy(dense0))
        assert binding.decompress_accumulate_batch([b.view for b in bufs], sizes, n, pg, dense) == 0
        assert binding.decode_status() == 0 and buf.intact()
        got = dense.cpu().numpy()
        assert np.allclose(got, odense, rtol=RTOL, atol=ATOL) and np.array_equal(got, odense), case


@pytest.mark.parametrize("workers", [1, 3])
@pytest.mark.parametrize("tiles", [5, 345])
def test_tiles_below_the_threshold_are_never_read_again(tiles, workers):
    # the kept entries sit in a few tiles; every other tile is non-zero but stays below the early-stop
    # threshold, so the encode pass lists only the hot tiles (and the last one, which carries the
    # header); the first and the last tile are cold, one gradient has no hot tile at all
    import gpu_util as G
    n = tiles * 16384 - 5000
    grads = []
    for w in range(workers):
        rng = np.random.default_rng(77 + 10 * tiles + w)
        v = (rng.standard_normal(n) * 1e-6).astype(np.float32)
        if w != 1:
            hot = rng.choice(np.arange(1, tiles - 1), size=max(1, tiles // 9), replace=False)
            for t in hot:
                k = int(rng.integers(1, 3000))
                idx = t * 16384 + rng.choice(16384, size=k, replace=False)
                v[idx] = (rng.standard_normal(k) * 1e-1).astype(np.float32)
        grads.append(v)
    S = float(np.abs(grads[0].astype(np.float64)).sum())
    base = float((S / 1e-3) ** (1.0 / 128.0))             # B_tau = 1e-3: far above the cold entries, below most hot ones
    pg, po = _params(base)
    binding.ensure_workspace(n, pg)
    cap = binding.compress_bound(n, pg)
    dg = [G.to_dev(v) for v in grads]
    bufs = [G.Guarded(cap, fill=0xA7) for _ in range(workers)]
    for rep in range(2):
        assert binding.compress_batch(dg, pg, [b.view for b in bufs]) == 0
        for w in range(workers):
            total, d, status = binding.stream_info(bufs[w].view)
            orc, ostream = oracle.compress(grads[w], po)
            assert status == orc == 0 and total == ostream.size and bufs[w].intact()
            assert np.array_equal(bufs[w].view[:total].cpu().numpy(), ostream), (w, rep)
            if w != 1:
                assert 0 < d < n // 10


@pytest.mark.parametrize("workers", [1, 2, 3, 5, 8, 10])
def test_sparse_adam_update_equals_the_oracles(workers):
    # the workers' streams decoded and one Adam step applied where the aggregated gradient is non-zero:
    # theta, m, v bit-equal to the oracle's, untouched coordinates untouched, the scratch vector back to zero;
    # two workers hold opposite values at shared keys (cancelled coordinates stay), tiles of every density
    import torch
    import gpu_util as G
    rng = np.random.default_rng(300 + workers)
    n = 41 * 16384 - 1234
    grads = [workloads.student_t_layers(n, seed=50 + w, blocks=7, lo=1e-4, hi=1e-1) for w in range(workers)]
    if workers >= 3:
        grads[2] = -grads[0]
    base = workloads.base_for_keep(grads[0], n // 25)
    pg, po = _params(base)
    binding.ensure_workspace(n, pg)
    cap = binding.compress_bound(n, pg)
    bufs = [G.Guarded(cap) for _ in range(workers)]
    assert binding.compress_batch([G.to_dev(v) for v in grads], pg, [b.view for b in bufs]) == 0
    streams, sizes = [], []
    for b in bufs:
        total, d, status = binding.stream_info(b.view)
        assert status == 0
        streams.append(b.view[:total].cpu().numpy()); sizes.append(total)
    theta0 = rng.standard_normal(n).astype(np.float32)
    m0 = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    v0 = (rng.standard_normal(n) ** 2 * 1e-6).astype(np.float32)
    lr, b1, b2, eps = 1e-3, 0.9, 0.999, 1e-8
    ot, om, ov = theta0.copy(), m0.copy(), v0.copy()
    assert oracle.sparse_adam_update(streams, n, po, lr, b1, b2, eps, ot, om, ov) == 0
    gt, gm, gv, gs = (G.Guarded(4 * n) for _ in range(4))
    theta, m, v, scratch = (x.view.view(torch.float32) for x in (gt, gm, gv, gs))
    theta.copy_(torch.from_numpy(theta0)); m.copy_(torch.from_numpy(m0)); v.copy_(torch.from_numpy(v0))
    for rep in range(2):                  # a second step right after: the scratch vector came back clean
        rc = binding.sparse_adam_update_batch([b.view for b in bufs], sizes, n, pg, binding.Adam(lr, b1, b2, eps),
                                              scratch, theta, m, v)
        assert rc == 0 and binding.decode_status() == 0
        assert all(x.intact() for x in (gt, gm, gv, gs))
        assert not bool(scratch.any().item())
        if rep == 1:
            assert oracle.sparse_adam_update(streams, n, po, lr, b1, b2, eps, ot, om, ov) == 0
        assert np.array_equal(theta.cpu().numpy(), ot) and np.array_equal(m.cpu().numpy(), om) and np.array_equal(v.cpu().numpy(), ov)
    changed = int((ot != theta0).sum())
    assert 0 < changed < n // 4
    if workers == 3:
        # coordinates kept by workers 0 and 2 alone cancel and must not move
        dense = np.zeros(n, np.float32)
        for s in streams:
            assert oracle.decompress_accumulate(s, n, po, dense) == 0
        assert np.array_equal(m0[dense == 0], om[dense == 0])


@pytest.mark.parametrize("group_log2, workers, shift", [(14, 2, 1), (14, 4, 3), (16, 1, 0), (16, 4, 0), (12, 3, 0), (10, 2, 2)])
def test_sparse_adam_update_other_group_sizes_and_unaligned_scratch(group_log2, workers, shift):
    # the update in one launch on the paths that the usual layout does not reach: groups wider than the slice a block
    # keeps in shared memory, a scratch vector that is not 16-byte aligned (both: aggregation in global memory, then
    # every stream again for the update), narrow groups; a key shared by all workers; theta, m, v bit-equal to the oracle's
    import torch
    import gpu_util as G
    rng = np.random.default_rng(900 + 10 * group_log2 + workers)
    n = 9 * 65536 + 4 * 777
    grads = [workloads.student_t_layers(n, seed=70 + w, blocks=5, lo=1e-4, hi=1e-1) for w in range(workers)]
    for g in grads[1:]:
        g[::97] = grads[0][::97]
    base = workloads.base_for_keep(grads[0], n // 12)
    pg, po = binding.params(base, 128, 2, group_log2), oracle.params(base, 128, 2, group_log2)
    binding.ensure_workspace(n, pg)
    cap = binding.compress_bound(n, pg)
    bufs = [G.Guarded(cap) for _ in range(workers)]
    streams, sizes = [], []
    for w in range(workers):
        assert binding.compress(G.to_dev(grads[w]), pg, bufs[w].view) == 0
        total, d, status = binding.stream_info(bufs[w].view)
        assert status == 0 and d > 0
        streams.append(bufs[w].view[:total].cpu().numpy()); sizes.append(total)
    theta0 = rng.standard_normal(n).astype(np.float32)
    m0 = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    v0 = (rng.standard_normal(n) ** 2 * 1e-6).astype(np.float32)
    lr, b1, b2, eps = 3e-3, 0.8, 0.99, 1e-7
    ot, om, ov = theta0.copy(), m0.copy(), v0.copy()
    assert oracle.sparse_adam_update(streams, n, po, lr, b1, b2, eps, ot, om, ov) == 0
    assert oracle.sparse_adam_update(streams, n, po, lr, b1, b2, eps, ot, om, ov) == 0
    theta, m, v = (torch.from_numpy(x).to(G.dev()) for x in (theta0, m0, v0))
    gs = G.Guarded(4 * (n + 4))
    scratch = gs.view.view(torch.float32)[shift:shift + n]
    for rep in range(2):
        rc = binding.sparse_adam_update_batch([b.view for b in bufs], sizes, n, pg, binding.Adam(lr, b1, b2, eps),
                                              scratch, theta, m, v)
        assert rc == 0 and binding.decode_status() == 0 and gs.intact()
        assert not bool(gs.view.any().item())
    assert np.array_equal(theta.cpu().numpy(), ot) and np.array_equal(m.cpu().numpy(), om) and np.array_equal(v.cpu().numpy(), ov)
    assert 0 < int((ot != theta0).sum()) < n // 2


@pytest.mark.parametrize("workers", [1, 3])
def test_model_update_on_damaged_streams_reports_the_decoders_status_and_stays_in_bounds(workers):
    # the one-launch update validates a group exactly as the aggregation does: on randomly damaged streams it reports
    # the status the oracle's decoder reports for the same streams and writes nowhere outside theta, m, v and the scratch
    import torch
    import gpu_util as G
    n = 6 * 16384 + 321
    rng = np.random.default_rng(4100 + workers)
    grads = [workloads.student_t_layers(n, seed=11 * w + 3, blocks=5, lo=1e-3, hi=1e-1) for w in range(workers)]
    b = workloads.base_for_keep(grads[0], n // 30)
    pg, po = _params(b)
    binding.ensure_workspace(n, pg)
    sound = [oracle.compress(v, po)[1] for v in grads]
    fixed = 64 + 8 * 7
    gt, gm, gv, gs = (G.Guarded(4 * n) for _ in range(4))
    theta, m, v, scratch = (x.view.view(torch.float32) for x in (gt, gm, gv, gs))
    h = binding.Adam(1e-3, 0.9, 0.999, 1e-8)
    gstate = G.Guarded(16 * n)
    seen = set()
    for case in range(36):
        streams = [s.copy() for s in sound]
        victim = case % workers
        s = streams[victim]
        region = case % 3
        for _ in range(int(rng.integers(1, 4))):
            pos = int(rng.integers(0, 64)) if region == 0 else (int(rng.integers(64, fixed)) if region == 1 else int(rng.integers(fixed, s.size)))
            s[pos] ^= np.uint8(rng.integers(1, 256))
        # the oracle's decoder, stream by stream: the first failing stream's status (streams are independent)
        expect = 0
        for t in streams:
            st = oracle.decompress_accumulate(t, n, po, np.zeros(n, np.float32))
            if st != 0 and expect == 0:
                expect = st
        bufs = [G.Guarded(t.size + (-t.size) % 16) for t in streams]
        for bf, t in zip(bufs, streams):
            bf.view[:t.size].copy_(torch.from_numpy(t))
        for x in (theta, m, v, scratch):
            x.zero_()
        rc = binding.sparse_adam_update_batch([bf.view for bf in bufs], [t.size for t in streams], n, pg, h, scratch, theta, m, v)
        assert rc == 0, case
        st = binding.decode_status()
        assert all(x.intact() for x in (gt, gm, gv, gs)) and all(bf.intact() for bf in bufs), case
        assert st == expect, (case, st, expect)
        seen.add(st)
        # the same streams through the call on the packed state
        gstate.view.zero_()
        rc = binding.sparse_adam_update_packed_batch([bf.view for bf in bufs], [t.size for t in streams], n, pg, h,
                                                     gstate.view.view(torch.float32))
        assert rc == 0 and binding.decode_status() == expect and gstate.intact() and all(bf.intact() for bf in bufs), case
    assert len(seen) >= 3


def test_three_hundred_launches_in_a_row_give_the_same_bytes():
    # every launch leaves the workspace as it found it: three gradients compressed in one launch, their streams decoded
    # and the model updated, 300 times back to back with nothing but the outputs cleared in between -- the streams, the
    # aggregated gradient and theta / m / v never differ from the first round's (which equal the oracle's)
    import torch
    import gpu_util as G
    n = 1_500_007
    host = [workloads.student_t_layers(n, seed=31 + w, blocks=6) for w in range(3)]
    b = workloads.base_for_keep(host[0], n // 120)
    pg, po = _params(b)
    binding.ensure_workspace(n, pg)
    grads = [G.to_dev(v) for v in host]
    cap = binding.compress_bound(n, pg)
    outs = [torch.zeros(cap, dtype=torch.uint8, device=G.dev()) for _ in range(3)]
    dense, theta, m, v, scratch = (torch.zeros(n, dtype=torch.float32, device=G.dev()) for _ in range(5))
    h = binding.Adam(1e-3, 0.9, 0.999, 1e-8)
    ref = None
    for it in range(300):
        for t in outs + [dense, theta, m, v]:
            t.zero_()
        assert binding.compress_batch(grads, pg, outs) == 0
        assert binding.decompress_accumulate_batch(outs, [cap] * 3, n, pg, dense) == 0
        assert binding.sparse_adam_update_batch(outs, [cap] * 3, n, pg, h, scratch, theta, m, v) == 0
        if ref is None:
            assert binding.decode_status() == 0
            for w in range(3):
                orc, ostream = oracle.compress(host[w], po)
                total, d, status = binding.stream_info(outs[w])
                assert status == orc == 0 and np.array_equal(outs[w][:total].cpu().numpy(), ostream)
            ref = [t.clone() for t in outs + [dense, theta, m, v]]
        elif it % 10 == 9 or it < 5:
            assert all(torch.equal(a, r) for a, r in zip(outs + [dense, theta, m, v], ref)), it
            assert binding.decode_status() == 0 and not bool(scratch.any().item())


@pytest.mark.parametrize("workers, n", [(1, 41 * 16384 - 1234), (2, 9 * 16384 + 3), (4, 41 * 16384 - 1234), (8, 20 * 16384 + 1)])
def test_model_update_on_the_packed_state_equals_the_oracles(workers, n):
    # the same step with theta, m, v and the scratch g interleaved four floats to a coordinate: theta, m, v bit-equal to
    # the oracle's on its three arrays, every g back to zero, two steps in a row, groups of every density, a last group
    # whose length is no multiple of four, keys shared by all workers, two workers that cancel
    import torch
    import gpu_util as G
    rng = np.random.default_rng(5200 + workers)
    grads = [workloads.student_t_layers(n, seed=90 + w, blocks=7, lo=1e-4, hi=1e-1) for w in range(workers)]
    for g in grads[1:]:
        g[::101] = grads[0][::101]
    if workers >= 4:
        grads[3] = -grads[1]
    base = workloads.base_for_keep(grads[0], n // 25)
    pg, po = _params(base)
    binding.ensure_workspace(n, pg)
    cap = binding.compress_bound(n, pg)
    bufs = [G.Guarded(cap) for _ in range(workers)]
    assert binding.compress_batch([G.to_dev(v) for v in grads], pg, [b.view for b in bufs]) == 0
    streams, sizes = [], []
    for b in bufs:
        total, d, status = binding.stream_info(b.view)
        assert status == 0
        streams.append(b.view[:total].cpu().numpy()); sizes.append(total)
    theta0 = rng.standard_normal(n).astype(np.float32)
    m0 = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    v0 = (rng.standard_normal(n) ** 2 * 1e-6).astype(np.float32)
    lr, b1, b2, eps = 1e-3, 0.9, 0.999, 1e-8
    ot, om, ov = theta0.copy(), m0.copy(), v0.copy()
    gstate = G.Guarded(16 * n)
    state = gstate.view.view(torch.float32)
    host = np.zeros((n, 4), np.float32)
    host[:, 0], host[:, 1], host[:, 2] = theta0, m0, v0
    state.copy_(torch.from_numpy(host.reshape(-1)))
    for rep in range(2):
        assert oracle.sparse_adam_update(streams, n, po, lr, b1, b2, eps, ot, om, ov) == 0
        rc = binding.sparse_adam_update_packed_batch([b.view for b in bufs], sizes, n, pg, binding.Adam(lr, b1, b2, eps), state)
        assert rc == 0 and binding.decode_status() == 0 and gstate.intact()
        got = state.cpu().numpy().reshape(n, 4)
        assert not got[:, 3].any()
        assert np.array_equal(got[:, 0], ot) and np.array_equal(got[:, 1], om) and np.array_equal(got[:, 2], ov)
    assert 0 < int((ot != theta0).sum()) < n // 2
    # what the call does not take
    p16 = binding.params(base, 128, 2, 16)
    binding.ensure_workspace(n, p16)
    assert binding.sparse_adam_update_packed_batch([b.view for b in bufs], sizes, n, p16, binding.Adam(lr, b1, b2, eps), state) == binding.E_NOT_IMPLEMENTED


def test_sparse_adam_update_single_stream_with_dense_tiles_and_bad_arguments():
    import torch
    import gpu_util as G
    rng = np.random.default_rng(77)
    n = 5 * 16384 + 100
    v_in = rng.standard_normal(n).astype(np.float32)
    v_in[3 * 16384:4 * 16384] = 0.0
    base = workloads.base_for_keep(v_in, n // 3)            # a third kept: whole blocks decode the groups
    pg, po = _params(base)
    binding.ensure_workspace(n, pg)
    buf = G.Guarded(binding.compress_bound(n, pg))
    assert binding.compress(G.to_dev(v_in), pg, buf.view) == 0
    total, d, status = binding.stream_info(buf.view)
    assert status == 0 and d > n // 4
    s = buf.view[:total].cpu().numpy()
    ot, om, ov = np.ones(n, np.float32), np.zeros(n, np.float32), np.zeros(n, np.float32)
    assert oracle.sparse_adam_update([s], n, po, 0.01, 0.9, 0.999, 1e-8, ot, om, ov) == 0
    theta = torch.ones(n, dtype=torch.float32, device=G.dev())
    m = torch.zeros(n, dtype=torch.float32, device=G.dev()); v = torch.zeros_like(m); scratch = torch.zeros_like(m)
    h = binding.Adam(0.01, 0.9, 0.999, 1e-8)
    assert binding.sparse_adam_update_batch([buf.view], [total], n, pg, h, scratch, theta, m, v) == 0
    assert binding.decode_status() == 0 and not bool(scratch.any().item())
    assert np.array_equal(theta.cpu().numpy(), ot) and np.array_equal(m.cpu().numpy(), om) and np.array_equal(v.cpu().numpy(), ov)
    import ctypes as C
    lib = binding.lib()
    ptrs = (C.c_void_p * 1)(int(buf.view.data_ptr())); sizes = (C.c_uint64 * 1)(total)
    assert lib.fastsgd_sparse_adam_update_batch(ptrs, sizes, 1, n, C.byref(pg), None, scratch.data_ptr(), theta.data_ptr(),
                                                m.data_ptr(), v.data_ptr(), None) == binding.E_NULL
    assert lib.fastsgd_sparse_adam_update_batch(ptrs, sizes, 1, n, C.byref(pg), C.byref(h), scratch.data_ptr(), None,
                                                m.data_ptr(), v.data_ptr(), None) == binding.E_NULL


def _gpu_bk(keys, l):
    """Algorithm 2 as printed, on the GPU -> (BK as a '0'/'1' string, M, index of bit offsets)."""
    import torch
    import gpu_util as G
    k = np.ascontiguousarray(keys, np.uint32)
    need = binding.key_encode_paper_bound(k.size, l)
    buf = G.Guarded(need, fill=0xC3)
    dk = torch.from_numpy(k.view(np.int32)).to(G.dev())
    assert binding.key_encode_paper(dk, l, buf.view) == 0
    raw = buf.view.cpu().numpy()
    assert buf.intact()
    M, l_got = int(raw[0:4].view(np.uint32)[0]), int(raw[4:8].view(np.uint32)[0])
    nbits = int(raw[8:16].view(np.uint64)[0])
    blocks = (k.size + 2047) // 2048
    index = raw[16:16 + 8 * blocks].view(np.uint64).copy()
    bits = np.unpackbits(raw[16 + 8 * blocks:16 + 8 * blocks + 4 * ((nbits + 31) // 32)])
    assert l_got == l and not bits[nbits:].any(), "padding bits must be zero"
    return "".join("01"[b] for b in bits[:nbits]), M, index


def test_paper_key_stream_worked_example_on_the_gpu():
    # the key list of the worked example under Fig. 3 (largest delta 232 -> M = 8, last key 578 -> '0011')
    keys = [10, 242, 300, 400, 575, 578]
    bk, M, index = _gpu_bk(keys, 2)
    obk, oM = oracle.key_encode_paper(keys, 2)
    assert M == oM == 8 and bk == obk and bk.endswith("0011") and list(index) == [0]


@pytest.mark.parametrize("l", [1, 2, 3, 4, 5])
@pytest.mark.parametrize("d", [0, 1, 2, 2047, 2048, 2049, 70_001])
def test_paper_key_stream_equals_the_oracles(d, l):
    rng = np.random.default_rng(1000 * l + d)
    if d % 2:
        gaps = rng.geometric(0.01, size=d).astype(np.int64)                     # smooth gaps
    else:
        gaps = np.where(rng.random(d) < 0.97, rng.integers(1, 9, d), rng.integers(1, 200_000, d)).astype(np.int64)   # mostly tiny, some huge
    if d:
        gaps[0] = 0 if d % 3 == 0 else gaps[0]                                  # a first key of 0
    keys = np.cumsum(gaps)
    assert d == 0 or keys[-1] < 2 ** 31
    bk, M, index = _gpu_bk(keys, l)
    obk, oM = oracle.key_encode_paper(keys, l)
    assert M == oM and len(bk) == len(obk) and bk == obk
    # the index: bit offset of every 2048th key = length of the oracle's BK over the keys before it
    for i, off in enumerate(index):
        if i and i % 16 == 0 or i == len(index) - 1:
            pre, _ = oracle.key_encode_paper(keys[:2048 * i], l) if i else ("", 0)
            if i and oracle.key_encode_paper(keys[:2048 * i], l)[1] == oM:
                assert int(off) == len(pre)


def test_paper_key_stream_on_compressed_gradient_keys_and_wide_deltas():
    # the kept keys of a compressed gradient, and keys spread over the whole 31-bit range (M = 31)
    n = 600_000
    v = workloads.student_t_layers(n, seed=4, blocks=9, lo=1e-4, hi=1e-1)
    rc, keys, codes, S = oracle.value_encode(v, workloads.base_for_keep(v, n // 50), 128)
    assert rc == 0 and keys.size > 5000
    for l in (2, 3):
        bk, M, _ = _gpu_bk(keys, l)
        obk, oM = oracle.key_encode_paper(keys, l)
        assert M == oM and bk == obk
    wide = np.array([0, 1, 2 ** 30 + 5, 2 ** 31 - 1], np.uint64)
    bk, M, _ = _gpu_bk(wide, 2)
    obk, oM = oracle.key_encode_paper(wide, 2)
    assert M == oM == 31 and bk == obk
    import ctypes as C
    assert binding.lib().fastsgd_key_encode_paper(None, 5, 2, None, 0, None) == binding.E_NULL
    assert binding.key_encode_paper_bound(10, 9) == 0


def _check_kv(keys, vals, n, b, l=2, tau=128, glog=14, cap=None):
    """fastsgd_compress_kv against the oracle's stream for the same pairs (= the dense vector's stream)."""
    import torch
    import gpu_util as G
    pg, po = binding.params(b, tau, l, glog), oracle.params(b, tau, l, glog)
    binding.ensure_workspace(n, pg)
    orc, ostream = oracle.compress_kv(keys, vals, n, po, cap)
    buf = G.Guarded(binding.compress_bound(n, pg) if cap is None else cap, fill=0x6B)
    dk = torch.from_numpy(np.ascontiguousarray(keys, np.uint32).view(np.int32)).to(G.dev())
    dv = torch.from_numpy(np.ascontiguousarray(vals, np.float32)).to(G.dev())
    for rep in range(2):
        assert binding.compress_kv(dk, dv, n, pg, buf.view) == 0
        total, d, status = binding.stream_info(buf.view)
        assert status == orc and total == ostream.size and buf.intact(), (status, orc, total, ostream.size)
        assert np.array_equal(buf.view[:total].cpu().numpy(), ostream), "stream differs"
    return ostream


@pytest.mark.parametrize("tiles", [1, 2, 7, 345, 700])
@pytest.mark.parametrize("density", [0.0, 3e-5, 1e-3, 0.05])
def test_key_value_input_equals_the_dense_path(tiles, density):
    rng = np.random.default_rng(int(tiles * 1000 + density * 1e6))
    n = tiles * 16384 - int(rng.integers(0, 16000)) if tiles > 1 else 9000
    cnt = int(density * n)
    if density == 0.0:
        cnt = [0, 1, 2, 3][tiles % 4]
    keys = np.sort(rng.choice(n, size=cnt, replace=False)).astype(np.uint64)
    vals = (rng.standard_t(3, cnt) * 1e-2).astype(np.float32)
    if cnt > 10:
        vals[rng.integers(0, cnt, cnt // 10)] = 0.0                   # pairs with a zero value
    dense = np.zeros(n, np.float32)
    dense[keys.astype(np.int64)] = vals
    b = workloads.base_for_keep(dense, max(1, int(0.7 * np.count_nonzero(dense)))) if np.count_nonzero(dense) else 1.1
    s = _check_kv(keys, vals, n, b)
    # and it is the dense call's stream
    import gpu_util as G
    pg, _ = _params(b)
    rc, status, gstream, intact = G.gpu_compress(dense, pg)
    assert rc == 0 and np.array_equal(gstream, s)


def test_key_value_input_with_dense_runs_and_every_flag_size():
    # runs of consecutive keys (tiles too dense for the per-warp lists), a first key of 0, a last key of n - 1
    rng = np.random.default_rng(12)
    n = 9 * 16384 + 77
    parts = [np.arange(0, 3000), np.arange(16384 * 2 + 100, 16384 * 3 + 900), rng.choice(np.arange(16384 * 5, n - 1), 400, replace=False), [n - 1]]
    keys = np.unique(np.concatenate(parts)).astype(np.uint64)
    vals = rng.standard_normal(keys.size).astype(np.float32)
    dense = np.zeros(n, np.float32)
    dense[keys.astype(np.int64)] = vals
    for l in (1, 3, 5):
        b = workloads.base_for_keep(dense, int(0.9 * keys.size))
        _check_kv(keys, vals, n, b, l=l)
    import ctypes as C
    import torch
    pg, _ = _params(1.1)
    out = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    assert binding.lib().fastsgd_compress_kv(None, None, 5, n, C.byref(pg), out.data_ptr(), out.numel(), None) == binding.E_NULL
    assert binding.lib().fastsgd_compress_kv(None, None, 0, n, C.byref(pg), None, 0, None) == binding.E_NULL


@pytest.mark.parametrize("glog", [4, 8, 12, 16, 20])
@pytest.mark.parametrize("l", [2, 5])
def test_key_value_input_other_group_sizes(glog, l):
    # the key-value encoder takes the group size as a parameter: runs, scattered pairs, a group that spans many chunks
    rng = np.random.default_rng(100 * glog + l)
    n = 2_500_003 if glog >= 12 else 300_007
    parts = [np.arange(5, 2600), rng.choice(n, n // 200, replace=False), np.arange(n - 40_000, n - 1, 3), [n - 1]]
    keys = np.unique(np.concatenate(parts)).astype(np.uint64)
    vals = (rng.standard_t(3, keys.size) * 1e-2).astype(np.float32)
    dense = np.zeros(n, np.float32)
    dense[keys.astype(np.int64)] = vals
    b = workloads.base_for_keep(dense, int(0.8 * keys.size))
    _check_kv(keys, vals, n, b, l=l, glog=glog)


@pytest.mark.parametrize("glog", [8, 12, 16, 20])
@pytest.mark.parametrize("keep_div", [300, 12])
def test_other_group_sizes_dense_input_and_decoder(glog, keep_div):
    # group sizes other than the fused encoder's 2^14: streams byte-equal to the oracle's, decoded sums bit-equal
    import gpu_util as G
    rng = np.random.default_rng(glog * 7 + keep_div)
    n = 3_000_017
    v = workloads.student_t_layers(n, seed=glog, blocks=11)
    v[rng.integers(0, n, n // 3)] = 0.0
    b = workloads.base_for_keep(v, n // keep_div)
    for l in (2, 3):
        pg, po = binding.params(b, 128, l, glog), oracle.params(b, 128, l, glog)
        orc, ostream = oracle.compress(v, po)
        rc, status, gstream, intact = G.gpu_compress(v, pg, fill=0x77)
        assert rc == 0 and intact and status == orc == 0
        assert gstream.size == ostream.size and np.array_equal(gstream, ostream)
        dense0 = rng.standard_normal(n).astype(np.float32)
        odense = dense0.copy()
        assert oracle.decompress_accumulate(ostream, n, po, odense) == 0
        rc, st, gdense, intact = G.gpu_decompress(gstream, n, pg, dense0)
        assert rc == 0 and st == 0 and intact
        assert np.allclose(gdense, odense, rtol=RTOL, atol=ATOL) and np.array_equal(gdense, odense)


def test_other_group_sizes_when_the_kept_list_does_not_fit():
    # general path: more kept entries than the workspace's list holds (4.5 M pairs): the dense walk takes over, same stream
    import gpu_util as G
    n = 6_300_001
    v = workloads.normal(n, seed=8)
    b = workloads.base_for_keep(v, int(0.8 * n))
    pg, po = binding.params(b, 128, 2, 12), oracle.params(b, 128, 2, 12)
    orc, ostream = oracle.compress(v, po)
    assert orc == 0 and int(np.frombuffer(ostream[24:32].tobytes(), np.uint64)[0]) > 4_700_000
    rc, status, gstream, intact = G.gpu_compress(v, pg, fill=0x31)
    assert rc == 0 and intact and status == 0
    assert gstream.size == ostream.size and np.array_equal(gstream, ostream)


def test_key_value_input_status_words_and_hostile_keys():
    import torch
    import gpu_util as G
    rng = np.random.default_rng(5)
    n = 6 * 16384 + 5
    keys = np.sort(rng.choice(n, 3000, replace=False)).astype(np.uint64)
    vals = rng.standard_normal(3000).astype(np.float32)
    dense = np.zeros(n, np.float32)
    dense[keys.astype(np.int64)] = vals
    b = workloads.base_for_keep(dense, 2500)
    pg, po = _params(b)
    # a capacity that holds header and directory but not the blobs; then one byte short of the stream; then exact
    full = _check_kv(keys, vals, n, b)
    for cap in (64 + 8 * 7, full.size - 4, full.size):
        s = _check_kv(keys, vals, n, b, cap=cap)
        assert (s.size == full.size) == (cap == full.size)
    # a value that is not finite; all values zero
    bad = vals.copy(); bad[17] = np.inf
    _check_kv(keys, bad, n, b)
    bad[17] = np.nan
    _check_kv(keys, bad, n, b)
    _check_kv(keys, np.zeros_like(vals), n, b)
    # keys that do not ascend, repeat, or reach beyond n: any stream, but nothing outside the buffers, and the next call is exact
    binding.ensure_workspace(n, pg)
    buf = G.Guarded(binding.compress_bound(n, pg), fill=0x6B)
    for hostile in (keys[::-1].copy(), np.repeat(keys[:1500], 2), np.concatenate([keys[:2990], np.arange(n, n + 10)]),
                    np.full(3000, 2 ** 32 - 1), rng.integers(0, 2 ** 32, 3000)):
        dk = torch.from_numpy(np.ascontiguousarray(hostile, np.uint64).astype(np.uint32).view(np.int32)).to(G.dev())
        dv = torch.from_numpy(vals).to(G.dev())
        assert binding.compress_kv(dk, dv, n, pg, buf.view) == 0
        torch.cuda.synchronize()
        assert buf.intact()
    _check_kv(keys, vals, n, b)


@pytest.mark.parametrize("keep_div", [500, 40, 3])
def test_randomly_damaged_streams_report_the_oracles_status(keep_div):
    # seeded random damage (one to three bytes anywhere in the stream, header and directory included) on sparse,
    # medium and dense streams: the decoder reports exactly the oracle's status and never leaves its buffers
    import gpu_util as G
    n = 6 * 16384 + 321
    rng = np.random.default_rng(900 + keep_div)
    v = workloads.student_t_layers(n, seed=keep_div, blocks=5, lo=1e-3, hi=1e-1)
    b = workloads.base_for_keep(v, n // keep_div)
    pg, po = _params(b)
    orc, st0 = oracle.compress(v, po)
    assert orc == 0
    fixed = 64 + 8 * 7
    seen = set()
    for case in range(60):
        s = st0.copy()
        region = case % 3                      # header, directory, blobs
        for _ in range(int(rng.integers(1, 4))):
            if region == 0:
                pos = int(rng.integers(0, 64))
            elif region == 1:
                pos = int(rng.integers(64, fixed))
            else:
                pos = int(rng.integers(fixed, st0.size))
            s[pos] ^= np.uint8(rng.integers(1, 256))
        expect = oracle.decompress_accumulate(s, n, po, np.zeros(n, np.float32))
        rc, st, dense, intact = G.gpu_decompress(s, n, pg)
        assert rc == 0 and intact, case
        assert st == expect, (case, st, expect)
        seen.add(st)
    assert len(seen) >= 3                      # several different outcomes, a sound decode among them or not
    rc, st, dense, intact = G.gpu_decompress(st0, n, pg)
    assert rc == 0 and st == 0 and intact
