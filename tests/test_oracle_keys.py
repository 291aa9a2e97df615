"""Pins of the oracle's gradient-key path (Sec. 3.3, Eq. 4, Algorithm 2) and of the stream
container: the paper's worked example, Python big-int strings, exhaustive round trips,
the closed-form space cost and a second, separately written reader / writer."""
import os

import numpy as np
import pytest

import oracle
import pyref

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _gold(name):
    out = {}
    for line in open(os.path.join(GOLD, name)):
        t = line.split()
        if t and not t[0].startswith("#"):
            out.setdefault(t[0], []).append(t[1:])
    return out


def test_fig3_worked_example():
    g = _gold("fig3_key_encoder.txt")
    max_delta, M, l = int(g["max_delta"][0][0]), int(g["M"][0][0]), int(g["l"][0][0])
    widths = [int(x) for x in g["widths"][0]]
    ranges = [int(x) for x in g["ranges"][0]]
    assert max(1, oracle.bitlen(max_delta)) == M
    assert oracle.widths(M, l) == widths
    # each level's range [ranges[f], ranges[f+1]) maps to flag f
    for f in range(4):
        assert oracle.length_flag(ranges[f], widths, l) == f
        assert oracle.length_flag(ranges[f + 1] - 1, widths, l) == f
    # a key list whose largest delta is 232 and whose last key 578 has delta 3
    last_key, last_delta = int(g["last_key"][0][0]), int(g["last_delta"][0][0])
    keys = [10, 242, 300, 400, 575, last_key]
    assert keys[1] - keys[0] == max_delta and keys[-1] - keys[-2] == last_delta
    bk, M_got = oracle.key_encode_paper(keys, l)
    assert M_got == M and bk.endswith(g["last_bits"][0][0])
    assert bk == pyref.alg2_paper(keys, l)[0]
    # plain binary strings quoted in the text: 3 -> '11', 5 -> '101'
    for value, s in g["binary"]:
        value = int(value)
        bkv, Mv = oracle.key_encode_paper([value], 1)       # one key: M = bitlen, widest level
        assert bkv[1:] == s and Mv == len(s)


def test_power_of_two_and_tiny_max_delta():
    # ceil(log2 maxDelta) would be one bit short for 2^m and zero for maxDelta <= 1
    for md, M in [(1, 1), (2, 2), (4, 3), (255, 8), (256, 9), (0, 1)]:
        bk, M_got = oracle.key_encode_paper([md], 2)
        assert M_got == M
        assert int(bk[2:], 2) == md


@pytest.mark.parametrize("l", [1, 2, 3, 4, 5])
def test_paper_sequence_against_python_strings(l):
    rng = np.random.default_rng(l)
    for _ in range(40):
        n = int(rng.integers(8, 5000))
        d = int(rng.integers(1, min(n, 64)))
        keys = np.sort(rng.choice(n, d, replace=False))
        bk, M = oracle.key_encode_paper(keys, l)
        ref, Mref = pyref.alg2_paper(keys.tolist(), l)
        assert (bk, M) == (ref, Mref)


@pytest.mark.parametrize("l", [1, 2, 3, 4, 5])
def test_single_group_stream_is_algorithm2_with_planes(l):
    # With T >= n a blob is Algorithm 2's output with flags and deltas stored as two planes:
    # re-interleaving them must give BK bit for bit.
    rng = np.random.default_rng(100 + l)
    for _ in range(30):
        glog = int(rng.integers(4, 13))
        n = int(rng.integers(2, (1 << glog) + 1))
        d = int(rng.integers(1, min(n, 200) + 1))
        keys = np.sort(rng.choice(n, d, replace=False))
        codes = rng.choice([-5, 3, 1, -128, 128, 77], d)
        p = oracle.params(1.1, 128, l, glog)
        rc, stream = oracle.write_stream(keys, codes, n, 1.0, p)
        assert rc == 0
        buf = stream.tobytes()
        a = int.from_bytes(buf[64:68], "little")
        off = int.from_bytes(buf[68:72], "little")
        count, M = a & 0xFFFFFF, a >> 24
        assert count == d and off == (64 + 8) // 4
        blob = buf[4 * off:]
        s = bin(int.from_bytes(blob, "big"))[2:].zfill(8 * len(blob))
        w = pyref.level_widths(M, l)
        flags = [s[8 * d + l * i: 8 * d + l * (i + 1)] for i in range(d)]
        pos, inter = 8 * d + l * d, ""
        for f in flags:
            wf = w[int(f, 2)]
            inter += f + s[pos:pos + wf]
            pos += wf
        bk, M_paper = oracle.key_encode_paper(keys, l)
        assert M == M_paper and inter == bk
        assert set(s[pos:]) <= {"0"}
        got_codes = [oracle.code_from_byte(blob[i]) for i in range(d)]
        assert got_codes == codes.tolist()


@pytest.mark.parametrize("glog", [2, 3, 4])
def test_round_trip_all_subsets(glog):
    # Keys must come back exactly (Sec. 3.3: the key codec is lossless): every non-empty subset of
    # {0..n-1} for n = 1, 5, 12 and 16 (65,535 subsets), groups of 4, 8 and 16 indices.
    p = oracle.params(1.1, 128, 2, glog)
    for n in (1, 5, 12, 16):
        for mask in range(1, 1 << n):
            keys = [i for i in range(n) if mask >> i & 1]
            codes = [(-1) ** i * (1 + (i * 37) % 128) for i in keys]
            rc, stream = oracle.write_stream(keys, codes, n, 2.5, p)
            assert rc == 0
            rc, k2, c2, S = oracle.parse(stream, n, p)
            assert rc == 0 and k2.tolist() == keys and c2.tolist() == codes and S == 2.5


@pytest.mark.parametrize("l", [1, 2, 3, 4, 5])
def test_round_trip_random_and_second_codec(l):
    # random subsets, n in [8, 64] and larger; a separately written Python writer must produce
    # the same bytes (one canonical stream per input) and a separate reader the same pairs
    rng = np.random.default_rng(7 * l)
    for trial in range(60):
        glog = int(rng.integers(2, 9))
        n = int(rng.integers(8, 65)) if trial % 2 else int(rng.integers(65, 3000))
        d = int(rng.integers(0, n + 1))
        keys = np.sort(rng.choice(n, d, replace=False)).tolist()
        codes = (rng.integers(1, 129, d) * rng.choice([-1, 1], d)).tolist()
        S, b, tau = 3.25, 1.25, 128
        p = oracle.params(b, tau, l, glog)
        rc, stream = oracle.write_stream(keys, codes, n, S, p)
        assert rc == 0
        assert stream.tobytes() == pyref.write_stream(keys, codes, n, S, b, tau, l, glog)
        hdr, k2, c2 = pyref.read_stream(stream.tobytes())
        assert k2 == keys and c2 == codes and hdr["d"] == d and hdr["S"] == S and hdr["b"] == b
        rc, k3, c3, S3 = oracle.parse(stream, n, p)
        assert rc == 0 and k3.tolist() == keys and c3.tolist() == codes
        assert stream.size <= oracle.compress_bound(n, p)


def test_space_cost_closed_form():
    # Sec. 3.4: evenly spaced keys cost ceil(log2(D_m/d)) + l bits each, values 8 bits each
    for line in open(os.path.join(GOLD, "space_cost.txt")):
        t = line.split()
        if not t or t[0].startswith("#"):
            continue
        Dm, d, l, key_bits, total_bits = map(int, t)
        s = Dm // d
        keys = [s * j for j in range(1, d)] + [s * d - 1]          # d keys, all deltas s except the last (s-1)
        bk, M = oracle.key_encode_paper(keys, l)
        assert len(bk) == d * key_bits
        assert 8 * d + len(bk) == total_bits
        # the container with one group spends the same bits plus header, directory and padding
        glog = max(1, (Dm - 1).bit_length())
        p = oracle.params(1.1, 128, l, glog)
        rc, stream = oracle.write_stream(keys, [1] * d, Dm, 1.0, p)
        assert rc == 0 and stream.size == 64 + 8 + 4 * ((total_bits + 31) // 32)


def test_compress_is_value_encode_then_stream():
    rng = np.random.default_rng(9)
    n = 40000
    v = (rng.standard_t(3, n) * 1e-3).astype(np.float32)
    b = 1.09
    p = oracle.params(b, 128, 2, 10)
    rc, keys, codes, S = oracle.value_encode(v, b, 128)
    rc2, stream = oracle.compress(v, p)
    assert rc == 0 and rc2 == 0 and keys.size > 100
    assert stream.tobytes() == pyref.write_stream(keys.tolist(), codes.tolist(), n, S, b, 128, 2, 10)
    # every kept code meets the threshold
    assert np.all((np.abs(codes) >= 1) & (np.abs(codes) <= 128))


def test_capacity_and_nonfinite_headers():
    rng = np.random.default_rng(10)
    n = 5000
    v = rng.standard_normal(n).astype(np.float32)
    p = oracle.params(1.2, 128, 2, 8)
    rc, full = oracle.compress(v, p)
    assert rc == 0
    rc, small = oracle.compress(v, p, cap=full.size - 4)
    assert rc == oracle.ERR_CAPACITY and small.size == 64
    hdr, k, c = pyref.read_stream(small.tobytes())
    assert hdr["status"] == oracle.ERR_CAPACITY and hdr["d"] == 0 and hdr["total"] == 64
    v[17] = np.inf
    rc, bad = oracle.compress(v, p)
    assert rc == oracle.ERR_NONFINITE and bad.size == 64
    hdr, k, c = pyref.read_stream(bad.tobytes())
    assert hdr["status"] == oracle.ERR_NONFINITE and hdr["S"] == 0.0
    dense = np.zeros(n, np.float32)
    assert oracle.decompress_accumulate(bad, n, p, dense) == oracle.DEC_BAD_STATUS
    assert not dense.any()


def _corrupt(stream, pos, value, width=4):
    s = stream.copy()
    s[pos:pos + width] = np.frombuffer(int(value).to_bytes(width, "little"), np.uint8)
    return s


def test_decoder_rejects_damaged_streams():
    rng = np.random.default_rng(12)
    n = 3000
    v = rng.standard_normal(n).astype(np.float32)
    p = oracle.params(1.07, 128, 2, 8)
    rc, st = oracle.compress(v, p)
    assert rc == 0
    G = (n + 255) // 256
    dense = np.zeros(n, np.float32)

    def run(s, nbytes=None, pp=p, nn=n):
        return oracle.decompress_accumulate(s, nn, pp, np.zeros(nn, np.float32), nbytes)

    assert run(st) == 0
    assert run(_corrupt(st, 0, 0x12345678)) == oracle.DEC_BAD_MAGIC
    assert run(_corrupt(st, 4, 2)) == oracle.DEC_BAD_VERSION
    assert run(_corrupt(st, 8, 3)) == oracle.DEC_BAD_STATUS
    assert run(st, nn=n + 1) in (oracle.DEC_N_MISMATCH,)
    assert run(st, pp=oracle.params(1.08, 128, 2, 8)) == oracle.DEC_PARAM_MISMATCH
    assert run(st, pp=oracle.params(1.07, 127, 2, 8)) == oracle.DEC_PARAM_MISMATCH
    assert run(st, pp=oracle.params(1.07, 128, 3, 8)) == oracle.DEC_PARAM_MISMATCH
    assert run(st, nbytes=st.size - 4) == oracle.DEC_TRUNCATED
    assert run(st, nbytes=10) == oracle.DEC_TRUNCATED
    # directory damage: a count larger than the group, a wrong offset, M out of range
    a0 = int.from_bytes(st[64:68].tobytes(), "little")
    assert run(_corrupt(st, 64, (a0 & 0xFF000000) | 257)) == oracle.DEC_BAD_DIRECTORY
    assert run(_corrupt(st, 64, (a0 & 0xFFFFFF) | (9 << 24))) == oracle.DEC_BAD_DIRECTORY
    off1 = int.from_bytes(st[76:80].tobytes(), "little")
    assert run(_corrupt(st, 76, off1 + 1)) == oracle.DEC_BAD_DIRECTORY
    # a key pushed past the end of its group: all deltas of the last group set to all ones
    last = G - 1
    offl = int.from_bytes(st[64 + 8 * last + 4:64 + 8 * last + 8].tobytes(), "little")
    al = int.from_bytes(st[64 + 8 * last:64 + 8 * last + 4].tobytes(), "little")
    cnt = al & 0xFFFFFF
    s2 = st.copy()
    s2[4 * offl + cnt:] = 0xFF                                   # flags -> widest, deltas -> max
    assert run(s2) in (oracle.DEC_BAD_KEY, oracle.DEC_BAD_DIRECTORY)
