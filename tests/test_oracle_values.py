"""Pins of the oracle's gradient-value path (Sec. 3.2, Eq. 2-3, Algorithm 1) against facts
that do not come from the oracle: the paper's worked example, exact rational arithmetic,
frexp, math.fsum, brute force and the paper's stated invariants."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
import pyref

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    for line in open(os.path.join(GOLD, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            yield line.split()


# ----------------------------------------------------------------- quantiser

def test_fig2_worked_example():
    # Sec. 3.2 Phase 2: b = 2, R = 6.1 -> L = 3.  Realised as sum = 6.1, |v| = 1.
    for b, R, L in _rows("fig2_quantiser.txt"):
        b, R, L = float(b), float(R), int(L)
        P, B = oracle.tables(R, b, 8)
        assert oracle.quantise(1.0, B, 8) == L
        assert math.ceil(math.log(R, b)) == L


def test_reciprocal_is_at_least_one_so_level_is_nonnegative():
    # Sec. 3.2 Phase 1, property 1: R(v_j) >= 1, hence L >= 0, and L = 0 only for |v| = sum.
    v = np.array([0.0, 0.0, -3.5, 0.0], np.float32)
    rc, keys, codes, s = oracle.value_encode(v, 1.1, 128)
    assert rc == 0 and s == 3.5
    assert keys.tolist() == [2] and codes.tolist() == [-1]     # L = 0 raised to 1, sign kept


def test_base2_power_of_two_sum_reduces_to_frexp():
    # b = 2 and sum = 2^s: ceil(log2(2^s/|v|)) = s - floor(log2|v|) unless |v| is a power of two
    rng = np.random.default_rng(1)
    vals = np.concatenate([rng.uniform(1e-6, 1.0, 2000), 2.0 ** -np.arange(0, 20)]).astype(np.float32)
    s = 5
    P, B = oracle.tables(2.0 ** s, 2.0, 64)
    for a in vals.tolist():
        m, e = math.frexp(a)               # a = m * 2^e, 0.5 <= m < 1
        expect = s - e + 1 if m != 0.5 else s - (e - 1)
        assert oracle.quantise(a, B, 64) == expect


def test_base2_any_sum_brute_force_with_ldexp():
    rng = np.random.default_rng(2)
    vals = rng.lognormal(-4, 2, 500).astype(np.float32)
    S = float(vals.astype(np.float64).sum())
    P, B = oracle.tables(S, 2.0, 100)
    for a in vals.tolist():
        k = 0
        while math.ldexp(a, k) < S:        # exact: scaling by 2^k
            k += 1
        assert oracle.quantise(a, B, 100) == k


@pytest.mark.parametrize("b", [1.1, 1.05, 1.5, 1.0371, 3.0])
def test_general_base_against_exact_rationals(b):
    # The table compare may differ from exact arithmetic only where |v| sits within rounding
    # distance of a boundary; on this random data it must not differ at all.
    rng = np.random.default_rng(3)
    v = (rng.standard_normal(4000) * 1e-3).astype(np.float32)
    S = oracle.abs_sum(v)
    tau = 128
    P, B = oracle.tables(S, b, tau)
    mism = 0
    for x in v.tolist():
        if x == 0.0:
            continue
        try:
            k = pyref.exact_level(x, S, b, kmax=tau)
        except OverflowError:
            k = tau + 1
        got = oracle.quantise(abs(x), B, tau)
        if got != k:
            # tolerated only within ~tau*2^-52 of a boundary
            r = Fraction(abs(x)) * Fraction(b) ** min(got, k) / Fraction(S)
            assert abs(float(r) - 1.0) < 200 * 2.0 ** -52
            mism += 1
    assert mism == 0


def test_exact_powers_are_inclusive():
    # R = b^k exactly gives L = k (ceiling of an integer)
    P, B = oracle.tables(1024.0, 2.0, 20)
    for k in range(0, 11):
        assert oracle.quantise(1024.0 / 2.0 ** k, B, 20) == k
        assert oracle.quantise(np.nextafter(1024.0 / 2.0 ** k, 0.0), B, 20) == k + 1


def test_order_reversal():
    # Sec. 3.2 Phase 1, property 2: bigger |v| -> smaller (or equal) code
    rng = np.random.default_rng(4)
    v = np.sort(np.abs(rng.standard_normal(3000)).astype(np.float32))
    P, B = oracle.tables(oracle.abs_sum(v), 1.1, 128)
    L = [oracle.quantise(float(a), B, 128) for a in v]
    assert all(L[i] >= L[i + 1] for i in range(len(L) - 1))


# -------------------------------------------------------------------- filter

@pytest.mark.parametrize("seed", range(4))
def test_filter_invariants(seed):
    rng = np.random.default_rng(seed)
    v = (rng.standard_t(3, 5000) * 1e-3).astype(np.float32)
    v[rng.integers(0, v.size, 50)] = 0.0
    b, tau = 1.07, 128
    rc, keys, codes, S = oracle.value_encode(v, b, tau)
    assert rc == 0
    P, B = oracle.tables(S, b, tau)
    tau_e = S / b ** tau
    a = np.abs(v).astype(np.float64)
    # kept <=> |v| >= tau_e (Algorithm 1), counted by an independent one-liner
    clear = np.abs(a / tau_e - 1.0) > 1e-9
    assert int(np.sum((a >= tau_e) & clear)) == int(np.sum(clear[keys.astype(np.int64)]))
    kept = np.zeros(v.size, bool)
    kept[keys.astype(np.int64)] = True
    assert np.all(a[kept & clear] >= tau_e) and np.all(a[~kept & clear] < tau_e)
    # every kept code lies within the threshold (Sec. 3.2 Phase 3) and carries the sign
    assert np.all(np.abs(codes) >= 1) and np.all(np.abs(codes) <= tau)
    assert np.all(np.sign(codes) == np.sign(v[keys.astype(np.int64)]))
    # each kept |v| >= sum / b^tau, so at most b^tau entries survive
    assert keys.size <= math.floor(b ** tau)
    assert np.all(np.diff(keys.astype(np.int64)) > 0)


def test_boundary_value_exactly_at_threshold_is_kept():
    # sum = 4 + 2^-5 * 0 ... build: values 1,1,1,1 -> sum 4; b = 2, tau = 3 -> tau_e = 0.5
    v = np.array([1, 1, 1, 0.5, 0.25, 0.25], np.float32)     # sum = 4.0, tau_e = 4/8 = 0.5
    rc, keys, codes, S = oracle.value_encode(v, 2.0, 3)
    assert S == 4.0
    assert keys.tolist() == [0, 1, 2, 3]                      # 0.5 >= tau_e kept (inclusive), 0.25 dropped
    assert codes.tolist() == [2, 2, 2, 3]                     # ceil(log2 4) = 2, ceil(log2 8) = 3


def test_zeros_and_all_zero():
    v = np.zeros(100, np.float32)
    v[3] = -0.0
    rc, keys, codes, S = oracle.value_encode(v, 1.1, 128)
    assert rc == 0 and S == 0.0 and keys.size == 0


def test_nonfinite_sum_is_reported():
    v = np.ones(10, np.float32)
    v[4] = np.inf
    rc, keys, codes, S = oracle.value_encode(v, 1.1, 128)
    assert rc == oracle.ERR_NONFINITE and keys.size == 0
    v[4] = np.nan
    assert oracle.value_encode(v, 1.1, 128)[0] == oracle.ERR_NONFINITE


def test_brute_force_tiny_inputs():
    # n in [8, 64]: Algorithm 1 restated with exact rationals on the oracle's own sum
    rng = np.random.default_rng(7)
    for trial in range(60):
        n = int(rng.integers(8, 65))
        v = (rng.standard_normal(n) * 10.0 ** rng.integers(-6, 3)).astype(np.float32)
        v[rng.random(n) < 0.2] = 0.0
        b = float(rng.choice([1.1, 1.3, 2.0]))
        tau = int(rng.choice([4, 16, 128]))
        rc, keys, codes, S = oracle.value_encode(v, b, tau)
        exp_keys, exp_codes = [], []
        for j, x in enumerate(v.tolist()):
            if x == 0.0:
                continue
            try:
                k = pyref.exact_level(x, S, b, kmax=tau)
            except OverflowError:
                continue
            exp_keys.append(j)
            exp_codes.append(int(math.copysign(max(k, 1), x)))
        assert keys.tolist() == exp_keys and codes.tolist() == exp_codes


# ----------------------------------------------------------------------- sum

def test_sum_tree_shape_by_hand():
    # (a+b)+(c+d) with a = 1, b = c = d = 2^-53: 1+2^-53 rounds to 1 (tie to even), 2^-53+2^-53 = 2^-52,
    # total 1+2^-52; a left-to-right sum would give exactly 1.
    t = 2.0 ** -53
    v = np.array([1.0, t, t, t], np.float32)
    assert oracle.abs_sum(v) == 1.0 + 2.0 ** -52
    assert ((1.0 + t) + t) + t == 1.0
    # n = 3 is padded with a zero: (1 + t) + (t + 0) = 1 + t -> rounds to 1
    assert oracle.abs_sum(v[:3]) == 1.0
    # n = 5: ((a+b)+(c+d)) + (((e+0)+(0+0))) with e = 2^-52: (1+2^-52) + 2^-52 = 1 + 2^-51
    v5 = np.array([1.0, t, t, t, 2.0 ** -52], np.float32)
    assert oracle.abs_sum(v5) == 1.0 + 2.0 ** -51
    # negative entries count by magnitude
    assert oracle.abs_sum(-v) == 1.0 + 2.0 ** -52


@pytest.mark.parametrize("n", [1, 2, 3, 7, 8, 9, 1000, 1024, 1025, 70001])
def test_sum_against_fsum_and_padding(n):
    rng = np.random.default_rng(n)
    v = (rng.standard_normal(n) * 10.0 ** rng.integers(-8, 4, n)).astype(np.float32)
    S = oracle.abs_sum(v)
    exact = math.fsum(abs(float(x)) for x in v)
    assert abs(S - exact) <= max(1, math.ceil(math.log2(n)) ) * 2.0 ** -53 * exact
    assert S == pyref.naive_tree_sum(v)
    assert oracle.abs_sum(np.concatenate([v, np.zeros(37, np.float32)])) == S


def test_sum_exact_on_dyadic_values():
    rng = np.random.default_rng(11)
    k = rng.integers(-1000, 1000, 5000)
    v = (k / 1024.0).astype(np.float32)
    assert oracle.abs_sum(v) == float(np.abs(k).sum()) / 1024.0


# -------------------------------------------------------------------- decode

@pytest.mark.parametrize("b", [1.1, 1.04, 2.0])
def test_decoded_value_underestimates_within_one_level(b):
    # Sec. 3.2: the ceiling makes the decoder underestimate; |v^| <= |v| < b |v^|
    rng = np.random.default_rng(5)
    n = 20000
    v = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    p = oracle.params(b, 128, 2, 10)
    rc, stream = oracle.compress(v, p)
    assert rc == 0
    dense = np.zeros(n, np.float32)
    assert oracle.decompress_accumulate(stream, n, p, dense) == 0
    rc, keys, codes, S = oracle.parse(stream, n, p)
    k = keys.astype(np.int64)
    assert np.all(dense[np.setdiff1d(np.arange(n), k)] == 0.0)
    vh, vo = dense[k].astype(np.float64), v[k].astype(np.float64)
    assert np.all(np.sign(vh) == np.sign(vo))
    ratio = np.abs(vh) / np.abs(vo)
    assert np.all(ratio <= 1.0)
    clamped = np.abs(codes) == 1            # L = 0 raised to 1 may lose one more level
    assert np.all(ratio[~clamped] > 1.0 / b - 1e-6)
    # phases 3-4: v^ = sum / b^L in double, rounded to float
    expect = np.array([S / b ** abs(int(q)) for q in codes])
    assert np.allclose(np.abs(vh), expect, rtol=1e-6, atol=0)


def test_accumulate_adds_workers_in_order():
    rng = np.random.default_rng(6)
    n = 5000
    p = oracle.params(1.08, 128, 2, 8)
    dense = rng.standard_normal(n).astype(np.float32)
    ref = dense.copy()
    for w in range(3):
        v = (rng.standard_normal(n) * 1e-2).astype(np.float32)
        rc, stream = oracle.compress(v, p)
        one = np.zeros(n, np.float32)
        assert oracle.decompress_accumulate(stream, n, p, one) == 0
        ref = ref + one                      # fp32 add, same order
        assert oracle.decompress_accumulate(stream, n, p, dense) == 0
    assert np.array_equal(dense, ref)
