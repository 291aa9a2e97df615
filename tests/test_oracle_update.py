"""Pins of the oracle's model update on decoded coordinates (Sec. 4.1: the two Adam equations
as printed, applied where the aggregated decoded gradient is non-zero).  Streams are built with
b = 2 and sum = 1, so that a code L decodes to exactly 2^-L."""
import numpy as np

import oracle


def _stream(keys, codes, n, po):
    rc, s = oracle.write_stream(np.array(keys, np.uint64), np.array(codes, np.int32), n, 1.0, po)
    assert rc == 0
    return s


def test_worked_example_with_exactly_representable_numbers():
    # g = 2^-1 at key 3.  beta1 = 1/2, m = 1/4: m' = 1/8 + 1/4 = 3/8.  beta2 = 3/4, v = 1/4:
    # v' = 3/16 + 1/4 * 1/4 = 1/4, sqrt = 1/2.  lr = 1/8: theta' = 1 - (1/8) / (1/2) * 3/8 = 1 - 3/32.
    po = oracle.params(2.0, 8, 2, 14)
    n = 40
    s = _stream([3], [1], n, po)
    theta, m, v = np.ones(n, np.float32), np.full(n, 0.25, np.float32), np.full(n, 0.25, np.float32)
    assert oracle.sparse_adam_update([s], n, po, 0.125, 0.5, 0.75, 0.0, theta, m, v) == 0
    assert theta[3] == np.float32(1.0 - 3.0 / 32.0) and m[3] == np.float32(0.375) and v[3] == np.float32(0.25)
    others = np.arange(n) != 3
    assert np.all(theta[others] == 1.0) and np.all(m[others] == 0.25) and np.all(v[others] == 0.25)


def test_streams_add_up_before_the_update_and_cancelled_coordinates_stay():
    po = oracle.params(2.0, 8, 2, 14)
    n = 100
    s1 = _stream([3, 7, 50], [1, -2, 3], n, po)       # +1/2, -1/4, +1/8
    s2 = _stream([7, 9, 50], [2, 3, 3], n, po)        # +1/4, +1/8, +1/8
    theta, m, v = np.zeros(n, np.float32), np.zeros(n, np.float32), np.zeros(n, np.float32)
    # beta1 = beta2 = 0, eps = 0: m' = g, v' = g^2, theta' = theta - lr * g / |g| = -lr * sign(g)
    assert oracle.sparse_adam_update([s1, s2], n, po, 0.5, 0.0, 0.0, 0.0, theta, m, v) == 0
    g = np.zeros(n, np.float32)
    g[3], g[9], g[50] = 0.5, 0.125, 0.25              # key 7: -1/4 + 1/4 = 0, untouched
    assert np.array_equal(m, g) and np.array_equal(v, g * g)
    assert np.array_equal(theta, np.where(g != 0, -0.5 * np.sign(g), 0).astype(np.float32))


def test_sign_descent_special_case_on_a_compressed_gradient():
    # with beta1 = beta2 = 0 and eps = 0 every touched coordinate moves by lr (up to rounding) against the sign of
    # its decoded value (sqrt(fl(g*g)) == |g| in IEEE arithmetic, no under- or overflow here); the touched set
    # is the set of kept keys, and m equals the decoded gradient bit for bit
    rng = np.random.default_rng(5)
    n = 50_000
    grad = (rng.standard_normal(n) * 1e-2).astype(np.float32)
    base = float(np.exp(np.log(np.abs(grad.astype(np.float64)).sum() / np.sort(np.abs(grad))[-n // 100]) / 128.0))
    po = oracle.params(base)
    rc, s = oracle.compress(grad, po)
    assert rc == 0
    rc, keys, codes, S = oracle.parse(s, n, po)
    theta = rng.standard_normal(n).astype(np.float32)
    theta0 = theta.copy()
    m, v = np.zeros(n, np.float32), np.zeros(n, np.float32)
    lr = np.float32(0.03125)
    assert oracle.sparse_adam_update([s], n, po, float(lr), 0.0, 0.0, 0.0, theta, m, v) == 0
    touched = np.zeros(n, bool)
    touched[keys.astype(np.int64)] = True
    assert 0 < touched.sum() < n // 50
    assert np.array_equal(theta[~touched], theta0[~touched]) and not m[~touched].any() and not v[~touched].any()
    sgn = np.sign(codes).astype(np.float32)
    # (lr / |g|) * g is lr up to two roundings, and the subtraction rounds once more
    k = keys.astype(np.int64)
    step = theta0[k].astype(np.float64) - theta[k].astype(np.float64)
    assert np.all(np.abs(step - float(lr) * sgn) <= float(lr) * 2.0 ** -22 + np.abs(theta0[k]) * 2.0 ** -23)
    dense = np.zeros(n, np.float32)
    assert oracle.decompress_accumulate(s, n, po, dense) == 0
    assert np.array_equal(m, dense)


def test_beta1_one_keeps_the_first_moment_and_errors_update_nothing():
    po = oracle.params(2.0, 8, 2, 14)
    n = 64
    s = _stream([5, 6], [2, -1], n, po)
    theta, m, v = np.zeros(n, np.float32), np.full(n, 0.5, np.float32), np.zeros(n, np.float32)
    assert oracle.sparse_adam_update([s], n, po, 1.0, 1.0, 0.0, 0.0, theta, m, v) == 0
    assert np.all(m == 0.5)                               # 1 * m + 0 * g
    assert theta[5] == np.float32(-0.5 / 0.25) and theta[6] == np.float32(-0.5 / 0.5)
    bad = s.copy()
    bad[0] ^= 0xFF                                        # magic
    t2, m2, v2 = np.zeros(n, np.float32), np.zeros(n, np.float32), np.zeros(n, np.float32)
    assert oracle.sparse_adam_update([s, bad], n, po, 1.0, 0.5, 0.5, 0.0, t2, m2, v2) != 0
    assert not t2.any() and not m2.any() and not v2.any()


def test_key_value_input_has_the_dense_vectors_stream_and_the_plain_sum():
    # values that are powers of two: the sum is exact in any order, so the header's sum is the plain total
    po = oracle.params(2.0, 16, 2, 14)
    n = 3 * 16384 + 9
    keys = np.array([0, 5, 16383, 16384, 40000, n - 1], np.uint64)
    vals = np.array([0.5, -0.25, 2.0, 0.0, -8.0, 1.0], np.float32)
    rc, s = oracle.compress_kv(keys, vals, n, po)
    assert rc == 0
    dense = np.zeros(n, np.float32)
    dense[keys.astype(np.int64)] = vals
    rc2, s2 = oracle.compress(dense, po)
    assert rc2 == 0 and np.array_equal(s, s2)
    rc3, pk, pc, S = oracle.parse(s, n, po)
    assert rc3 == 0 and S == 11.75
    assert set(pk.tolist()) <= set(keys[vals != 0].tolist())          # a zero value is never kept
    # order and range of the keys are part of the contract
    assert oracle.compress_kv(np.array([5, 5], np.uint64), np.ones(2, np.float32), n, po)[0] != 0
    assert oracle.compress_kv(np.array([7, 3], np.uint64), np.ones(2, np.float32), n, po)[0] != 0
    assert oracle.compress_kv(np.array([n], np.uint64), np.ones(1, np.float32), n, po)[0] != 0
    rc4, s4 = oracle.compress_kv(np.zeros(0, np.uint64), np.zeros(0, np.float32), n, po)
    assert rc4 == 0 and np.array_equal(s4, oracle.compress(np.zeros(n, np.float32), po)[1])
