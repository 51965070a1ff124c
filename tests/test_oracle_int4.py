"""Pins of the oracle's 4-bit group-wise weights (Section 6 outlook): the same Q as Eq. 6 with range [-7, 7]."""
import numpy as np

from oracle import quasar_oracle as qo


def test_hand_rows_and_zero_group():
    row = np.zeros((1, 256), np.float32)
    row[0, :4] = [-7, 3.5, 2.5, 7]                 # first group: delta = 7/7 = 1; ties go to even: 4 and 2
    row[0, 128:132] = [7 / 16, -3.5 / 16, 1.5 / 16, 0.8 / 16]   # second group: delta = (7/16)/7 = 2^-4 exactly
    q, d = qo.quantize_int4(row)
    assert list(q[0, :4]) == [-7, 4, 2, 7] and d[0, 0] == np.float32(1.0)
    assert d[0, 1] == np.float32(2.0 ** -4)
    assert list(q[0, 128:132]) == [7, -4, 2, 1]   # -3.5 -> -4 and 1.5 -> 2 (ties to even); 0.8 -> 1
    z, dz = qo.quantize_int4(np.zeros((2, 128), np.float32))
    assert np.all(z == 0) and np.all(dz == 1.0)


def test_error_bound_range_and_idempotence():
    rng = np.random.default_rng(0)
    w = qo.bf16_round(rng.normal(size=(33, 512)) * 0.02).astype(np.float32)
    q, d = qo.quantize_int4(w)
    assert q.min() >= -7 and q.max() <= 7
    assert np.all(np.abs(q.reshape(33, 4, 128)).max(2) == 7)
    deq = q.reshape(33, 4, 128).astype(np.float64) * d.astype(np.float64)[:, :, None]
    err = np.abs(w.reshape(33, 4, 128).astype(np.float64) - deq)
    assert np.all(err <= d.astype(np.float64)[:, :, None] * (0.5 + 2.0 ** -22))
    q2, d2 = qo.quantize_int4(deq.reshape(33, 512).astype(np.float32))
    assert np.array_equal(q, q2) and np.array_equal(d, d2)


def test_pack_unpack_round_trip_and_nibble_order():
    codes = np.array([[-7, 7, 0, -1, 3, -8, 1, 2]], np.int8)
    p = qo.pack_int4(codes)
    assert list(p[0]) == [0x79, 0xF0, 0x83, 0x21]     # low nibble = even channel, two's complement nibbles
    assert np.array_equal(qo.unpack_int4(p), codes)
    rng = np.random.default_rng(1)
    c = rng.integers(-7, 8, (5, 256)).astype(np.int8)
    assert np.array_equal(qo.unpack_int4(qo.pack_int4(c)), c)


def test_linear_against_the_dequantised_product():
    rng = np.random.default_rng(2)
    w = qo.bf16_round(rng.normal(size=(10, 384)) * 0.02).astype(np.float32)
    x = qo.bf16_round(rng.normal(size=(3, 384)))
    q, d = qo.quantize_int4(w)
    deq = (q.reshape(10, 3, 128).astype(np.float64) * d.astype(np.float64)[:, :, None]).reshape(10, 384)
    y = qo.linear_int4(x, q, d)
    ref = np.zeros((3, 10))
    for m in range(3):
        for n in range(10):
            for k in range(384):
                ref[m, n] += x[m, k] * deq[n, k]
    assert np.allclose(y, ref, rtol=1e-12, atol=1e-14)
    # the result is within the quantisation bound of the full-precision product
    exact = x @ w.astype(np.float64).T
    bound = np.abs(x) @ np.repeat(d.astype(np.float64), 128, axis=1).T * 0.5
    assert np.all(np.abs(y - exact) <= bound * (1 + 1e-6))
