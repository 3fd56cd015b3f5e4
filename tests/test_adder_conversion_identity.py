"""The identity behind the kernels' fast fixed-point conversions, checked in numpy float32 (IEEE
round-to-nearest-even, as the GPU's adder): for |x| < 2^22 the float sum x + 1.5 * 2^23 has the
integer nearest to x (ties to even) in its low mantissa bits, the float with bits 0x4B400000 + i is
1.5 * 2^23 + i, and the range test on the sum's exponent accepts exactly the sums in [2^23, 2^24)."""
import numpy as np

M = np.float32(12582912.0)            # 1.5 * 2^23
BITS = 0x4B400000


def by_adder(x):
    y = (x.astype(np.float32) + M).astype(np.float32)
    b = y.view(np.uint32)
    ok = (b & np.uint32(0xFF800000)) == np.uint32(0x4B000000)
    return (b.astype(np.int64) - BITS), ok


def samples():
    rng = np.random.default_rng(5)
    parts = [rng.uniform(-2.0 ** 22, 2.0 ** 22, 200000), rng.normal(0, 3e4, 200000), rng.normal(0, 2.0, 100000),
             np.arange(-4096, 4096) + 0.5, np.arange(-4096, 4096) * 0.25,
             np.array([0.0, -0.0, 0.5, -0.5, 1.5, 2.5, -1.5, -2.5, 2.0 ** 22 - 1, 2.0 ** 22 - 0.5, -(2.0 ** 22), -(2.0 ** 22) + 0.5,
                       4194303.5, 4194302.5, -4194303.5])]
    return np.concatenate(parts).astype(np.float32)


def test_float_to_nearest_integer_through_the_adder():
    x = samples()
    got, ok = by_adder(x)
    ref = np.rint(x.astype(np.float64)).astype(np.int64)      # numpy rint: ties to even
    inside = np.abs(x.astype(np.float64)) < 2.0 ** 22 - 0.5
    assert ok[inside].all()
    assert np.array_equal(got[ok], ref[ok])
    assert (got[ok] >= -2 ** 22).all() and (got[ok] < 2 ** 22).all()


def test_out_of_range_values_are_sent_to_the_conversion_instruction():
    x = np.array([2.0 ** 22, 2.0 ** 22 + 1, 2.0 ** 23, 1e9, -2.0 ** 22 - 1, -2.0 ** 23, -1e9, np.inf, -np.inf, np.nan, 3e38], np.float32)
    with np.errstate(invalid="ignore", over="ignore"):
        _, ok = by_adder(x)
    assert not ok.any()


def test_integer_to_float_through_the_adder():
    i = np.concatenate([np.arange(-2 ** 22, 2 ** 22, 997), np.array([-2 ** 22, 2 ** 22 - 1, 0, -1, 1])]).astype(np.int64)
    b = (i + BITS).astype(np.uint32)
    assert ((b & np.uint32(0xFF800000)) == np.uint32(0x4B000000)).all()
    f = (b.view(np.float32) - M).astype(np.float32)
    assert np.array_equal(f.astype(np.int64), i) and np.array_equal(f, i.astype(np.float32))
    # outside [-2^22, 2^22) the exponent test fails, also after the 32-bit wrap of the addition
    out = np.array([2 ** 22, 2 ** 22 + 5, -2 ** 22 - 1, 2 ** 30, -2 ** 31, 2 ** 31 - 1], np.int64)
    bo = ((out + BITS) & 0xFFFFFFFF).astype(np.uint32)
    assert not ((bo & np.uint32(0xFF800000)) == np.uint32(0x4B000000)).any()
