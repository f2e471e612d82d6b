"""Pins for the oracle's binary16 codec (CPU only).

The codec is checked against things other than itself: values fixed by the IEEE
format definition (tests/golden/*.txt), numpy's independent float16
implementation over all 65536 bit patterns, and the host CPU's own conversion
(struct 'e' format) on random probes.
"""
import os
import struct

import numpy as np

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                yield line


def test_decode_known_values(oracle_lib):
    for line in _rows("f16_known_values.txt"):
        h, expr = line.split(None, 1)
        want = float(eval(expr))
        got = float(oracle_lib.f16_bits_to_f64(np.array([int(h, 16)], dtype=np.uint16))[0])
        assert got == want and np.signbit(got) == np.signbit(want), (h, got, want)


def test_decode_exhaustive_vs_numpy(oracle_lib):
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    got = oracle_lib.f16_bits_to_f64(bits)
    want = bits.view(np.float16).astype(np.float64)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))
    # NaN patterns are exactly exponent 31 with a non-zero fraction
    assert nan.sum() == 2 * 1023


def test_encode_golden_rounding(oracle_lib):
    for line in _rows("f64_to_f16_rounding.txt"):
        expr, h = line.rsplit(None, 1)
        got = int(oracle_lib.f64_to_f16_bits(np.array([float(eval(expr))]))[0])
        assert got == int(h, 16), (expr, hex(got), h)


def test_encode_roundtrip_all_patterns(oracle_lib):
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    vals = oracle_lib.f16_bits_to_f64(bits)
    keep = ~np.isnan(vals)
    back = oracle_lib.f64_to_f16_bits(vals[keep])
    assert np.array_equal(back, bits[keep])


def test_encode_midpoints_and_neighbours(oracle_lib):
    """Every midpoint between adjacent finite binary16 values rounds to the even neighbour;
    a nudge either way rounds to the nearer one."""
    bits = np.arange(0, 0x7bff, dtype=np.uint16)          # positive finite, excluding the largest
    lo = oracle_lib.f16_bits_to_f64(bits)
    hi = oracle_lib.f16_bits_to_f64(bits + 1)
    mid = (lo + hi) / 2                                    # exact in fp64
    even = np.where(bits & 1, bits + 1, bits).astype(np.uint16)
    assert np.array_equal(oracle_lib.f64_to_f16_bits(mid), even)
    assert np.array_equal(oracle_lib.f64_to_f16_bits(np.nextafter(mid, 0.0)), bits)
    assert np.array_equal(oracle_lib.f64_to_f16_bits(np.nextafter(mid, np.inf)), bits + 1)
    assert np.array_equal(oracle_lib.f64_to_f16_bits(-mid), even | 0x8000)


def test_encode_random_vs_numpy_and_struct(oracle_lib):
    rng = np.random.default_rng(12345)
    x = np.concatenate([
        rng.uniform(-70000, 70000, 20000),
        rng.uniform(-1, 1, 20000),
        rng.uniform(-1, 1, 20000) * 2.0 ** rng.integers(-30, 0, 20000),
    ])
    got = oracle_lib.f64_to_f16_bits(x)
    with np.errstate(over="ignore"):
        want = x.astype(np.float16).view(np.uint16)       # numpy: one correctly rounded step
    assert np.array_equal(got, want)
    for v, g in zip(x[::997], got[::997]):
        try:
            w = struct.unpack("<H", struct.pack("<e", v))[0]
        except OverflowError:
            w = 0x7c00 | (0x8000 if v < 0 else 0)
        assert int(g) == w
