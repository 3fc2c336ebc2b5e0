"""Pins for the oracle's number-format code: every 16-bit pattern, every tie."""
from decimal import Decimal
from fractions import Fraction

import numpy as np
import pytest
import torch

import refnum

DTYPES16 = [0, 1]  # bf16, fp16


@pytest.mark.parametrize("dtype", DTYPES16)
def test_decode_all_patterns_matches_library(oracle_lib, dtype):
    bits = np.arange(65536, dtype=np.int64).astype(np.uint16)
    got = oracle_lib.decode16(bits, dtype)
    want = refnum.decode_bits(bits, dtype)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))


@pytest.mark.parametrize("dtype", DTYPES16)
def test_encode_roundtrips_every_pattern(oracle_lib, dtype):
    bits = np.arange(65536, dtype=np.int64).astype(np.uint16)
    vals = refnum.decode_bits(bits, dtype)
    keep = ~np.isnan(vals)
    assert np.array_equal(oracle_lib.encode16_from_f64(vals[keep], dtype), bits[keep])
    assert np.array_equal(oracle_lib.encode16_from_f32(vals[keep].astype(np.float32), dtype), bits[keep])


@pytest.mark.parametrize("dtype", DTYPES16)
def test_every_midpoint_rounds_to_even_and_neighbours_round_to_nearest(oracle_lib, dtype):
    vals, bits = refnum.finite_table(dtype)
    a, b = vals[:-1], vals[1:]
    mid = (a + b) / 2  # exact in float64
    even = np.where((bits[:-1] & 1) == 0, bits[:-1], bits[1:])
    got = oracle_lib.encode16_from_f64(mid, dtype)
    # a tie that lands on zero keeps the sign of the value being rounded
    want = np.where((even == 0) & np.signbit(mid), np.uint16(0x8000), even)
    assert np.array_equal(got, want)
    below = np.nextafter(mid, -np.inf)
    above = np.nextafter(mid, np.inf)
    gb = oracle_lib.encode16_from_f64(below, dtype)
    ga = oracle_lib.encode16_from_f64(above, dtype)
    wb = np.where((bits[:-1] == 0) & np.signbit(below), np.uint16(0x8000), bits[:-1])
    assert np.array_equal(gb, wb)
    wa = np.where((bits[1:] == 0) & np.signbit(above), np.uint16(0x8000), bits[1:])
    assert np.array_equal(ga, wa)


@pytest.mark.parametrize("dtype", DTYPES16)
def test_overflow_threshold(oracle_lib, dtype):
    vals, bits = refnum.finite_table(dtype)
    top, ulp = vals[-1], vals[-1] - vals[-2]
    inf = 0x7F80 if dtype == 0 else 0x7C00
    thr = top + ulp / 2
    probe = np.array([thr, np.nextafter(thr, 0.0), -thr, np.nextafter(-thr, 0.0), 1e300, -1e300,
                      np.inf, -np.inf])
    got = oracle_lib.encode16_from_f64(probe, dtype)
    want = np.array([inf, bits[-1], 0x8000 | inf, 0x8000 | int(bits[-1]), inf, 0x8000 | inf, inf,
                     0x8000 | inf], dtype=np.uint16)
    assert np.array_equal(got, want)


@pytest.mark.parametrize("dtype", DTYPES16)
def test_f32_to_16_matches_library_conversion(oracle_lib, dtype):
    g = np.random.Generator(np.random.Philox(key=[11, dtype]))
    raw = g.integers(0, 2**32, size=1_000_000, dtype=np.uint64).astype(np.uint32)
    f = raw.view(np.float32)
    f = f[~np.isnan(f)]
    # add values concentrated near the format's own range, subnormals included
    extra = (g.standard_normal(200_000) * np.exp(g.uniform(-25, 12, 200_000))).astype(np.float32)
    f = np.concatenate([f, extra])
    want = torch.from_numpy(f).to(refnum.TORCH_16[dtype]).view(torch.int16).numpy().view(np.uint16)
    got = oracle_lib.encode16_from_f32(f, dtype)
    assert np.array_equal(got, want)


@pytest.mark.parametrize("dtype", DTYPES16)
def test_f64_direct_rounding_matches_exact_bracket_search(oracle_lib, dtype):
    g = np.random.Generator(np.random.Philox(key=[12, dtype]))
    v = g.standard_normal(20_000) * np.exp(g.uniform(-110 if dtype == 0 else -22, 14, 20_000))
    got = oracle_lib.encode16_from_f64(v, dtype)
    assert np.array_equal(got, refnum.round_array(v, dtype))
    # a few with exact rational arithmetic as well
    for x in v[:300]:
        assert int(oracle_lib.encode16_from_f64(np.array([x]), dtype)[0]) == refnum.round_exact(Fraction(float(x)), dtype)


def test_direct_rounding_differs_from_rounding_through_binary32(oracle_lib):
    # 1 + 2^-8 is the bf16 tie between 1 and 1 + 2^-7; the 2^-30 breaks the tie upward,
    # but is lost when the value first passes through binary32.
    v = 1.0 + 2.0**-8 + 2.0**-30
    assert int(oracle_lib.encode16_from_f64(np.array([v]), 0)[0]) == 0x3F81
    assert int(oracle_lib.encode16_from_f32(np.array([np.float32(v)]), 0)[0]) == 0x3F80
    assert refnum.round_exact(Decimal(v), 0) == 0x3F81


def test_ulp_compare_pins(oracle_lib):
    c = oracle_lib.compare_y
    u16 = lambda *a: np.array(a, dtype=np.uint16)
    assert c(u16(0x0000), u16(0x8000), 0) == (0, 0)          # +0 == -0
    assert c(u16(0x3F80), u16(0x3F81), 0) == (1, 0)
    assert c(u16(0x0001), u16(0x8001), 1) == (2, 0)          # across zero
    assert c(u16(0x3C00), u16(0x3C03), 1) == (3, 1)
    assert c(u16(0x7FC0), u16(0x7FC1), 0) == (0, 0)          # NaN vs NaN
    assert c(u16(0x7FC0), u16(0x3F80), 0)[1] == 1
    # the lattice is that of the finite values: an overflowed output is not one step from the largest finite value
    assert c(u16(0x7BFF), u16(0x7C00), 1) == (65535, 1)      # fp16 max finite vs +inf
    assert c(u16(0x7F7F), u16(0x7F80), 0) == (65535, 1)      # bf16 max finite vs +inf
    assert c(u16(0x7C00), u16(0x7C00), 1) == (0, 0)          # +inf vs +inf
    assert c(u16(0x7C00), u16(0xFC00), 1) == (65535, 1)      # +inf vs -inf
    assert c(u16(0xFF80), u16(0xFF80), 0) == (0, 0)          # -inf vs -inf (bf16)
    assert c(u16(0x7BFF), u16(0x7BFE), 1) == (1, 0)          # the two largest finite values stay adjacent
    worst, bad = c(np.array([1.0, 2.0, 0.0], np.float32), np.array([1.0, 2.00001, 0.0], np.float32))
    assert bad == 0 and 4e-6 < worst < 6e-6
    worst, bad = c(np.array([1.0], np.float32), np.array([1.0001], np.float32))
    assert bad == 1
    inf = float("inf")
    worst, bad = c(np.array([3.4e38, inf, inf], np.float32), np.array([inf, inf, -inf], np.float32))
    assert bad == 2 and worst == inf                          # binary32: an infinity matches only itself
    assert oracle_lib.bit_mismatches(u16(1, 2, 3), u16(1, 2, 4), 0) == 1
