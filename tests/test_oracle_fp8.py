"""Pins of the fp8-output variant's oracle: the e4m3 codec exhaustively, and the operator's closed forms."""
import math

import numpy as np
import pytest
import torch

TD = {0: torch.bfloat16, 1: torch.float16, 2: torch.float32}


def _library_table():
    """All 256 e4m3 patterns decoded by torch's own conversion."""
    bits = torch.arange(256, dtype=torch.int16).to(torch.uint8)
    return bits.numpy(), bits.view(torch.float8_e4m3fn).to(torch.float64).numpy()


def test_decode_all_patterns_matches_library(oracle_lib):
    bits, want = _library_table()
    got = oracle_lib.decode_e4m3(bits)
    nan = np.isnan(want)
    assert nan.sum() == 2 and np.array_equal(np.isnan(got), nan)       # 0x7F and 0xFF only
    assert np.array_equal(got[~nan], want[~nan]) and np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))
    assert got[0x7E] == 448.0 and got[0x01] == 2.0**-9 and got[0x08] == 2.0**-6


def test_encode_roundtrip_midpoints_and_saturation(oracle_lib):
    bits, vals = _library_table()
    finite = ~np.isnan(vals)
    assert np.array_equal(oracle_lib.encode_e4m3(vals[finite]), bits[finite])
    pos = np.sort(vals[finite & (bits < 0x80)])                          # 0 ... 448
    pos_bits = oracle_lib.encode_e4m3(pos)
    mid = (pos[:-1] + pos[1:]) / 2
    even = np.where((pos_bits[:-1] & 1) == 0, pos_bits[:-1], pos_bits[1:])
    assert np.array_equal(oracle_lib.encode_e4m3(mid), even)
    assert np.array_equal(oracle_lib.encode_e4m3(np.nextafter(mid, np.inf)), pos_bits[1:])
    assert np.array_equal(oracle_lib.encode_e4m3(np.nextafter(mid, -np.inf)), pos_bits[:-1])
    assert np.array_equal(oracle_lib.encode_e4m3(-mid), even | 0x80)
    # saturation: everything from 448 upwards, including the tie 464 that would round to "512", is 0x7E
    sat = oracle_lib.encode_e4m3(np.array([448.0, 450.0, 464.0, 480.0, 1e9, np.inf, -1e9]))
    assert sat.tolist() == [0x7E, 0x7E, 0x7E, 0x7E, 0x7E, 0x7E, 0xFE]
    assert (oracle_lib.encode_e4m3(np.array([np.nan]))[0] & 0x7F) == 0x7F
    assert oracle_lib.encode_e4m3(np.array([2.0**-11, -2.0**-12, 0.0])).tolist() == [0x00, 0x80, 0x00]  # ties to even, tiny


def test_compare_e4m3_pins(oracle_lib):
    a = np.array([0x00, 0x38, 0x7E, 0x81, 0x7F], dtype=np.uint8)
    b = np.array([0x80, 0x39, 0x7C, 0x01, 0xFF], dtype=np.uint8)
    assert oracle_lib.compare_e4m3(a, b, tol_steps=1) == (2, 2)  # +0 == -0; 1 step; 2 steps; across zero 2 steps; NaN == NaN


@pytest.mark.parametrize("dtype", [0, 1, 2])
def test_operator_closed_forms(oracle_lib, dtype):
    H, c, eps = 40, 1.5, 0.25
    w = torch.linspace(-2.0, 2.0, H, dtype=torch.float64).to(TD[dtype])
    x = torch.full((2, H), c / 2, dtype=torch.float64).to(TD[dtype])
    q, scale, ro = oracle_lib.add_rmsnorm_fp8(x, x, w, eps)
    y = w.double().numpy() * c / math.sqrt(c * c + eps)                  # constant row, as for the plain operator
    sc = np.abs(y).max() / 448.0
    assert np.array_equal(scale.numpy(), np.full(2, np.float32(sc)))
    assert np.array_equal(q.numpy()[0], oracle_lib.encode_e4m3(y / sc)) and np.array_equal(q.numpy()[0], q.numpy()[1])
    assert int(q[0, 0]) == 0xFE and int(q[0, -1]) == 0x7E                # the extremes of w map to -448 and +448
    assert np.all(ro.double().numpy() == c)
    # one-hot row: that element is +-448, everything else is zero; the scale carries the magnitude
    xo = torch.zeros(1, 24, dtype=TD[dtype]); xo[0, 5] = -3.0
    q, scale, _ = oracle_lib.add_rmsnorm_fp8(xo, torch.zeros_like(xo), torch.ones(24, dtype=TD[dtype]), eps)
    want = np.zeros(24, dtype=np.uint8); want[5] = 0xFE
    assert np.array_equal(q.numpy()[0] & 0x7F | (q.numpy()[0] & 0x80) * (q.numpy()[0] != 0x80), want)
    assert abs(float(scale[0]) - 3.0 / math.sqrt(9.0 / 24 + eps) / 448.0) < 1e-9
    # a row of zeros: the floor keeps the scale positive and the codes zero
    z = torch.zeros(1, 8, dtype=TD[dtype])
    q, scale, _ = oracle_lib.add_rmsnorm_fp8(z, z, torch.ones(8, dtype=TD[dtype]), 1e-6)
    assert float(scale[0]) == float(np.float32(1e-12 / 448.0)) and np.all((q.numpy() & 0x7F) == 0)


@pytest.mark.parametrize("dtype", [0, 1, 2])
def test_dequantised_output_reproduces_the_plain_oracle(oracle_lib, dtype):
    from paper_2601_12698_b200 import synth
    name = {0: "bf16", 1: "fp16", 2: "fp32"}[dtype]
    x, r, w = synth.make_inputs(33, 1000, name, seed=17)
    q, scale, ro = oracle_lib.add_rmsnorm_fp8(x, r, w, 1e-6)
    y_plain, r_plain = oracle_lib.add_rmsnorm(x, r, w, 1e-6)
    assert torch.equal(ro, r_plain)                                      # the residual output is the same contract
    s = (x.float() + r.float()).double()   # the binary32 sum, as the operator defines it
    y64 = s * torch.rsqrt(s.pow(2).mean(-1, keepdim=True) + float(np.float32(1e-6))) * w.double()
    amax = y64.abs().amax(-1)
    assert torch.allclose(scale.double(), amax / 448.0, rtol=1.2e-7, atol=0)   # binary32 storage of the scale
    deq = torch.from_numpy(oracle_lib.decode_e4m3(q.numpy())) * (amax / 448.0)[:, None]
    # half an e4m3 step: 2^-4 relative for normal codes, half the subnormal quantum (2^-10 of the scale) below
    step = torch.maximum(y64.abs() * 2.0**-4, (amax / 448.0)[:, None] * 2.0**-10)
    assert bool(((deq - y64).abs() <= step * (1 + 1e-9)).all())
    assert bool((q.view(-1).to(torch.int32) & 0x7F).max() == 0x7E)       # every row reaches full scale
    # library cross-check of the codes: torch's own e4m3 conversion of y/scale (no value exceeds 448 here)
    lib_codes = (y64 / (amax / 448.0)[:, None]).to(torch.float32).to(torch.float8_e4m3fn).view(torch.uint8)
    assert oracle_lib.compare_e4m3(q, lib_codes, tol_steps=0)[1] <= q.numel() // 2000  # fp32 pre-rounding may flip ties
    assert oracle_lib.compare_e4m3(q, lib_codes, tol_steps=1)[1] == 0
