"""Pins of the silu_and_mul oracle: closed forms, the row layout, exact evaluation, a library evaluation."""
import math
from decimal import Decimal, getcontext

import numpy as np
import pytest
import torch

import refnum

getcontext().prec = 80
TD = {0: torch.bfloat16, 1: torch.float16, 2: torch.float32}


def _bits(t, dtype):
    return t.numpy() if dtype == 2 else t.view(torch.int16).numpy().view(np.uint16)


def _expect(v64, dtype):
    v64 = np.asarray(v64, dtype=np.float64)
    return v64.astype(np.float32) if dtype == 2 else refnum.round_array(v64, dtype)


def _row(gate, up, dtype):
    return torch.tensor([list(gate) + list(up)], dtype=torch.float64).to(TD[dtype])


@pytest.mark.parametrize("dtype", [0, 1, 2])
def test_closed_forms(oracle_lib, dtype):
    # silu(0) = 0 whatever the value half holds; a zero value half gives zero
    out = oracle_lib.silu_and_mul(_row([0.0, 0.0, 2.0], [5.0, -3.0, 0.0], dtype))
    assert np.all(out.double().numpy() == 0.0)
    # large gates: silu(g) = g exactly in fp64 once exp(-g) < 2^-53, so out = g * u rounded once
    x = _row([40.0, 64.0, 100.0], [0.5, -3.0, 1.25], dtype)
    want = x[0, :3].double().numpy() * x[0, 3:].double().numpy()
    assert np.array_equal(_bits(oracle_lib.silu_and_mul(x), dtype)[0], _expect(want, dtype))
    # very negative gates: silu(g) -> -0
    out = oracle_lib.silu_and_mul(_row([-800.0], [1.0], dtype))
    assert float(out[0, 0]) == 0.0
    # silu(g) - silu(-g) = g: checked in fp32 storage where rounding is fine enough to see it
    if dtype == 2:
        g = np.linspace(-12.0, 12.0, 97)
        pos = oracle_lib.silu_and_mul(_row(g, np.ones_like(g), dtype)).double().numpy()[0]
        neg = oracle_lib.silu_and_mul(_row(-g, np.ones_like(g), dtype)).double().numpy()[0]
        assert np.allclose(pos - neg, g.astype(np.float32).astype(np.float64), rtol=0, atol=2e-6)
        # silu(ln 3) = ln 3 / (1 + 1/3) = 0.75 ln 3
        ln3 = float(np.float32(math.log(3.0)))
        v = float(oracle_lib.silu_and_mul(_row([ln3], [1.0], dtype))[0, 0])
        assert abs(v - ln3 / (1 + math.exp(-ln3))) <= 2.0**-24 * v
        assert abs(v - 0.75 * math.log(3.0)) < 2e-7


@pytest.mark.parametrize("dtype", [0, 1, 2])
def test_which_half_is_the_gate_and_rows_do_not_mix(oracle_lib, dtype):
    # gate = 50 (silu = identity), value = 2  ->  100; swapped halves would give silu(2) * 50 = 88.08
    x = _row([50.0, 50.0], [2.0, 2.0], dtype)
    assert oracle_lib.silu_and_mul(x).double().tolist() == [[100.0, 100.0]]
    g = np.random.Generator(np.random.Philox(key=[51, dtype]))
    x = torch.from_numpy(g.standard_normal((5, 14)) * 3).to(TD[dtype])
    full = oracle_lib.silu_and_mul(x)
    for t in range(5):
        assert np.array_equal(_bits(oracle_lib.silu_and_mul(x[t:t + 1].contiguous()), dtype)[0], _bits(full, dtype)[t])
    # column j of the output depends on columns j and d + j only
    y = x.clone(); y[:, 3] = 0
    changed = (_bits(oracle_lib.silu_and_mul(y), dtype) != _bits(full, dtype)).any(0)
    assert changed.tolist() == [False, False, False, True, False, False, False]
    assert oracle_lib.silu_and_mul(x, threads=3).equal(full)


@pytest.mark.parametrize("dtype", [0, 1, 2])
def test_tiny_shapes_against_80_digit_arithmetic(oracle_lib, dtype):
    g = np.random.Generator(np.random.Philox(key=[52, dtype]))
    x = torch.from_numpy(g.standard_normal((3, 8)) * np.array([0.01, 1.0, 20.0])[:, None]).to(TD[dtype])
    out = oracle_lib.silu_and_mul(x)
    xs = x.double().numpy()
    for t in range(3):
        for j in range(4):
            gd, ud = Decimal(float(xs[t, j])), Decimal(float(xs[t, 4 + j]))
            exact = gd / (1 + (-gd).exp()) * ud
            if dtype == 2:
                got = float(out[t, j])
                lo, hi = np.nextafter(np.float32(got), np.float32(-np.inf)), np.nextafter(np.float32(got), np.float32(np.inf))
                err = abs(Decimal(got) - exact)
                assert err <= abs(Decimal(float(lo)) - exact) and err <= abs(Decimal(float(hi)) - exact)
            else:
                assert (int(out.view(torch.int16)[t, j]) & 0xFFFF) == refnum.round_exact(exact, dtype)


@pytest.mark.parametrize("dtype,T,d", [(0, 64, 1376), (1, 9, 11008), (2, 7, 4096)])
def test_float64_library_evaluation(oracle_lib, dtype, T, d):
    g = np.random.Generator(np.random.Philox(key=[53, dtype]))
    x = torch.from_numpy(g.standard_normal((T, 2 * d)) * 2.5).to(TD[dtype])
    out = oracle_lib.silu_and_mul(x, threads=4)
    xd = x.double()
    want = torch.nn.functional.silu(xd[:, :d]) * xd[:, d:]
    if dtype == 2:
        rel = ((out.double() - want).abs() / want.abs().clamp_min(1e-300)).max().item()
        assert rel <= 2.0**-24 * (1 + 1e-6)
    else:
        got = _bits(out, dtype)
        exp = refnum.round_array(want.numpy(), dtype)
        assert np.count_nonzero(got != exp) <= max(1, got.size // 100_000)
        assert oracle_lib.compare_y(got, exp, dtype)[0] <= 1


def test_argument_checks(oracle_lib):
    assert oracle_lib.silu_and_mul(torch.zeros(0, 8)).shape == (0, 4)
    with pytest.raises(ValueError):
        oracle_lib.silu_and_mul(torch.zeros(2, 7))
