"""Closed forms and invariants that pin the oracle's operator arithmetic.

Each case is chosen so that one plausible mistake fails it: eps outside the square
root, division by H-1, a missing weight, a weight indexed by row, the rounded
residual used where the un-rounded one belongs, a dropped residual term.
"""
import math

import numpy as np
import pytest
import torch

import refnum

EPS_BIG = 0.25  # exactly representable; large enough that its placement changes every output bit


def _t(a, dtype):
    return torch.tensor(a, dtype=torch.float64).to({0: torch.bfloat16, 1: torch.float16, 2: torch.float32}[dtype])


def _vals(t):
    return t.to(torch.float64).numpy()


def _expect(y64, dtype):
    """Round expected float64 values to the output dtype without the oracle's codec."""
    y64 = np.asarray(y64, dtype=np.float64)
    if dtype == 2:
        return y64.astype(np.float32)
    return refnum.round_array(y64, dtype)


def _bits(t, dtype):
    if dtype == 2:
        return t.numpy()
    return t.view(torch.int16).numpy().view(np.uint16)


@pytest.mark.parametrize("dtype", [0, 1, 2])
@pytest.mark.parametrize("c", [1.5, -3.0, 0.0078125])
def test_constant_row(oracle_lib, dtype, c):
    H = 37
    x = _t(np.full((2, H), 0.5 * c), dtype)
    r = _t(np.full((2, H), 0.5 * c), dtype)  # halves are exact, so s == c exactly
    w = _t(np.linspace(-2.0, 2.0, H), dtype)
    y, ro = oracle_lib.add_rmsnorm(x, r, w, EPS_BIG)
    assert np.array_equal(_vals(ro), np.full((2, H), c))
    want = _vals(w)[None, :] * c / math.sqrt(c * c + EPS_BIG)
    assert np.array_equal(_bits(y, dtype), _expect(np.repeat(want, 2, 0), dtype))
    # sign(c) * |c| form of the same statement
    want2 = _vals(w) * math.copysign(1.0, c) * abs(c) / math.sqrt(c * c + EPS_BIG)
    assert np.array_equal(_bits(y, dtype)[0], _expect(want2, dtype))


@pytest.mark.parametrize("dtype", [0, 1, 2])
def test_one_hot_row_divides_by_h(oracle_lib, dtype):
    H, k, a = 24, 5, 3.0
    x = np.zeros((1, H)); x[0, k] = a
    w = np.linspace(0.5, 1.5, H)
    y, ro = oracle_lib.add_rmsnorm(_t(x, dtype), _t(np.zeros((1, H)), dtype), _t(w, dtype), EPS_BIG)
    want = np.zeros(H)
    want[k] = _vals(_t(w, dtype))[k] * a / math.sqrt(a * a / H + EPS_BIG)
    assert np.array_equal(_bits(y, dtype)[0], _expect(want, dtype))
    assert np.array_equal(_vals(ro)[0], x[0])


@pytest.mark.parametrize("dtype", [0, 1, 2])
def test_x_equals_minus_r_gives_positive_zero_residual_and_zero_output(oracle_lib, dtype):
    g = np.random.Generator(np.random.Philox(key=[21, dtype]))
    x = _t(g.standard_normal((3, 19)), dtype)
    w = _t(g.standard_normal(19), dtype)
    y, ro = oracle_lib.add_rmsnorm(x, -x, w, 1e-6)
    if dtype == 2:
        assert np.array_equal(ro.numpy().view(np.uint32), np.zeros((3, 19), np.uint32))
    else:
        assert np.array_equal(_bits(ro, dtype), np.zeros((3, 19), np.uint16))
    assert np.all(_vals(y) == 0.0)


@pytest.mark.parametrize("dtype", [0, 1, 2])
def test_alternating_unit_row_has_unit_mean_square(oracle_lib, dtype):
    H = 50
    s = np.where(np.arange(H) % 2 == 0, 1.0, -1.0)
    w = np.linspace(0.25, 4.0, H)
    y, _ = oracle_lib.add_rmsnorm(_t(s[None] * 0.75, dtype), _t(s[None] * 0.25, dtype), _t(w, dtype), EPS_BIG)
    want = _vals(_t(w, dtype)) * s / math.sqrt(1.0 + EPS_BIG)
    assert np.array_equal(_bits(y, dtype)[0], _expect(want, dtype))


def test_unit_weight_rows_have_rms_close_to_one(oracle_lib):
    g = np.random.Generator(np.random.Philox(key=[22, 0]))
    x = torch.from_numpy(g.standard_normal((16, 4096)).astype(np.float32))
    r = torch.from_numpy(g.standard_normal((16, 4096)).astype(np.float32))
    eps = 1e-6
    y, _ = oracle_lib.add_rmsnorm(x, r, torch.ones(4096), eps)
    s = x.double() + r.double()
    ms = (s * s).mean(-1)
    rms_y = y.double().pow(2).mean(-1).sqrt()
    want = (ms / (ms + float(np.float32(eps)))).sqrt()
    assert torch.allclose(rms_y, want, rtol=1e-7, atol=0)
    assert torch.all((rms_y - 1).abs() < 1e-6)


@pytest.mark.parametrize("dtype", [0, 1, 2])
@pytest.mark.parametrize("k", [-3, 4])
def test_power_of_two_scale_invariance_without_eps(oracle_lib, dtype, k):
    g = np.random.Generator(np.random.Philox(key=[23, dtype]))
    x = _t(g.standard_normal((4, 33)), dtype)
    r = _t(g.standard_normal((4, 33)), dtype)
    w = _t(g.standard_normal(33), dtype)
    y0, r0 = oracle_lib.add_rmsnorm(x, r, w, 0.0)
    y1, r1 = oracle_lib.add_rmsnorm(x * 2.0**k, r * 2.0**k, w, 0.0)
    assert np.array_equal(_bits(y0, dtype), _bits(y1, dtype))
    assert np.array_equal(_vals(r0) * 2.0**k, _vals(r1))


@pytest.mark.parametrize("dtype", [0, 1, 2])
def test_rows_are_independent_and_columns_permute(oracle_lib, dtype):
    g = np.random.Generator(np.random.Philox(key=[24, dtype]))
    T, H = 7, 45
    x, r, w = _t(g.standard_normal((T, H)), dtype), _t(g.standard_normal((T, H)), dtype), _t(g.standard_normal(H), dtype)
    y, ro = oracle_lib.add_rmsnorm(x, r, w, 1e-6)
    # each row alone, and rows in reverse order
    for t in range(T):
        yt, rt = oracle_lib.add_rmsnorm(x[t:t + 1], r[t:t + 1], w, 1e-6)
        assert np.array_equal(_bits(yt, dtype)[0], _bits(y, dtype)[t])
        assert np.array_equal(_bits(rt, dtype)[0], _bits(ro, dtype)[t])
    yr, _ = oracle_lib.add_rmsnorm(x.flip(0), r.flip(0), w, 1e-6)
    assert np.array_equal(_bits(yr, dtype), _bits(y, dtype)[::-1])
    # permuting columns of x, r and w together permutes y (fp64 sum order changes: allow 1 ulp, rarely)
    p = torch.from_numpy(g.permutation(H))
    yp, rp = oracle_lib.add_rmsnorm(x[:, p].contiguous(), r[:, p].contiguous(), w[p].contiguous(), 1e-6)
    assert np.array_equal(_bits(rp, dtype), _bits(ro[:, p].contiguous(), dtype))
    worst, bad = oracle_lib.compare_y(yp, y[:, p].contiguous(), tol_ulp=1, tol_rel=2e-7)
    assert bad == 0


@pytest.mark.parametrize("dtype", [0, 1])
def test_residual_is_fp32_add_then_one_rounding_to_dtype(oracle_lib, dtype):
    """r' is the binary32 sum (library addition) rounded once more to the dtype."""
    g = np.random.Generator(np.random.Philox(key=[25, dtype]))
    x = _t(g.standard_normal((64, 512)) * np.exp(g.uniform(-8, 8, (64, 512))), dtype)
    r = _t(g.standard_normal((64, 512)) * np.exp(g.uniform(-8, 8, (64, 512))), dtype)
    w = _t(np.ones(512), dtype)
    _, ro = oracle_lib.add_rmsnorm(x, r, w, 1e-6)
    s32 = x.float().numpy() + r.float().numpy()  # library binary32 addition
    want_two_step = refnum.round_array(s32.astype(np.float64), dtype)
    assert np.array_equal(_bits(ro, dtype), want_two_step)
    assert torch.equal(ro, (x.float() + r.float()).to(ro.dtype))


@pytest.mark.parametrize("dtype", [0, 1])
def test_norm_reading_switch_changes_y_by_at_most_one_ulp_here(oracle_lib, dtype):
    g = np.random.Generator(np.random.Philox(key=[26, dtype]))
    x, r, w = _t(g.standard_normal((32, 1024)), dtype), _t(g.standard_normal((32, 1024)), dtype), _t(1 + 0.1 * g.standard_normal(1024), dtype)
    y_a, r_a = oracle_lib.add_rmsnorm(x, r, w, 1e-6)
    y_b, r_b = oracle_lib.add_rmsnorm(x, r, w, 1e-6, norm_from_rounded=True)
    assert torch.equal(r_a, r_b)
    worst, bad = oracle_lib.compare_y(y_b, y_a, tol_ulp=1)
    assert bad == 0 and worst == 1  # the readings do differ, by one step at most
    # and the rounded reading equals running the un-rounded one on inputs (r', 0)
    y_c, _ = oracle_lib.add_rmsnorm(r_a, torch.zeros_like(r_a), w, 1e-6)
    assert torch.equal(y_b, y_c)


def test_argument_checks_and_empty_batch(oracle_lib):
    w = torch.ones(8)
    y, ro = oracle_lib.add_rmsnorm(torch.zeros(0, 8), torch.zeros(0, 8), w, 1e-6)
    assert y.shape == (0, 8) and ro.shape == (0, 8)
    with pytest.raises(ValueError):
        oracle_lib.add_rmsnorm(torch.zeros(2, 8), torch.zeros(2, 7), w, 1e-6)
    with pytest.raises(TypeError):
        oracle_lib.add_rmsnorm(torch.zeros(2, 8), torch.zeros(2, 8).half(), w, 1e-6)


def test_threads_do_not_change_results(oracle_lib):
    g = np.random.Generator(np.random.Philox(key=[27, 0]))
    x, r, w = _t(g.standard_normal((37, 300)), 0), _t(g.standard_normal((37, 300)), 0), _t(g.standard_normal(300), 0)
    y1, r1 = oracle_lib.add_rmsnorm(x, r, w, 1e-6, threads=1)
    y5, r5 = oracle_lib.add_rmsnorm(x, r, w, 1e-6, threads=5)
    assert torch.equal(y1, y5) and torch.equal(r1, r5)
