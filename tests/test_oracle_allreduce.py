"""Pins of the oracle for the tensor-parallel form of the fused add + RMSNorm (x given as N parts summed in
binary32 in rank order): the N = 1 special case, exact rational arithmetic with a hand-written binary32 rounding,
a float32 library chain, closed forms where the order of the binary32 additions shows, and planted mistakes."""
import math
import os
from decimal import Decimal, getcontext
from fractions import Fraction

import numpy as np
import pytest
import torch

import refnum

getcontext().prec = 80
TD = {0: torch.bfloat16, 1: torch.float16, 2: torch.float32}


def round_to_binary32(v: Fraction) -> Fraction:
    """Nearest binary32 value of an exact rational, ties to even (no overflow handling: callers stay in range)."""
    if v == 0:
        return Fraction(0)
    sign = -1 if v < 0 else 1
    a = abs(v)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    if Fraction(2) ** (e + 1) <= a:
        e += 1
    e = max(e, -126)                      # subnormals share the spacing of the smallest normal binade
    quantum = Fraction(2) ** (e - 23)
    q, rem = divmod(a, quantum)
    q = int(q)
    if rem * 2 > quantum or (rem * 2 == quantum and (q & 1)):
        q += 1
    return sign * q * quantum


def test_round_to_binary32_helper_against_known_values():
    assert round_to_binary32(Fraction(2 ** 24 + 1)) == 2 ** 24          # tie, even mantissa below
    assert round_to_binary32(Fraction(2 ** 24 + 3)) == 2 ** 24 + 4      # tie, even mantissa above
    assert round_to_binary32(Fraction(1, 3)) == Fraction(11184811, 2 ** 25)
    assert round_to_binary32(Fraction(-5, 2)) == Fraction(-5, 2)
    assert round_to_binary32(Fraction(1, 2 ** 149)) == Fraction(1, 2 ** 149)
    assert round_to_binary32(Fraction(1, 2 ** 150)) == 0                 # tie to even at the bottom


def _dec(fr: Fraction) -> Decimal:
    return Decimal(fr.numerator) / Decimal(fr.denominator)


def _exact(parts, r, w, eps32):
    """Per element: the binary32 chain as an exact Fraction, and y as an 80-digit Decimal."""
    N, T, H = parts.shape
    p64, r64, w64 = parts.double().numpy(), r.double().numpy(), w.double().numpy()
    all_s, all_y = [], []
    for t in range(T):
        s = []
        for j in range(H):
            a = Fraction(float(p64[0, t, j]))
            for k in range(1, N):
                a = round_to_binary32(a + Fraction(float(p64[k, t, j])))
            s.append(round_to_binary32(a + Fraction(float(r64[t, j]))))
        ms = sum(v * v for v in s) / H
        denom = (_dec(ms) + Decimal(float(eps32))).sqrt()
        all_s.append(s)
        all_y.append([_dec(s[j]) * Decimal(float(w64[j])) / denom for j in range(H)])
    return all_s, all_y


@pytest.mark.parametrize("dtype", [0, 1, 2])
@pytest.mark.parametrize("N,T,H", [(2, 1, 1), (3, 2, 3), (4, 1, 8), (8, 2, 5)])
def test_tiny_shapes_against_exact_arithmetic(oracle_lib, dtype, N, T, H):
    g = np.random.Generator(np.random.Philox(key=[71, dtype * 1000 + N * 100 + T * 10 + H]))
    for trial in range(4):
        # wide magnitude spread between the parts so that the binary32 additions really round
        mag = np.exp(g.uniform(-9, 9, (N, T, H))) if trial % 2 == 0 else np.ones((N, T, H))
        parts = torch.from_numpy(g.standard_normal((N, T, H)) * mag).to(TD[dtype])
        r = torch.from_numpy(g.standard_normal((T, H))).to(TD[dtype])
        w = torch.from_numpy(1 + 0.5 * g.standard_normal(H)).to(TD[dtype])
        eps = [1e-6, 1e-2][trial % 2]
        y, ro = oracle_lib.allreduce_add_rmsnorm(parts, r, w, eps)
        s, yex = _exact(parts, r, w, np.float32(eps))
        for t in range(T):
            for j in range(H):
                if dtype == 2:
                    assert Fraction(float(ro[t, j])) == s[t][j]
                    got = np.float32(y[t, j])
                    err = abs(Decimal(float(got)) - yex[t][j])
                    for nb in (np.nextafter(got, np.float32(-np.inf)), np.nextafter(got, np.float32(np.inf))):
                        assert err <= abs(Decimal(float(nb)) - yex[t][j])
                else:
                    assert (int(ro.view(torch.int16)[t, j]) & 0xFFFF) == refnum.round_exact(s[t][j], dtype)
                    assert (int(y.view(torch.int16)[t, j]) & 0xFFFF) == refnum.round_exact(yex[t][j], dtype)


@pytest.mark.parametrize("dtype", [0, 1, 2])
def test_one_part_is_the_plain_operator(oracle_lib, dtype):
    g = np.random.Generator(np.random.Philox(key=[72, dtype]))
    x = torch.from_numpy(g.standard_normal((7, 130)) * 3).to(TD[dtype])
    r = torch.from_numpy(g.standard_normal((7, 130))).to(TD[dtype])
    w = torch.from_numpy(1 + 0.2 * g.standard_normal(130)).to(TD[dtype])
    y1, r1 = oracle_lib.allreduce_add_rmsnorm(x[None], r, w, 1e-6)
    y0, r0 = oracle_lib.add_rmsnorm(x, r, w, 1e-6)
    assert torch.equal(y1.view(torch.int16) if dtype < 2 else y1, y0.view(torch.int16) if dtype < 2 else y0)
    assert torch.equal(r1.view(torch.int16) if dtype < 2 else r1, r0.view(torch.int16) if dtype < 2 else r0)


def _library_chain(parts, r):
    a = parts[0].float()
    for k in range(1, parts.shape[0]):
        a = a + parts[k].float()
    return a + r.float()


@pytest.mark.parametrize("dtype", [0, 1, 2])
@pytest.mark.parametrize("N", [2, 4, 8])
def test_library_float32_chain_and_float64_norm(oracle_lib, dtype, N):
    g = np.random.Generator(np.random.Philox(key=[73, dtype * 10 + N]))
    T, H = 9, 517
    parts = torch.from_numpy(g.standard_normal((N, T, H)) * np.exp(g.uniform(-6, 4, (N, T, H)))).to(TD[dtype])
    r = torch.from_numpy(g.standard_normal((T, H))).to(TD[dtype])
    w = torch.from_numpy(1 + 0.3 * g.standard_normal(H)).to(TD[dtype])
    y, ro = oracle_lib.allreduce_add_rmsnorm(parts, r, w, 1e-6, threads=3)
    s32 = _library_chain(parts, r)
    assert torch.equal(ro, s32.to(TD[dtype]))
    s = s32.double()
    y64 = s * torch.rsqrt(s.pow(2).mean(-1, keepdim=True) + float(np.float32(1e-6))) * w.double()
    if dtype == 2:
        assert torch.allclose(y.double(), y64, rtol=1e-7, atol=0)
    else:
        got = y.view(torch.int16).numpy().view(np.uint16)
        assert np.count_nonzero(got != refnum.round_array(y64.numpy(), dtype)) <= 2  # fp64 near-ties only
    # threads only split rows
    y1, r1 = oracle_lib.allreduce_add_rmsnorm(parts, r, w, 1e-6, threads=1)
    assert torch.equal(y1.view(torch.int32 if dtype == 2 else torch.int16), y.view(torch.int32 if dtype == 2 else torch.int16))
    assert torch.equal(r1.view(torch.int32 if dtype == 2 else torch.int16), ro.view(torch.int32 if dtype == 2 else torch.int16))


def test_order_of_the_binary32_additions_is_rank_order(oracle_lib):
    # parts (2^24, 1, -2^24), residual 0: rank order gives fl(2^24 + 1) = 2^24, then 0; any exact or reordered
    # evaluation gives 1.  bf16 holds all three values exactly.
    H = 4
    for dtype in (0, 2):
        parts = torch.zeros(3, 1, H, dtype=TD[dtype])
        parts[0, 0, 0], parts[1, 0, 0], parts[2, 0, 0] = 2.0 ** 24, 1.0, -(2.0 ** 24)
        parts[0, 0, 1], parts[1, 0, 1], parts[2, 0, 1] = 2.0 ** 24, -(2.0 ** 24), 1.0     # the same set, benign order
        parts[0, 0, 2] = 2.0
        r = torch.zeros(1, H, dtype=TD[dtype]); r[0, 3] = 3.0
        w = torch.ones(H, dtype=TD[dtype])
        y, ro = oracle_lib.allreduce_add_rmsnorm(parts, r, w, 0.0)
        assert ro.float().tolist() == [[0.0, 1.0, 2.0, 3.0]]
        want = np.array([0.0, 1.0, 2.0, 3.0]) / math.sqrt(14.0 / 4)
        if dtype == 2:
            assert np.allclose(y.double().numpy()[0], want, rtol=1e-7, atol=0)
        else:
            assert np.array_equal(y.view(torch.int16).numpy().view(np.uint16)[0], refnum.round_array(want, dtype))
    # the residual joins last: fl(fl(1 + 2^-24) + 2^-24) = 1 in rank order, but r first would give 1 + 2^-23
    parts = torch.tensor([[[1.0]], [[2.0 ** -24]]], dtype=torch.float32)
    r = torch.tensor([[2.0 ** -24]], dtype=torch.float32)
    _, ro = oracle_lib.allreduce_add_rmsnorm(parts, r, torch.ones(1), 0.0)
    assert float(ro) == 1.0
    parts = torch.tensor([[[2.0 ** -24]], [[2.0 ** -24]]], dtype=torch.float32)
    _, ro = oracle_lib.allreduce_add_rmsnorm(parts, torch.tensor([[1.0]]), torch.ones(1), 0.0)
    assert float(ro) == 1.0 + 2.0 ** -23


def test_constant_parts_closed_form(oracle_lib):
    # every part holds c / N (exact in each format for N a power of two): s = c + 0, y_j = w_j c / sqrt(c^2 + eps)
    c, eps, H = 1.5, 0.25, 33
    for dtype in (0, 1):
        for N in (2, 4, 8):
            w = torch.linspace(-2, 2, H, dtype=torch.float64).to(TD[dtype])
            parts = torch.full((N, 2, H), c / N, dtype=TD[dtype])
            y, ro = oracle_lib.allreduce_add_rmsnorm(parts, torch.zeros(2, H, dtype=TD[dtype]), w, eps)
            assert torch.all(ro.double() == c)
            want = refnum.round_array(np.repeat((w.double().numpy() * c / math.sqrt(c * c + eps))[None], 2, 0), dtype)
            assert np.array_equal(y.view(torch.int16).numpy().view(np.uint16), want)


def test_argument_errors(oracle_lib):
    x = np.zeros((2, 3, 4), np.float32)
    with pytest.raises(ValueError):
        oracle_lib.allreduce_add_rmsnorm(x, np.zeros((3, 5), np.float32), np.zeros(4, np.float32), 1e-6)
    with pytest.raises(ValueError):
        oracle_lib.allreduce_add_rmsnorm(x[0], np.zeros((3, 4), np.float32), np.zeros(4, np.float32), 1e-6)
    y, ro = oracle_lib.allreduce_add_rmsnorm(np.zeros((2, 0, 4), np.float32), np.zeros((0, 4), np.float32),
                                             np.zeros(4, np.float32), 1e-6)
    assert y.shape == (0, 4) and ro.shape == (0, 4)


# ---- the pins must be able to fail -----------------------------------------------------------------------------

MUTATIONS = {
    "reversed_rank_order": ("for (int k = 1; k < job->n_parts; ++k) {\n                const float part = load32(job->x_parts, (int64_t)k * part_stride",
                            "for (int k = 1; k < job->n_parts; ++k) {\n                const float part = load32(job->x_parts, (int64_t)(job->n_parts - k) * part_stride"),
    "fp64_accumulation_rounded_once": ("            float a = load32(job->x_parts, base + j, job->dtype);",
                                       "            double a = load32(job->x_parts, base + j, job->dtype);"),
    "last_part_dropped": ("for (int k = 1; k < job->n_parts; ++k) {", "for (int k = 1; k < job->n_parts - (job->n_parts > 2); ++k) {"),
    "part_stride_is_one_row": ("const int64_t part_stride = job->n_tokens * H;", "const int64_t part_stride = H;"),
    "residual_dropped": ("const float s32 = a + load32(job->r, base + j, job->dtype);", "const float s32 = a;"),
    "divide_by_parts": ("sqrt(acc / (double)H + job->eps)", "sqrt(acc / (double)(H * job->n_parts) + job->eps)"),
    "weight_dropped": ("s[j] * (double)load32(job->w, j, job->dtype) / denom", "s[j] / denom"),
    "eps_outside_sqrt": ("sqrt(acc / (double)H + job->eps)", "(sqrt(acc / (double)H) + job->eps)"),
}


def _pins(o) -> bool:
    try:
        test_order_of_the_binary32_additions_is_rank_order(o)
        test_constant_parts_closed_form(o)
        test_library_float32_chain_and_float64_norm(o, 0, 4)
        test_tiny_shapes_against_exact_arithmetic(o, 2, 3, 2, 3)
    except AssertionError:
        return False
    return True


def _build_mutant(oracle_lib, out_dir: str, old: str, new: str) -> str:
    here = os.path.dirname(oracle_lib.__file__)
    hits = 0
    for f in oracle_lib.SOURCES + oracle_lib.HEADERS:
        text = open(os.path.join(here, f)).read()
        if f == "allreduce_add_rmsnorm_oracle.c":
            hits += text.count(old)
            text = text.replace(old, new)
        with open(os.path.join(out_dir, f), "w") as out:
            out.write(text)
    assert hits == 1, f"mutation anchor found {hits} times: {old}"
    return oracle_lib.compile_sources(out_dir, os.path.join(out_dir, "mutant.so"))


def test_real_oracle_passes_the_condensed_pins(oracle_lib):
    assert _pins(oracle_lib)


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_is_caught(oracle_lib, tmp_path, name):
    old, new = MUTATIONS[name]
    so = _build_mutant(oracle_lib, str(tmp_path), old, new)
    saved = oracle_lib._lib
    try:
        oracle_lib._lib = oracle_lib._bind(so)
        assert not _pins(oracle_lib), f"pins did not notice: {name}"
    finally:
        oracle_lib._lib = saved
