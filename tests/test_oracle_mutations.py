"""The pins must be able to fail: plant one mistake at a time in a copy of the oracle's C source
(on the CPU), build it, and check that the core pins reject it while the real source passes."""
import math
import os

import numpy as np
import pytest
import torch

import refnum

MUTATIONS = {
    "divide_by_h_minus_1": ("acc / (double)H", "acc / (double)(H - 1)"),
    "eps_outside_sqrt": ("sqrt(ms + job->eps)", "(sqrt(ms) + job->eps)"),
    "weight_dropped": ("s[j] * wj / denom", "s[j] / denom"),
    "residual_dropped": ("const float s32 = xf + rf;", "const float s32 = xf;"),
    "residual_sign": ("const float s32 = xf + rf;", "const float s32 = xf - rf;"),
    "sum_not_squared": ("acc += used * used;", "acc += used;"),
    "ties_away_from_zero": ("(rem == 0.5 && (n & 1u))", "(rem == 0.5)"),
    "truncating_encode": ("if (rem > 0.5 ||", "if (rem > 2.0 ||"),
    "weight_indexed_by_row": ("wj = decode16(((const uint16_t*)job->w)[j], f);",
                              "wj = decode16(((const uint16_t*)job->w)[t % H], f);"),
    "output_row_ignored": ("((uint16_t*)job->y)[base + j] = encode16(y64, f);",
                           "((uint16_t*)job->y)[j] = encode16(y64, f);"),
    "add_in_double_then_round_direct": ("const uint16_t rb = encode16((double)s32, f);",
                                        "const uint16_t rb = encode16((double)xf * 1.0000001 + (double)rf, f);"),
    "rounded_residual_in_norm": ("if (job->norm_from_rounded)", "if (1)"),
    "subnormal_flush": ("bits = (uint32_t)n; /* subnormal", "bits = 0; /* subnormal"),
}


def _core_pins(o) -> bool:
    """A condensed set of the pins (bf16 and fp16), True when all hold."""
    bf, hf = torch.bfloat16, torch.float16
    try:
        for dtype, td in ((0, bf), (1, hf)):
            H = 37
            c, eps = 1.5, 0.25
            w = torch.linspace(-2, 2, H, dtype=torch.float64).to(td)
            x = torch.full((3, H), c / 2, dtype=td)
            y, ro = o.add_rmsnorm(x, x, w, eps)
            want = refnum.round_array(np.repeat((w.double().numpy() * c / math.sqrt(c * c + eps))[None], 3, 0), dtype)
            if not np.array_equal(y.view(torch.int16).numpy().view(np.uint16), want):
                return False
            # one-hot row: the mean divides by H
            xo = torch.zeros(1, 24, dtype=td); xo[0, 5] = 3.0
            wo = torch.linspace(0.5, 1.5, 24, dtype=torch.float64).to(td)
            y, _ = o.add_rmsnorm(xo, torch.zeros_like(xo), wo, eps)
            want = np.zeros(24); want[5] = float(wo[5]) * 3.0 / math.sqrt(9.0 / 24 + eps)
            if not np.array_equal(y.view(torch.int16).numpy().view(np.uint16)[0], refnum.round_array(want, dtype)):
                return False
            # library evaluation, ragged shape, two readings of the residual
            g = np.random.Generator(np.random.Philox(key=[41, dtype]))
            x = torch.from_numpy(g.standard_normal((5, 300)) * np.exp(g.uniform(-12, 3, (5, 300)))).to(td)
            r = torch.from_numpy(g.standard_normal((5, 300)) * np.exp(g.uniform(-12, 3, (5, 300)))).to(td)
            w = torch.from_numpy(1 + 0.3 * g.standard_normal(300)).to(td)
            y, ro = o.add_rmsnorm(x, r, w, 1e-6)
            s32 = x.float() + r.float()
            if not torch.equal(ro, s32.to(td)):
                return False
            s = s32.double()
            y64 = s * torch.rsqrt(s.pow(2).mean(-1, keepdim=True) + float(np.float32(1e-6))) * w.double()
            got = y.view(torch.int16).numpy().view(np.uint16)
            if np.count_nonzero(got != refnum.round_array(y64.numpy(), dtype)) > 1:
                return False
            # ties and subnormals of the codec
            vals, bits = refnum.finite_table(dtype)
            mid = (vals[:-1] + vals[1:]) / 2
            even = np.where((bits[:-1] & 1) == 0, bits[:-1], bits[1:])
            even = np.where((even == 0) & np.signbit(mid), np.uint16(0x8000), even)
            if not np.array_equal(o.encode16_from_f64(mid, dtype), even):
                return False
            above = np.nextafter(mid, np.inf)
            wa = np.where((bits[1:] == 0) & np.signbit(above), np.uint16(0x8000), bits[1:])
            if not np.array_equal(o.encode16_from_f64(above, dtype), wa):
                return False
    except Exception:
        return False
    return True


def _build_mutant(oracle_lib, out_dir: str, old: str, new: str,
                  targets=("add_rmsnorm_oracle.c", "number_formats.h")) -> str:
    """Copy the oracle's C sources into out_dir with one replacement applied, and compile them."""
    here = os.path.dirname(oracle_lib.__file__)
    hits = 0
    for f in oracle_lib.SOURCES + oracle_lib.HEADERS:
        text = open(os.path.join(here, f)).read()
        if f in targets:
            hits += text.count(old)
            text = text.replace(old, new)
        with open(os.path.join(out_dir, f), "w") as out:
            out.write(text)
    assert hits >= 1, f"mutation anchor not found: {old}"
    return oracle_lib.compile_sources(out_dir, os.path.join(out_dir, "mutant.so"))


def test_real_oracle_passes_core_pins(oracle_lib):
    assert _core_pins(oracle_lib)


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_is_caught(oracle_lib, tmp_path, name):
    old, new = MUTATIONS[name]
    so = _build_mutant(oracle_lib, str(tmp_path), old, new)
    saved = oracle_lib._lib
    try:
        oracle_lib._lib = oracle_lib._bind(so)
        assert not _core_pins(oracle_lib), f"pins did not notice: {name}"
    finally:
        oracle_lib._lib = saved


SILU_MUTATIONS = {
    "exp_sign": ("exp(-g)", "exp(g)"),
    "value_dropped": ("(1.0 + exp(-g)) * u", "(1.0 + exp(-g))"),
    "halves_swapped": ("const double v = g / (1.0 + exp(-g)) * u;", "const double v = u / (1.0 + exp(-u)) * g;"),
    "value_from_gate_half": ("t * 2 * d + d + j", "t * 2 * d + j"),
    "sigmoid_denominator": ("(1.0 + exp(-g))", "(2.0 + exp(-g))"),
    "gate_always_from_row_zero": ("load_elem(job->x, t * 2 * d + j, job->dtype)", "load_elem(job->x, j, job->dtype)"),
}


def _silu_pins(o) -> bool:
    try:
        for dtype, td in ((0, torch.bfloat16), (1, torch.float16)):
            x = torch.tensor([[50.0, 0.0, 1.5, -2.0, 2.0, 7.0, -3.0, 0.5],
                              [-1.0, 3.0, 60.0, 0.25, 4.0, 1.0, 0.5, -8.0]], dtype=torch.float64).to(td)
            out = o.silu_and_mul(x)
            xd = x.double()
            want = torch.nn.functional.silu(xd[:, :4]) * xd[:, 4:]
            if not np.array_equal(out.view(torch.int16).numpy().view(np.uint16), refnum.round_array(want.numpy(), dtype)):
                return False
            g = np.random.Generator(np.random.Philox(key=[61, dtype]))
            x = torch.from_numpy(g.standard_normal((6, 600)) * 3).to(td)
            xd = x.double()
            want = torch.nn.functional.silu(xd[:, :300]) * xd[:, 300:]
            got = o.silu_and_mul(x).view(torch.int16).numpy().view(np.uint16)
            if np.count_nonzero(got != refnum.round_array(want.numpy(), dtype)) > 1:
                return False
    except Exception:
        return False
    return True


def test_real_silu_oracle_passes_its_pins(oracle_lib):
    assert _silu_pins(oracle_lib)


@pytest.mark.parametrize("name", sorted(SILU_MUTATIONS))
def test_planted_silu_mistake_is_caught(oracle_lib, tmp_path, name):
    old, new = SILU_MUTATIONS[name]
    so = _build_mutant(oracle_lib, str(tmp_path), old, new, targets=("silu_and_mul_oracle.c",))
    saved = oracle_lib._lib
    try:
        oracle_lib._lib = oracle_lib._bind(so)
        assert not _silu_pins(oracle_lib), f"pins did not notice: {name}"
    finally:
        oracle_lib._lib = saved


MERGE_MUTATIONS = {
    "second_weight_is_first": ("(wa * a + wb * b) / D", "(wa * a + wa * b) / D"),
    "not_normalised": ("(wa * a + wb * b) / D", "(wa * a + wb * b)"),
    "log_dropped": ("(float)(m + log(D))", "(float)(m + D)"),
    "shift_dropped": ("wb = exp(sb - m)", "wb = exp(sb)"),
    "lse_indexed_by_token": ("const double sa = (double)s_a[row], sb = (double)s_b[row];",
                             "const double sa = (double)s_a[t], sb = (double)s_b[row];"),
    "parts_swapped_weights": ("const double wa = exp(sa - m), wb = exp(sb - m)", "const double wa = exp(sb - m), wb = exp(sa - m)"),
    "empty_case_returns_garbage": ("s_out[row] = -INFINITY;", "s_out[row] = 0.0f;"),
}


def _merge_pins(o) -> bool:
    try:
        for dtype, td in ((0, torch.bfloat16), (2, torch.float32)):
            g = torch.Generator().manual_seed(5)
            n, h, d, k1, k2 = 4, 3, 8, 9, 5
            q = torch.randn(n, h, d, generator=g, dtype=torch.float64)
            K = torch.randn(h, k1 + k2, d, generator=g, dtype=torch.float64)
            V = torch.randn(h, k1 + k2, d, generator=g, dtype=torch.float64)

            def attend(lo, hi):
                logits = torch.einsum("nhd,hkd->nhk", q, K[:, lo:hi]) / math.sqrt(d)
                return torch.einsum("nhk,hkd->nhd", torch.softmax(logits, -1), V[:, lo:hi]), torch.logsumexp(logits, -1)
            (o1, l1), (o2, l2), (oo, ll) = attend(0, k1), attend(k1, k1 + k2), attend(0, k1 + k2)
            v, so = o.merge_attn_states(o1.to(td), l1.float(), o2.to(td), l2.float())
            if not torch.allclose(v.double(), oo, rtol=0, atol=0.04 if dtype == 0 else 1e-5):
                return False
            if not torch.allclose(so.double(), ll, rtol=0, atol=2e-6):
                return False
            empty = torch.full((n, h), float("-inf"))
            v, so = o.merge_attn_states(o1.to(td), empty, o2.to(td), empty)
            if not (torch.equal(so, empty) and bool((v == 0).all())):
                return False
    except Exception:
        return False
    return True


def test_real_merge_oracle_passes_its_pins(oracle_lib):
    assert _merge_pins(oracle_lib)


@pytest.mark.parametrize("name", sorted(MERGE_MUTATIONS))
def test_planted_merge_mistake_is_caught(oracle_lib, tmp_path, name):
    old, new = MERGE_MUTATIONS[name]
    so = _build_mutant(oracle_lib, str(tmp_path), old, new, targets=("merge_attn_states_oracle.c",))
    saved = oracle_lib._lib
    try:
        oracle_lib._lib = oracle_lib._bind(so)
        assert not _merge_pins(oracle_lib), f"pins did not notice: {name}"
    finally:
        oracle_lib._lib = saved


FP8_MUTATIONS = {
    "scale_from_448_wrong": ("(amax > 1e-12 ? amax : 1e-12) / 448.0", "(amax > 1e-12 ? amax : 1e-12) / 240.0"),
    "amax_without_abs": ("if (fabs(y[j]) > amax) amax = fabs(y[j]);", "if (y[j] > amax) amax = y[j];"),
    "weight_left_out_of_amax": ("y[j] = y[j] * (double)load32(w, j, dtype) / denom;\n            if (fabs(y[j]) > amax) amax = fabs(y[j]);",
                                "if (fabs(y[j] / denom) > amax) amax = fabs(y[j] / denom);\n            y[j] = y[j] * (double)load32(w, j, dtype) / denom;"),
    "ties_away": ("if (rem > 0.5 || (rem == 0.5 && (n & 1u))) n += 1;\n    uint32_t bits = E < emin", "if (rem >= 0.5) n += 1;\n    uint32_t bits = E < emin"),
    "saturation_threshold": ("if (a >= 448.0) return (uint8_t)(sign | 0x7Eu);", "if (a >= 480.0) return (uint8_t)(sign | 0x7Eu);"),
    "exponent_bias": ("((uint32_t)(E + 7) << 3)", "((uint32_t)(E + 8) << 3)"),
    "scale_per_tensor": ("        double amax = 0.0;\n        for (int64_t j = 0; j < hidden; ++j) {\n            y[j] = y[j] *",
                         "        static double amax = 0.0;\n        for (int64_t j = 0; j < hidden; ++j) {\n            y[j] = y[j] *"),
}


def _fp8_pins(o) -> bool:
    try:
        bits = torch.arange(256, dtype=torch.int16).to(torch.uint8)
        vals = bits.view(torch.float8_e4m3fn).to(torch.float64).numpy()
        fin = ~np.isnan(vals)
        if not np.array_equal(o.encode_e4m3(vals[fin]), bits.numpy()[fin]):
            return False
        pos = np.sort(vals[fin & (bits.numpy() < 0x80)])
        pb = o.encode_e4m3(pos)
        mid = (pos[:-1] + pos[1:]) / 2
        if not np.array_equal(o.encode_e4m3(mid), np.where((pb[:-1] & 1) == 0, pb[:-1], pb[1:])):
            return False
        if o.encode_e4m3(np.array([464.0, 470.0])).tolist() != [0x7E, 0x7E]:
            return False
        g = np.random.Generator(np.random.Philox(key=[81, 0]))
        x = torch.from_numpy(g.standard_normal((6, 200)) * np.array([0.1, 1, 5, 1, 30, 1])[:, None]).to(torch.bfloat16)
        r = torch.from_numpy(g.standard_normal((6, 200))).to(torch.bfloat16)
        w = torch.from_numpy(-1.0 - 0.5 * np.abs(g.standard_normal(200))).to(torch.bfloat16)  # negative weights
        q, scale, _ = o.add_rmsnorm_fp8(x, r, w, 1e-6)
        s = (x.float() + r.float()).double()
        y = s * torch.rsqrt(s.pow(2).mean(-1, keepdim=True) + float(np.float32(1e-6))) * w.double()
        amax = y.abs().amax(-1)
        if not torch.allclose(scale.double(), amax / 448.0, rtol=1.2e-7, atol=0):
            return False
        want = o.encode_e4m3((y / (amax / 448.0)[:, None]).numpy())
        if np.count_nonzero(q.numpy() != want) > 1:
            return False
    except Exception:
        return False
    return True


def test_real_fp8_oracle_passes_its_pins(oracle_lib):
    assert _fp8_pins(oracle_lib)


@pytest.mark.parametrize("name", sorted(FP8_MUTATIONS))
def test_planted_fp8_mistake_is_caught(oracle_lib, tmp_path, name):
    old, new = FP8_MUTATIONS[name]
    so = _build_mutant(oracle_lib, str(tmp_path), old, new, targets=("add_rmsnorm_fp8_oracle.c",))
    saved = oracle_lib._lib
    try:
        oracle_lib._lib = oracle_lib._bind(so)
        assert not _fp8_pins(oracle_lib), f"pins did not notice: {name}"
    finally:
        oracle_lib._lib = saved
