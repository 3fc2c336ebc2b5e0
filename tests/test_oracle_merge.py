"""Pins of the merge_attn_states oracle: closed forms, symmetries, and the defining property that merged
partial attentions equal attention over the concatenated keys."""
import math

import numpy as np
import pytest
import torch

import refnum

TD = {0: torch.bfloat16, 1: torch.float16, 2: torch.float32}
NEG_INF = float("-inf")


def _bits(t, dtype):
    return t.numpy() if dtype == 2 else t.view(torch.int16).numpy().view(np.uint16)


def _round(v64, dtype):
    v64 = np.asarray(v64, dtype=np.float64)
    return v64.astype(np.float32) if dtype == 2 else refnum.round_array(v64, dtype)


def _rand(shape, dtype, key):
    g = np.random.Generator(np.random.Philox(key=key))
    return torch.from_numpy(g.standard_normal(shape)).to(TD[dtype])


@pytest.mark.parametrize("dtype", [0, 1, 2])
def test_closed_forms(oracle_lib, dtype):
    n, h, d = 2, 3, 8
    va, vb = _rand((n, h, d), dtype, [71, dtype]), _rand((n, h, d), dtype, [72, dtype])
    s = torch.tensor([[0.5, -2.0, 7.25], [3.0, 0.0, -1.5]], dtype=torch.float32)
    # equal log-sum-exps: the mean, and s + ln 2
    v, so = oracle_lib.merge_attn_states(va, s, vb, s)
    assert np.array_equal(_bits(v, dtype), _round((va.double() + vb.double()).numpy() / 2, dtype))
    assert np.array_equal(so.numpy(), (s.double() + math.log(2.0)).numpy().astype(np.float32))
    # an empty part (-inf) returns the other part unchanged
    empty = torch.full_like(s, NEG_INF)
    v, so = oracle_lib.merge_attn_states(va, s, vb, empty)
    assert torch.equal(v, va) and torch.equal(so, s)
    v, so = oracle_lib.merge_attn_states(va, empty, vb, s)
    assert torch.equal(v, vb) and torch.equal(so, s)
    # both empty: zeros and -inf
    v, so = oracle_lib.merge_attn_states(va, empty, vb, empty)
    assert np.all(v.double().numpy() == 0.0) and torch.equal(so, empty)
    # s_a - s_b = ln 3 (in binary32): weights 3/4 and 1/4 up to the rounding of ln 3
    ln3 = float(np.float32(math.log(3.0)))
    sa = torch.full((n, h), ln3, dtype=torch.float32)
    v, so = oracle_lib.merge_attn_states(va, sa, vb, torch.zeros(n, h))
    wa = math.exp(ln3) / (math.exp(ln3) + 1.0)
    assert np.array_equal(_bits(v, dtype), _round((wa * va.double() + (1 - wa) * vb.double()).numpy(), dtype))
    assert abs(wa - 0.75) < 1e-8 and abs(float(so[0, 0]) - math.log(4.0)) < 2e-7
    # far-apart log-sum-exps: the heavier part wins exactly in fp64
    v, so = oracle_lib.merge_attn_states(va, torch.full((n, h), 50.0), vb, torch.full((n, h), -50.0))
    assert torch.equal(v, va) and float(so[0, 0]) == 50.0


@pytest.mark.parametrize("dtype", [0, 1, 2])
def test_symmetry_shift_and_independence(oracle_lib, dtype):
    n, h, d = 3, 4, 16
    va, vb = _rand((n, h, d), dtype, [73, dtype]), _rand((n, h, d), dtype, [74, dtype])
    sa, sb = _rand((n, h), 2, [75, dtype]) * 3, _rand((n, h), 2, [76, dtype]) * 3
    v, so = oracle_lib.merge_attn_states(va, sa, vb, sb)
    v2, so2 = oracle_lib.merge_attn_states(vb, sb, va, sa)
    assert torch.equal(v, v2) and torch.equal(so, so2)
    # a common power-of-two shift of both log-sum-exps is exact in binary32 here: only s_out moves
    v3, so3 = oracle_lib.merge_attn_states(va, sa + 64.0, vb, sb + 64.0)
    if torch.equal((sa + 64.0) - 64.0, sa) and torch.equal((sb + 64.0) - 64.0, sb):
        assert torch.equal(v3, v)
    assert torch.allclose(so3, so + 64.0, rtol=0, atol=1e-5)
    # every (token, head) row stands alone, and uses its own pair of log-sum-exps
    for t in range(n):
        for k in range(h):
            vr, sr = oracle_lib.merge_attn_states(va[t:t + 1, k:k + 1].contiguous(), sa[t:t + 1, k:k + 1].contiguous(),
                                                  vb[t:t + 1, k:k + 1].contiguous(), sb[t:t + 1, k:k + 1].contiguous())
            assert np.array_equal(_bits(vr, dtype)[0, 0], _bits(v, dtype)[t, k]) and float(sr) == float(so[t, k])


@pytest.mark.parametrize("dtype", [0, 1, 2])
def test_merging_partial_attention_equals_attention_over_all_keys(oracle_lib, dtype):
    """Float64 library softmax attention over keys K1 and K2 separately, merged by the oracle, against the same
    attention over the concatenation [K1; K2]."""
    g = torch.Generator().manual_seed(77 + dtype)
    n, h, d, k1, k2 = 5, 3, 16, 11, 7
    q = torch.randn(n, h, d, generator=g, dtype=torch.float64)
    K = torch.randn(h, k1 + k2, d, generator=g, dtype=torch.float64)
    V = torch.randn(h, k1 + k2, d, generator=g, dtype=torch.float64)

    def attend(lo, hi):
        logits = torch.einsum("nhd,hkd->nhk", q, K[:, lo:hi]) / math.sqrt(d)
        return torch.einsum("nhk,hkd->nhd", torch.softmax(logits, -1), V[:, lo:hi]), torch.logsumexp(logits, -1)
    (o1, l1), (o2, l2), (o, l) = attend(0, k1), attend(k1, k1 + k2), attend(0, k1 + k2)
    # the partial results are stored in the kernel's types: outputs in dtype, log-sum-exps in binary32
    o1s, o2s, l1s, l2s = o1.to(TD[dtype]), o2.to(TD[dtype]), l1.float(), l2.float()
    v, so = oracle_lib.merge_attn_states(o1s, l1s, o2s, l2s)
    tol = {0: 2.0**-7, 1: 2.0**-10, 2: 1e-6}[dtype]
    assert torch.allclose(v.double(), o, rtol=0, atol=tol * 4)
    assert torch.allclose(so.double(), l, rtol=0, atol=2e-6)
    # and with exact inputs the merge is exact to fp64 accuracy (fp32 storage of the result only)
    if dtype == 2:
        wa = torch.exp(l1 - torch.maximum(l1, l2)); wb = torch.exp(l2 - torch.maximum(l1, l2))
        ref = (wa[..., None] * o1s.double() + wb[..., None] * o2s.double()) / (wa + wb)[..., None]
        assert torch.allclose(v.double(), ref, rtol=1e-6, atol=1e-7)


def test_mixed_compare_pins(oracle_lib):
    ref = torch.tensor([1.0, 0.001, -2.0, 0.0], dtype=torch.bfloat16)
    got = ref.clone(); got.view(torch.int16)[0] += 2          # 2 ulp: passes on ulps
    assert oracle_lib.compare_mixed(got, ref, tol=2.0, tol_abs=0.0)[1] == 0
    got.view(torch.int16)[0] += 1                               # 3 ulp of 1.0 = 0.0234: fails both
    assert oracle_lib.compare_mixed(got, ref, tol=2.0, tol_abs=1e-3)[1] == 1
    got = ref.clone(); got[1] = 0.0012                          # many ulps, tiny absolute difference
    assert oracle_lib.compare_mixed(got, ref, tol=2.0, tol_abs=1e-3)[1] == 0
    assert oracle_lib.compare_mixed(got, ref, tol=2.0, tol_abs=1e-5)[1] == 1
    a, b = torch.tensor([1.0, 1e-9]), torch.tensor([1.000001, 0.0])
    assert oracle_lib.compare_mixed(a, b, tol=1e-5, tol_abs=1e-8)[1] == 0
    assert oracle_lib.compare_mixed(a, b, tol=1e-7, tol_abs=1e-10)[1] == 2
    # an overflowed 16-bit output is no neighbour of the largest finite value; equal infinities match
    top = torch.tensor([65504.0, float("inf"), float("inf")], dtype=torch.float16)
    inf = torch.tensor([float("inf"), float("inf"), float("-inf")], dtype=torch.float16)
    assert oracle_lib.compare_mixed(top, inf, tol=2.0, tol_abs=1e-5)[1] == 2


def test_argument_checks(oracle_lib):
    v = torch.zeros(2, 3, 4); s = torch.zeros(2, 3)
    with pytest.raises(ValueError):
        oracle_lib.merge_attn_states(v, torch.zeros(2, 4), v, s)
    with pytest.raises(TypeError):
        oracle_lib.merge_attn_states(v, s.double().numpy(), v, s)
    out, so = oracle_lib.merge_attn_states(torch.zeros(0, 3, 4), torch.zeros(0, 3), torch.zeros(0, 3, 4), torch.zeros(0, 3))
    assert out.shape == (0, 3, 4) and so.shape == (0, 3)
