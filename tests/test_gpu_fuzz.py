"""Randomised parity: random shapes (ragged row counts, odd vector counts, every alignment class), random dtypes and a
random sample of each shape's hard-feasible thetas, against the CPU oracle.  Seeded: the cases are the same every run."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu
EPS = 1e-6


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2601_12698_b200 import binding
    torch.cuda.set_device(0)
    return binding


def _cases(n, seed):
    g = np.random.Generator(np.random.Philox(key=[seed, 0]))
    out = []
    for _ in range(n):
        dtype = ["bf16", "fp16", "fp32"][int(g.integers(0, 3))]
        eb = 4 if dtype == "fp32" else 2
        align = [16, 16, 16, 8, 4, 2][int(g.integers(0, 6))]      # bytes the row length is a multiple of
        if align < eb:
            align = eb
        units = int(g.integers(1, 24576 // align + 1)) if g.random() < 0.5 else int(g.integers(1, 600))
        H = units * align // eb
        T = int(g.integers(1, 40)) if g.random() < 0.7 else int(g.integers(40, 700))
        out.append((dtype, T, max(H, 1)))
    return out


@pytest.mark.parametrize("dtype,T,H", _cases(48, seed=2024))
def test_random_shapes_and_thetas_match_oracle(B, oracle_lib, dtype, T, H):
    from paper_2601_12698_b200 import synth
    x, r, w = synth.make_inputs(T, H, dtype, seed=H * 31 + T)
    y_ref, r_ref = oracle_lib.add_rmsnorm(x, r, w, EPS)
    xd, rd, wd = x.cuda(), r.cuda(), w.cuda()
    y, ro = torch.empty_like(xd), torch.empty_like(xd)
    shape = B.shape_of(T, H, dtype, B._ptr_align(xd, rd, wd, y, ro))
    thetas = B.tuner_derive_feasible(shape, heuristics=0)
    assert thetas, "every shape has at least the narrow fall-back"
    g = np.random.Generator(np.random.Philox(key=[T, H]))
    picks = [thetas[int(i)] for i in g.choice(len(thetas), size=min(25, len(thetas)), replace=False)]
    y_ref_d, r_ref_d = y_ref.cuda(), r_ref.cuda()
    for th in picks:
        y.fill_(float("nan")); ro.fill_(float("nan"))
        B.rmsnorm_template_launch(th, xd, rd, wd, y, ro, EPS)
        _, r_bad = B.tuner_compare(ro, r_ref_d, B.RT_CMP_BITS)
        if dtype == "fp32":
            worst, y_bad = B.tuner_compare(y, y_ref_d, B.RT_CMP_REL32, 1e-5)
        else:
            worst, y_bad = B.tuner_compare(y, y_ref_d, B.RT_CMP_ULP16, 2.0)
        assert r_bad == 0 and y_bad == 0, (repr(th), r_bad, y_bad, worst)
    assert B.rt_device_status() == 0
