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


def _allreduce_cases(n, seed):
    g = np.random.Generator(np.random.Philox(key=[seed, 1]))
    out = []
    for _ in range(n):
        dtype = ["bf16", "fp16", "fp32"][int(g.integers(0, 3))]
        eb = 4 if dtype == "fp32" else 2
        vectors = int(g.integers(1, 1536)) if g.random() < 0.5 else int(g.integers(1, 64))
        H = vectors * 16 // eb
        T = int(g.integers(1, 60))
        n_parts = [2, 4, 8][int(g.integers(0, 3))]
        lo = int(g.integers(0, T))
        rows = int(g.integers(0, T - lo + 1))
        out.append((dtype, T, H, n_parts, lo, rows, int(g.integers(1, 9)), int(g.integers(1, 9))))
    return out


@pytest.mark.parametrize("dtype,T,H,n_parts,lo,rows,n_y,n_r", _allreduce_cases(36, seed=2025))
def test_random_allreduce_fused_launches_match_oracle(B, oracle_lib, dtype, T, H, n_parts, lo, rows, n_y, n_r):
    """Random part counts, row blocks inside a larger tensor and destination counts of the all-reduce-fused norm."""
    from paper_2601_12698_b200 import synth
    _, r, w = synth.make_inputs(T, H, dtype, seed=H * 17 + T)
    parts = synth.make_parts(0, T, H, dtype, H * 17 + T, n_parts)
    y_ref, r_ref = oracle_lib.allreduce_add_rmsnorm(parts, r, w, EPS)
    pd, rd, wd = parts.cuda(), r.cuda(), w.cuda()
    shape = B.shape_of(max(rows, 1), H, dtype, op=B.RT_OP_ADD_RMSNORM_ALLREDUCE, n_parts=n_parts)
    thetas = B.tuner_derive_feasible(shape, heuristics=0)
    assert thetas
    g = np.random.Generator(np.random.Philox(key=[T, H + n_parts]))
    picks = [thetas[int(i)] for i in g.choice(len(thetas), size=min(8, len(thetas)), replace=False)]
    mode, tol = (B.RT_CMP_REL32, 1e-5) if dtype == "fp32" else (B.RT_CMP_ULP16, 2.0)
    block = slice(lo, lo + rows)
    y_ref_d, r_ref_d = y_ref[block].contiguous().cuda(), r_ref[block].contiguous().cuda()
    for th in picks:
        ys = [torch.full_like(rd, 5.0) for _ in range(n_y)]
        ros = [torch.full_like(rd, 5.0) for _ in range(n_r)]
        B.rmsnorm_allreduce_template_launch(th, [pd[k] for k in range(n_parts)], rd, wd, ys, ros, lo, rows, EPS)
        for dst, ref, m, t in [(d, y_ref_d, mode, tol) for d in ys] + [(d, r_ref_d, B.RT_CMP_BITS, 0.0) for d in ros]:
            if rows:
                worst, bad = B.tuner_compare(dst[block].contiguous(), ref, m, t)
                assert bad == 0, (repr(th), worst)
            outside = torch.cat([dst[:lo], dst[lo + rows:]])
            assert bool((outside == 5.0).all()), repr(th)
    assert B.rt_device_status() == 0
