"""Parity on the shapes the workload list and the paper name, and on inputs chosen to stress the fp32 sum of squares.

1. The five decode shapes {1, 4, 16, 64, 256} x 4096 (bf16) and the thirteen (m, n) shapes of the paper's
   Experimental Setup ("Kernels"), every feasible theta each.
2. Rows with a closed form - constants (among them values whose square is not representable), one-hot rows, +-1 rows,
   ones with a single 1e4 outlier, rows at the edge of the fp16 range - at real widths, all three dtypes, every
   hard-feasible theta, so that each stage runs with the largest per-thread element count it admits (384 for fp32
   rows of 12288 elements on 32 threads).  A per-thread chain of fp32 additions rounds one-sidedly on exactly such
   rows; the fp32 tolerance of 1e-5 has to hold there too, and the worst error seen is printed."""
import pytest
import torch

pytestmark = pytest.mark.gpu

TD = {"bf16": torch.bfloat16, "fp16": torch.float16, "fp32": torch.float32}
EPS = 1e-6


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2601_12698_b200 import binding
    torch.cuda.set_device(0)
    return binding


def _run_all(B, oracle_lib, x, r, w, dtype, thetas, eps=EPS):
    """Launch every theta; returns (number run, failures, worst y error seen)."""
    y_ref, r_ref = oracle_lib.add_rmsnorm(x, r, w, eps)
    xd, rd, wd = x.cuda(), r.cuda(), w.cuda()
    y_ref_d, r_ref_d = y_ref.cuda(), r_ref.cuda()
    y, ro = torch.empty_like(xd), torch.empty_like(xd)
    failures, worst_seen = [], 0.0
    for th in thetas:
        y.fill_(float("nan")); ro.fill_(float("nan"))
        B.rmsnorm_template_launch(th, xd, rd, wd, y, ro, eps)
        _, r_bad = B.tuner_compare(ro, r_ref_d, B.RT_CMP_BITS)
        if dtype == "fp32":
            worst, y_bad = B.tuner_compare(y, y_ref_d, B.RT_CMP_REL32, 1e-5)
        else:
            worst, y_bad = B.tuner_compare(y, y_ref_d, B.RT_CMP_ULP16, 2.0)
        worst_seen = max(worst_seen, worst)
        if r_bad or y_bad:
            failures.append((repr(th), r_bad, y_bad, worst))
    assert B.rt_device_status() == 0
    return len(thetas), failures, worst_seen


def _named_shapes():
    from paper_2601_12698_b200 import synth
    out = [("bf16", t, 4096, 1) for t in (1, 4, 16, 64, 256)]                        # the decode configuration
    out += [("fp32", m, n, 40) for m, n in synth.PAPER_SHAPES_FP32]
    out += [(d, m, n, 41) for d in ("bf16", "fp16") for m, n in synth.PAPER_SHAPES_16BIT]
    return out


@pytest.mark.parametrize("dtype,T,H,seed", _named_shapes())
def test_named_shapes_every_feasible_theta(B, oracle_lib, dtype, T, H, seed):
    from paper_2601_12698_b200 import synth
    x, r, w = synth.make_inputs(T, H, dtype, seed=seed)
    # the decode shapes take every hard-feasible theta; the larger paper shapes the set the search works on
    thetas = B.tuner_derive_feasible(B.shape_of(T, H, dtype), heuristics=0 if T <= 256 and H <= 4096 else B.RT_PRUNE_DEFAULT)
    n, failures, worst = _run_all(B, oracle_lib, x, r, w, dtype, thetas)
    assert n > 50 and not failures, f"{len(failures)} of {n} configurations differ: {failures[:5]}"


def _closed_form_rows(dtype: str, H: int):
    """(x, r, w): rows whose x + r is a constant, one-hot, +-1, ones with one outlier, or at the edge of the range."""
    td = TD[dtype]
    rows = []
    for c in (1.0, 0.1, 3.3, 1.7, 1.4142135, 0.70710678, 1.6202135, 1e-3, 300.0, -2.5):
        rows.append(torch.full((H,), c))                               # constant: y = w c / sqrt(c^2 + eps)
    for k in (0, H // 3, H - 1):
        e = torch.zeros(H); e[k] = 7.0
        rows.append(e)                                                 # one-hot: every other y is exactly 0
    alt = torch.ones(H); alt[1::2] = -1.0
    rows.append(alt)                                                   # +-1: mean square exactly 1
    out = torch.ones(H); out[H // 2] = 1e4
    rows.append(out)                                                   # ones with one outlier of 1e4
    big = 60000.0 if dtype == "fp16" else 1e15
    rows.append(torch.full((H,), big)); rows.append(torch.full((H,), -big))   # the edge of the fp16 range / squares of 1e30
    rows.append(torch.full((H,), 2.0 ** -14 if dtype == "fp16" else 1e-18))   # tiny squares: eps dominates
    s = torch.stack(rows)
    g = torch.Generator().manual_seed(H)
    x = (s * 0.75).to(td)                                              # two addends whose binary32 sum is the row
    r = (s.to(td).float() - x.float()).to(td)
    w = (1.0 + 0.1 * torch.randn(H, generator=g)).to(td)
    return x.contiguous(), r.contiguous(), w.contiguous()


@pytest.mark.parametrize("dtype", ["bf16", "fp16", "fp32"])
@pytest.mark.parametrize("H", [4096, 8192, 12288])
def test_closed_form_rows_through_every_stage(B, oracle_lib, dtype, H):
    x, r, w = _closed_form_rows(dtype, H)
    T = x.shape[0]
    thetas = B.tuner_derive_feasible(B.shape_of(T, H, dtype), heuristics=0)   # hard rules only: the widest net
    per_thread = max(H // t.threads_per_row // max(1, t.cluster_size) for t in thetas)
    assert per_thread >= (384 if H == 12288 else 128)
    assert {t.stage for t in thetas} == {0, 1, 2, 4}
    n, failures, worst = _run_all(B, oracle_lib, x, r, w, dtype, thetas)
    print(f"closed-form rows {dtype} H={H}: {n} thetas, up to {per_thread} elements per thread, worst y error {worst:.3g}")
    assert not failures, f"{len(failures)} of {n} configurations differ: {failures[:5]}"
    if dtype == "fp32":
        assert worst <= 5e-6          # half the tolerance: the chain of additions is one per vector, not per element


def test_closed_forms_hold_on_the_device(B):
    """The same rows against the closed forms themselves (no oracle in between): constant rows give
    w c / sqrt(c^2 + eps), one-hot rows are zero off the hot column, +-1 rows give +-w / sqrt(1 + eps)."""
    H = 8192
    x, r, w = _closed_form_rows("fp32", H)
    xd, rd, wd = x.cuda(), r.cuda(), w.cuda()
    y, ro = torch.empty_like(xd), torch.empty_like(xd)
    B.rmsnorm_template_launch(B.make_params(threads_per_row=256, vec_bytes=32, unroll=2), xd, rd, wd, y, ro, EPS)
    y, s, w64 = y.cpu().double(), (x.double() + r.double()), w.double()
    for row in range(10):                                               # the constants
        c = s[row, 0]
        want = w64 * c / torch.sqrt(c * c + float(torch.tensor(EPS, dtype=torch.float32)))
        assert torch.allclose(y[row], want, rtol=2e-6, atol=0)
    for row, k in zip((10, 11, 12), (0, H // 3, H - 1)):
        assert float(y[row].abs().sum() - y[row, k].abs()) == 0.0
        assert abs(float(y[row, k]) - float(w64[k] * 7.0 / (49.0 / H + 1e-6) ** 0.5)) <= 2e-6 * abs(float(y[row, k]))
    assert torch.allclose(y[13], s[13] * w64 / (1.0 + 1e-6) ** 0.5, rtol=2e-6, atol=0)


@pytest.mark.parametrize("dtype,T,H", [("fp32", 3, 57856), ("bf16", 3, 57856), ("bf16", 2, 462336), ("fp32", 2, 200000)])
def test_the_longest_rows_the_template_serves(B, oracle_lib, dtype, T, H):
    """Maximum sizes: the longest row one CTA serves (57 856 elements, shared-memory stage), the longest a cluster of 8
    serves (462 336), and a length in between - every theta the deriver offers."""
    from paper_2601_12698_b200 import synth
    x, r, w = synth.make_inputs(T, H, dtype, seed=50)
    thetas = B.tuner_derive_feasible(B.shape_of(T, H, dtype), heuristics=0)
    assert thetas and (H <= 57856 or {t.cluster_size for t in thetas} <= {4, 8})
    n, failures, worst = _run_all(B, oracle_lib, x, r, w, dtype, thetas)
    assert not failures, f"{len(failures)} of {n} configurations differ: {failures[:5]}"
    # one element more than the chip holds is refused, and nothing is launched
    before = B.rt_launch_count()
    assert B.tuner_derive_feasible(B.shape_of(T, 462336 + 64, dtype), heuristics=0) == []
    assert B.rt_launch_count() == before
