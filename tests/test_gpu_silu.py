"""silu_and_mul: every feasible theta against the CPU oracle, refusals, the search, a full-size workload."""
import pytest
import torch

pytestmark = pytest.mark.gpu
TD = {"bf16": torch.bfloat16, "fp16": torch.float16, "fp32": torch.float32}


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2601_12698_b200 import binding
    torch.cuda.set_device(0)
    return binding


def _check(B, oracle_lib, out, ref, dtype, what):
    worst, bad = oracle_lib.compare_y(out.cpu(), ref, tol_ulp=2, tol_rel=1e-5)
    assert bad == 0, (what, worst)


@pytest.mark.parametrize("dtype", ["bf16", "fp16", "fp32"])
@pytest.mark.parametrize("T,d", [(1, 8), (3, 64), (2, 1000), (5, 4096), (130, 1024), (3, 11008), (2, 13824), (2, 3076),
                                 (2, 3074), (3, 3073)])
def test_every_feasible_theta_matches_oracle(B, oracle_lib, dtype, T, d):
    from paper_2601_12698_b200 import synth
    x = synth.make_gate_up(0, T, d, dtype, seed=200 + d % 89)
    x[0, : min(4, d)] = torch.tensor([0.0, -60.0, 45.0, -100.0][: min(4, d)]).to(TD[dtype])  # exact zero and the tails
    ref = oracle_lib.silu_and_mul(x)
    xd = x.cuda()
    n = T * d
    full = torch.full((n + 128,), -7.0, dtype=TD[dtype], device="cuda")
    out = full[64:64 + n].view(T, d)
    shape = B.shape_of(T, d, dtype, B._ptr_align(xd, out), op=B.RT_OP_SILU_AND_MUL)
    thetas = B.tuner_derive_feasible(shape, heuristics=0)
    assert thetas and {t.stage for t in thetas} <= {0, 2} and {t.reduce for t in thetas} == {0}
    ref_d = ref.cuda()
    bad = []
    for th in thetas:
        out.fill_(float("nan"))
        B.silu_and_mul_template_launch(th, xd, out)
        if dtype == "fp32":
            worst, n_bad = B.tuner_compare(out, ref_d, B.RT_CMP_REL32, 1e-5)
        else:
            worst, n_bad = B.tuner_compare(out, ref_d, B.RT_CMP_ULP16, 2.0)
        if n_bad:
            bad.append((repr(th), worst, n_bad))
    assert B.rt_device_status() == 0
    assert bool((full[:64] == -7.0).all()) and bool((full[64 + n:] == -7.0).all()), "wrote outside the output"
    assert not bad, f"{len(bad)} of {len(thetas)} differ: {bad[:4]}"
    # the device comparator's verdict is the oracle comparator's
    _check(B, oracle_lib, out, ref, dtype, "last theta")


def test_refusals(B):
    x = torch.zeros(4, 8192, dtype=torch.bfloat16, device="cuda")
    out = torch.full((4, 4096), 3.0, dtype=torch.bfloat16, device="cuda")
    before = B.rt_launch_count()
    for th in (B.make_params(reduce=B.RT_REDUCE_SMEM), B.make_params(reduce=B.RT_REDUCE_CLUSTER, cluster_size=2),
               B.make_params(stage=B.RT_STAGE_SMEM_LDG), B.make_params(threads_per_row=1024, rows_per_cta=2),
               B.make_params(unroll=3)):
        st = B.lib.silu_and_mul_template_launch(B.byref(th), x.data_ptr(), out.data_ptr(), 4, 4096, B.RT_BF16, None)
        assert st == B.RT_ERR_INFEASIBLE, repr(th)
    th = B.make_params()
    assert B.lib.silu_and_mul_template_launch(B.byref(th), None, out.data_ptr(), 4, 4096, 0, None) == B.RT_ERR_NULL
    assert B.lib.silu_and_mul_template_launch(B.byref(th), x.data_ptr(), out.data_ptr(), 4, 4097, 0, None) == B.RT_ERR_ALIGN
    assert B.lib.silu_and_mul_template_launch(B.byref(th), x.data_ptr(), out.data_ptr(), 4, 4096, 9, None) == B.RT_ERR_DTYPE
    assert B.lib.silu_and_mul_template_launch(B.byref(th), None, None, 0, 4096, 0, None) == B.RT_OK
    torch.cuda.synchronize()
    assert B.rt_launch_count() == before and bool((out == 3.0).all())


@pytest.mark.parametrize("name", ["silu_bf16_64x11008", "silu_fp32_2048x8192", "silu_bf16_16384x14336"])
def test_search_and_full_size_parity(B, oracle_lib, name):
    from paper_2601_12698_b200 import synth
    wl = synth.workloads()[name]
    (x,) = synth.make_workload_inputs(wl)
    n_ref = min(wl.n_tokens, 256)
    ref = oracle_lib.silu_and_mul(x[:n_ref], threads=8)
    xd = x.cuda()
    out = torch.empty(wl.n_tokens, wl.hidden, dtype=xd.dtype, device="cuda")
    stream = torch.cuda.Stream()
    ws = B.make_workspace(xd, None, None, out, None, ref.cuda(), None, 0.0, n_ref_tokens=n_ref, stream=stream)
    shape = B.shape_of(wl.n_tokens, wl.hidden, wl.dtype, op=B.RT_OP_SILU_AND_MUL)
    res, log = B.tuner_search(shape, B.make_budget(max_evals=24, warmup=2, iters=5, repeats=1, top_k=2), ws)
    assert res.n_failed_gate == 0 and res.evals_used <= 24
    rows = sorted({0, 1, wl.n_tokens // 2, wl.n_tokens - 1} |
                  {int(v) for v in torch.randint(0, wl.n_tokens, (16,), generator=torch.Generator().manual_seed(9))})
    ref_rows = oracle_lib.silu_and_mul(x[rows].contiguous())
    feasible = B.tuner_derive_feasible(shape)
    picks = [res.best] + [t for t in feasible if t.stage == 0][:1] + [t for t in feasible if t.stage == 2][:1]
    for th in picks:
        out.fill_(float("nan"))
        B.silu_and_mul_template_launch(th, xd, out)
        _check(B, oracle_lib, out[rows], ref_rows, wl.dtype, repr(th))
        assert not bool(torch.isnan(out).any())
    assert B.rt_device_status() == 0
