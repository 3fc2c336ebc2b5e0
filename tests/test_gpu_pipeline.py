"""The persistent TMA pipeline stage (RT_STAGE_TMA_PIPELINE): a grid of resident CTAs walking over row blocks with a
ring of shared-memory stages.  Shapes here give every CTA several blocks, so the ring wraps and each stage's mbarrier
goes through several phases; the row count leaves a ragged last block and a ragged last round."""
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


def _pipeline_thetas(B, shape):
    mask = B.RT_PRUNE_DEFAULT & ~B.RT_PRUNE_PIPELINE_STAGE & ~B.RT_PRUNE_DUPLICATES
    return [t for t in B.tuner_derive_feasible(shape, heuristics=mask) if t.stage == B.RT_STAGE_TMA_PIPELINE]


@pytest.mark.parametrize("dtype,T,H", [("bf16", 20011, 512), ("fp16", 9001, 1544), ("fp32", 6007, 1024), ("bf16", 3, 8192),
                                       ("bf16", 1, 4096), ("fp32", 1500, 12288)])
def test_pipeline_stage_matches_oracle(B, oracle_lib, dtype, T, H):
    from paper_2601_12698_b200 import synth
    x, r, w = synth.make_inputs(T, H, dtype, seed=500 + H % 83)
    y_ref, r_ref = oracle_lib.add_rmsnorm(x, r, w, EPS, threads=8)
    xd, rd, wd = x.cuda(), r.cuda(), w.cuda()
    y_ref_d, r_ref_d = y_ref.cuda(), r_ref.cuda()
    shape = B.shape_of(T, H, dtype)
    thetas = _pipeline_thetas(B, shape)
    assert thetas and {t.unroll for t in thetas} == ({1, 2, 4} if H < 12288 else {1, 2})
    limits = B.rt_query_limits()
    if T > 15000:  # the point of this shape: several row blocks per resident CTA whatever the block shape, so the ring wraps
        assert T > 4 * 32 * limits.sm_count
    y, ro = torch.empty_like(xd), torch.empty_like(xd)
    failures = []
    for th in thetas:
        y.fill_(float("nan")); ro.fill_(float("nan"))
        B.rmsnorm_template_launch(th, xd, rd, wd, y, ro, EPS)
        _, r_bad = B.tuner_compare(ro, r_ref_d, B.RT_CMP_BITS)
        if dtype == "fp32":
            worst, y_bad = B.tuner_compare(y, y_ref_d, B.RT_CMP_REL32, 1e-5)
        else:
            worst, y_bad = B.tuner_compare(y, y_ref_d, B.RT_CMP_ULP16, 2.0)
        if r_bad or y_bad:
            failures.append((repr(th), r_bad, y_bad, worst))
    assert B.rt_device_status() == 0
    assert not failures, f"{len(failures)} of {len(thetas)} configurations differ: {failures[:5]}"
    # in place (y over x, r_out over r): a stage is read completely before its rows are written
    for th in thetas[::7]:
        x2, r2 = x.cuda(), r.cuda()
        B.rmsnorm_template_launch(th, x2, r2, wd, x2, r2, EPS)
        assert B.tuner_compare(r2, r_ref_d, B.RT_CMP_BITS)[1] == 0, repr(th)
        mode, tol = (B.RT_CMP_REL32, 1e-5) if dtype == "fp32" else (B.RT_CMP_ULP16, 2.0)
        assert B.tuner_compare(x2, y_ref_d, mode, tol)[1] == 0, repr(th)


def test_pipeline_stage_in_the_search_only_on_request(B, oracle_lib):
    from paper_2601_12698_b200 import synth
    wl = synth.Workload("t", "bf16", 4096, 2048, seed=12)
    x, r, w = synth.make_workload_inputs(wl)
    y_ref, r_ref = oracle_lib.add_rmsnorm(x, r, w, wl.eps, threads=8)
    t = dict(x=x.cuda(), r=r.cuda(), w=w.cuda(), y_ref=y_ref.cuda(), r_ref=r_ref.cuda())
    t["y"], t["r_out"] = torch.empty_like(t["x"]), torch.empty_like(t["x"])
    stream = torch.cuda.Stream()
    ws = B.make_workspace(t["x"], t["r"], t["w"], t["y"], t["r_out"], t["y_ref"], t["r_ref"], wl.eps, stream=stream)
    shape = B.shape_of(wl.n_tokens, wl.hidden, wl.dtype)
    pipe = B.RT_STAGE_TMA_PIPELINE
    res, log = B.tuner_search(shape, B.make_budget(max_evals=40, warmup=1, iters=3, repeats=1, top_k=2), ws)
    assert pipe not in {rec.params.stage for rec in log}
    mask = B.RT_PRUNE_DEFAULT & ~B.RT_PRUNE_PIPELINE_STAGE
    res, log = B.tuner_search(shape, B.make_budget(max_evals=60, warmup=1, iters=3, repeats=1, top_k=2, heuristics=mask), ws)
    mine = [rec for rec in log if rec.params.stage == pipe]
    assert mine and all(rec.status == 0 and rec.r_bad == 0 and rec.y_bad == 0 for rec in mine)
    assert res.n_failed_gate == 0 and B.rt_device_status() == 0


def test_pipeline_stage_reports_an_expired_wait(B):
    """The ring's bounded waits give up like the one-row TMA stage's: no copy is posted, the poll limit is a few hundred."""
    T, H = 2000, 1024
    xd = torch.zeros(T, H, dtype=torch.bfloat16, device="cuda")
    wd = torch.ones(H, dtype=torch.bfloat16, device="cuda")
    y, ro = torch.empty_like(xd), torch.empty_like(xd)
    th = B.make_params(threads_per_row=128, stage=B.RT_STAGE_TMA_PIPELINE, unroll=2)
    try:
        assert B.lib.rt_set_option(B.RT_OPTION_TMA_WAIT_POLL_LIMIT, 200) == B.RT_OK
        assert B.lib.rt_set_option(B.RT_OPTION_DEBUG_DROP_TMA_COPIES, 1) == B.RT_OK
        B.rmsnorm_template_launch(th, xd, xd, wd, y, ro, EPS)
        torch.cuda.synchronize()
        assert B.rt_device_status() == B.RT_ERR_DEVICE_TIMEOUT and B.rt_device_status() == 0
    finally:
        assert B.lib.rt_set_option(B.RT_OPTION_DEBUG_DROP_TMA_COPIES, 0) == B.RT_OK
        assert B.lib.rt_set_option(B.RT_OPTION_TMA_WAIT_POLL_LIMIT, 1 << 24) == B.RT_OK
    B.rmsnorm_template_launch(th, xd, xd, wd, y, ro, EPS)
    torch.cuda.synchronize()
    assert B.rt_device_status() == 0 and bool((ro == 0).all()) and bool((y == 0).all())
