"""merge_attn_states: every feasible theta against the CPU oracle, edge cases, refusals, search, full size."""
import pytest
import torch

pytestmark = pytest.mark.gpu
TD = {"bf16": torch.bfloat16, "fp16": torch.float16, "fp32": torch.float32}
NEG_INF = float("-inf")


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2601_12698_b200 import binding
    torch.cuda.set_device(0)
    return binding


def _tol(dtype):
    return 1e-5 if dtype == "fp32" else 2.0


def _assert_close(oracle_lib, v, s, v_ref, s_ref, dtype, what):
    worst, bad = oracle_lib.compare_mixed(v.cpu(), v_ref, tol=_tol(dtype), tol_abs=1e-5)
    assert bad == 0, (what, "v_out", worst)
    worst, bad = oracle_lib.compare_mixed(s.cpu(), s_ref, tol=1e-5, tol_abs=1e-5)
    assert bad == 0, (what, "s_out", worst)


@pytest.mark.parametrize("dtype", ["bf16", "fp16", "fp32"])
@pytest.mark.parametrize("n,h,d", [(1, 1, 8), (3, 2, 64), (5, 32, 128), (2, 40, 128), (2, 32, 256), (130, 8, 64), (3, 5, 100),
                                   (2, 7, 66), (2, 3, 33)])
def test_every_feasible_theta_matches_oracle(B, oracle_lib, dtype, n, h, d):
    from paper_2601_12698_b200 import synth
    va, sa, vb, sb = synth.make_merge_inputs(0, n, h, d, dtype, seed=300 + d)
    # edge cases in the first rows: an empty part, both empty, far-apart and equal log-sum-exps
    sa, sb = sa.clone(), sb.clone()
    sa[0, 0] = NEG_INF
    if h > 1:
        sa[0, 1] = NEG_INF; sb[0, 1] = NEG_INF
    if n > 1:
        sa[1, 0] = 60.0; sb[1, 0] = -60.0
        sa[1, -1] = sb[1, -1]
    v_ref, s_ref = oracle_lib.merge_attn_states(va, sa, vb, sb)
    dev = [t.cuda() for t in (va, sa, vb, sb)]
    n_el = n * h * d
    full = torch.full((n_el + 128,), -7.0, dtype=TD[dtype], device="cuda")
    v_out = full[64:64 + n_el].view(n, h, d)
    s_full = torch.full((n * h + 16,), -7.0, dtype=torch.float32, device="cuda")
    s_out = s_full[8:8 + n * h].view(n, h)
    shape = B.shape_of(n, h * d, dtype, B._ptr_align(dev[0], dev[2], v_out), op=B.RT_OP_MERGE_ATTN_STATES, head_dim=d)
    thetas = B.tuner_derive_feasible(shape, heuristics=0)
    assert thetas and {t.stage for t in thetas} <= {0, 2} and {t.reduce for t in thetas} == {0}
    v_ref_d, s_ref_d = v_ref.cuda(), s_ref.cuda()
    bad = []
    for th in thetas:
        v_out.fill_(float("nan")); s_out.fill_(float("nan"))
        B.merge_attn_states_template_launch(th, dev[0], dev[1], dev[2], dev[3], v_out, s_out)
        worst_v, bad_v = B.tuner_compare_mixed(v_out, v_ref_d, _tol(dtype), 1e-5)
        worst_s, bad_s = B.tuner_compare_mixed(s_out, s_ref_d, 1e-5, 1e-5)
        if bad_v or bad_s:
            bad.append((repr(th), worst_v, bad_v, worst_s, bad_s))
    assert B.rt_device_status() == 0
    assert bool((full[:64] == -7.0).all()) and bool((full[64 + n_el:] == -7.0).all()), "wrote outside v_out"
    assert bool((s_full[:8] == -7.0).all()) and bool((s_full[8 + n * h:] == -7.0).all()), "wrote outside s_out"
    assert not bad, f"{len(bad)} of {len(thetas)} differ: {bad[:3]}"
    _assert_close(oracle_lib, v_out, s_out, v_ref, s_ref, dtype, "last theta")  # the oracle's own comparator agrees
    # exact special cases, bit for bit: an empty part returns the other part; both empty give zeros and -inf
    assert torch.equal(v_out[0, 0].cpu(), vb[0, 0]) and float(s_out[0, 0]) == float(sb[0, 0])
    if h > 1:
        assert bool((v_out[0, 1] == 0).all()) and float(s_out[0, 1]) == NEG_INF
    if n > 1:
        assert torch.equal(v_out[1, 0].cpu(), va[1, 0]) and float(s_out[1, 0]) == 60.0


def test_mixed_comparator_agrees_with_oracle(B, oracle_lib):
    g = torch.Generator().manual_seed(4)
    ref = torch.randn(5000, generator=g).bfloat16()
    got = ref.clone()
    idx = torch.randperm(5000, generator=g)[:300]
    got.view(torch.int16)[idx] += torch.randint(-4, 5, (300,), generator=g).to(torch.int16)
    for tol, tol_abs in ((2.0, 0.0), (2.0, 1e-3), (0.0, 1e-2)):
        worst_o, bad_o = oracle_lib.compare_mixed(got, ref, tol=tol, tol_abs=tol_abs)
        worst_d, bad_d = B.tuner_compare_mixed(got.cuda(), ref.cuda(), tol, tol_abs)
        assert bad_d == bad_o and abs(worst_d - worst_o) <= 1e-6 * max(worst_o, 1e-9)
    a = torch.randn(4097, generator=g)
    b = a * (1 + 3e-5 * torch.randn(4097, generator=g))
    for tol, tol_abs in ((1e-5, 0.0), (1e-5, 1e-5), (1e-7, 1e-7)):
        assert B.tuner_compare_mixed(b.cuda(), a.cuda(), tol, tol_abs)[1] == oracle_lib.compare_mixed(b, a, tol=tol, tol_abs=tol_abs)[1]


def test_refusals(B):
    n, h, d = 4, 8, 128
    v = torch.zeros(n, h, d, dtype=torch.bfloat16, device="cuda")
    s = torch.zeros(n, h, dtype=torch.float32, device="cuda")
    out = torch.full_like(v, 3.0); so = torch.full_like(s, 3.0)
    call = B.lib.merge_attn_states_template_launch
    before = B.rt_launch_count()
    args = (v.data_ptr(), s.data_ptr(), v.data_ptr(), s.data_ptr(), out.data_ptr(), so.data_ptr())
    for th in (B.make_params(reduce=B.RT_REDUCE_SMEM), B.make_params(stage=B.RT_STAGE_SMEM_LDG),
               B.make_params(reduce=B.RT_REDUCE_CLUSTER, cluster_size=2), B.make_params(threads_per_row=1024, rows_per_cta=2)):
        assert call(B.byref(th), *args, n, h, d, B.RT_BF16, None) == B.RT_ERR_INFEASIBLE
    th = B.make_params()
    assert call(B.byref(th), *args, n, h, 100, B.RT_BF16, None) == B.RT_ERR_ALIGN       # heads of 200 bytes, 16-byte vectors
    assert call(B.byref(th), *args, n, 0, d, B.RT_BF16, None) == B.RT_ERR_SHAPE
    assert call(B.byref(th), None, *args[1:], n, h, d, B.RT_BF16, None) == B.RT_ERR_NULL
    assert call(B.byref(th), *args, n, h, d, 6, None) == B.RT_ERR_DTYPE
    assert call(B.byref(th), args[0], s.data_ptr() + 2, *args[2:], n, h, d, B.RT_BF16, None) == B.RT_ERR_ALIGN
    assert call(B.byref(th), None, None, None, None, None, None, 0, h, d, B.RT_BF16, None) == B.RT_OK
    torch.cuda.synchronize()
    assert B.rt_launch_count() == before and bool((out == 3.0).all()) and bool((so == 3.0).all())


@pytest.mark.parametrize("name", ["merge_bf16_512x40x128", "merge_bf16_768x32x256", "merge_bf16_32768x32x128"])
def test_search_and_full_size_parity(B, oracle_lib, name):
    from paper_2601_12698_b200 import synth
    wl = synth.workloads()[name]
    h, d = wl.hidden // wl.head_dim, wl.head_dim
    va, sa, vb, sb = synth.make_workload_inputs(wl)
    n_ref = min(wl.n_tokens, 256)
    v_ref, s_ref = oracle_lib.merge_attn_states(va[:n_ref].contiguous(), sa[:n_ref].contiguous(),
                                                vb[:n_ref].contiguous(), sb[:n_ref].contiguous())
    dev = [t.cuda() for t in (va, sa, vb, sb)]
    v_out, s_out = torch.empty_like(dev[0]), torch.empty_like(dev[1])
    stream = torch.cuda.Stream()
    ws = B.make_workspace(dev[0], dev[2], dev[1], v_out, s_out, v_ref.cuda(), s_ref.cuda(), 0.0, n_ref_tokens=n_ref,
                          stream=stream, aux=dev[3])
    shape = B.shape_of(wl.n_tokens, wl.hidden, wl.dtype, op=B.RT_OP_MERGE_ATTN_STATES, head_dim=d)
    res, log = B.tuner_search(shape, B.make_budget(max_evals=24, warmup=2, iters=5, repeats=1, top_k=2), ws)
    assert res.n_failed_gate == 0 and res.evals_used <= 24
    rows = sorted({0, 1, wl.n_tokens // 2, wl.n_tokens - 1} |
                  {int(v) for v in torch.randint(0, wl.n_tokens, (16,), generator=torch.Generator().manual_seed(9))})
    v_rows, s_rows = oracle_lib.merge_attn_states(va[rows].contiguous(), sa[rows].contiguous(), vb[rows].contiguous(),
                                                  sb[rows].contiguous())
    feasible = B.tuner_derive_feasible(shape)
    for th in [res.best] + [t for t in feasible if t.stage == 0][:1] + [t for t in feasible if t.stage == 2][:1]:
        v_out.fill_(float("nan")); s_out.fill_(float("nan"))
        B.merge_attn_states_template_launch(th, dev[0], dev[1], dev[2], dev[3], v_out, s_out)
        _assert_close(oracle_lib, v_out[rows], s_out[rows], v_rows, s_rows, wl.dtype, repr(th))
        assert not bool(torch.isnan(v_out).any()) and not bool(torch.isnan(s_out).any())
    assert B.rt_device_status() == 0
