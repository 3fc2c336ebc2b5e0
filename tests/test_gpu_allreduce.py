"""The tensor-parallel form of the norm (all-reduce folded into the kernel) against the CPU oracle.

One GPU stands in for the whole group: the partial inputs and the output tensors of all ranks live on this GPU and
each rank's launch (its own block of rows, all ranks' partials in, all ranks' outputs out) runs one after the other.
No launch waits on another, so this is the same code path a group of GPUs runs with peer-mapped pointers."""
import pytest
import torch

pytestmark = pytest.mark.gpu
EPS = 1e-6
INT_VIEW = {"bf16": torch.int16, "fp16": torch.int16, "fp32": torch.int32}


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2601_12698_b200 import binding
    torch.cuda.set_device(0)
    return binding


def _inputs(T, H, dtype, n_parts, seed):
    from paper_2601_12698_b200 import synth
    _, r, w = synth.make_inputs(T, H, dtype, seed)
    parts = synth.make_parts(0, T, H, dtype, seed, n_parts)
    if T > 2:
        parts[:, 1].zero_(); r[1].zero_()                     # a row of zeros
        parts[:, 2] *= 64.0                                     # a loud row: binary32 sums that really round
    return parts, r, w


def _assert_matches(oracle_lib, y, ro, y_ref, r_ref, what):
    assert oracle_lib.bit_mismatches(ro.cpu(), r_ref) == 0, (what, "r_out")
    worst, bad = oracle_lib.compare_y(y.cpu(), y_ref)
    assert bad == 0, (what, "y", worst)


@pytest.mark.parametrize("dtype", ["bf16", "fp16", "fp32"])
@pytest.mark.parametrize("n_parts", [2, 4, 8])
@pytest.mark.parametrize("T,H", [(1, 8), (3, 64), (37, 1000), (5, 4096), (130, 1024), (11, 8192)])
def test_group_emulated_on_one_gpu_every_theta(B, oracle_lib, dtype, n_parts, T, H):
    from paper_2601_12698_b200 import dp
    parts, r, w = _inputs(T, H, dtype, n_parts, seed=500 + H % 71 + n_parts)
    y_ref, r_ref = oracle_lib.allreduce_add_rmsnorm(parts, r, w, EPS)
    pd, rd, wd = parts.cuda(), r.cuda(), w.cuda()
    x_parts = [pd[k] for k in range(n_parts)]
    y_ref_d, r_ref_d = y_ref.cuda(), r_ref.cuda()
    shape = B.shape_of(max(1, (T + n_parts - 1) // n_parts), H, dtype, op=B.RT_OP_ADD_RMSNORM_ALLREDUCE, n_parts=n_parts)
    thetas = B.tuner_derive_feasible(shape, heuristics=0)
    assert thetas and {t.stage for t in thetas} == {0} and 16 in {t.vec_bytes for t in thetas} and \
        {t.vec_bytes for t in thetas} <= {16, 32}
    # guard bands around every destination
    n = T * H
    y_full = torch.zeros(n_parts, n + 256, dtype=pd.dtype, device="cuda")
    r_full = torch.zeros(n_parts, n + 256, dtype=pd.dtype, device="cuda")
    y_outs = [y_full[k, 128:128 + n].view(T, H) for k in range(n_parts)]
    r_outs = [r_full[k, 128:128 + n].view(T, H) for k in range(n_parts)]
    bad = []
    for th in thetas:
        for t in y_outs + r_outs:
            t.fill_(float("nan"))
        for rank in range(n_parts):
            sh = dp.strong_shard(T, rank, n_parts)
            B.rmsnorm_allreduce_template_launch(th, x_parts, rd, wd, y_outs, r_outs, sh.row_begin, sh.rows, EPS)
        for k in range(n_parts):
            _, r_bad = B.tuner_compare(r_outs[k].contiguous(), r_ref_d, B.RT_CMP_BITS)
            worst, y_bad = B.tuner_compare(y_outs[k].contiguous(), y_ref_d,
                                           B.RT_CMP_REL32 if dtype == "fp32" else B.RT_CMP_ULP16, 1e-5 if dtype == "fp32" else 2.0)
            if r_bad or y_bad:
                bad.append((repr(th), k, r_bad, y_bad, worst))
        # every rank holds the same bits: each row was computed once and sent to all
        for k in range(1, n_parts):
            assert torch.equal(y_outs[k].view(INT_VIEW[dtype]), y_outs[0].view(INT_VIEW[dtype])), repr(th)
    assert not bad, f"{len(bad)} differ: {bad[:3]}"
    assert bool((y_full[:, :128] == 0).all()) and bool((y_full[:, 128 + n:] == 0).all()), "wrote outside y"
    assert bool((r_full[:, :128] == 0).all()) and bool((r_full[:, 128 + n:] == 0).all()), "wrote outside r_out"
    _assert_matches(oracle_lib, y_outs[-1], r_outs[-1], y_ref, r_ref, "last theta")


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_one_shot_form_and_in_place_residual(B, oracle_lib, dtype):
    T, H, n_parts = 67, 5120, 4
    parts, r, w = _inputs(T, H, dtype, n_parts, seed=611)
    y_ref, r_ref = oracle_lib.allreduce_add_rmsnorm(parts, r, w, EPS)
    pd, wd = parts.cuda(), w.cuda()
    x_parts = [pd[k] for k in range(n_parts)]
    th = B.make_params(threads_per_row=256, unroll=2)
    # one destination, all rows, the residual updated in place
    rd = r.cuda()
    y = torch.full_like(rd, float("nan"))
    B.rmsnorm_allreduce_template_launch(th, x_parts, rd, wd, [y], [rd], 0, T, EPS)
    _assert_matches(oracle_lib, y, rd, y_ref, r_ref, "one shot, in place")
    # a block of rows only: the others stay untouched
    rd = r.cuda()
    y = torch.full_like(rd, 7.0)
    ro = torch.full_like(rd, 7.0)
    B.rmsnorm_allreduce_template_launch(th, x_parts, rd, wd, [y], [ro], 20, 30, EPS)
    _assert_matches(oracle_lib, y[20:50], ro[20:50], y_ref[20:50].contiguous(), r_ref[20:50].contiguous(), "rows 20..50")
    assert bool((y[:20] == 7.0).all()) and bool((y[50:] == 7.0).all()) and bool((ro[:20] == 7.0).all()) and bool((ro[50:] == 7.0).all())
    # no rows: nothing is launched
    before = B.rt_launch_count()
    B.rmsnorm_allreduce_template_launch(th, x_parts, rd, wd, [y], [ro], 5, 0, EPS)
    assert B.rt_launch_count() == before


def test_order_of_the_sum_is_rank_order(B):
    # parts (2^24, 1, 0, -2^24) in binary32: rank order gives fl(2^24 + 1) = 2^24 and then 0, any exact sum gives 1
    H = 8
    parts = torch.zeros(4, 1, H, dtype=torch.float32)
    parts[0, 0, 0], parts[1, 0, 0], parts[3, 0, 0] = 2.0 ** 24, 1.0, -(2.0 ** 24)
    parts[0, 0, 1], parts[1, 0, 1], parts[3, 0, 1] = 2.0 ** 24, -(2.0 ** 24), 1.0
    pd = parts.cuda()
    r = torch.zeros(1, H, device="cuda"); r[0, 2] = 3.0
    w = torch.ones(H, device="cuda")
    y = torch.empty_like(r); ro = torch.empty_like(r)
    B.rmsnorm_allreduce_template_launch(B.make_params(threads_per_row=32), [pd[k] for k in range(4)], r, w, [y], [ro], 0, 1, 0.0)
    assert ro.cpu().tolist() == [[0.0, 1.0, 3.0, 0.0, 0.0, 0.0, 0.0, 0.0]]


def test_refusals(B):
    T, H = 8, 4096
    x = [torch.zeros(T, H, dtype=torch.bfloat16, device="cuda") for _ in range(4)]
    r = torch.zeros(T, H, dtype=torch.bfloat16, device="cuda"); w = torch.ones(H, dtype=torch.bfloat16, device="cuda")
    y = torch.full_like(r, 9.0); ro = torch.full_like(r, 9.0)
    vp = B.c_void_p

    def arr(ts):
        return (vp * len(ts))(*[t.data_ptr() if t is not None else None for t in ts])

    def call(th, xs=x, n_parts=None, r_=r, w_=w, ys=(y,), ros=(ro,), n_y=None, n_r=None, row_begin=0, rows=T, hidden=H,
             dtype=B.RT_BF16):
        return B.lib.rmsnorm_allreduce_template_launch(
            B.byref(th), arr(list(xs)) if xs is not None else None, len(xs) if n_parts is None else n_parts,
            r_.data_ptr() if r_ is not None else None, w_.data_ptr(), arr(list(ys)), len(ys) if n_y is None else n_y,
            arr(list(ros)), len(ros) if n_r is None else n_r, row_begin, rows, hidden, EPS, dtype, None)

    th = B.make_params()
    before = B.rt_launch_count()
    for bad in (B.make_params(vec_bytes=8), B.make_params(reduce=B.RT_REDUCE_SMEM), B.make_params(stage=B.RT_STAGE_SMEM_TMA),
                B.make_params(stage=B.RT_STAGE_SMEM_LDG), B.make_params(reduce=B.RT_REDUCE_CLUSTER, cluster_size=2),
                B.make_params(unroll=3), B.make_params(threads_per_row=48)):
        assert call(bad) == B.RT_ERR_INFEASIBLE, repr(bad)
    assert call(th, xs=x[:3]) == B.RT_ERR_SHAPE                        # three parts
    assert call(th, n_y=0) == B.RT_ERR_SHAPE and call(th, n_r=0) == B.RT_ERR_SHAPE
    assert call(th, ys=[y] * 9) == B.RT_ERR_SHAPE and call(th, ros=[ro] * 9) == B.RT_ERR_SHAPE
    assert call(th, row_begin=-1) == B.RT_ERR_SHAPE and call(th, rows=-2) == B.RT_ERR_SHAPE
    assert call(th, ys=[x[1]]) == B.RT_ERR_SHAPE and call(th, ros=[ro, x[3]]) == B.RT_ERR_SHAPE   # would overwrite a part
    assert call(th, xs=x[:3] + [None]) == B.RT_ERR_NULL
    assert call(th, r_=None) == B.RT_ERR_NULL
    assert call(th, xs=None, n_parts=4) == B.RT_ERR_NULL
    assert call(th, ys=[y, None]) == B.RT_ERR_NULL
    assert call(th, hidden=4100) == B.RT_ERR_ALIGN
    off = torch.zeros(T * H + 8, dtype=torch.bfloat16, device="cuda")[4:4 + T * H].view(T, H)   # 8-byte aligned only
    assert call(th, xs=[off] + x[1:]) == B.RT_ERR_ALIGN
    assert call(th, dtype=7) == B.RT_ERR_DTYPE
    # a 32-thread row of 1024 vectors would keep 32 vectors per thread: no such instance
    x8 = [torch.zeros(2, 8192, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    r8 = torch.zeros(2, 8192, dtype=torch.bfloat16, device="cuda"); w8 = torch.ones(8192, dtype=torch.bfloat16, device="cuda")
    assert call(B.make_params(threads_per_row=32), xs=x8, r_=r8, w_=w8, ys=[r8.clone()], ros=[r8.clone()], rows=2,
                hidden=8192) == B.RT_ERR_INFEASIBLE
    torch.cuda.synchronize()
    assert B.rt_launch_count() == before and bool((y == 9.0).all()) and bool((ro == 9.0).all())


def test_residual_stays_with_the_owner_of_the_rows(B, oracle_lib):
    """The usual group form: y goes to every rank, the new residual only to the rank that owns the rows."""
    from paper_2601_12698_b200 import dp
    T, H, n_parts = 45, 2048, 4
    parts, r, w = _inputs(T, H, "bf16", n_parts, seed=633)
    y_ref, r_ref = oracle_lib.allreduce_add_rmsnorm(parts, r, w, EPS)
    pd, wd = parts.cuda(), w.cuda()
    x_parts = [pd[k] for k in range(n_parts)]
    residual = [r.cuda() for _ in range(n_parts)]                      # every rank's copy of the residual stream
    y_outs = [torch.full((T, H), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(n_parts)]
    th = B.make_params(threads_per_row=256)
    for rank in range(n_parts):
        sh = dp.strong_shard(T, rank, n_parts)
        B.rmsnorm_allreduce_template_launch(th, x_parts, residual[rank], wd, y_outs, [residual[rank]], sh.row_begin, sh.rows, EPS)
    for rank in range(n_parts):
        sh = dp.strong_shard(T, rank, n_parts)
        worst, bad = oracle_lib.compare_y(y_outs[rank].cpu(), y_ref)
        assert bad == 0, (rank, worst)
        own = slice(sh.row_begin, sh.row_end)
        assert oracle_lib.bit_mismatches(residual[rank][own].cpu().contiguous(), r_ref[own].contiguous()) == 0
        others = torch.ones(T, dtype=torch.bool); others[own] = False
        assert torch.equal(residual[rank].cpu()[others].view(torch.int16), r[others].view(torch.int16))  # untouched


@pytest.mark.parametrize("name", ["c2ar8_decode_bf16_64x8192", "c3ar4_prefill_bf16_4096x8192"])
def test_search_on_the_stacked_workspace_and_sampled_parity(B, oracle_lib, name):
    from paper_2601_12698_b200 import synth
    wl = synth.workloads()[name]
    parts, r, w = synth.make_workload_inputs(wl)
    n_ref = min(wl.n_tokens, 128)
    y_ref, r_ref = oracle_lib.allreduce_add_rmsnorm(parts[:, :n_ref].contiguous(), r[:n_ref].contiguous(), w, wl.eps)
    pd, rd, wd = parts.cuda(), r.cuda(), w.cuda()
    y = torch.empty_like(rd); ro = torch.empty_like(rd)
    stream = torch.cuda.Stream()
    ws = B.make_workspace(pd, rd, wd, y, ro, y_ref.cuda(), r_ref.cuda(), wl.eps, n_ref_tokens=n_ref, stream=stream)
    shape = B.shape_of(wl.n_tokens, wl.hidden, wl.dtype, op=B.RT_OP_ADD_RMSNORM_ALLREDUCE, n_parts=wl.n_parts)
    res, log = B.tuner_search(shape, B.make_budget(max_evals=20, warmup=2, iters=5, repeats=1, top_k=2), ws)
    assert res.n_failed_gate == 0 and 1 <= res.evals_used <= 20 and res.best_us > 0
    feasible = {t.key() for t in B.tuner_derive_feasible(shape)}
    assert res.best.key() in feasible
    rows = sorted({0, 1, wl.n_tokens // 2, wl.n_tokens - 1} |
                  {int(v) for v in torch.randint(0, wl.n_tokens, (12,), generator=torch.Generator().manual_seed(5))})
    y_rows, r_rows = oracle_lib.allreduce_add_rmsnorm(parts[:, rows].contiguous(), r[rows].contiguous(), w, wl.eps)
    y.fill_(float("nan")); ro.fill_(float("nan"))
    B.rmsnorm_allreduce_template_launch(res.best, [pd[k] for k in range(wl.n_parts)], rd, wd, [y], [ro], 0, wl.n_tokens, wl.eps)
    _assert_matches(oracle_lib, y[rows], ro[rows], y_rows, r_rows, repr(res.best))
    assert not bool(torch.isnan(y.float()).any()) and not bool(torch.isnan(ro.float()).any())


def test_shipped_table_drives_the_launch(B, oracle_lib):
    table = B.SpecTable.default()
    assert B.RT_OP_ADD_RMSNORM_ALLREDUCE in table.generals
    for n_parts, T, H in ((8, 64, 8192), (4, 300, 8192), (2, 9, 1024)):
        parts, r, w = _inputs(T, H, "bf16", n_parts, seed=650 + n_parts)
        y_ref, r_ref = oracle_lib.allreduce_add_rmsnorm(parts, r, w, EPS)
        pd, rd, wd = parts.cuda(), r.cuda(), w.cuda()
        y, ro = torch.full_like(rd, float("nan")), torch.full_like(rd, float("nan"))
        theta = table.launch_rmsnorm_allreduce([pd[k] for k in range(n_parts)], rd, wd, [y], [ro], 0, T, EPS)
        shape = B.shape_of(T, H, "bf16", op=B.RT_OP_ADD_RMSNORM_ALLREDUCE, n_parts=n_parts)
        assert B.tuner_check_params(shape, theta) == B.RT_OK
        if (n_parts, T, H) == (8, 64, 8192):
            assert table.lookup(shape)[1] == "table_exact"
        _assert_matches(oracle_lib, y, ro, y_ref, r_ref, (n_parts, T, H, repr(theta)))
