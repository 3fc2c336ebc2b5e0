"""Parity of the CUDA template against the CPU oracle, through the C ABI (needs a B200)."""
import numpy as np
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


def _synth():
    from paper_2601_12698_b200 import synth
    return synth


def _padded(shape, dtype, pad=64):
    """An output buffer with canary words before and after: (view, full, check)."""
    n = int(np.prod(shape))
    full = torch.full((n + 2 * pad,), -7.0, dtype=dtype, device="cuda")
    view = full[pad:pad + n].view(*shape)

    def intact():
        return bool((full[:pad] == -7.0).all().item() and (full[pad + n:] == -7.0).all().item())
    return view, full, intact


def _gate(B, oracle, y, ro, y_ref_d, r_ref_d, dtype):
    """(r_bad, y_bad, y_worst) computed by the library's device comparator."""
    _, r_bad = B.tuner_compare(ro, r_ref_d, B.RT_CMP_BITS)
    if dtype == "fp32":
        worst, y_bad = B.tuner_compare(y, y_ref_d, B.RT_CMP_REL32, 1e-5)
    else:
        worst, y_bad = B.tuner_compare(y, y_ref_d, B.RT_CMP_ULP16, 2.0)
    return r_bad, y_bad, worst


SMALL_SHAPES = [(1, 8), (3, 64), (2, 1000), (5, 4096), (257, 1024), (128, 4096), (3, 5120), (2, 6152), (2, 6148),
                (3, 7168), (2, 8192), (2, 12288)]


@pytest.mark.parametrize("dtype", ["bf16", "fp16", "fp32"])
@pytest.mark.parametrize("T,H", SMALL_SHAPES)
def test_every_feasible_theta_matches_oracle(B, oracle_lib, dtype, T, H):
    synth = _synth()
    x, r, w = synth.make_inputs(T, H, dtype, seed=100 + H % 97)
    y_ref, r_ref = oracle_lib.add_rmsnorm(x, r, w, EPS)
    xd, rd, wd = x.cuda(), r.cuda(), w.cuda()
    y_ref_d, r_ref_d = y_ref.cuda(), r_ref.cuda()
    shape = B.shape_of(T, H, dtype, B._ptr_align(xd, rd, wd))
    # all hard-feasible points, heuristics off: the widest net
    thetas = B.tuner_derive_feasible(shape, heuristics=0)
    assert len(thetas) > 0
    y, y_full, y_ok = _padded((T, H), TD[dtype])
    ro, ro_full, ro_ok = _padded((T, H), TD[dtype])
    shape_out = B.shape_of(T, H, dtype, B._ptr_align(xd, rd, wd, y, ro))
    failures = []
    n_run = 0
    for th in thetas:
        if B.tuner_check_params(shape_out, th) != B.RT_OK:
            continue  # the padded outputs may be less aligned than the inputs
        y.fill_(float("nan")); ro.fill_(float("nan"))
        B.rmsnorm_template_launch(th, xd, rd, wd, y, ro, EPS)
        r_bad, y_bad, worst = _gate(B, oracle_lib, y, ro, y_ref_d, r_ref_d, dtype)
        n_run += 1
        if r_bad or y_bad:
            failures.append((repr(th), r_bad, y_bad, worst))
    assert B.rt_device_status() == 0
    assert y_ok() and ro_ok(), "a kernel wrote outside its output"
    assert n_run > 0
    assert not failures, f"{len(failures)} of {n_run} configurations differ: {failures[:5]}"


RAGGED_SHAPES = [(1, 1), (9, 1), (5, 3), (9, 7), (4, 9), (7, 33), (5, 1001), (3, 4097), (5, 6145), (4, 6146), (3, 6148),
                 (5, 6152), (2, 12289), (5, 4096), (6, 17), (33, 31)]


@pytest.mark.parametrize("dtype", ["bf16", "fp16", "fp32"])
@pytest.mark.parametrize("T,H", RAGGED_SHAPES)
def test_ragged_row_stage_matches_oracle(B, oracle_lib, dtype, T, H):
    """Rows of any byte length through the aligned-chunk stage: every block shape and unroll depth that passes the
    hard rules, written between canaries (the end chunks of a row are shared with its neighbours, or reach past
    the tensor), then in place."""
    synth = _synth()
    x, r, w = synth.make_inputs(T, H, dtype, seed=300 + H % 89)
    y_ref, r_ref = oracle_lib.add_rmsnorm(x, r, w, EPS)
    xd, rd, wd = x.cuda(), r.cuda(), w.cuda()
    y_ref_d, r_ref_d = y_ref.cuda(), r_ref.cuda()
    y, _, y_ok = _padded((T, H), TD[dtype])
    ro, _, ro_ok = _padded((T, H), TD[dtype])
    shape = B.shape_of(T, H, dtype, B._ptr_align(xd, rd, wd, y, ro))
    thetas = [B.make_params(threads_per_row=tpr, rows_per_cta=rpc, unroll=u, vec_bytes=vb, stage=B.RT_STAGE_REG_REALIGN)
              for vb in (16, 32) for tpr in (32, 64, 128, 256, 512, 1024) for rpc in (1, 2, 4, 8) for u in (1, 2, 4)]
    thetas = [th for th in thetas if B.tuner_check_params(shape, th) == B.RT_OK]
    assert {th.vec_bytes for th in thetas} == {16, 32}
    # the deriver offers a chunk width exactly on the rows that width does not divide
    offered = {t.key() for t in B.tuner_derive_feasible(shape, heuristics=0) if t.stage == B.RT_STAGE_REG_REALIGN}
    row_bytes = H * (4 if dtype == "fp32" else 2)
    assert offered == {t.key() for t in thetas if row_bytes % t.vec_bytes != 0}
    failures = []
    for th in thetas:
        y.fill_(float("nan")); ro.fill_(float("nan"))
        B.rmsnorm_template_launch(th, xd, rd, wd, y, ro, EPS)
        r_bad, y_bad, worst = _gate(B, oracle_lib, y, ro, y_ref_d, r_ref_d, dtype)
        if r_bad or y_bad:
            failures.append((repr(th), r_bad, y_bad, worst))
    assert B.rt_device_status() == 0
    assert y_ok() and ro_ok(), "a kernel wrote outside its output"
    assert not failures, f"{len(failures)} of {len(thetas)} configurations differ: {failures[:5]}"
    # in place: y over x and r_out over r, neighbours' rows untouched where a chunk is shared
    for th in thetas[::5]:
        x2, r2 = x.cuda(), r.cuda()
        B.rmsnorm_template_launch(th, x2, r2, wd, x2, r2, EPS)
        r_bad, y_bad, _ = _gate(B, oracle_lib, x2, r2, y_ref_d, r_ref_d, dtype)
        assert (r_bad, y_bad) == (0, 0), repr(th)


@pytest.mark.parametrize("dtype", ["bf16", "fp16", "fp32"])
def test_device_comparator_agrees_with_oracle_comparator(B, oracle_lib, dtype):
    """The gate's own metric is checked against the oracle's comparison routine on perturbed data."""
    synth = _synth()
    x, r, w = synth.make_inputs(37, 515 if dtype != "fp32" else 513, dtype, seed=5)
    y_ref, r_ref = oracle_lib.add_rmsnorm(x, r, w, EPS)
    g = torch.Generator().manual_seed(1)
    got = y_ref.clone()
    flat = got.view(-1)
    idx = torch.randperm(flat.numel(), generator=g)[:200]
    if dtype == "fp32":
        flat[idx] = flat[idx] * (1 + 3e-5 * torch.randn(200, generator=g))
        worst_o, bad_o = oracle_lib.compare_y(got, y_ref, tol_rel=1e-5)
        worst_d, bad_d = B.tuner_compare(got.cuda(), y_ref.cuda(), B.RT_CMP_REL32, 1e-5)
        assert bad_d == bad_o and bad_o > 0
        assert abs(worst_d - worst_o) <= 1e-6 * worst_o
    else:
        bits = flat.view(torch.int16)
        bits[idx] = bits[idx] + torch.randint(-4, 5, (200,), generator=g).to(torch.int16)
        worst_o, bad_o = oracle_lib.compare_y(got, y_ref, tol_ulp=2)
        worst_d, bad_d = B.tuner_compare(got.cuda(), y_ref.cuda(), B.RT_CMP_ULP16, 2.0)
        assert (int(worst_d), bad_d) == (worst_o, bad_o) and bad_o > 0
    n_diff = oracle_lib.bit_mismatches(got, y_ref)
    _, bad_bits = B.tuner_compare(got.cuda(), y_ref.cuda(), B.RT_CMP_BITS)
    assert bad_bits == n_diff
    # odd element count (a trailing half word) and an exact match
    a = y_ref.view(-1)[:1001].contiguous().cuda()
    assert B.tuner_compare(a, a.clone(), B.RT_CMP_BITS) == (0.0, 0)
    if dtype != "fp32":
        b = a.clone(); b[-1] = -b[-1] if float(b[-1]) != 0 else 1.0
        assert B.tuner_compare(a, b, B.RT_CMP_BITS)[1] == 1


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_in_place_aliasing_and_determinism(B, oracle_lib, dtype):
    synth = _synth()
    T, H = 33, 4096
    x, r, w = synth.make_inputs(T, H, dtype, seed=7)
    y_ref, r_ref = oracle_lib.add_rmsnorm(x, r, w, EPS)
    wd = w.cuda()
    shape = B.shape_of(T, H, dtype)
    for th in B.tuner_derive_feasible(shape)[::7]:
        xd, rd = x.cuda(), r.cuda()
        B.rmsnorm_template_launch(th, xd, rd, wd, xd, rd, EPS)  # y over x, r_out over r
        assert oracle_lib.bit_mismatches(rd.cpu(), r_ref) == 0, repr(th)
        assert oracle_lib.compare_y(xd.cpu(), y_ref)[1] == 0, repr(th)
        # the same theta twice gives the same bits
        x2, r2 = x.cuda(), r.cuda()
        y2, o2 = torch.empty_like(x2), torch.empty_like(x2)
        B.rmsnorm_template_launch(th, x2, r2, wd, y2, o2, EPS)
        assert torch.equal(y2.view(torch.int32 if dtype == "fp32" else torch.int16),
                           xd.view(torch.int32 if dtype == "fp32" else torch.int16)), repr(th)


def test_refusals_launch_nothing(B):
    T, H = 4, 4096
    x = torch.zeros(T, H, dtype=torch.bfloat16, device="cuda")
    w = torch.ones(H, dtype=torch.bfloat16, device="cuda")
    y = torch.full_like(x, 5.0); ro = torch.full_like(x, 5.0)
    before = B.rt_launch_count()
    cases = [
        (B.make_params(threads_per_row=1024, rows_per_cta=2), B.RT_ERR_INFEASIBLE),       # 2048 threads
        (B.make_params(threads_per_row=48), B.RT_ERR_INFEASIBLE),                          # not a power of two
        (B.make_params(threads_per_row=32, vec_bytes=16), B.RT_ERR_INFEASIBLE),            # 16 vectors/thread... register stage cap
        (B.make_params(reduce=B.RT_REDUCE_CLUSTER, cluster_size=3), B.RT_ERR_INFEASIBLE),
        (B.make_params(reduce=B.RT_REDUCE_SHFL, cluster_size=2), B.RT_ERR_INFEASIBLE),
        (B.make_params(unroll=3), B.RT_ERR_INFEASIBLE),
        (B.make_params(vec_bytes=12), B.RT_ERR_INFEASIBLE),
        (B.make_params(stage=7), B.RT_ERR_INFEASIBLE),
    ]
    for th, want in cases:
        st = B.lib.rmsnorm_template_launch(B.byref(th), x.data_ptr(), x.data_ptr(), w.data_ptr(), y.data_ptr(),
                                           ro.data_ptr(), T, H, EPS, B.RT_BF16, None)
        if th.threads_per_row == 32 and th.vec_bytes == 16:
            assert st in (B.RT_OK, want)
            continue
        assert st == want, (repr(th), st)
    # misaligned pointer for the vector width, and for TMA
    xo = torch.zeros(T * H + 8, dtype=torch.bfloat16, device="cuda")[4:4 + T * H].view(T, H)  # 8-byte aligned
    st = B.lib.rmsnorm_template_launch(B.byref(B.make_params(vec_bytes=16)), xo.data_ptr(), x.data_ptr(), w.data_ptr(),
                                       y.data_ptr(), ro.data_ptr(), T, H, EPS, B.RT_BF16, None)
    assert st == B.RT_ERR_ALIGN
    st = B.lib.rmsnorm_template_launch(B.byref(B.make_params(vec_bytes=8, stage=B.RT_STAGE_SMEM_TMA)), xo.data_ptr(),
                                       x.data_ptr(), w.data_ptr(), y.data_ptr(), ro.data_ptr(), T, H, EPS, B.RT_BF16, None)
    assert st == B.RT_ERR_ALIGN
    # row length not a multiple of the vector
    st = B.lib.rmsnorm_template_launch(B.byref(B.make_params(vec_bytes=16)), x.data_ptr(), x.data_ptr(), w.data_ptr(),
                                       y.data_ptr(), ro.data_ptr(), 2, 4100, EPS, B.RT_BF16, None)
    assert st == B.RT_ERR_ALIGN
    # NULL, dtype, shape
    th = B.make_params()
    assert B.lib.rmsnorm_template_launch(B.byref(th), None, x.data_ptr(), w.data_ptr(), y.data_ptr(), ro.data_ptr(), T, H, EPS, 0, None) == B.RT_ERR_NULL
    assert B.lib.rmsnorm_template_launch(B.byref(th), x.data_ptr(), x.data_ptr(), w.data_ptr(), y.data_ptr(), ro.data_ptr(), T, H, EPS, 5, None) == B.RT_ERR_DTYPE
    assert B.lib.rmsnorm_template_launch(B.byref(th), x.data_ptr(), x.data_ptr(), w.data_ptr(), y.data_ptr(), ro.data_ptr(), -1, H, EPS, 0, None) == B.RT_ERR_SHAPE
    assert B.lib.rmsnorm_template_launch(B.byref(th), x.data_ptr(), x.data_ptr(), w.data_ptr(), y.data_ptr(), ro.data_ptr(), T, 0, EPS, 0, None) == B.RT_ERR_SHAPE
    # an empty batch is a successful no-op
    assert B.lib.rmsnorm_template_launch(B.byref(th), None, None, None, None, None, 0, H, EPS, 0, None) == B.RT_OK
    torch.cuda.synchronize()
    launched = B.rt_launch_count() - before
    assert launched <= 1  # only the possibly-feasible 32-thread case may have run
    if launched == 0:
        assert bool((y == 5.0).all()) and bool((ro == 5.0).all())


def test_narrow_fallback_for_rows_that_fit_no_wide_vector(B, oracle_lib):
    synth = _synth()
    for H, want_vec in ((6146, 4), (6145, 2)):
        x, r, w = synth.make_inputs(9, H, "fp16", seed=11)
        y_ref, r_ref = oracle_lib.add_rmsnorm(x, r, w, EPS)
        xd, rd, wd = x.cuda(), r.cuda(), w.cuda()
        shape = B.shape_of(9, H, "fp16")
        thetas = [t for t in B.tuner_derive_feasible(shape) if t.stage != B.RT_STAGE_REG_REALIGN]  # the row-vector stages
        assert thetas and all(t.vec_bytes == want_vec for t in thetas)
        for th in thetas:
            y, ro = torch.empty_like(xd), torch.empty_like(xd)
            B.rmsnorm_template_launch(th, xd, rd, wd, y, ro, EPS)
            assert oracle_lib.bit_mismatches(ro.cpu(), r_ref) == 0
            assert oracle_lib.compare_y(y.cpu(), y_ref)[1] == 0
        for vb in (8, 16):
            assert B.tuner_check_params(shape, B.make_params(vec_bytes=vb)) == B.RT_ERR_ALIGN


def test_extreme_values_and_subnormal_outputs(B, oracle_lib):
    """fp16 rows whose outputs land in the subnormal range, and rows of zeros (rsqrt(eps) path)."""
    T, H = 6, 2048
    g = torch.Generator().manual_seed(3)
    x = (torch.randn(T, H, generator=g) * 200).half()
    r = (torch.randn(T, H, generator=g) * 200).half()
    x[1].zero_(); r[1].zero_()
    x[2] = x[2] * 0 + 60000.0; r[2] = r[2] * 0 + 10000.0      # fp16 overflow of the residual: inf in r', as in the oracle
    w = (torch.randn(H, generator=g) * 1e-4).half()            # tiny weights: subnormal y
    y_ref, r_ref = oracle_lib.add_rmsnorm(x, r, w, EPS)
    xd, rd, wd = x.cuda(), r.cuda(), w.cuda()
    for th in B.tuner_derive_feasible(B.shape_of(T, H, "fp16"))[::11]:
        y, ro = torch.empty_like(xd), torch.empty_like(xd)
        B.rmsnorm_template_launch(th, xd, rd, wd, y, ro, EPS)
        assert oracle_lib.bit_mismatches(ro.cpu(), r_ref) == 0, repr(th)
        assert oracle_lib.compare_y(y.cpu(), y_ref)[1] == 0, repr(th)


def test_host_buffer_entry_point(B, oracle_lib):
    synth = _synth()
    T, H = 1000, 2048
    x, r, w = synth.make_inputs(T, H, "bf16", seed=13)
    y_ref, r_ref = oracle_lib.add_rmsnorm(x, r, w, EPS)
    xp, rp, wp = x.pin_memory(), r.pin_memory(), w.pin_memory()
    y, ro = torch.empty_like(xp).pin_memory(), torch.empty_like(xp).pin_memory()
    for chunk in (0, 64, 333, 5000):
        nbytes = B.rmsnorm_host_workspace_bytes(T, H, "bf16", chunk)
        ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        y.zero_(); ro.zero_()
        B.rmsnorm_template_run_host(B.make_params(), xp, rp, wp, y, ro, EPS, ws, chunk)
        assert oracle_lib.bit_mismatches(ro, r_ref) == 0
        assert oracle_lib.compare_y(y, y_ref)[1] == 0
    small = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.TunerError) as e:
        B.rmsnorm_template_run_host(B.make_params(), xp, rp, wp, y, ro, EPS, small)
    assert e.value.status == B.RT_ERR_CAPACITY


def test_more_than_2_to_31_elements(B, oracle_lib):
    """A batch whose element count and byte offsets exceed 32 bits: rows are a 4096-row seeded block repeated on the
    device, and sampled rows from the whole range (the far end above all) are checked against the oracle."""
    synth = _synth()
    H, block, reps = 8192, 4096, 66                      # 270 336 rows, 2.21e9 elements, 4.4 GB per tensor
    T = block * reps
    x, r, w = synth.make_inputs(block, H, "bf16", seed=77)
    y_ref, r_ref = oracle_lib.add_rmsnorm(x, r, w, EPS, threads=8)
    xd = x.cuda().repeat(reps, 1); rd = r.cuda().repeat(reps, 1); wd = w.cuda()
    assert xd.numel() > 2**31 and xd.shape == (T, H)
    y, ro = torch.empty_like(xd), torch.empty_like(xd)
    rows = sorted({0, 1, block - 1, block, 131072, 131073, 262143, 262144, T - 2, T - 1} |
                  {int(v) for v in torch.randint(0, T, (48,), generator=torch.Generator().manual_seed(1))})
    idx = torch.tensor(rows)
    shape = B.shape_of(T, H, "bf16")
    feasible = B.tuner_derive_feasible(shape)
    picks = [next(t for t in feasible if t.stage == s) for s in (0, 1, 2)] + [B.make_params(threads_per_row=256, rows_per_cta=4)]
    for th in picks:
        y.fill_(float("nan")); ro.fill_(float("nan"))
        B.rmsnorm_template_launch(th, xd, rd, wd, y, ro, EPS)
        assert oracle_lib.bit_mismatches(ro[idx].cpu(), r_ref[idx % block]) == 0, repr(th)
        assert oracle_lib.compare_y(y[idx].cpu(), y_ref[idx % block])[1] == 0, repr(th)
        assert not bool(torch.isnan(y[-4096:]).any()) and not bool(torch.isnan(ro[-4096:]).any())
    # the device comparator over the whole far half (offsets past 2^32 bytes)
    half = (reps // 2) * block
    want = y_ref.cuda().repeat(reps - reps // 2, 1)
    assert B.tuner_compare(y[half:], want, B.RT_CMP_ULP16, 2.0)[1] == 0
    assert B.rt_device_status() == 0


def test_programmatic_launch_option_does_not_change_results(B):
    """Back-to-back in-place launches (each consumes what the previous one wrote) with and without the
    programmatic-stream-serialization attribute: the bits must agree, in a plain stream and inside a CUDA graph."""
    from paper_2601_12698_b200 import synth
    x, r, w = synth.make_inputs(64, 4096, "bf16", seed=77)
    w = (w * 0 + 1).to(w.dtype)
    thetas = [B.make_params(threads_per_row=512), B.make_params(threads_per_row=256, stage=B.RT_STAGE_SMEM_TMA),
              B.make_params(threads_per_row=128, reduce=B.RT_REDUCE_CLUSTER, cluster_size=4)]
    opt = B.RT_OPTION_PROGRAMMATIC_LAUNCH
    results = {}
    try:
        for value in (0, 1):
            assert B.lib.rt_set_option(opt, value) == B.RT_OK
            for mode in ("stream", "graph"):
                xd, rd, wd = x.cuda(), r.cuda(), w.cuda()
                stream = torch.cuda.Stream()
                stream.wait_stream(torch.cuda.current_stream())

                def chain():
                    for i in range(12):  # y over x, r' over r: every launch depends on the one before
                        B.rmsnorm_template_launch(thetas[i % len(thetas)], xd, rd, wd, xd, rd, 1e-6, stream=stream)
                if mode == "graph":
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, stream=stream):
                        chain()
                    g.replay()
                    torch.cuda.synchronize()
                else:
                    chain()
                    stream.synchronize()
                results[(value, mode)] = (xd.cpu().view(torch.int16).clone(), rd.cpu().view(torch.int16).clone())
    finally:
        assert B.lib.rt_set_option(opt, 1) == B.RT_OK
    base = results[(0, "stream")]
    for key, got in results.items():
        assert torch.equal(got[0], base[0]) and torch.equal(got[1], base[1]), key
    assert B.rt_device_status() == 0
