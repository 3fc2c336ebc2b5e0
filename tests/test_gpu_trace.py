"""The instrumented instances: the same outputs as the plain ones, and stamps that are ordered and plausible."""
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2601_12698_b200 import binding
    torch.cuda.set_device(0)
    return binding


@pytest.mark.parametrize("dtype,T,H,theta", [
    ("bf16", 1, 4096, dict(threads_per_row=512)),
    ("bf16", 128, 4096, dict(threads_per_row=256)),                                    # two vectors per thread
    ("bf16", 16, 4096, dict(threads_per_row=512, reduce=1)),
    ("bf16", 4, 4096, dict(threads_per_row=128, reduce=2, cluster_size=4)),
    ("bf16", 64, 4096, dict(threads_per_row=256, stage=2)),
    ("fp32", 37, 4096, dict(threads_per_row=1024)),
])
def test_traced_launch_matches_oracle_and_stamps_are_ordered(B, oracle_lib, dtype, T, H, theta):
    from paper_2601_12698_b200 import synth
    x, r, w = synth.make_inputs(T, H, dtype, seed=31)
    y_ref, r_ref = oracle_lib.add_rmsnorm(x, r, w, 1e-6)
    xd, rd, wd = x.cuda(), r.cuda(), w.cuda()
    y, ro = torch.empty_like(xd), torch.empty_like(xd)
    th = B.make_params(**theta)
    words = B.rmsnorm_trace_words(th, T, H, dtype)
    assert words > 0 and words % B.RT_TRACE_WORDS == 0
    trace = torch.full((words,), -1, dtype=torch.int64, device="cuda")
    B.rmsnorm_template_launch_traced(th, xd, rd, wd, y, ro, 1e-6, trace)
    torch.cuda.synchronize()
    assert oracle_lib.bit_mismatches(ro.cpu(), r_ref) == 0 and oracle_lib.compare_y(y.cpu(), y_ref)[1] == 0
    t = trace.view(-1, B.RT_TRACE_WORDS).cpu()
    assert bool((t[:, 0] <= t[:, 6]).all())                                            # nanosecond timer: entry before exit
    for a, b in zip(range(1, 5), range(2, 6)):
        assert bool((t[:, a] <= t[:, b]).all()), (a, b)                               # cycle stamps in phase order
    assert bool(((t[:, 5] - t[:, 1]) < 2_000_000).all())                              # a launch of microseconds, not seconds
    assert int(t[:, 7].max()) < B.rt_query_limits().sm_count
    assert B.rt_device_status() == 0


def test_traced_launch_refusals(B):
    x = torch.zeros(4, 4096, dtype=torch.bfloat16, device="cuda")
    w = torch.ones(4096, dtype=torch.bfloat16, device="cuda")
    y, ro = torch.empty_like(x), torch.empty_like(x)
    trace = torch.zeros(4 * 8, dtype=torch.int64, device="cuda")
    before = B.rt_launch_count()
    with pytest.raises(B.TunerError) as e:                                            # no instrumented instance of this theta
        B.rmsnorm_template_launch_traced(B.make_params(vec_bytes=32, threads_per_row=256), x, x, w, y, ro, 1e-6, trace)
    assert e.value.status == B.RT_ERR_INFEASIBLE
    with pytest.raises(B.TunerError) as e:                                            # trace buffer too small
        B.rmsnorm_template_launch_traced(B.make_params(threads_per_row=512), x, x, w, y, ro, 1e-6, trace[:8])
    assert e.value.status == B.RT_ERR_CAPACITY
    assert B.rmsnorm_trace_words(B.make_params(threads_per_row=48), 4, 4096, "bf16") == -1
    assert B.rt_launch_count() == before


def test_phase_table_of_a_decode_shape(B):
    from paper_2601_12698_b200 import trace
    res = trace.run("c2_decode_bf16_16x4096", "512,1,16,1,0,0,1", launches=60, replays=2)
    for mode in ("l2_warm", "cold"):
        info = res["modes"][mode]
        assert 0.5 < info["sm_ghz_from_stamps"] < 2.2
        assert len(info["phases"]) == 4 and all(ph["cycles_median_cta"] >= 0 for ph in info["phases"])
        assert 0.0 < info["released_to_stored_ns_slowest_cta"] < info["launch_period_ns"] * 1.5 < 30000
    assert "released -> stored" in trace.render(res)
