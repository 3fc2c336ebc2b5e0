"""The bounded device-side wait, made to run out on purpose in the one way that harms nothing: the TMA stage posts no
copy (a host-set diagnostic switch), its mbarrier is initialised and never completed, and the poll limit is lowered to
a few hundred polls.  The wait gives up within microseconds, writes the status word, and the launch completes through
every barrier: the context stays usable, which the second half of each test shows."""
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


class _expiring_waits:
    def __init__(self, B, polls=300):
        self.B, self.polls = B, polls

    def __enter__(self):
        B = self.B
        self.old = B.lib.rt_get_option(B.RT_OPTION_TMA_WAIT_POLL_LIMIT)
        assert B.lib.rt_set_option(B.RT_OPTION_TMA_WAIT_POLL_LIMIT, self.polls) == B.RT_OK
        assert B.lib.rt_set_option(B.RT_OPTION_DEBUG_DROP_TMA_COPIES, 1) == B.RT_OK

    def __exit__(self, *exc):
        B = self.B
        assert B.lib.rt_set_option(B.RT_OPTION_DEBUG_DROP_TMA_COPIES, 0) == B.RT_OK
        assert B.lib.rt_set_option(B.RT_OPTION_TMA_WAIT_POLL_LIMIT, self.old) == B.RT_OK


def test_options_are_validated(B):
    assert B.lib.rt_get_option(B.RT_OPTION_TMA_WAIT_POLL_LIMIT) == 1 << 24
    assert B.lib.rt_get_option(B.RT_OPTION_DEBUG_DROP_TMA_COPIES) == 0
    assert B.lib.rt_set_option(B.RT_OPTION_TMA_WAIT_POLL_LIMIT, 0) == B.RT_ERR_SHAPE
    assert B.lib.rt_set_option(B.RT_OPTION_TMA_WAIT_POLL_LIMIT, (1 << 24) + 1) == B.RT_ERR_SHAPE
    assert B.lib.rt_set_option(B.RT_OPTION_DEBUG_DROP_TMA_COPIES, 2) == B.RT_ERR_SHAPE
    assert B.lib.rt_set_option(99, 0) == B.RT_ERR_SHAPE and B.lib.rt_get_option(99) == -1


def test_an_expired_wait_sets_the_status_word_and_the_context_survives(B, oracle_lib):
    from paper_2601_12698_b200 import synth
    T, H = 8, 4096
    x, r, w = synth.make_inputs(T, H, "bf16", seed=5)
    y_ref, r_ref = oracle_lib.add_rmsnorm(x, r, w, EPS)
    xd, rd, wd = x.cuda(), r.cuda(), w.cuda()
    y, ro = torch.empty_like(xd), torch.empty_like(xd)
    tma = B.make_params(threads_per_row=256, stage=B.RT_STAGE_SMEM_TMA)
    reg = B.make_params(threads_per_row=256)
    assert B.rt_device_status() == 0
    with _expiring_waits(B):
        B.rmsnorm_template_launch(tma, xd, rd, wd, y, ro, EPS)
        torch.cuda.synchronize()                                   # the launch completes: no hang, no fault
        assert B.rt_device_status() == B.RT_ERR_DEVICE_TIMEOUT
        assert B.rt_device_status() == 0                           # reading clears the word
        # a stage without bulk copies has nothing to wait for: it is unaffected by the switch
        B.rmsnorm_template_launch(reg, xd, rd, wd, y, ro, EPS)
        assert B.rt_device_status() == 0
        assert oracle_lib.bit_mismatches(ro.cpu(), r_ref) == 0 and oracle_lib.compare_y(y.cpu(), y_ref)[1] == 0
    # switch off again: the same TMA launch now lands its copies and matches the oracle
    y.fill_(float("nan")); ro.fill_(float("nan"))
    B.rmsnorm_template_launch(tma, xd, rd, wd, y, ro, EPS)
    assert B.rt_device_status() == 0
    assert oracle_lib.bit_mismatches(ro.cpu(), r_ref) == 0 and oracle_lib.compare_y(y.cpu(), y_ref)[1] == 0


def test_the_tuner_skips_a_candidate_whose_wait_expired(B, oracle_lib):
    """tuner_evaluate reports such a candidate through its record (not as a failure of the call), and a search goes
    on with the candidates that have no bulk copies and returns one of them."""
    from paper_2601_12698_b200 import synth
    wl = synth.Workload("t", "bf16", 32, 4096, seed=8)
    x, r, w = synth.make_workload_inputs(wl)
    y_ref, r_ref = oracle_lib.add_rmsnorm(x, r, w, wl.eps)
    t = dict(x=x.cuda(), r=r.cuda(), w=w.cuda(), y_ref=y_ref.cuda(), r_ref=r_ref.cuda())
    t["y"], t["r_out"] = torch.empty_like(t["x"]), torch.empty_like(t["x"])
    stream = torch.cuda.Stream()
    ws = B.make_workspace(t["x"], t["r"], t["w"], t["y"], t["r_out"], t["y_ref"], t["r_ref"], wl.eps, stream=stream)
    shape = B.shape_of(wl.n_tokens, wl.hidden, wl.dtype)
    proto = B.make_budget(warmup=1, iters=3, repeats=1)
    tma = B.make_params(threads_per_row=256, stage=B.RT_STAGE_SMEM_TMA)
    with _expiring_waits(B):
        rec = B.tuner_evaluate(shape, tma, proto, ws)
        assert rec.status == B.RT_ERR_DEVICE_TIMEOUT
        assert B.rt_device_status() == 0                           # the evaluator read and cleared the word itself
        res, log = B.tuner_search(shape, B.make_budget(max_evals=40, warmup=1, iters=3, repeats=1, top_k=2), ws)
        by_stage = {}
        for rec in log:
            by_stage.setdefault(rec.params.stage, set()).add(rec.status)
        assert by_stage[B.RT_STAGE_SMEM_TMA] == {B.RT_ERR_DEVICE_TIMEOUT}       # logged and skipped, every one
        assert by_stage[B.RT_STAGE_REG] == {B.RT_OK}
        assert res.best.stage != B.RT_STAGE_SMEM_TMA and res.n_failed_gate == sum(1 for rec in log if rec.status != 0)
        recs, blocks = B.tuner_retest_interleaved(shape, [tma, B.make_params()], proto, ws, 2)
        assert [rec.status for rec in recs] == [B.RT_ERR_DEVICE_TIMEOUT, B.RT_OK]
        assert {blk.theta_index for blk in blocks} == {1}
    rec = B.tuner_evaluate(shape, tma, proto, ws)
    assert rec.status == B.RT_OK and rec.us > 0 and B.rt_device_status() == 0
