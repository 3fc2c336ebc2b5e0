"""The search on a synthetic cost function with a known optimum (host only): grid + hill-climb logic,
budget accounting, seeds, gate failures, exhaustive mode."""
import math

import pytest

from paper_2601_12698_b200 import binding as B


@pytest.fixture(scope="module")
def L():
    return B.sm100_nominal_limits()


SHAPE = (16384, 8192, "bf16")


def _cost_factory(opt, noise=None, counter=None):
    """Separable bowl over the ordered axes with a preferred stage/reduction: minimum 100 us at `opt`."""
    def cost(p):
        if counter is not None:
            counter.append(p.key())
        t = 100.0
        t += 12.0 * abs(math.log2(p.threads_per_row) - math.log2(opt["tpr"]))
        t += 7.0 * abs(math.log2(p.rows_per_cta) - math.log2(opt["rpc"]))
        t += 5.0 * abs(math.log2(p.unroll) - math.log2(opt["unroll"]))
        t += 9.0 * abs(math.log2(p.vec_bytes) - math.log2(opt["vec"]))
        t += 0.0 if p.stage == opt["stage"] else 15.0
        t += 0.0 if p.reduce == opt["reduce"] else 4.0
        if noise is not None:
            t *= 1.0 + noise(p)
        return t
    return cost


OPTIMA = [dict(tpr=256, rpc=1, unroll=1, vec=16, stage=2, reduce=0),
          dict(tpr=128, rpc=2, unroll=2, vec=16, stage=0, reduce=1),
          dict(tpr=512, rpc=1, unroll=4, vec=8, stage=1, reduce=0),
          dict(tpr=128, rpc=4, unroll=4, vec=16, stage=1, reduce=0)]


@pytest.mark.parametrize("opt", OPTIMA)
def test_guided_search_finds_the_known_optimum_within_budget(L, opt):
    s = B.shape_of(*SHAPE)
    feasible = B.tuner_derive_feasible(s, L)
    target = [t for t in feasible if (t.threads_per_row, t.rows_per_cta, t.unroll, t.vec_bytes, t.stage, t.reduce) ==
              (opt["tpr"], opt["rpc"], opt["unroll"], opt["vec"], opt["stage"], opt["reduce"])]
    assert target, "the planted optimum must be feasible"
    calls = []
    budget = 80
    res, log = B.tuner_search_with(s, L, B.make_budget(max_evals=budget, top_k=3), _cost_factory(opt, counter=calls))
    assert res.best.key() == target[0].key(), (res.best, res.best_us)
    assert abs(res.best_us - 100.0) < 1e-3
    assert res.evals_used == len(calls) == len(log) <= budget
    assert res.n_candidates == len(feasible) and budget < len(feasible) / 4
    assert [r.eval_index for r in log] == list(range(len(log)))
    phases = [r.phase for r in log]
    assert phases == sorted(phases[:-3]) + [3, 3, 3]  # grid, then climb, then exactly top_k re-tests
    # nothing but the re-tested finalists is evaluated twice
    first = [r.params.key() for r in log if r.phase != 3]
    assert len(set(first)) == len(first)


def test_exhaustive_mode_visits_every_candidate_once(L):
    s = B.shape_of(128, 4096, "bf16")
    feasible = B.tuner_derive_feasible(s, L)
    calls = []
    res, log = B.tuner_search_with(s, L, B.make_budget(max_evals=len(feasible), top_k=0, strategy=B.RT_SEARCH_EXHAUSTIVE),
                                   _cost_factory(dict(tpr=128, rpc=1, unroll=2, vec=16, stage=0, reduce=0), counter=calls))
    assert res.evals_used == len(feasible) and sorted(calls) == sorted(t.key() for t in feasible)
    assert all(r.phase == 4 for r in log) and abs(res.best_us - 100.0) < 1e-3
    # a budget smaller than the set stops early and says so through evals_used
    res2, _ = B.tuner_search_with(s, L, B.make_budget(max_evals=50, top_k=0, strategy=B.RT_SEARCH_EXHAUSTIVE),
                                  _cost_factory(dict(tpr=128, rpc=1, unroll=2, vec=16, stage=0, reduce=0)))
    assert res2.evals_used == 50


def test_budget_is_never_exceeded_and_tiny_budgets_still_return(L):
    s = B.shape_of(*SHAPE)
    cost = _cost_factory(OPTIMA[0])
    for budget in (1, 2, 3, 5, 8, 13, 40):
        res, log = B.tuner_search_with(s, L, B.make_budget(max_evals=budget, top_k=5), cost)
        assert 1 <= res.evals_used <= budget and len(log) == res.evals_used
        assert res.best_us >= 100.0
    with pytest.raises(B.TunerError) as e:
        B.tuner_search_with(s, L, B.make_budget(max_evals=0), cost)
    assert e.value.status == B.RT_ERR_BUDGET


def test_seeds_are_evaluated_first_and_help(L):
    s = B.shape_of(*SHAPE)
    opt = OPTIMA[1]
    seed = B.make_params(threads_per_row=opt["tpr"], rows_per_cta=opt["rpc"], vec_bytes=opt["vec"], unroll=opt["unroll"],
                         stage=opt["stage"], reduce=opt["reduce"])
    infeasible_seed = B.make_params(threads_per_row=1024, rows_per_cta=8)
    res, log = B.tuner_search_with(s, L, B.make_budget(max_evals=12, top_k=2, seeds=[infeasible_seed, seed]),
                                   _cost_factory(opt))
    assert log[0].phase == 0 and log[0].params.key() == seed.key()  # the infeasible seed is skipped silently
    assert sum(1 for r in log if r.phase == 0) == 1
    assert res.best.key() == seed.key() and abs(res.best_us - 100.0) < 1e-3
    # the same tiny budget without the seed does not reach the optimum
    cold, _ = B.tuner_search_with(s, L, B.make_budget(max_evals=12, top_k=2), _cost_factory(opt))
    assert cold.best_us > 100.0


def test_candidates_that_fail_the_gate_are_skipped_and_counted(L):
    s = B.shape_of(*SHAPE)
    base = _cost_factory(OPTIMA[0])

    def cost(p):  # every TMA candidate "fails parity", NaN for the shared-memory tree
        if p.stage == B.RT_STAGE_SMEM_TMA:
            return -1.0
        if p.reduce == B.RT_REDUCE_SMEM:
            return float("nan")
        return base(p)
    res, log = B.tuner_search_with(s, L, B.make_budget(max_evals=80, top_k=3), cost)
    assert res.best.stage != B.RT_STAGE_SMEM_TMA and res.best.reduce != B.RT_REDUCE_SMEM
    failed = [r for r in log if r.status != B.RT_OK]
    assert res.n_failed_gate == len(failed) > 0 and all(r.status == B.RT_ERR_MISMATCH for r in failed)
    assert abs(res.best_us - 115.0) < 1e-3  # the best point outside the failing stage
    with pytest.raises(B.TunerError) as e:
        B.tuner_search_with(s, L, B.make_budget(max_evals=20), lambda p: -1.0)
    assert e.value.status == B.RT_ERR_MISMATCH


def test_search_tolerates_timing_noise(L):
    """3% multiplicative noise, deterministic per theta: the winner is within 3% of the optimum."""
    s = B.shape_of(*SHAPE)

    def noise(p):
        h = hash(p.key()) & 0xFFFF
        return 0.03 * (h / 65535.0 - 0.5)
    res, _ = B.tuner_search_with(s, L, B.make_budget(max_evals=80, top_k=5), _cost_factory(OPTIMA[0], noise=noise))
    clean = _cost_factory(OPTIMA[0])(res.best)
    assert clean <= 103.0 + 7.0  # at most one small axis step away


def test_empty_feasible_set_is_an_error_not_a_crash(L):
    # fp32 rows of 3 elements: 12 bytes, only 4-byte vectors; with 2-byte pointer alignment nothing fits
    s = B.shape_of(4, 3, "fp32", min_ptr_align=2)
    with pytest.raises(B.TunerError) as e:
        B.tuner_search_with(s, L, B.make_budget(max_evals=10), lambda p: 1.0)
    assert e.value.status == B.RT_ERR_INFEASIBLE


def test_a_small_budget_still_touches_every_stage_and_reduction_mode(L):
    """The coarse grid is cut mode by mode: with room for 12 grid points every (stage, reduction) pair of the prefill
    shape (3 x 2) is visited before any pair is visited a third time."""
    s = B.shape_of(*SHAPE)
    res, log = B.tuner_search_with(s, L, B.make_budget(max_evals=30, top_k=5), _cost_factory(OPTIMA[0]))
    grid = [r for r in log if r.phase == 1]
    assert len(grid) == 12
    modes = [(r.params.stage, r.params.reduce) for r in grid]
    assert set(modes[:6]) == {(st, rd) for st in (0, 1, 2) for rd in (0, 1)}
    assert all(modes.count(m) == 2 for m in set(modes))
    # the first point of every mode is the one where a thread owns one vector of the row (8192 bf16 elements are 512
    # vectors of 32 bytes), one row per CTA, unroll 1
    assert all(r.params.threads_per_row == 512 and r.params.rows_per_cta == 1 and r.params.unroll == 1 for r in grid[:6])
    # and the grid's levels of threads per row are every other one counted from there
    assert {r.params.threads_per_row for r in grid} <= {128, 512}
    # a row split over a cluster of 8 moves the centre with the slice: 768 vectors / 8 = 96 -> 128 threads; whole rows: 1024
    s2 = B.shape_of(16, 12288, "bf16")
    _, log2 = B.tuner_search_with(s2, L, B.make_budget(max_evals=60, top_k=5), _cost_factory(OPTIMA[0]))
    first = {}
    for r in log2:
        if r.phase == 1:
            first.setdefault((r.params.stage, r.params.reduce, r.params.cluster_size), r.params.threads_per_row)
    assert first[(0, 2, 8)] == 128 and first[(0, 0, 1)] == 1024


def test_an_optimum_two_steps_from_every_leader_is_reached_with_leftover_budget(L):
    """A narrower vector that only pays with a deeper unroll: both one-step moves towards it are worse than the
    three leaders, so the climb gets there only because the frontier widens once the leaders are expanded."""
    s = B.shape_of(64, 11008, "bf16", op=B.RT_OP_SILU_AND_MUL)
    base = _cost_factory(dict(tpr=1024, rpc=1, unroll=1, vec=16, stage=0, reduce=0))

    def cost(p):
        if (p.threads_per_row, p.rows_per_cta, p.vec_bytes, p.unroll, p.stage) == (1024, 1, 8, 4, 0):
            return 90.0                                   # the planted optimum, 10% under the bowl's minimum
        return base(p)

    feasible = B.tuner_derive_feasible(s, L)
    assert any((t.threads_per_row, t.rows_per_cta, t.vec_bytes, t.unroll, t.stage) == (1024, 1, 8, 4, 0) for t in feasible)
    res, log = B.tuner_search_with(s, L, B.make_budget(max_evals=64, top_k=3), cost)
    assert (res.best.threads_per_row, res.best.vec_bytes, res.best.unroll, res.best.stage) == (1024, 8, 4, 0)
    assert res.evals_used <= 64
    # with the budget of a single frontier it stays on the bowl's minimum
    small, _ = B.tuner_search_with(s, L, B.make_budget(max_evals=20, top_k=2), cost)
    assert small.evals_used <= 20


def test_the_fastest_point_of_another_stage_is_climbed_from_while_the_leaders_keep_improving(L):
    """The shape of a sweep recorded on fp32 32768 x 12288: the shared-memory stage is a wide shallow bowl whose
    points keep the three leaders busy for the whole budget, the register stage is a narrow one whose optimum
    (512 threads per row) lies between two levels of the coarse grid and 2 % under the other stage's best.  The
    register stage's fastest grid point is within 3 % of the leader, so it gets an expansion of its own."""
    s = B.shape_of(32768, 12288, "fp32")

    def cost(p):
        lt, lr, lu = math.log2(p.threads_per_row), math.log2(p.rows_per_cta), math.log2(p.unroll)
        wide = 0.0 if p.vec_bytes == 32 else 6.0
        tree = 0.0 if p.reduce == 0 else 9.0
        if p.stage == 1:      # shallow: 0.4 % per level around 256 x 2, unroll 2
            return 100.0 + 0.4 * (abs(lt - 8) + abs(lr - 1) + abs(lu - 1)) + wide + tree
        if p.stage == 0:      # narrow: 98 at 512 x 1, unroll 2; 2.5 per level of threads per row
            return 98.0 + 4.0 * abs(lt - 9) + 6.0 * lr + 1.0 * abs(lu - 1) + wide + tree
        return 112.0 + wide + tree

    feasible = B.tuner_derive_feasible(s, L)
    assert any(t.key() == (512, 1, 32, 2, 0, 0, 1) for t in feasible)
    res, log = B.tuner_search_with(s, L, B.make_budget(max_evals=64, top_k=5), cost)
    grid = [r.params for r in log if r.phase == 1]  # 1: the coarse grid
    assert not any(p.stage == 0 and p.threads_per_row == 512 for p in grid)      # the grid itself does not see it
    assert res.best.key() == (512, 1, 32, 2, 0, 0, 1) and res.best_us == pytest.approx(98.0)


RAGGED_OPTIMA = [dict(tpr=256, rpc=1, unroll=4, vec=16, stage=3, reduce=0),   # 16-byte chunks of the ragged-row stage
                 dict(tpr=1024, rpc=1, unroll=4, vec=2, stage=0, reduce=0),   # the 2-byte row vectors of the register stage
                 dict(tpr=128, rpc=2, unroll=1, vec=32, stage=3, reduce=0)]   # 32-byte chunks


@pytest.mark.parametrize("opt", RAGGED_OPTIMA)
def test_guided_search_crosses_between_stages_of_different_vector_width(L, opt):
    """Rows of 6145 fp16 elements: the row-vector stage has 2-byte vectors only, the ragged-row stage 16- and 32-byte
    chunks.  The coarse grid must hold points of both stages (each at its own widest width) and the climb must be able
    to step from one to the other, whichever side the optimum is on."""
    s = B.shape_of(8192, 6145, "fp16")
    feasible = B.tuner_derive_feasible(s, L)
    assert {(t.stage, t.vec_bytes) for t in feasible} == {(0, 2), (3, 16), (3, 32)}
    target = [t for t in feasible if (t.threads_per_row, t.rows_per_cta, t.unroll, t.vec_bytes, t.stage, t.reduce) ==
              (opt["tpr"], opt["rpc"], opt["unroll"], opt["vec"], opt["stage"], opt["reduce"])]
    assert target, "the planted optimum must be feasible"

    def cost(p):  # the bowl of _cost_factory with a vector term inside the ragged-row stage only (elsewhere the width is tied to the stage)
        t = 100.0 + 12.0 * abs(math.log2(p.threads_per_row) - math.log2(opt["tpr"]))
        t += 7.0 * abs(math.log2(p.rows_per_cta) - math.log2(opt["rpc"])) + 5.0 * abs(math.log2(p.unroll) - math.log2(opt["unroll"]))
        t += 3.0 if p.stage == 3 and opt["stage"] == 3 and p.vec_bytes != opt["vec"] else 0.0
        return t + (0.0 if p.stage == opt["stage"] else 15.0)

    res, log = B.tuner_search_with(s, L, B.make_budget(max_evals=24, top_k=2), cost)
    assert res.best.key() == target[0].key(), (res.best, res.best_us)
    grid = [r for r in log if r.phase == 1]  # RT_PHASE_GRID
    assert {(r.params.stage, r.params.vec_bytes) for r in grid} == {(0, 2), (3, 32)}   # each stage at its widest width
    # a search that starts from a seed on one side still reaches the other
    seed = B.make_params(threads_per_row=1024, vec_bytes=2, unroll=1) if opt["stage"] == 3 else \
        B.make_params(threads_per_row=512, unroll=1, stage=B.RT_STAGE_REG_REALIGN)
    res2, _ = B.tuner_search_with(s, L, B.make_budget(max_evals=24, top_k=2, seeds=[seed]), cost)
    assert res2.best.key() == target[0].key()


def test_a_finalist_that_fails_its_retest_drops_out_and_the_runner_up_is_confirmed(L):
    """A candidate that passes its gate once and fails it the second time (what a race in a stage would look like) is
    the fastest by its first measurement.  The Top-K re-test must not return it: it drops out, the next runner-up is
    re-tested in its place, and the winner is the fastest candidate that passed twice."""
    s = B.shape_of(*SHAPE)
    opt = OPTIMA[0]
    base = _cost_factory(opt)
    seen = {}

    def cost(p):
        n = seen[p.key()] = seen.get(p.key(), 0) + 1
        flaky = (p.threads_per_row, p.rows_per_cta, p.unroll, p.vec_bytes, p.stage, p.reduce) == \
            (opt["tpr"], opt["rpc"], opt["unroll"], opt["vec"], opt["stage"], opt["reduce"])
        if flaky:
            return 100.0 if n == 1 else -1.0
        return base(p)
    res, log = B.tuner_search_with(s, L, B.make_budget(max_evals=80, top_k=3), cost)
    topk = [r for r in log if r.phase == 3]
    assert [r.status for r in topk] == [B.RT_ERR_MISMATCH, 0, 0]    # budget spent: no replacement, but no flaky winner
    assert res.best.key() != topk[0].params.key() and res.best_us == pytest.approx(min(r.us for r in topk[1:]))
    seen.clear()
    res, log = B.tuner_search_with(s, L, B.make_budget(max_evals=600, top_k=3), cost)   # the climb ends with budget to spare
    topk = [r for r in log if r.phase == 3]
    assert len(topk) == 4                                   # three finalists, one replacement
    assert topk[0].status == B.RT_ERR_MISMATCH and [r.status for r in topk[1:]] == [0, 0, 0]
    flaky_key = topk[0].params.key()
    assert res.best.key() != flaky_key and seen[flaky_key] == 2
    assert res.best_us == pytest.approx(min(r.us for r in topk[1:]))
    assert res.n_failed_gate == 1 and res.evals_used == len(log) < 600
    # every finalist failing its re-test leaves the best of the rest
    always = {}

    def cost2(p):
        n = always[p.key()] = always.get(p.key(), 0) + 1
        return base(p) if n == 1 else -1.0
    res2, log2 = B.tuner_search_with(s, L, B.make_budget(max_evals=600, top_k=2), cost2)
    assert [r.status for r in log2 if r.phase == 3] == [B.RT_ERR_MISMATCH] * 4
    assert res2.best_us > 100.0 and always[res2.best.key()] == 1


def test_a_photo_finish_in_the_retest_does_not_overturn_the_first_ranking(L):
    """The optimum reads 4 % slow for the length of the re-test (the callback's evaluator scores a finalist by the mean
    of its two times: 104.1 against the runner-up's 104.0).  Re-test times within 0.5 % are a tie, and a tie goes to the
    finalist that led by the first measurement; a finalist that loses its re-test by more than that loses."""
    s = B.shape_of(*SHAPE)
    opt = OPTIMA[0]
    base = _cost_factory(opt)

    def is_opt(p):
        return (p.threads_per_row, p.rows_per_cta, p.unroll, p.vec_bytes, p.stage, p.reduce) == \
            (opt["tpr"], opt["rpc"], opt["unroll"], opt["vec"], opt["stage"], opt["reduce"])

    for second, opt_wins in ((108.2, True), (112.0, False)):
        seen = {}

        def cost(p):
            n = seen[p.key()] = seen.get(p.key(), 0) + 1
            return second if is_opt(p) and n == 2 else base(p)
        res, log = B.tuner_search_with(s, L, B.make_budget(max_evals=80, top_k=3), cost)
        topk = [r for r in log if r.phase == 3]
        assert is_opt(topk[0].params) and topk[0].us == pytest.approx(second) and topk[1].us == pytest.approx(104.0)
        assert is_opt(res.best) == opt_wins, (second, res.best, res.best_us)
        assert res.best_us == pytest.approx(0.5 * (100.0 + second) if opt_wins else 104.0)
