"""SelectGeneral and the specialised-table lookup (host only)."""
import math
import random

import pytest

from oracle import selection
from paper_2601_12698_b200 import binding as B


def test_oracle_selection_pins():
    # hand-computed: T* = (10, 18); c0: sqrt(1 * 18/20) = 0.948683..., c1: sqrt(10/12 * 1) = 0.912870...
    best, score, scores = selection.select_general([[10.0, 20.0], [12.0, 18.0]])
    assert best == 0 and abs(score - math.sqrt(0.9)) < 1e-15 and abs(scores[1] - math.sqrt(10 / 12)) < 1e-15
    # three candidates with the same geometric mean: the first wins the tie
    best, score, scores = selection.select_general([[1.0, 4.0], [2.0, 2.0], [4.0, 1.0]])
    assert best == 0 and all(abs(s - 0.5) < 1e-15 for s in scores)
    # a candidate that is best on every shape scores exactly 1
    assert selection.select_general([[3.0, 5.0, 7.0], [4.0, 5.0, 8.0]])[:2] == (0, 1.0)
    # rescaling one shape's times (a bigger problem) does not change the ranking; an arithmetic mean of
    # times would flip it here
    a = [[10.0, 1000.0], [14.0, 800.0]]
    b = [[10.0, 1.0], [14.0, 0.8]]
    assert selection.select_general(a)[0] == selection.select_general(b)[0] == 0  # sqrt(0.8) > sqrt(10/14)
    assert sum(a[0]) > sum(a[1]) and sum(b[0]) < sum(b[1])
    # a candidate that cannot run on some shape is not eligible, however fast elsewhere
    best, _, scores = selection.select_general([[1.0, float("nan")], [5.0, 5.0], [0.5, -1.0]])
    assert best == 1 and scores[0] == 0.0 and scores[2] == 0.0
    assert selection.select_general([[1.0, -1.0], [float("inf"), 2.0]])[0] is None


def test_library_selection_matches_oracle():
    rng = random.Random(7)
    for trial in range(200):
        n_c, n_x = rng.randint(1, 9), rng.randint(1, 6)
        t = [[rng.choice([rng.uniform(1.0, 500.0)] * 9 + [-1.0]) for _ in range(n_x)] for _ in range(n_c)]
        want_best, want_score, want_scores = selection.select_general(t)
        if want_best is None:
            with pytest.raises(B.TunerError) as e:
                B.tuner_select_general(t)
            assert e.value.status == B.RT_ERR_INFEASIBLE
            continue
        best, score, scores = B.tuner_select_general(t)
        assert best == want_best
        assert abs(score - want_score) <= 2e-6 * want_score
        assert all(abs(a - b) <= 2e-6 * max(b, 1e-9) for a, b in zip(scores, want_scores))


def test_selection_argument_errors():
    import ctypes
    best = ctypes.c_int32(0)
    t = (ctypes.c_float * 2)(1.0, 2.0)
    assert B.lib.tuner_select_general(None, 1, 2, ctypes.byref(best), None, None) == B.RT_ERR_NULL
    assert B.lib.tuner_select_general(t, 0, 2, ctypes.byref(best), None, None) == B.RT_ERR_SHAPE
    assert B.lib.tuner_select_general(t, 1, 2, ctypes.byref(best), None, None) == B.RT_OK and best.value == 0


def test_table_lookup_prefers_exact_then_nearest_then_general():
    L = B.sm100_nominal_limits()
    th_small = B.make_params(threads_per_row=512, stage=B.RT_STAGE_REG)
    th_big = B.make_params(threads_per_row=256, stage=B.RT_STAGE_SMEM_TMA)
    th_fp32 = B.make_params(threads_per_row=512, unroll=4)
    general = B.make_params(threads_per_row=256, unroll=4)
    table = B.SpecTable([(B.shape_of(128, 4096, "bf16"), th_small, 2.0), (B.shape_of(16384, 8192, "bf16"), th_big, 160.0),
                         (B.shape_of(32768, 12288, "fp32"), th_fp32, 950.0)], general)
    assert table.lookup(B.shape_of(128, 4096, "bf16"), L) == (th_small, "table_exact") or \
        table.lookup(B.shape_of(128, 4096, "bf16"), L)[0].key() == th_small.key()
    theta, src = table.lookup(B.shape_of(16384, 8192, "bf16"), L)
    assert (theta.key(), src) == (th_big.key(), "table_exact")
    # nearest: 4 x octaves of hidden + octaves of tokens
    theta, src = table.lookup(B.shape_of(8192, 8192, "bf16"), L)
    assert (theta.key(), src) == (th_big.key(), "table_nearest")
    theta, src = table.lookup(B.shape_of(64, 4096, "bf16"), L)
    assert (theta.key(), src) == (th_small.key(), "table_nearest")
    theta, src = table.lookup(B.shape_of(16384, 4096, "bf16"), L)  # hidden matches the small entry: 7 vs 4 octaves
    assert (theta.key(), src) == (th_big.key(), "table_nearest")
    theta, src = table.lookup(B.shape_of(300, 5120, "bf16"), L)     # 4*0.32+1.23 vs 4*0.68+5.77
    assert (theta.key(), src) == (th_small.key(), "table_nearest")
    # bf16 and fp16 entries serve each other (same element size, a quarter of an octave further away than an entry of
    # the query's own type); an element size the table lacks falls back to the general configuration
    theta, src = table.lookup(B.shape_of(8192, 5120, "fp16"), L)
    assert (theta.key(), src) == (th_big.key(), "table_nearest")
    theta, src = table.lookup(B.shape_of(128, 4096, "fp16"), L)           # same shape, other 16-bit type: nearest, not exact
    assert (theta.key(), src) == (th_small.key(), "table_nearest")
    both = B.SpecTable([(B.shape_of(128, 4096, "bf16"), th_small, 2.0), (B.shape_of(160, 4096, "fp16"), th_big, 2.1)], general)
    assert both.lookup(B.shape_of(128, 4096, "fp16"), L)[0].key() == th_small.key()   # 0.25 for the type < 0.32 for the rows
    assert both.lookup(B.shape_of(150, 4096, "fp16"), L)[0].key() == th_big.key()     # 0.09 for the rows < 0.23 + 0.25
    only32 = B.SpecTable([(B.shape_of(32768, 12288, "fp32"), th_fp32, 950.0)], general)
    theta, src = only32.lookup(B.shape_of(8192, 5120, "fp16"), L)
    assert (theta.key(), src) == (general.key(), "general")
    # an entry whose theta is not launchable for the query is skipped: rows of 6148 fp16 take no 16-byte vectors
    t16 = B.SpecTable([(B.shape_of(8192, 6152, "fp16"), B.make_params(vec_bytes=16), 66.0)],
                      B.make_params(vec_bytes=8, threads_per_row=512))
    theta, src = t16.lookup(B.shape_of(8192, 6148, "fp16"), L)
    assert (theta.vec_bytes, src) == (8, "general")
    # nothing usable at all: a point of the feasible set - on rows that are not 16-byte multiples the ragged-row stage
    theta, src = B.SpecTable([], None).lookup(B.shape_of(64, 6146, "fp16"), L)
    assert src == "feasible_set" and (theta.stage, theta.vec_bytes, theta.threads_per_row, theta.rows_per_cta) == \
        (B.RT_STAGE_REG_REALIGN, 16, 256, 1)
    theta, src = B.SpecTable([], None).lookup(B.shape_of(64, 6146, "fp16", min_ptr_align=4), L)  # pointers rule it out
    assert src == "feasible_set" and (theta.stage, theta.vec_bytes) == (B.RT_STAGE_REG, 4)
    theta, src = B.SpecTable([], None).lookup(B.shape_of(64, 4096, "fp16"), L)
    assert src == "feasible_set" and theta.stage == B.RT_STAGE_REG and theta.vec_bytes == 32  # the widest that fits
    # an entry tuned on ragged rows serves other ragged rows of its dtype, never rows that are 16-byte multiples
    ragged = B.make_params(unroll=4, stage=B.RT_STAGE_REG_REALIGN)
    tr = B.SpecTable([(B.shape_of(8192, 6145, "fp16"), ragged, 65.0), (B.shape_of(8192, 5120, "fp16"), th_fp32, 51.0)], general)
    theta, src = tr.lookup(B.shape_of(4096, 6146, "fp16"), L)
    assert (theta.key(), src) == (ragged.key(), "table_nearest")
    theta, src = tr.lookup(B.shape_of(8192, 5121, "fp16"), L)  # the aligned neighbour's theta cannot run here
    assert (theta.key(), src) == (ragged.key(), "table_nearest")
    theta, src = tr.lookup(B.shape_of(8192, 6144, "fp16"), L)  # 6145 is nearer, but its theta is for ragged rows
    assert (theta.key(), src) == (th_fp32.key(), "table_nearest")
    # JSON round trip
    again = B.SpecTable.from_json(table.to_json())
    assert [(s.n_tokens, s.hidden, s.dtype, t.key()) for s, t, _ in again.entries] == \
           [(s.n_tokens, s.hidden, s.dtype, t.key()) for s, t, _ in table.entries]
    assert again.general.key() == general.key()


def test_shipped_table_loads_and_every_entry_is_feasible_for_its_shape():
    L = B.sm100_nominal_limits()
    table = B.SpecTable.default()
    assert len(table.entries) >= 20 and table.general is not None
    for shape, theta, us in table.entries:
        assert B.tuner_check_params(shape, theta, L) == B.RT_OK and us > 0
        got, source = table.lookup(shape, L)
        assert got.key() == theta.key() and source == "table_exact"
    # every kernel has a general configuration, and it runs on every shape of its kernel in the table
    assert set(table.generals) == {0, 1, 2, 3, 4}
    # (rows that are not 16-byte multiples are served by their own entries: the general 16-byte vectors do not divide them)
    assert all(B.tuner_check_params(s, table.generals[int(s.op)], L) == B.RT_OK for s, _, _ in table.entries
               if (s.hidden * (4 if s.dtype == B.RT_FP32 else 2)) % 16 == 0)


def test_merging_tables_keeps_what_was_not_tuned_again():
    from paper_2601_12698_b200 import binding as B
    from paper_2601_12698_b200 import tune
    th = lambda tpr: B.make_params(threads_per_row=tpr)
    old = B.SpecTable([(B.shape_of(16, 4096, "bf16"), th(512), 1.6), (B.shape_of(8192, 5120, "fp16"), th(256), 52.0),
                       (B.shape_of(64, 11008, "bf16", op=B.RT_OP_SILU_AND_MUL), th(1024), 2.3)],
                      generals={B.RT_OP_ADD_RMSNORM: th(512), B.RT_OP_SILU_AND_MUL: th(1024)}, device_name="old device")
    new = B.SpecTable([(B.shape_of(8192, 5120, "fp16"), th(128), 51.0), (B.shape_of(8192, 6145, "fp16"), th(64), 63.0)],
                      generals={B.RT_OP_ADD_RMSNORM: th(128)}, device_name="new device")
    merged = tune.merge_tables(old, new)
    got = [(int(s.op), int(s.n_tokens), int(s.hidden), t.threads_per_row, round(us, 1)) for s, t, us in merged.entries]
    assert got == [(0, 16, 4096, 512, 1.6), (0, 8192, 5120, 128, 51.0), (1, 64, 11008, 1024, 2.3), (0, 8192, 6145, 64, 63.0)]
    assert merged.generals[B.RT_OP_ADD_RMSNORM].threads_per_row == 128 and merged.generals[B.RT_OP_SILU_AND_MUL].threads_per_row == 1024
    assert tune.merge_tables(old, new, keep_general=True).generals[B.RT_OP_ADD_RMSNORM].threads_per_row == 512
    assert merged.device_name == "new device"
    # the merged table round-trips through its JSON form
    again = B.SpecTable.from_json(merged.to_json())
    assert [(t.key(), round(us, 1)) for _, t, us in again.entries] == [(t.key(), round(us, 1)) for _, t, us in merged.entries]
