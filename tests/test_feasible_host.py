"""The feasible-region deriver on the documented sm_100a limits (no GPU needed)."""
import pytest

from paper_2601_12698_b200 import binding as B


@pytest.fixture(scope="module")
def L():
    return B.sm100_nominal_limits()


def _keys(thetas):
    return {t.key() for t in thetas}


SHAPES = [(128, 4096, "bf16"), (1, 4096, "bf16"), (16384, 8192, "bf16"), (8192, 5120, "fp16"), (8192, 6152, "fp16"),
          (8192, 6148, "fp16"), (32768, 12288, "fp32"), (64, 6146, "fp16"), (64, 6145, "fp16"), (3, 8, "fp32")]


@pytest.mark.parametrize("T,H,dtype", SHAPES)
def test_every_emitted_theta_passes_the_hard_rules_and_counts_add_up(L, T, H, dtype):
    s = B.shape_of(T, H, dtype)
    feasible = B.tuner_derive_feasible(s, L)
    assert feasible, "empty feasible set"
    assert len(_keys(feasible)) == len(feasible)  # no duplicates
    for th in feasible:
        assert B.tuner_check_params(s, th, L) == B.RT_OK
        assert th.threads_per_row * th.rows_per_cta <= 1024
        if th.stage == B.RT_STAGE_REG_REALIGN:  # aligned 16- or 32-byte chunks over rows that the chunk does not divide
            assert th.vec_bytes in (16, 32) and th.reduce == B.RT_REDUCE_SHFL and (H * (4 if dtype == "fp32" else 2)) % th.vec_bytes != 0
        else:
            assert (H * (4 if dtype == "fp32" else 2)) % th.vec_bytes == 0
        assert (th.reduce == B.RT_REDUCE_CLUSTER) == (th.cluster_size > 1)
    c = B.tuner_derive_counts(s, L)
    assert c["feasible"] == len(feasible)
    assert sum(v for k, v in c.items() if k != "raw") == c["raw"] == len(B.tuner_raw_grid(s))


def test_heuristics_only_remove_points(L):
    s = B.shape_of(128, 4096, "bf16")
    wide = _keys(B.tuner_derive_feasible(s, L, heuristics=0))
    for mask in (B.RT_PRUNE_IDLE_THREADS, B.RT_PRUNE_DUPLICATES, B.RT_PRUNE_CLUSTER_WAVES, B.RT_PRUNE_IDLE_ROWS,
                 B.RT_PRUNE_BYTES_IN_FLIGHT, B.RT_PRUNE_DEFAULT):
        narrow = _keys(B.tuner_derive_feasible(s, L, heuristics=mask))
        assert narrow <= wide
    assert len(_keys(B.tuner_derive_feasible(s, L))) < len(wide)


def test_the_bytes_in_flight_rule_follows_littles_law_and_only_where_it_can(L):
    """On a batch of two waves or more, a theta that keeps less than 32 KB of input in flight per SM goes; the figure
    is recomputed here from the 48 KB rows, the block shape and the resident CTAs that the registers allow."""
    without = B.RT_PRUNE_DEFAULT & ~B.RT_PRUNE_BYTES_IN_FLIGHT
    s = B.shape_of(32768, 12288, "fp32")
    wide, narrow = _keys(B.tuner_derive_feasible(s, L, heuristics=without)), _keys(B.tuner_derive_feasible(s, L))
    assert narrow < wide and len(wide) - len(narrow) > 100
    gone = wide - narrow
    # register stage, 128 threads x 1 row, 32-byte vectors, unroll 1: 128 x 32 B x 2 inputs = 8 KB per CTA; three such
    # CTAs per SM (12 vectors of fp32 per thread cost registers) stay under 32 KB - the closest any pruned point came
    # to an optimum in the recorded sweeps (1.22 of it)
    assert (128, 1, 32, 1, 0, 0, 1) in gone and (512, 1, 32, 2, 0, 0, 1) in narrow and (256, 2, 32, 2, 1, 0, 1) in narrow
    # the bulk-copy stage requests whole rows: 2 x 48 KB per CTA, never pruned by this rule
    assert not any(k[4] == B.RT_STAGE_SMEM_TMA for k in gone)
    # a pruned point's CTA itself asks for less than 32 KB (threads x vector x unroll x 2 inputs)
    assert all(k[0] * k[1] * k[2] * k[3] * 2 < 32 * 1024 for k in gone)
    # fewer than two waves: the batch bounds what is in flight, the rule is void (decode and the small configuration)
    for shape in (B.shape_of(128, 4096, "bf16"), B.shape_of(256, 4096, "bf16"), B.shape_of(64, 8192, "bf16", op=B.RT_OP_SILU_AND_MUL)):
        assert _keys(B.tuner_derive_feasible(shape, L, heuristics=without)) == _keys(B.tuner_derive_feasible(shape, L))
    # rows so narrow that no theta reaches the threshold: all stay
    s = B.shape_of(1 << 20, 64, "bf16")
    assert _keys(B.tuner_derive_feasible(s, L, heuristics=without)) == _keys(B.tuner_derive_feasible(s, L)) != set()
    # the fall-back vector widths are exempt (nothing wider exists for the row), the ragged-row stage is not
    s = B.shape_of(8192, 6145, "fp16")
    wide, narrow = B.tuner_derive_feasible(s, L, heuristics=without), B.tuner_derive_feasible(s, L)
    assert {t.key() for t in wide if t.vec_bytes == 2} == {t.key() for t in narrow if t.vec_bytes == 2} != set()
    assert len([t for t in narrow if t.stage == B.RT_STAGE_REG_REALIGN]) < len([t for t in wide if t.stage == B.RT_STAGE_REG_REALIGN])
    # merge_attn_states is left alone
    s = B.shape_of(32768, 4096, "bf16", op=B.RT_OP_MERGE_ATTN_STATES, head_dim=128)
    assert _keys(B.tuner_derive_feasible(s, L, heuristics=without)) == _keys(B.tuner_derive_feasible(s, L))


def test_idle_threads_are_pruned_from_half_the_row_on(L):
    """5120 bf16 elements are 320 32-byte vectors: 512 threads per row (one vector per thread, 192 idle) stay - measured
    the fastest on 32 x 5120 -, 1024 (more than half idle) go; on a power-of-two vector count nothing is in between."""
    f = _keys(B.tuner_derive_feasible(B.shape_of(32, 5120, "bf16"), L))
    assert (512, 1, 32, 1, 0, 0, 1) in f and (1024, 1, 32, 1, 0, 0, 1) not in f and (1024, 1, 16, 1, 0, 0, 1) in f
    wide = _keys(B.tuner_derive_feasible(B.shape_of(32, 5120, "bf16"), L, heuristics=B.RT_PRUNE_DEFAULT & ~B.RT_PRUNE_IDLE_THREADS))
    assert (1024, 1, 32, 1, 0, 0, 1) in wide
    f = _keys(B.tuner_derive_feasible(B.shape_of(128, 4096, "bf16"), L))     # 256 vectors of 32 bytes
    assert (256, 1, 32, 1, 0, 0, 1) in f and (512, 1, 32, 1, 0, 0, 1) not in f


def test_rules_bite_where_they_should(L):
    ragged = B.RT_STAGE_REG_REALIGN

    def row_vectors(f):  # the stages whose vectors must divide the row
        return [t for t in f if t.stage != ragged]

    # 6148 fp16: row bytes = 8 mod 16 -> only 8-byte row vectors, no TMA stage; the ragged-row stage keeps 16-byte chunks
    f = B.tuner_derive_feasible(B.shape_of(8192, 6148, "fp16"), L)
    assert {t.vec_bytes for t in row_vectors(f)} == {8} and {t.stage for t in f} == {0, 1, ragged}
    assert {t.vec_bytes for t in f if t.stage == ragged} == {16, 32}
    # rows of 8192 bf16 elements: all three widths of the vector axis, for every kernel
    f = B.tuner_derive_feasible(B.shape_of(16384, 8192, "bf16"), L)
    assert {t.vec_bytes for t in f} == {8, 16, 32} and {t.stage for t in f if t.vec_bytes == 32} == {0, 1, 2}
    assert B.tuner_check_params(B.shape_of(16384, 8192, "bf16", min_ptr_align=16), B.make_params(vec_bytes=32), L) == B.RT_ERR_ALIGN
    assert B.tuner_check_params(B.shape_of(64, 8192, "bf16", op=B.RT_OP_SILU_AND_MUL), B.make_params(vec_bytes=32), L) == B.RT_OK
    assert B.tuner_check_params(B.shape_of(64, 8192, "bf16", op=B.RT_OP_ADD_RMSNORM_FP8), B.make_params(vec_bytes=32), L) == B.RT_OK
    assert B.tuner_check_params(B.shape_of(64, 8192, "bf16", op=B.RT_OP_ADD_RMSNORM_ALLREDUCE, n_parts=2),
                                B.make_params(vec_bytes=32), L) == B.RT_OK
    # 6152 fp16: 769 16-byte vectors (no 32-byte row vectors): both widths in the three aligned stages, and the
    # ragged-row stage with the 32-byte chunks that the row length does not divide into
    f = B.tuner_derive_feasible(B.shape_of(8192, 6152, "fp16"), L)
    assert {t.vec_bytes for t in row_vectors(f)} == {8, 16} and {t.stage for t in f} == {0, 1, 2, ragged}
    assert {t.vec_bytes for t in f if t.stage == ragged} == {32}
    # rows that fit no 8-byte vector fall back to the widest narrow width, or take the ragged-row stage
    for hidden, narrow in ((6146, 4), (6145, 2)):
        f = B.tuner_derive_feasible(B.shape_of(64, hidden, "fp16"), L)
        assert {t.vec_bytes for t in row_vectors(f)} == {narrow} and {t.stage for t in row_vectors(f)} == {0}
        assert any(t.stage == ragged for t in f)
    # pointers that are only 8-byte aligned remove the 16-byte vectors, TMA and the ragged-row stage
    f = B.tuner_derive_feasible(B.shape_of(128, 4096, "bf16", min_ptr_align=8), L)
    assert {t.vec_bytes for t in f} == {8} and not {B.RT_STAGE_SMEM_TMA, ragged} & {t.stage for t in f}
    f = B.tuner_derive_feasible(B.shape_of(128, 4100, "bf16", min_ptr_align=8), L)
    assert f and {t.vec_bytes for t in f} == {8} and ragged not in {t.stage for t in f}
    # the ragged-row stage: add_rmsnorm only, 16-byte chunks, shuffle reduction, one CTA per row; it also runs on
    # aligned rows (where the deriver does not offer it)
    s_odd = B.shape_of(64, 6145, "fp16")
    assert B.tuner_check_params(s_odd, B.make_params(stage=ragged), L) == B.RT_OK
    assert B.tuner_check_params(s_odd, B.make_params(stage=ragged, vec_bytes=8), L) == B.RT_ERR_INFEASIBLE
    assert B.tuner_check_params(s_odd, B.make_params(stage=ragged, reduce=B.RT_REDUCE_SMEM), L) == B.RT_ERR_INFEASIBLE
    assert B.tuner_check_params(s_odd, B.make_params(stage=ragged, reduce=B.RT_REDUCE_CLUSTER, cluster_size=2), L) == B.RT_ERR_INFEASIBLE
    assert B.tuner_check_params(s_odd, B.make_params(stage=5), L) == B.RT_ERR_INFEASIBLE
    assert B.tuner_check_params(B.shape_of(64, 6145, "fp16", min_ptr_align=8), B.make_params(stage=ragged), L) == B.RT_ERR_ALIGN
    assert B.tuner_check_params(B.shape_of(128, 4096, "bf16"), B.make_params(stage=ragged), L) == B.RT_OK
    assert B.tuner_check_params(B.shape_of(64, 6145, "fp16", op=B.RT_OP_SILU_AND_MUL), B.make_params(stage=ragged), L) == B.RT_ERR_INFEASIBLE
    # a 32-thread row of fp32 12289 would keep 96 chunks per thread: no instance that large
    assert B.tuner_check_params(B.shape_of(64, 12289, "fp32"), B.make_params(threads_per_row=32, stage=ragged), L) == B.RT_ERR_INFEASIBLE
    # a single token: one row per CTA only; clusters are allowed (too few rows to fill the SMs)
    f = B.tuner_derive_feasible(B.shape_of(1, 4096, "bf16"), L)
    assert {t.rows_per_cta for t in f} == {1} and 8 in {t.cluster_size for t in f}
    # the prefill shape fills the machine with whole rows: no cluster split survives
    f = B.tuner_derive_feasible(B.shape_of(16384, 8192, "bf16"), L)
    assert {t.cluster_size for t in f} == {1}
    # register stage: a 32-thread row of 1024 vectors would need 32 vectors per thread (256 fp32): rejected
    s = B.shape_of(16384, 8192, "bf16")
    assert B.tuner_check_params(s, B.make_params(threads_per_row=32), L) == B.RT_ERR_INFEASIBLE
    assert b"register" in B.lib.rt_last_error()
    # shared-memory stage: 8 rows of fp32 12288 need 8 * 48 KB
    s5 = B.shape_of(32768, 12288, "fp32")
    assert B.tuner_check_params(s5, B.make_params(threads_per_row=128, rows_per_cta=8, stage=B.RT_STAGE_SMEM_LDG), L) == B.RT_ERR_INFEASIBLE
    assert b"shared memory" in B.lib.rt_last_error()
    assert B.tuner_check_params(s5, B.make_params(threads_per_row=128, rows_per_cta=2, stage=B.RT_STAGE_SMEM_TMA), L) == B.RT_OK
    assert B.tuner_check_params(s5, B.make_params(threads_per_row=128, rows_per_cta=4, stage=B.RT_STAGE_SMEM_TMA), L) == B.RT_ERR_INFEASIBLE


def test_argument_errors(L):
    import ctypes
    n = ctypes.c_int32(0)
    assert B.lib.tuner_derive_feasible_ex(None, ctypes.byref(L), 15, None, 0, ctypes.byref(n)) == B.RT_ERR_NULL
    bad = B.shape_of(4, 64, 7)
    assert B.lib.tuner_derive_feasible_ex(ctypes.byref(bad), ctypes.byref(L), 15, None, 0, ctypes.byref(n)) == B.RT_ERR_DTYPE
    bad = B.shape_of(-1, 64, "bf16")
    assert B.lib.tuner_derive_feasible_ex(ctypes.byref(bad), ctypes.byref(L), 15, None, 0, ctypes.byref(n)) == B.RT_ERR_SHAPE
    bad = B.shape_of(4, 0, "bf16")
    assert B.lib.tuner_derive_feasible_ex(ctypes.byref(bad), ctypes.byref(L), 15, None, 0, ctypes.byref(n)) == B.RT_ERR_SHAPE
    ok = B.shape_of(4, 4096, "bf16")
    assert B.lib.tuner_derive_feasible_ex(ctypes.byref(ok), ctypes.byref(L), 15, None, 5, ctypes.byref(n)) == B.RT_ERR_NULL
    # a small capacity still reports the full count
    arr = (B.rt_params * 3)()
    assert B.lib.tuner_derive_feasible_ex(ctypes.byref(ok), ctypes.byref(L), 15, arr, 3, ctypes.byref(n)) == B.RT_OK
    assert n.value > 3


def test_silu_and_mul_grid_has_no_reduction_axis(L):
    s = B.shape_of(16384, 14336, "bf16", op=B.RT_OP_SILU_AND_MUL)
    raw = B.tuner_raw_grid(s)
    assert {t.reduce for t in raw} == {0} and {t.cluster_size for t in raw} == {1} and {t.stage for t in raw} == {0, 2}
    f = B.tuner_derive_feasible(s, L)
    assert f and {t.stage for t in f} == {0, 2} and {t.vec_bytes for t in f} == {32, 16, 8}
    for th in f:
        assert B.tuner_check_params(s, th, L) == B.RT_OK
    c = B.tuner_derive_counts(s, L)
    assert c["feasible"] == len(f) and sum(v for k, v in c.items() if k != "raw") == c["raw"] == len(raw)
    # the other kernel's thetas are not this kernel's
    assert B.tuner_check_params(s, B.make_params(reduce=B.RT_REDUCE_SMEM), L) == B.RT_ERR_INFEASIBLE
    assert B.tuner_check_params(s, B.make_params(stage=B.RT_STAGE_SMEM_LDG), L) == B.RT_ERR_INFEASIBLE
    # d = 3073 fp16: 2-byte fall-back only; the TMA stage needs 16-byte rows
    f = B.tuner_derive_feasible(B.shape_of(8, 3073, "fp16", op=B.RT_OP_SILU_AND_MUL), L)
    assert f and {t.vec_bytes for t in f} == {2} and {t.stage for t in f} == {0}
    assert B.tuner_check_params(B.shape_of(8, 4096, "bf16", op=7), B.make_params(), L) == B.RT_ERR_SHAPE


def test_merge_attn_states_grid(L):
    s = B.shape_of(512, 40 * 128, "bf16", op=B.RT_OP_MERGE_ATTN_STATES, head_dim=128)
    f = B.tuner_derive_feasible(s, L)
    assert f and {t.stage for t in f} == {0, 2} and {t.reduce for t in f} == {0} and {t.vec_bytes for t in f} == {32, 16, 8}
    assert all(B.tuner_check_params(s, t, L) == B.RT_OK for t in f)
    # heads of 72 bf16 elements (144 bytes): 16-byte vectors fit a head, 32-byte ones would straddle two
    f72 = B.tuner_derive_feasible(B.shape_of(64, 8 * 72, "bf16", op=B.RT_OP_MERGE_ATTN_STATES, head_dim=72), L)
    assert f72 and {t.vec_bytes for t in f72} == {16, 8}
    # a vector may not straddle two heads: heads of 66 bf16 elements (132 bytes) allow 4-byte vectors only
    f = B.tuner_derive_feasible(B.shape_of(4, 7 * 66, "bf16", op=B.RT_OP_MERGE_ATTN_STATES, head_dim=66), L)
    assert f and {t.vec_bytes for t in f} == {4}
    assert B.tuner_check_params(B.shape_of(4, 7 * 66, "bf16", op=B.RT_OP_MERGE_ATTN_STATES, head_dim=66),
                                B.make_params(vec_bytes=8), L) == B.RT_ERR_ALIGN
    # head_dim must divide hidden
    assert B.tuner_check_params(B.shape_of(4, 1000, "bf16", op=B.RT_OP_MERGE_ATTN_STATES, head_dim=128), B.make_params(), L) == B.RT_ERR_SHAPE
    assert B.tuner_check_params(B.shape_of(4, 1024, "bf16", op=B.RT_OP_MERGE_ATTN_STATES, head_dim=0), B.make_params(), L) == B.RT_ERR_SHAPE


def test_fp8_output_norm_grid(L):
    s = B.shape_of(16384, 8192, "bf16", op=B.RT_OP_ADD_RMSNORM_FP8)
    f = B.tuner_derive_feasible(s, L)
    assert f and {t.vec_bytes for t in f} == {16, 32} and {t.stage for t in f} == {0, 2} and {t.reduce for t in f} == {0}
    assert all(B.tuner_check_params(s, t, L) == B.RT_OK for t in f)
    # rows of 4104 bf16 elements: 16-byte vectors only
    f16 = B.tuner_derive_feasible(B.shape_of(64, 4104, "bf16", op=B.RT_OP_ADD_RMSNORM_FP8), L)
    assert f16 and {t.vec_bytes for t in f16} == {16}
    assert B.tuner_check_params(B.shape_of(64, 4096, "fp32", op=B.RT_OP_ADD_RMSNORM_FP8), B.make_params(), L) == B.RT_ERR_DTYPE
    assert B.tuner_check_params(s, B.make_params(vec_bytes=8), L) == B.RT_ERR_INFEASIBLE
    # rows that are not 16-byte multiples have no instance of this variant
    assert B.tuner_derive_feasible(B.shape_of(64, 6148, "fp16", op=B.RT_OP_ADD_RMSNORM_FP8), L) == []


def test_allreduce_fused_norm_grid(L):
    s = B.shape_of(4096, 8192, "bf16", op=B.RT_OP_ADD_RMSNORM_ALLREDUCE, n_parts=4)
    f = B.tuner_derive_feasible(s, L)
    assert f and {t.vec_bytes for t in f} == {16, 32} and {t.stage for t in f} == {0} and {t.reduce for t in f} == {0}
    assert all(B.tuner_check_params(s, t, L) == B.RT_OK for t in f)
    # at most 256 bytes of x in flight per thread: four parts of 32-byte vectors allow unroll 1 and 2 only
    assert {t.unroll for t in f if t.vec_bytes == 32} == {1, 2} and {t.unroll for t in f if t.vec_bytes == 16} == {1, 2, 4}
    c = B.tuner_derive_counts(s, L)
    assert c["feasible"] == len(f) and sum(v for k, v in c.items() if k != "raw") == c["raw"] == len(B.tuner_raw_grid(s))
    # eight parts leave no instance with four vectors per part in flight
    s8 = B.shape_of(4096, 8192, "bf16", op=B.RT_OP_ADD_RMSNORM_ALLREDUCE, n_parts=8)
    f8 = B.tuner_derive_feasible(s8, L)
    assert f8 and 4 not in {t.unroll for t in f8} and len(f8) < len(f)
    # the part count is 2, 4 or 8
    for bad in (0, 1, 3, 16):
        assert B.tuner_check_params(B.shape_of(64, 4096, "bf16", op=B.RT_OP_ADD_RMSNORM_ALLREDUCE, n_parts=bad),
                                    B.make_params(), L) == B.RT_ERR_SHAPE
    # the other stages, reductions and vector widths are not this variant's
    assert B.tuner_check_params(s, B.make_params(stage=B.RT_STAGE_SMEM_TMA), L) == B.RT_ERR_INFEASIBLE
    assert B.tuner_check_params(s, B.make_params(reduce=B.RT_REDUCE_SMEM), L) == B.RT_ERR_INFEASIBLE
    assert B.tuner_check_params(s, B.make_params(vec_bytes=8), L) == B.RT_ERR_INFEASIBLE
    # rows that are not 16-byte multiples have no instance
    assert B.tuner_derive_feasible(B.shape_of(64, 6148, "fp16", op=B.RT_OP_ADD_RMSNORM_ALLREDUCE, n_parts=2), L) == []
    # fp32 rows work too
    assert B.tuner_derive_feasible(B.shape_of(64, 4096, "fp32", op=B.RT_OP_ADD_RMSNORM_ALLREDUCE, n_parts=2), L)


def test_the_pipeline_stage_is_derived_only_on_request(L):
    """RT_STAGE_TMA_PIPELINE is part of the raw grid and passes the hard rules, but the default mask leaves it out of
    the feasible set (it has won on no shape measured); clearing RT_PRUNE_PIPELINE_STAGE brings it in."""
    pipe = B.RT_STAGE_TMA_PIPELINE
    s = B.shape_of(16384, 8192, "bf16")
    assert pipe in {t.stage for t in B.tuner_raw_grid(s)}
    assert pipe not in {t.stage for t in B.tuner_derive_feasible(s, L)}
    with_pipe = B.tuner_derive_feasible(s, L, heuristics=B.RT_PRUNE_DEFAULT & ~B.RT_PRUNE_PIPELINE_STAGE)
    mine = [t for t in with_pipe if t.stage == pipe]
    assert mine and {t.unroll for t in mine} == {1, 2, 4} and {t.reduce for t in mine} == {0, 1}
    assert {t.cluster_size for t in mine} == {1} and {t.vec_bytes for t in mine} == {8, 16, 32}
    assert _keys([t for t in with_pipe if t.stage != pipe]) == _keys(B.tuner_derive_feasible(s, L))
    c_default, c_with = B.tuner_derive_counts(s, L), B.tuner_derive_counts(s, L, B.RT_PRUNE_DEFAULT & ~B.RT_PRUNE_PIPELINE_STAGE)
    assert c_with["feasible"] - c_default["feasible"] == len(mine) == c_default["heuristics"] - c_with["heuristics"]
    # hard rules: one CTA per row, add_rmsnorm only, 16-byte rows and pointers, the ring must fit in shared memory
    ok = B.make_params(stage=pipe, unroll=2)
    assert B.tuner_check_params(s, ok, L) == B.RT_OK
    assert B.tuner_check_params(s, B.make_params(stage=pipe, reduce=B.RT_REDUCE_CLUSTER, cluster_size=2), L) == B.RT_ERR_INFEASIBLE
    assert B.tuner_check_params(B.shape_of(64, 8192, "bf16", op=B.RT_OP_SILU_AND_MUL), ok, L) == B.RT_ERR_INFEASIBLE
    assert B.tuner_check_params(B.shape_of(64, 6148, "fp16"), B.make_params(stage=pipe, vec_bytes=8), L) == B.RT_ERR_ALIGN
    assert B.tuner_check_params(B.shape_of(64, 8192, "bf16", min_ptr_align=8), B.make_params(stage=pipe, vec_bytes=8), L) == B.RT_ERR_ALIGN
    s5 = B.shape_of(32768, 12288, "fp32")            # 96 KB per row and stage
    assert B.tuner_check_params(s5, B.make_params(stage=pipe, unroll=2), L) == B.RT_OK
    assert B.tuner_check_params(s5, B.make_params(stage=pipe, unroll=4), L) == B.RT_ERR_INFEASIBLE
    assert b"shared memory" in B.lib.rt_last_error()
    # decode shapes: a CTA walks over one row block, so a deeper ring is the same kernel again (pruned as a duplicate)
    few = B.tuner_derive_feasible(B.shape_of(16, 4096, "bf16"), L, heuristics=B.RT_PRUNE_DEFAULT & ~B.RT_PRUNE_PIPELINE_STAGE)
    assert {t.unroll for t in few if t.stage == pipe} == {1}


def test_the_longest_row_the_template_serves(L):
    """The header states the limit: 57 856 elements in one CTA, 462 336 over a cluster of 8 (shared-memory stage)."""
    for dtype in ("bf16", "fp32"):
        f = B.tuner_derive_feasible(B.shape_of(4, 57856, dtype), L, heuristics=0)
        assert {(t.stage, t.cluster_size) for t in f if t.cluster_size == 1} == {(B.RT_STAGE_SMEM_LDG, 1)}
        assert not [t for t in B.tuner_derive_feasible(B.shape_of(4, 57856 + 64, dtype), L, heuristics=0) if t.cluster_size == 1]
        assert B.tuner_derive_feasible(B.shape_of(4, 462336, dtype), L, heuristics=0)
        assert B.tuner_derive_feasible(B.shape_of(4, 462336 + 64, dtype), L, heuristics=0) == []
    # the register stages end at 128 elements per thread within the CTA's 64 K registers
    f = B.tuner_derive_feasible(B.shape_of(4, 32768, "bf16"), L, heuristics=0)
    assert any(t.stage == B.RT_STAGE_REG and t.cluster_size == 1 for t in f)
    f = B.tuner_derive_feasible(B.shape_of(4, 32768 + 64, "bf16"), L, heuristics=0)
    assert not any(t.stage == B.RT_STAGE_REG and t.cluster_size == 1 for t in f)
