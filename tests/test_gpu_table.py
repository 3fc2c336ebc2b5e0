"""D_spec / theta_gen on the device: tuning a few shapes, persistence, and rmsnorm_launch_auto parity."""
import json

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


@pytest.fixture(scope="module")
def tuned(B):
    from paper_2601_12698_b200 import tune
    table, report = tune.tune([("bf16", 64, 4096), ("bf16", 2048, 8192), ("fp16", 512, 5120)], budget=24, top_k=2)
    return table, report


def test_tuning_builds_a_table_and_a_general_configuration(B, tuned, tmp_path):
    table, report = tuned
    assert len(table.entries) == 3 and table.general is not None
    assert 0.5 < report["general_geomean_vs_specialised"] <= 1.0 + 1e-6
    assert all(g >= s * 0.97 for g, s in zip(report["general_us"], report["specialised_us"]))
    # an entry is within half a percent of the fastest configuration measured on its shape when every finalist was
    # timed on every shape
    assert all(s * 0.998 <= us <= s / 0.995 + 1e-3 for (_, _, us), s in zip(table.entries, report["specialised_us"]))
    path = tmp_path / "table.json"
    path.write_text(json.dumps(table.to_json()))
    again = B.SpecTable.from_json(json.loads(path.read_text()))
    assert [t.key() for _, t, _ in again.entries] == [t.key() for _, t, _ in table.entries]
    assert again.general.key() == table.general.key()


@pytest.mark.parametrize("dtype,T,H,want_source", [
    ("bf16", 64, 4096, "table_exact"), ("bf16", 2048, 8192, "table_exact"), ("bf16", 77, 4096, "table_nearest"),
    ("bf16", 4096, 7168, "table_nearest"), ("fp16", 300, 6152, "nearest_or_general"), ("fp16", 300, 6148, None),
    ("fp32", 33, 12288, "general_or_feasible"), ("fp16", 9, 6146, "feasible_set"), ("bf16", 1, 8, None)])
def test_launch_auto_matches_the_oracle(B, oracle_lib, tuned, dtype, T, H, want_source):
    from paper_2601_12698_b200 import synth
    table, _ = tuned
    x, r, w = synth.make_inputs(T, H, dtype, seed=31)
    y_ref, r_ref = oracle_lib.add_rmsnorm(x, r, w, EPS)
    xd, rd, wd = x.cuda(), r.cuda(), w.cuda()
    y, ro = torch.empty_like(xd), torch.empty_like(xd)
    used = table.launch(xd, rd, wd, y, ro, EPS)
    torch.cuda.synchronize()
    assert oracle_lib.bit_mismatches(ro.cpu(), r_ref) == 0, repr(used)
    assert oracle_lib.compare_y(y.cpu(), y_ref)[1] == 0, repr(used)
    shape = B.shape_of(T, H, dtype, B._ptr_align(xd, rd, wd, y, ro))
    assert B.tuner_check_params(shape, used) == B.RT_OK
    theta, source = table.lookup(shape)
    assert theta.key() == used.key()
    if want_source == "nearest_or_general":  # rows of 6152 fp16 take no 32-byte vectors: an entry that uses them is skipped
        assert source in ("table_nearest", "general")
    elif want_source == "general_or_feasible":
        assert source in ("general", "feasible_set")
    elif want_source is not None:
        assert source == want_source
    assert B.rt_device_status() == 0


def test_tuning_and_auto_launch_for_the_other_kernels(B, oracle_lib):
    from paper_2601_12698_b200 import synth, tune
    table, report = tune.tune([("silu", "bf16", (64, 2048)), ("silu", "bf16", (512, 5504)), ("merge", "bf16", (128, 8, 128)),
                               ("fp8", "bf16", (256, 4096))], budget=16, top_k=2)
    assert set(table.generals) == {B.RT_OP_SILU_AND_MUL, B.RT_OP_MERGE_ATTN_STATES, B.RT_OP_ADD_RMSNORM_FP8}
    assert 0.5 < report["kernels"]["silu"]["general_geomean_vs_specialised"] <= 1.0 + 1e-6
    again = B.SpecTable.from_json(table.to_json())
    assert {op: th.key() for op, th in again.generals.items()} == {op: th.key() for op, th in table.generals.items()}
    # silu_and_mul on a shape that is not in the table
    x = synth.make_gate_up(0, 100, 2048, "bf16", seed=3)
    out = torch.empty(100, 2048, dtype=torch.bfloat16, device="cuda")
    used = again.launch_silu_and_mul(x.cuda(), out)
    assert oracle_lib.compare_y(out.cpu(), oracle_lib.silu_and_mul(x))[1] == 0 and used.reduce == 0
    # merge_attn_states, exact shape
    va, sa, vb, sb = synth.make_merge_inputs(0, 128, 8, 128, "bf16", seed=3)
    vo, so = torch.empty_like(va, device="cuda"), torch.empty_like(sa, device="cuda")
    again.launch_merge_attn_states(va.cuda(), sa.cuda(), vb.cuda(), sb.cuda(), vo, so)
    v_ref, s_ref = oracle_lib.merge_attn_states(va, sa, vb, sb)
    assert oracle_lib.compare_mixed(vo.cpu(), v_ref)[1] == 0 and oracle_lib.compare_mixed(so.cpu(), s_ref, tol=1e-5)[1] == 0
    # the fp8-output norm on another token count
    xx, rr, ww = synth.make_inputs(77, 4096, "bf16", seed=3)
    q = torch.empty(77, 4096, dtype=torch.uint8, device="cuda"); sc = torch.empty(77, device="cuda")
    ro = torch.empty(77, 4096, dtype=torch.bfloat16, device="cuda")
    again.launch_rmsnorm_fp8(xx.cuda(), rr.cuda(), ww.cuda(), q, sc, ro, EPS)
    q_ref, sc_ref, r_ref = oracle_lib.add_rmsnorm_fp8(xx, rr, ww, EPS)
    assert oracle_lib.compare_e4m3(q.cpu(), q_ref)[1] == 0 and oracle_lib.compare_y(sc.cpu(), sc_ref)[1] == 0
    assert oracle_lib.bit_mismatches(ro.cpu(), r_ref) == 0


@pytest.mark.parametrize("dtype,T,H,want_stage", [
    ("fp16", 100, 6145, 3), ("fp16", 8192, 6146, 3), ("bf16", 7, 4099, 3), ("fp32", 50, 4097, 3), ("bf16", 33, 1001, 3),
    ("fp16", 100, 6144, None), ("bf16", 16, 4096, None)])
def test_shipped_table_serves_ragged_rows_with_the_ragged_row_stage(B, oracle_lib, dtype, T, H, want_stage):
    """The table shipped with the package: rows that are not 16-byte multiples get an entry tuned on such rows (the
    ragged-row stage), rows that are never do; either way the launch matches the oracle."""
    from paper_2601_12698_b200 import synth
    table = B.SpecTable.default()
    x, r, w = synth.make_inputs(T, H, dtype, seed=47)
    y_ref, r_ref = oracle_lib.add_rmsnorm(x, r, w, EPS)
    xd, rd, wd = x.cuda(), r.cuda(), w.cuda()
    y, ro = torch.empty_like(xd), torch.empty_like(xd)
    used = table.launch(xd, rd, wd, y, ro, EPS)
    torch.cuda.synchronize()
    assert oracle_lib.bit_mismatches(ro.cpu(), r_ref) == 0, repr(used)
    assert oracle_lib.compare_y(y.cpu(), y_ref)[1] == 0, repr(used)
    if want_stage is None:
        assert used.stage != B.RT_STAGE_REG_REALIGN
    else:
        assert used.stage == want_stage and used.vec_bytes in (16, 32)
    assert B.rt_device_status() == 0
