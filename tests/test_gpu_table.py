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
    path = tmp_path / "table.json"
    path.write_text(json.dumps(table.to_json()))
    again = B.SpecTable.from_json(json.loads(path.read_text()))
    assert [t.key() for _, t, _ in again.entries] == [t.key() for _, t, _ in table.entries]
    assert again.general.key() == table.general.key()


@pytest.mark.parametrize("dtype,T,H,want_source", [
    ("bf16", 64, 4096, "table_exact"), ("bf16", 2048, 8192, "table_exact"), ("bf16", 77, 4096, "table_nearest"),
    ("bf16", 4096, 7168, "table_nearest"), ("fp16", 300, 6152, "table_nearest"), ("fp16", 300, 6148, None),
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
    if want_source == "general_or_feasible":
        assert source in ("general", "feasible_set")
    elif want_source is not None:
        assert source == want_source
    assert B.rt_device_status() == 0
