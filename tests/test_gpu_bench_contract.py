"""bench.py's own arm on a GPU: one JSON line with every key of the contract, on a small workload with a fixed theta
(the tuner is skipped) and on one with a short search."""
import json
import os
import subprocess
import sys

import pytest
import torch

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*args):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1, out.stdout
    return json.loads(lines[0])


def _check_contract(d, workload, steps, warmup):
    assert d["metric"] == "fused_add_rmsnorm_hbm_gbs" and d["unit"] == "GB/s" and d["value"] > 0
    assert d["n_gpus"] == 1 and d["steps"] == steps and d["warmup"] == warmup and d["ms_per_step"] > 0
    assert d["higher_is_better"] is True and d["scaling"] == "weak" and d["vs_baseline"] is None
    assert d["data"] == "synthetic" and d["dtype"] in ("bf16", "fp16", "fp32")
    assert d["config"]["workload"] == workload and "model" not in d["config"] and d["config"]["l2"]
    assert d["gpu_launches"] == steps  # one launch of the library's kernel per step, counted by the library
    roof = d["roofline"]
    assert roof["bound"] == "hbm" and roof["unit"] == "GB/s" and roof["peak"] > 0
    assert abs(roof["frac"] - roof["achieved"] / roof["peak"]) < 1e-9 and roof["peak_kind"] in ("of measured", "of fallback")
    assert roof["traffic"] is None or roof["traffic"] > 0
    # value = algorithmic bytes per launch / measured time per launch
    assert abs(d["value"] - roof["algorithmic_bytes_per_launch"] / (d["ms_per_step"] * 1e-3) / 1e9) < 1e-6 * d["value"]
    e2e = d["e2e"]
    assert e2e["unit"] == "GB/s" and 0 < e2e["value"] and e2e["h2d_bytes_per_step"] > 0 and e2e["d2h_bytes_per_step"] > 0
    assert e2e["value"] != d["value"]
    clocks = d["clocks"]
    assert clocks["sm_max_mhz"] >= clocks["sm_mhz"] > 0 and isinstance(clocks["reasons"], list)
    cpu = d["cpu_baseline"]
    assert cpu["kind"] == "oracle" and cpu["value"] > 0 and cpu["cores"] >= 1 and cpu["sample"]
    par = d["parity"]
    assert par["r_out_bit_mismatches"] == 0 and par["y_beyond_tolerance"] == 0 and par["rows_checked"] > 0


def test_fixed_theta_line_keeps_the_contract():
    d = _run("--workload", "c2_decode_bf16_256x4096", "--steps", "40", "--warmup", "3", "--e2e-steps", "2",
             "--theta", "512,1,16,1,0,0,1")
    _check_contract(d, "c2_decode_bf16_256x4096", 40, 3)
    assert d["config"]["theta"] == {"threads_per_row": 512, "rows_per_cta": 1, "vec_bytes": 16, "unroll": 1, "stage": 0,
                                    "reduce": 0, "cluster_size": 1}


def test_searched_line_on_ragged_rows_reports_the_tuner():
    """Rows of 6145 fp16 elements (a small feasible set, so the sweep is short): the line carries the search report and
    the search's pick is the ragged-row stage."""
    d = _run("--workload", "c4x_fp16_8192x6145", "--steps", "30", "--warmup", "3", "--e2e-steps", "2", "--search-budget", "24")
    _check_contract(d, "c4x_fp16_8192x6145", 30, 3)
    t = d["tuner"]
    assert t["feasible"] > 0 and t["raw_grid"] >= t["feasible"] and t["search_evals_used"] <= 24 and t["failed_gate"] == 0
    assert t["search_best"] == d["config"]["theta"] and t["search_best"]["stage"] == 3
    assert 1.0 <= t["search_vs_exhaustive"] < 1.1          # the guided winner is a member of the re-tested set
    assert d["roofline"]["frac"] > 0.75
    # the side-by-side re-test: every candidate with its spread and clock, the per-round ratios, the shipped table's pick
    rt = t["retest"]
    assert len(rt["per_round_ratio_min_median_max"]) == 3 and rt["per_round_ratio_min_median_max"][0] >= 1.0
    assert any(c["from"] == "guided" for c in rt["candidates"]) and all(c["us"] > 0 and c["spread"] >= 0 for c in rt["candidates"])
    assert t["shipped_table"]["source"] == "table_exact" and t["shipped_table"]["vs_exhaustive"] >= 1.0
    assert set(t["sweep_best_per_stage"]) == {"reg", "reg_realign"}
    assert d["cpu_baseline"]["single_thread"]["cores"] == 1 and d["cpu_baseline"]["single_thread"]["value"] > 0
    assert d["clocks"]["samples"] >= 1 and d["roofline"]["traffic_capture"] is None or "kernel_sha256_16_now" in d["roofline"]["traffic_capture"]


def test_a_search_resumes_from_its_log_and_ad_hoc_shapes_run(tmp_path):
    """--log writes the search log, --resume seeds the next search with its fastest thetas (evaluated first, phase
    'seed'); the workload is an ad-hoc shape the shipped table has no entry for, so the table's answer is a neighbour's;
    --sweep-heuristics widens the exhaustive sweep alone."""
    log = str(tmp_path / "search.jsonl")
    d = _run("--workload", "bf16:700x4096", "--steps", "20", "--warmup", "3", "--e2e-steps", "2", "--search-budget", "20",
             "--retest-rounds", "3", "--log", log)
    assert d["config"]["workload"] == "adhoc_bf16_700x4096" and d["tuner"]["shipped_table"]["source"] == "table_nearest"
    first = d["tuner"]["search_best"]
    d2 = _run("--workload", "bf16:700x4096", "--steps", "20", "--warmup", "3", "--e2e-steps", "2", "--search-budget", "20",
              "--retest-rounds", "3", "--resume", log, "--log", log + ".2", "--sweep-heuristics", "18")
    assert d2["tuner"]["resumed_seeds"] >= 8
    # the sweep alone ran over the hard-feasible set (duplicates and the pipeline stage aside), the search over the default one
    assert d2["tuner"]["sweep_heuristics"] == 18 and d2["tuner"]["exhaustive_evals"] > d2["tuner"]["feasible"] == d["tuner"]["feasible"]
    assert d["tuner"]["sweep_heuristics"] == 63 and d["tuner"]["exhaustive_evals"] == d["tuner"]["feasible"]
    phases = [json.loads(line)["phase"] for line in open(log + ".2") if '"guided"' in line]
    assert phases[0] == "seed" and phases.count("seed") >= 4
    assert d2["tuner"]["search_best_us"] <= 1.1 * d["tuner"]["search_best_us"] and first
