"""Host-side parts of bench.py that need no GPU: the N-rank launcher, resuming a search from its log, the choice of
finalists, the clock-sample windows and the ncu traffic table."""
import importlib.util
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _bench():
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_plain_start_with_gpus_2_runs_two_ranks_and_prints_one_line():
    """`python bench.py --gpus 2` without a launcher starts the ranks itself; on the reference arm (no GPU needed)
    rank 0 alone prints, and the line says n_gpus = 2."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                          "--warmup", "0", "--workload", "c2_decode_bf16_4x4096"], capture_output=True, text=True,
                         check=True, cwd=ROOT, env=env)
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2
    assert d["config"]["n_tokens_per_gpu"] == 4 and d["config"]["hidden"] == 4096


def test_spawned_ranks_rendezvous_as_one_group(tmp_path):
    """The launcher's environment is what torch.distributed needs: two ranks find each other over gloo on 127.0.0.1
    and a failure of one rank ends the launcher with its exit code."""
    bench = _bench()
    script = tmp_path / "rank.py"
    script.write_text(textwrap.dedent("""
        import os, sys
        import torch, torch.distributed as dist
        dist.init_process_group("gloo")
        t = torch.tensor([float(os.environ["RANK"]) + 1.0])
        dist.all_reduce(t)
        assert os.environ["LOCAL_RANK"] == os.environ["RANK"] and os.environ["MASTER_ADDR"] == "127.0.0.1"
        open(os.path.join(sys.argv[1], "rank%s.txt" % os.environ["RANK"]), "w").write("%d %d %g" % (
            dist.get_rank(), dist.get_world_size(), t.item()))
        dist.destroy_process_group()
        sys.exit(int(sys.argv[2]) if os.environ["RANK"] == "1" else 0)
    """))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_PORT")}
    old = dict(os.environ)
    try:
        os.environ.clear()
        os.environ.update(env)
        assert bench.spawn_ranks(2, [str(tmp_path), "0"], script=str(script), timeout_s=120) == 0
        assert sorted(p.name for p in tmp_path.glob("rank*.txt")) == ["rank0.txt", "rank1.txt"]
        assert (tmp_path / "rank0.txt").read_text() == "0 2 3" and (tmp_path / "rank1.txt").read_text() == "1 2 3"
        assert bench.spawn_ranks(2, [str(tmp_path), "7"], script=str(script), timeout_s=120) == 7
    finally:
        os.environ.clear()
        os.environ.update(old)


def _rec(workload, theta, us, status=0):
    names = ("threads_per_row", "rows_per_cta", "vec_bytes", "unroll", "stage", "reduce", "cluster_size")
    return json.dumps({"search": "guided", "workload": workload, "status": status, "us": us, "params": dict(zip(names, theta))})


def test_resume_reads_a_search_log_back_as_seeds(tmp_path):
    bench = _bench()
    log = tmp_path / "log.jsonl"
    a, b, c, d = (256, 1, 32, 2, 0, 0, 1), (512, 1, 16, 1, 2, 0, 1), (128, 2, 16, 4, 0, 1, 1), (64, 1, 8, 1, 1, 0, 1)
    log.write_text("\n".join([_rec("wl", b, 120.0), _rec("wl", a, 101.0), _rec("wl", a, 99.5), _rec("wl", c, 90.0, status=7),
                              _rec("other", d, 5.0), "", _rec("wl", c, 0.0)]) + "\n")
    seeds = bench.resume_seeds(str(log), "wl")
    # this workload's thetas first, fastest first (a theta's best time counts); failed and untimed records are dropped;
    # thetas of other workloads follow
    assert [s.key() for s in seeds] == [a, b, d]
    assert [s.key() for s in bench.resume_seeds(str(log), "wl", k=1)] == [a, d]


def test_fastest_of_takes_the_last_record_of_each_theta():
    bench = _bench()
    from paper_2601_12698_b200 import binding as B

    def rec(theta, us, status=0):
        r = B.rt_eval_record()
        r.params = B.rt_params(*theta)
        r.us, r.status = us, status
        return r
    a, b, c = (256, 1, 32, 2, 0, 0, 1), (512, 1, 16, 1, 2, 0, 1), (128, 2, 16, 4, 0, 1, 1)
    log = [rec(a, 100.0), rec(b, 105.0), rec(c, 90.0, status=7), rec(a, 110.0)]   # a's re-test was slower
    assert [t.key() for t in bench.fastest_of(log, 8)] == [b, a]
    assert [t.key() for t in bench.fastest_of(log, 1)] == [b]


def test_clock_windows_pick_the_samples_of_an_interval():
    bench = _bench()
    cs = bench.ClockSampler.__new__(bench.ClockSampler)
    cs.proc, cs.max_mhz, cs._parsed = None, 1965, 0
    cs.samples = [(10.0 + 0.001 * i, 1965 if i < 50 else 1500, 0x4 if i >= 50 else 0) for i in range(100)]
    w = cs.window(10.0, 10.0495)
    assert w["sm_mhz"] == 1965 and w["samples"] == 50 and w["reasons"] == [] and "window" not in w
    w = cs.window(10.05, 10.2)
    assert w["sm_mhz"] == 1500 and w["sm_min_mhz"] == 1500 and w["reasons"] == ["sw_power_cap"]
    w = cs.window(10.0601, 10.0602)  # an interval between two samples: widened to the nearest ones, and says so
    assert w["samples"] == 3 and w["sm_mhz"] == 1500 and "window" in w
    assert cs.median_mhz(10.0203, 10.0204) == 1965
    cs.samples = []
    assert cs.window(0.0, 1.0) == {"sm_mhz": None, "sm_max_mhz": 1965, "reasons": [], "samples": 0}


def test_traffic_figures_are_tied_to_the_kernel_they_were_captured_on():
    bench = _bench()
    wl, theta = "c3_prefill_bf16_16384x8192", (512, 1, 32, 1, 0, 0, 1)
    nbytes, captured_on = bench.NCU_TRAFFIC[wl][theta]
    traffic, info = bench.ncu_traffic(wl, theta)
    assert info["bytes_per_launch"] == nbytes and info["kernel_sha256_16_now"] == bench.kernel_source_hash()
    assert (traffic == nbytes) == (captured_on == bench.kernel_source_hash())  # null once the kernel has changed
    assert bench.ncu_traffic(wl, (32, 8, 8, 1, 1, 1, 1)) == (None, None)
    # every stored figure is at most the workload's algorithmic bytes plus a few percent (no re-reads), and short of
    # them by no more than the share of the outputs that can still be dirty in L2 when the kernel ends
    from paper_2601_12698_b200 import synth
    for name, table in bench.NCU_TRAFFIC.items():
        alg = synth.workloads()[name].algorithmic_bytes
        assert all(alg - 60e6 < v[0] < 1.02 * alg for v in table.values())


def test_phase_analysis_of_synthetic_stamps():
    """trace.analyse on stamps built by hand: 1.5 GHz, phases of 300 / 900 / 450 / 150 cycles, a launch every 2000 ns."""
    import torch
    from paper_2601_12698_b200 import trace
    launches, ctas = 40, 3
    t = torch.zeros((launches, ctas, 8), dtype=torch.int64)
    for k in range(launches):
        for c in range(ctas):
            ns0 = 1_000_000 + 2000 * k + 10 * c
            cyc0 = 5_000_000 + int(1.5 * (ns0 - 1_000_000)) + 7 * c
            marks = [cyc0, cyc0 + 300, cyc0 + 1200, cyc0 + 1650 + 30 * c, cyc0 + 1800 + 30 * c]
            t[k, c] = torch.tensor([ns0, *marks, ns0 + 1300, 5])
    info = trace.analyse(t, launches, ctas, skip=4)
    assert abs(info["sm_ghz_from_stamps"] - 1.5) < 0.01
    assert [round(ph["cycles_median_cta"]) for ph in info["phases"]] == [300, 900, 480, 150]
    assert [round(ph["cycles_slowest_cta"]) for ph in info["phases"]] == [300, 900, 510, 150]
    assert info["launch_period_ns"] == 2000 and abs(info["released_to_stored_ns_slowest_cta"] - 1560 / 1.5) < 8
    assert abs(info["outside_the_kernel_ns"] - (2000 - 1560 / 1.5)) < 8
    assert info["next_launch_resident_before_exit_ns"] == (1300 + 20) - 2000


def test_replay_of_a_recorded_sweep(tmp_path):
    """replay.py: the guided search over a sweep log's times; a budget that covers the set finds the optimum exactly."""
    import math
    from paper_2601_12698_b200 import binding as B
    from paper_2601_12698_b200 import replay, synth
    wl = synth.workloads()["c2_decode_bf16_16x4096"]
    shape = replay.shape_of_workload(wl)
    feasible = B.tuner_derive_feasible(shape, B.sm100_nominal_limits())
    names = [name for name, _ in B.rt_params._fields_]
    cost = lambda t: 2.0 + 0.3 * abs(math.log2(t.threads_per_row) - 9) + 0.1 * (t.unroll - 1) + 0.2 * t.stage + 0.05 * t.reduce
    log = tmp_path / "sweep.jsonl"
    with open(log, "w") as f:
        for t in feasible:
            f.write(json.dumps({"search": "exhaustive", "workload": wl.name, "status": 0, "us": cost(t),
                                "params": dict(zip(names, t.key()))}) + "\n")
        f.write(json.dumps({"search": "guided", "workload": wl.name, "status": 0, "us": 0.1,
                            "params": dict(zip(names, feasible[0].key()))}) + "\n")      # not part of the sweep: ignored
        f.write(json.dumps({"search": "exhaustive", "workload": wl.name, "status": 7, "us": 0.1,
                            "params": dict(zip(names, feasible[1].key()))}) + "\n")      # failed its gate: ignored
    times = replay.load_sweep(str(log))[wl.name]
    assert len(times) == len(feasible) and min(times.values()) >= 2.0
    rows = replay.replay(times, shape, [4, 64, 4 * len(feasible)])
    assert [b for b, _, _ in rows] == [4, 64, 4 * len(feasible)]
    assert all(ratio >= 1.0 for _, ratio, _ in rows) and rows[0][2] <= 4 and rows[1][2] <= 64
    assert rows[1][1] < 1.1 and rows[2][1] == 1.0
