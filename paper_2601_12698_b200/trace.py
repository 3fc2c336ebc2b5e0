"""Phase breakdown of one launch of the norm on a latency-bound shape, from the instrumented instances.

    python -m paper_2601_12698_b200.trace --workload c2_decode_bf16_1x4096 [--theta tpr,rpc,vec,unroll,stage,reduce,cluster]
                                          [--launches 200] [--json out.json]

A CUDA graph of `launches` instrumented launches (each with its own slice of the trace buffer) is replayed; every CTA's
first thread stamps SM cycles at entry, when the previous launch has completed, when its share of x and r has arrived,
after the row reduction and after its last store (rmsnorm_template_launch_traced).  Printed per phase: the median over
launches of the CTA-wise median and maximum, in cycles and - with the SM clock recovered from the stamps themselves - in
nanoseconds, for L2-warm launches (the same buffers every time) and for cold ones (a ring of buffer sets larger than
L2).  The launch period (exit to exit of consecutive launches) minus the released-to-stored span is what the kernel
itself cannot shorten: scheduling of the dependent launch, the flush of the previous one, and the exit.
All arithmetic here is bookkeeping on time stamps; the operator runs in the library.
"""
from __future__ import annotations

import argparse
import json
import statistics
import sys

PHASES = ("entry -> released by the previous launch", "released -> x and r arrived and summed",
          "arrived -> row reduced", "reduced -> last store issued")


def _median(v):
    return statistics.median(v) if v else float("nan")


def analyse(tr, launches: int, ctas: int, skip: int = 8) -> dict:
    """tr: int64 tensor [launches, ctas, 8] of stamps (host).  Launches before `skip` are left out (graph warm-up)."""
    rows = tr.tolist()
    # SM clock from the stamps: cycles over nanoseconds between two launches whose CTA 0 ran on the same SM
    ratios = []
    for a in range(skip, launches):
        for b in range(launches - 1, a + 16, -1):
            if rows[a][0][7] == rows[b][0][7] and rows[b][0][0] > rows[a][0][0]:
                ratios.append((rows[b][0][1] - rows[a][0][1]) / (rows[b][0][0] - rows[a][0][0]))
                break
    ghz = _median(ratios)
    per_phase_med, per_phase_max, active, period, overlap = [[] for _ in PHASES], [[] for _ in PHASES], [], [], []
    for k in range(skip, launches):
        spans = [[rows[k][c][2 + p] - rows[k][c][1 + p] for c in range(ctas)] for p in range(len(PHASES))]
        for p, s in enumerate(spans):
            per_phase_med[p].append(_median(s))
            per_phase_max[p].append(max(s))
        active.append(max(rows[k][c][5] - rows[k][c][2] for c in range(ctas)))
        if k + 1 < launches:
            period.append(max(rows[k + 1][c][6] for c in range(ctas)) - max(rows[k][c][6] for c in range(ctas)))
            # how long the next launch's first CTA was already resident before this launch's last CTA left
            overlap.append(max(rows[k][c][6] for c in range(ctas)) - min(rows[k + 1][c][0] for c in range(ctas)))
    out = {"sm_ghz_from_stamps": ghz, "launches_used": launches - skip, "ctas": ctas, "phases": []}
    for p, name in enumerate(PHASES):
        med, mx = _median(per_phase_med[p]), _median(per_phase_max[p])
        out["phases"].append({"phase": name, "cycles_median_cta": med, "cycles_slowest_cta": mx,
                              "ns_median_cta": med / ghz, "ns_slowest_cta": mx / ghz})
    out["released_to_stored_ns_slowest_cta"] = _median(active) / ghz
    out["launch_period_ns"] = _median(period)
    out["next_launch_resident_before_exit_ns"] = _median(overlap)
    out["outside_the_kernel_ns"] = out["launch_period_ns"] - out["released_to_stored_ns_slowest_cta"]
    return out


def run(workload: str, theta_text: str = "", launches: int = 200, replays: int = 5) -> dict:
    import torch
    from . import binding as B
    from . import synth
    if not torch.cuda.is_available():
        raise RuntimeError("the phase trace needs a CUDA device")
    wl = synth.workloads()[workload]
    if wl.op != "add_rmsnorm":
        raise SystemExit("instrumented instances exist for add_rmsnorm only")
    T, H = wl.n_tokens, wl.hidden
    x, r, w = synth.make_workload_inputs(wl)
    if theta_text:
        theta = B.rt_params(*[int(v) for v in theta_text.split(",")])
    else:
        theta = B.SpecTable.default().lookup(B.shape_of(T, H, wl.dtype))[0]
    words = B.rmsnorm_trace_words(theta, T, H, wl.dtype)
    if words < 0:
        raise SystemExit(f"{theta!r} is infeasible on {workload}")
    ctas = words // B.RT_TRACE_WORDS
    limits = B.rt_query_limits()
    sets_cold = int(min(4096, -(-3 * limits.l2_bytes // wl.algorithmic_bytes)))
    stream = torch.cuda.Stream()
    floor = B.tuner_launch_floor(B.make_budget(warmup=20, iters=100, repeats=5, use_graph=True), stream=stream)
    result = {"workload": workload, "theta": theta.as_dict(), "empty_kernel_in_graph_us": floor, "modes": {}}
    for mode, sets in (("l2_warm", 1), ("cold", sets_cold)):
        ring = lambda t: t.cuda().unsqueeze(0).repeat(sets, 1, 1).contiguous()
        xd, rd, wd = ring(x), ring(r), w.cuda()
        yd, od = torch.empty_like(xd), torch.empty_like(xd)
        trace = torch.zeros((launches, ctas, B.RT_TRACE_WORDS), dtype=torch.int64, device="cuda")
        B.rmsnorm_template_launch_traced(theta, xd[0], rd[0], wd, yd[0], od[0], wl.eps, trace[0], stream=stream)  # refusals show here
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for k in range(launches):
                s = k % sets
                B.rmsnorm_template_launch_traced(theta, xd[s], rd[s], wd, yd[s], od[s], wl.eps, trace[k], stream=stream)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(replays):
            e0.record(); graph.replay(); e1.record()
        torch.cuda.synchronize()
        info = analyse(trace.cpu(), launches, ctas)
        info["event_us_per_launch_with_stamps"] = e0.elapsed_time(e1) * 1e3 / launches
        info["ring_sets"] = sets
        # the same graph without the stamps, for what the stamps themselves cost
        plain = torch.cuda.CUDAGraph()
        with torch.cuda.graph(plain, stream=stream):
            for k in range(launches):
                s = k % sets
                B.rmsnorm_template_launch(theta, xd[s], rd[s], wd, yd[s], od[s], wl.eps, stream=stream)
        for _ in range(replays):
            e0.record(); plain.replay(); e1.record()
        torch.cuda.synchronize()
        info["event_us_per_launch_plain"] = e0.elapsed_time(e1) * 1e3 / launches
        result["modes"][mode] = info
    if B.rt_device_status() != 0:
        raise RuntimeError("device status word set")
    return result


def render(res: dict) -> str:
    lines = [f"{res['workload']}  theta {list(res['theta'].values())}  empty kernel in a graph {res['empty_kernel_in_graph_us']:.3f} us"]
    for mode, info in res["modes"].items():
        lines.append(f"-- {mode} ({info['ring_sets']} buffer set(s), {info['ctas']} CTAs, SM clock from stamps "
                     f"{info['sm_ghz_from_stamps'] * 1e3:.0f} MHz): {info['event_us_per_launch_plain']:.3f} us per launch by "
                     f"events ({info['event_us_per_launch_with_stamps']:.3f} with stamps)")
        for ph in info["phases"]:
            lines.append(f"   {ph['phase']:<44} {ph['cycles_median_cta']:8.0f} cycles = {ph['ns_median_cta']:7.0f} ns"
                         f"   (slowest CTA {ph['ns_slowest_cta']:7.0f} ns)")
        lines.append(f"   released -> stored, slowest CTA {info['released_to_stored_ns_slowest_cta']:7.0f} ns;  launch period "
                     f"{info['launch_period_ns']:7.0f} ns;  outside the kernel {info['outside_the_kernel_ns']:7.0f} ns;  next launch "
                     f"resident {info['next_launch_resident_before_exit_ns']:7.0f} ns before this one exits")
    return "\n".join(lines)


def main(argv=None) -> None:
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--workload", default="c2_decode_bf16_1x4096")
    ap.add_argument("--theta", default="", help="tpr,rpc,vec,unroll,stage,reduce,cluster (default: the shipped table's)")
    ap.add_argument("--launches", type=int, default=200)
    ap.add_argument("--json", default="")
    args = ap.parse_args(argv)
    res = run(args.workload, args.theta, args.launches)
    print(render(res))
    if args.json:
        with open(args.json, "w") as f:
            json.dump(res, f, indent=1)


if __name__ == "__main__":
    main(sys.argv[1:])
