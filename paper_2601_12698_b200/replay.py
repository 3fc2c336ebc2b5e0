"""Replay the guided search over a recorded exhaustive sweep (host only, no GPU).

    python -m paper_2601_12698_b200.replay SEARCH_LOG.jsonl [--budgets 8,16,24,32,48,64,96] [--top-k 5]

SEARCH_LOG.jsonl is what ``bench.py --log`` writes: one record per evaluated theta of the exhaustive sweep (and of the
guided search, which is ignored here).  The sweep's measured times become the cost function of ``tuner_search_with``
(a lookup: a theta the sweep did not time counts as failing its gate), and the guided search is run over it once per
budget.  Printed per budget: the time of the theta the search returns divided by the sweep's optimum, and the
evaluations it used - how much of the optimum a budget buys, free of re-timing noise.  The feasible set is derived
from the documented sm_100 limits and the compiler's report on the library as compiled, so the replay runs on any machine.
"""
from __future__ import annotations

import argparse
import json
import sys

from . import binding as B
from . import synth


def load_sweep(path: str) -> dict:
    """workload -> {theta key: microseconds} from the log's exhaustive-sweep records that passed their gate."""
    fields = [name for name, _ in B.rt_params._fields_]
    out: dict = {}
    with open(path) as f:
        for line in f:
            line = line.strip()
            if not line:
                continue
            rec = json.loads(line)
            if rec.get("search") != "exhaustive" or rec.get("status") != 0 or not rec.get("us"):
                continue
            key = tuple(int(rec["params"][k]) for k in fields)
            out.setdefault(rec["workload"], {})[key] = float(rec["us"])
    return out


def shape_of_workload(wl) -> B.rt_shape:
    op = {"add_rmsnorm": B.RT_OP_ADD_RMSNORM, "silu_and_mul": B.RT_OP_SILU_AND_MUL,
          "merge_attn_states": B.RT_OP_MERGE_ATTN_STATES, "add_rmsnorm_fp8": B.RT_OP_ADD_RMSNORM_FP8,
          "add_rmsnorm_allreduce": B.RT_OP_ADD_RMSNORM_ALLREDUCE}[wl.op]
    return B.shape_of(wl.n_tokens, wl.hidden, wl.dtype, op=op, head_dim=wl.head_dim, n_parts=wl.n_parts)


def workload_named(name: str):
    """A workload of synth.workloads(), or the ad-hoc norm shapes bench.py names adhoc_<dtype>_<tokens>x<hidden>."""
    table = synth.workloads()
    if name in table:
        return table[name]
    parts = name.split("_")
    if len(parts) == 3 and parts[0] == "adhoc" and parts[1] in synth.DTYPE_BYTES and "x" in parts[2]:
        tokens, hidden = (int(v) for v in parts[2].split("x"))
        return synth.Workload(name, parts[1], tokens, hidden, seed=9)
    return None


def replay(times: dict, shape: B.rt_shape, budgets, top_k: int = 5) -> list:
    """[(budget, ratio of the returned theta's time to the sweep's optimum, evaluations used)]."""
    limits = B.sm100_nominal_limits()
    best = min(times.values())
    rows = []
    for budget in budgets:
        res, _ = B.tuner_search_with(shape, limits, B.make_budget(max_evals=budget, top_k=top_k),
                                     lambda p: times.get(p.key(), -1.0))
        rows.append((budget, times[res.best.key()] / best, res.evals_used))
    return rows


def main(argv=None) -> None:
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("logs", nargs="+")
    ap.add_argument("--budgets", default="8,16,24,32,48,64,96")
    ap.add_argument("--top-k", type=int, default=5)
    args = ap.parse_args(argv)
    budgets = [int(v) for v in args.budgets.split(",")]
    print("workload | swept | " + " | ".join(f"budget {b}" for b in budgets))
    for path in args.logs:
        for name, times in load_sweep(path).items():
            wl = workload_named(name)
            if wl is None:
                print(f"{name}: not a workload this tool knows, skipped", file=sys.stderr)
                continue
            rows = replay(times, shape_of_workload(wl), budgets, args.top_k)
            print(f"{name} | {len(times)} | " + " | ".join(f"{ratio:.3f} ({used})" for _, ratio, used in rows))


if __name__ == "__main__":
    main(sys.argv[1:])
