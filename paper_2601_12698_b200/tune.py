"""Tune the template on this GPU: a specialised table D_spec and a general configuration theta_gen.

    python -m paper_2601_12698_b200.tune --shapes bf16:128x4096,bf16:16384x8192,fp32:2048x8192 \
        --budget 64 --out rmsnorm_table.json

For every shape: seeded synthetic inputs, a guided search (Algorithm 1: DeriveFeasibleSpace, Search), then
SelectGeneral over the shapes' finalists timed on every shape and BuildSpecialized as a JSON table that
``binding.SpecTable`` loads for ``rmsnorm_launch_auto``.

The correctness gate needs reference outputs.  As in the paper's protocol (every candidate is compared with
the original kernel S_ref on identical inputs), the reference here is the library's plainest instance -
registers, shuffle reduction, unroll 1, one row per CTA - run on the same inputs; that instance is itself
checked against the CPU oracle by the test-suite, which this tool does not use.
"""
from __future__ import annotations

import argparse
import json
import sys

import torch

from . import binding as B
from . import synth


def parse_shapes(text: str):
    out = []
    for item in text.split(","):
        dtype, dims = item.strip().split(":")
        t, h = dims.lower().split("x")
        out.append((dtype, int(t), int(h)))
    return out


def reference_theta(shape: B.rt_shape) -> B.rt_params:
    """The plainest feasible instance: S_ref of the gate."""
    plain = [t for t in B.tuner_derive_feasible(shape) if t.stage == B.RT_STAGE_REG and t.reduce == B.RT_REDUCE_SHFL
             and t.unroll == 1 and t.rows_per_cta == 1]
    if not plain:
        raise RuntimeError("no plain register-stage instance is feasible for this shape")
    return max(plain, key=lambda t: (t.vec_bytes, -t.threads_per_row))


class ShapeProblem:
    """Device buffers of one shape: inputs, outputs, reference outputs from S_ref."""

    def __init__(self, dtype: str, n_tokens: int, hidden: int, seed: int, eps: float, stream):
        self.dtype, self.n_tokens, self.hidden, self.eps = dtype, n_tokens, hidden, eps
        x, r, w = synth.make_inputs(n_tokens, hidden, dtype, seed)
        self.x, self.r, self.w = x.cuda(), r.cuda(), w.cuda()
        self.y, self.r_out = torch.empty_like(self.x), torch.empty_like(self.x)
        self.y_ref, self.r_ref = torch.empty_like(self.x), torch.empty_like(self.x)
        self.shape = B.shape_of(n_tokens, hidden, dtype, B._ptr_align(self.x, self.r, self.w, self.y, self.r_out))
        self.ref_theta = reference_theta(self.shape)
        B.rmsnorm_template_launch(self.ref_theta, self.x, self.r, self.w, self.y_ref, self.r_ref, eps, stream=stream)
        stream.synchronize()
        self.ws = B.make_workspace(self.x, self.r, self.w, self.y, self.r_out, self.y_ref, self.r_ref, eps, stream=stream)
        limits = B.rt_query_limits()
        self.use_graph = 4 * x.numel() * x.element_size() <= 2 * limits.l2_bytes


def tune(shapes, budget: int = 64, top_k: int = 5, finalists: int = 3, seed: int = 0, eps: float = 1e-6, verbose=False):
    """Returns (SpecTable, report dict)."""
    stream = torch.cuda.Stream()
    problems, per_shape, candidates = [], [], {}
    for dtype, t, h in shapes:
        p = ShapeProblem(dtype, t, h, seed, eps, stream)
        res, log = B.tuner_search(p.shape, B.make_budget(max_evals=budget, top_k=top_k, use_graph=p.use_graph), p.ws)
        ranked = sorted((rec for rec in log if rec.status == B.RT_OK), key=lambda rec: rec.us)
        seen = []
        for rec in ranked:
            if rec.params.key() not in seen:
                seen.append(rec.params.key())
            if len(seen) == finalists:
                break
        for key in [res.best.key()] + seen:
            candidates.setdefault(key, B.rt_params(*key))
        per_shape.append((p.shape, res.best, res.best_us, res.evals_used))
        problems.append((dtype, t, h))
        if verbose:
            print(f"{dtype}:{t}x{h}: {res.best} {res.best_us:.2f} us ({res.evals_used} evaluations)", file=sys.stderr)
        del p
        torch.cuda.empty_cache()

    # SelectGeneral: every finalist timed on every shape (paper protocol), then the geometric-mean choice
    cand = list(candidates.values())
    times = [[-1.0] * len(problems) for _ in cand]
    for xi, (dtype, t, h) in enumerate(problems):
        p = ShapeProblem(dtype, t, h, seed, eps, stream)
        proto = B.make_budget(warmup=20, iters=100, repeats=3, use_graph=p.use_graph)
        for ci, th in enumerate(cand):
            if B.tuner_check_params(p.shape, th) != B.RT_OK:
                continue
            rec = B.tuner_evaluate(p.shape, th, proto, p.ws)
            if rec.status == B.RT_OK:
                times[ci][xi] = rec.us
        del p
        torch.cuda.empty_cache()
    general, report = None, {"shapes": [f"{d}:{t}x{h}" for d, t, h in problems]}
    try:
        gi, score, scores = B.tuner_select_general(times)
        general = cand[gi]
        report.update({"general": general.as_dict(), "general_geomean_vs_specialised": round(score, 4),
                       "general_us": [round(v, 3) for v in times[gi]]})
    except B.TunerError as err:
        report["general"] = None
        report["general_error"] = str(err)
    best_per_shape = [min((times[c][x] for c in range(len(cand)) if times[c][x] > 0), default=-1.0)
                      for x in range(len(problems))]
    report["specialised_us"] = [round(v, 3) for v in best_per_shape]
    report["specialised"] = [th.as_dict() for _, th, _, _ in per_shape]
    report["evaluations"] = [n for _, _, _, n in per_shape]
    table = B.SpecTable([(s, th, us) for s, th, us, _ in per_shape], general, torch.cuda.get_device_name())
    return table, report


def main() -> None:
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--shapes", required=True, help="comma-separated dtype:TOKENSxHIDDEN, e.g. bf16:128x4096")
    ap.add_argument("--budget", type=int, default=64, help="kernel evaluations per shape")
    ap.add_argument("--out", default="", help="write the table as JSON here")
    ap.add_argument("--seed", type=int, default=0)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("tuning needs a CUDA device")
    table, report = tune(parse_shapes(args.shapes), budget=args.budget, seed=args.seed, verbose=True)
    if args.out:
        with open(args.out, "w") as f:
            json.dump(table.to_json(), f, indent=1)
    print(json.dumps(report))


if __name__ == "__main__":
    main()
