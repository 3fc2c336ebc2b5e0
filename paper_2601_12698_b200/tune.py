"""Tune the template on this GPU: a specialised table D_spec and a general configuration theta_gen.

    python -m paper_2601_12698_b200.tune --shapes bf16:128x4096,bf16:16384x8192,fp32:2048x8192 \
        --budget 64 --out rmsnorm_table.json
    python -m paper_2601_12698_b200.tune --shapes silu/bf16:4096x14336,merge/bf16:512x32x128,fp8/bf16:4096x8192
    python -m paper_2601_12698_b200.tune --shapes allreduce/bf16:4096x8192x4

For every (kernel, shape): seeded synthetic inputs, a guided search (Algorithm 1: DeriveFeasibleSpace, Search),
then, per kernel, SelectGeneral over the shapes' finalists timed on every shape, and BuildSpecialized as a JSON table that
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


PREHEAT_MS = 300

OPS = {"norm": B.RT_OP_ADD_RMSNORM, "silu": B.RT_OP_SILU_AND_MUL, "merge": B.RT_OP_MERGE_ATTN_STATES,
       "fp8": B.RT_OP_ADD_RMSNORM_FP8, "allreduce": B.RT_OP_ADD_RMSNORM_ALLREDUCE}


def parse_shapes(text: str):
    """[kernel/]dtype:dims, comma separated.  kernel: norm (default, TOKENSxHIDDEN), silu (TOKENSxD),
    merge (TOKENSxHEADSxHEAD_DIM), fp8 (the norm with e4m3 output, TOKENSxHIDDEN), allreduce (the norm with its x
    given as PARTS partial inputs, TOKENSxHIDDENxPARTS)."""
    out = []
    for item in text.split(","):
        item = item.strip()
        kernel, rest = item.split("/") if "/" in item else ("norm", item)
        dtype, dims = rest.split(":")
        out.append((kernel, dtype, tuple(int(v) for v in dims.lower().split("x"))))
    return out


def reference_theta(shape: B.rt_shape) -> B.rt_params:
    """The plainest feasible instance: S_ref of the gate."""
    plain = [t for t in B.tuner_derive_feasible(shape) if t.stage == B.RT_STAGE_REG and t.reduce == B.RT_REDUCE_SHFL
             and t.unroll == 1 and t.rows_per_cta == 1]
    if not plain:
        raise RuntimeError("no plain register-stage instance is feasible for this shape")
    return max(plain, key=lambda t: (t.vec_bytes, -t.threads_per_row))


class ShapeProblem:
    """Device buffers of one (kernel, shape): inputs, outputs, reference outputs from S_ref."""

    def __init__(self, kernel: str, dtype: str, dims: tuple, seed: int, eps: float, stream):
        self.kernel, self.dtype, self.dims, self.eps = kernel, dtype, dims, eps
        op = OPS[kernel]
        n_tokens = dims[0]
        if kernel == "silu":
            d = dims[1]
            x = synth.make_gate_up(0, n_tokens, d, dtype, seed).cuda()
            y, y_ref = (torch.empty(n_tokens, d, dtype=x.dtype, device="cuda") for _ in range(2))
            self.shape = B.shape_of(n_tokens, d, dtype, B._ptr_align(x, y), op=op)
            self.ref_theta = reference_theta(self.shape)
            B.silu_and_mul_template_launch(self.ref_theta, x, y_ref, stream=stream)
            self.ws = B.make_workspace(x, None, None, y, None, y_ref, None, eps, stream=stream)
            moved = 3 * x.element_size() * n_tokens * d
            self.keep = (x, y, y_ref)
        elif kernel == "merge":
            h, d = dims[1], dims[2]
            va, sa, vb, sb = (t.cuda() for t in synth.make_merge_inputs(0, n_tokens, h, d, dtype, seed))
            vo, vo_ref, so, so_ref = torch.empty_like(va), torch.empty_like(va), torch.empty_like(sa), torch.empty_like(sa)
            self.shape = B.shape_of(n_tokens, h * d, dtype, B._ptr_align(va, vb, vo), op=op, head_dim=d)
            self.ref_theta = reference_theta(self.shape)
            B.merge_attn_states_template_launch(self.ref_theta, va, sa, vb, sb, vo_ref, so_ref, stream=stream)
            self.ws = B.make_workspace(va, vb, sa, vo, so, vo_ref, so_ref, eps, stream=stream, aux=sb)
            moved = 3 * va.element_size() * va.numel()
            self.keep = (va, sa, vb, sb, vo, vo_ref, so, so_ref)
        elif kernel == "allreduce":
            hidden, n_parts = dims[1], dims[2]
            _, r, w = (t.cuda() for t in synth.make_inputs(n_tokens, hidden, dtype, seed))
            parts = synth.make_parts(0, n_tokens, hidden, dtype, seed, n_parts).cuda()  # [parts, tokens, hidden]
            y, y_ref, r_out, r_ref = (torch.empty_like(r) for _ in range(4))
            self.shape = B.shape_of(n_tokens, hidden, dtype, B._ptr_align(parts, r, w, y, r_out), op=op, n_parts=n_parts)
            self.ref_theta = reference_theta(self.shape)
            B.rmsnorm_allreduce_template_launch(self.ref_theta, [parts[k] for k in range(n_parts)], r, w, [y_ref], [r_ref],
                                                0, n_tokens, eps, stream=stream)
            self.ws = B.make_workspace(parts, r, w, y, r_out, y_ref, r_ref, eps, stream=stream)
            moved = (n_parts + 3) * r.element_size() * r.numel()
            self.keep = (parts, r, w, y, y_ref, r_out, r_ref)
        else:
            hidden = dims[1]
            x, r, w = (t.cuda() for t in synth.make_inputs(n_tokens, hidden, dtype, seed))
            r_out, r_ref = torch.empty_like(x), torch.empty_like(x)
            if kernel == "fp8":
                y, y_ref = (torch.empty(n_tokens, hidden, dtype=torch.uint8, device="cuda") for _ in range(2))
                sc, sc_ref = (torch.empty(n_tokens, dtype=torch.float32, device="cuda") for _ in range(2))
                self.shape = B.shape_of(n_tokens, hidden, dtype, B._ptr_align(x, r, w, r_out), op=op)
                self.ref_theta = reference_theta(self.shape)
                B.rmsnorm_fp8_template_launch(self.ref_theta, x, r, w, y_ref, sc_ref, r_ref, eps, stream=stream)
                self.ws = B.make_workspace(x, r, w, y, r_out, y_ref, r_ref, eps, stream=stream, aux_out=sc, aux_ref=sc_ref)
                self.keep = (x, r, w, y, y_ref, r_out, r_ref, sc, sc_ref)
            else:
                y, y_ref = torch.empty_like(x), torch.empty_like(x)
                self.shape = B.shape_of(n_tokens, hidden, dtype, B._ptr_align(x, r, w, y, r_out), op=op)
                self.ref_theta = reference_theta(self.shape)
                B.rmsnorm_template_launch(self.ref_theta, x, r, w, y_ref, r_ref, eps, stream=stream)
                self.ws = B.make_workspace(x, r, w, y, r_out, y_ref, r_ref, eps, stream=stream)
                self.keep = (x, r, w, y, y_ref, r_out, r_ref)
            moved = 4 * x.element_size() * x.numel()
        stream.synchronize()
        # up to half of L2: a CUDA graph of 100 launches on the same buffers (L2-warm, launch gaps out of the way);
        # above that plain back-to-back launches on a pre-heated device
        self.use_graph = moved <= B.rt_query_limits().l2_bytes // 2

    @property
    def label(self) -> str:
        return f"{self.kernel}/{self.dtype}:" + "x".join(str(v) for v in self.dims)


def tune(shapes, budget: int = 64, top_k: int = 5, finalists: int = 3, seed: int = 0, eps: float = 1e-6, verbose=False):
    """shapes: [(kernel, dtype, dims)] or, for the norm, [(dtype, n_tokens, hidden)].  Returns (SpecTable, report)."""
    shapes = [s if isinstance(s[2], tuple) else ("norm", s[0], (s[1], s[2])) for s in shapes]
    stream = torch.cuda.Stream()
    per_shape, candidates = [], {}  # candidates: kernel -> {theta key: theta}
    for kernel, dtype, dims in shapes:
        p = ShapeProblem(kernel, dtype, dims, seed, eps, stream)
        # bandwidth-bound shapes are searched on a loaded device (see rt_budget.preheat_ms)
        res, log = B.tuner_search(p.shape, B.make_budget(max_evals=budget, top_k=top_k, use_graph=p.use_graph,
                                                         preheat_ms=0 if p.use_graph else PREHEAT_MS), p.ws)
        ranked = sorted((rec for rec in log if rec.status == B.RT_OK), key=lambda rec: rec.us)
        seen = []
        for rec in ranked:
            if rec.params.key() not in seen:
                seen.append(rec.params.key())
            if len(seen) == finalists:
                break
        for key in [res.best.key()] + seen:
            candidates.setdefault(kernel, {}).setdefault(key, B.rt_params(*key))
        per_shape.append((p.shape, res.best, res.best_us, res.evals_used, p.label))
        if verbose:
            print(f"{p.label}: {res.best} {res.best_us:.2f} us ({res.evals_used} evaluations)", file=sys.stderr)
        del p
        torch.cuda.empty_cache()

    # SelectGeneral, kernel by kernel: every finalist timed on every shape of its kernel (paper protocol), then
    # the geometric-mean choice
    generals, report = {}, {"shapes": [label for *_, label in per_shape], "kernels": {}}
    for kernel, cand_map in candidates.items():
        cand = list(cand_map.values())
        mine = [(k, d, dims) for k, d, dims in shapes if k == kernel]
        times = [[-1.0] * len(mine) for _ in cand]
        for xi, (k, dtype, dims) in enumerate(mine):
            p = ShapeProblem(k, dtype, dims, seed, eps, stream)
            proto = B.make_budget(warmup=20, iters=100, repeats=3, use_graph=p.use_graph,
                                  preheat_ms=0 if p.use_graph else PREHEAT_MS // 4)
            for ci, th in enumerate(cand):
                if B.tuner_check_params(p.shape, th) != B.RT_OK:
                    continue
                rec = B.tuner_evaluate(p.shape, th, proto, p.ws)
                if rec.status == B.RT_OK:
                    times[ci][xi] = rec.us
            del p
            torch.cuda.empty_cache()
        entry = {"specialised_us": [round(min((times[c][x] for c in range(len(cand)) if times[c][x] > 0), default=-1.0), 3)
                                    for x in range(len(mine))]}
        # BuildSpecialized: a shape's entry is its own search's winner, unless another shape's finalist beat it by more
        # than half a percent when every finalist was timed on every shape (less than that is timing noise, and often
        # the very same kernel under another name: an unroll deeper than the vectors a thread owns)
        labels = [f"{k}/{d}:" + "x".join(str(v) for v in dims) for k, d, dims in mine]
        keys = [c.key() for c in cand]
        for i, (shape_i, th_i, us_i, n_i, label_i) in enumerate(per_shape):
            if label_i not in labels:
                continue
            x = labels.index(label_i)
            timed = [(times[c][x], c) for c in range(len(cand)) if times[c][x] > 0]
            if not timed:
                continue
            us_best, c_best = min(timed)
            us_own = times[keys.index(th_i.key())][x]
            if us_own > 0 and us_best >= 0.995 * us_own:
                per_shape[i] = (shape_i, th_i, us_own, n_i, label_i)
            else:
                per_shape[i] = (shape_i, cand[c_best], us_best, n_i, label_i)
        try:
            gi, score, _ = B.tuner_select_general(times)
            generals[OPS[kernel]] = cand[gi]
            entry.update({"general": cand[gi].as_dict(), "general_geomean_vs_specialised": round(score, 4),
                          "general_us": [round(v, 3) for v in times[gi]]})
        except B.TunerError as err:
            entry.update({"general": None, "general_error": str(err)})
        report["kernels"][kernel] = entry
    norm = report["kernels"].get("norm", {})
    report.update({k: norm.get(k) for k in ("general", "general_geomean_vs_specialised", "general_us", "specialised_us")})
    report["specialised"] = [th.as_dict() for _, th, _, _, _ in per_shape]
    report["evaluations"] = [n for _, _, _, n, _ in per_shape]
    table = B.SpecTable([(s, th, us) for s, th, us, _, _ in per_shape], None, torch.cuda.get_device_name(), generals)
    return table, report


def merge_tables(old: "B.SpecTable", new: "B.SpecTable", keep_general: bool = False) -> "B.SpecTable":
    """The entries of `old` with those of `new` laid over them (same kernel, dtype, shape, head size and part count:
    the new entry wins), old entries first in their order; general configurations of `new` win unless keep_general."""
    key = lambda s: (int(s.op), int(s.dtype), int(s.n_tokens), int(s.hidden), int(s.head_dim), int(s.n_parts))
    fresh = {key(s): (s, th, us) for s, th, us in new.entries}
    entries = [fresh.pop(key(s), (s, th, us)) for s, th, us in old.entries] + list(fresh.values())
    generals = dict(old.generals)
    for op, th in new.generals.items():
        if not (keep_general and op in generals):
            generals[op] = th
    return B.SpecTable(entries, None, new.device_name or old.device_name, generals)


def main() -> None:
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--shapes", required=True, help="comma-separated [kernel/]dtype:dims, e.g. bf16:128x4096,"
                    "silu/bf16:4096x14336,merge/bf16:512x32x128,fp8/bf16:4096x8192")
    ap.add_argument("--budget", type=int, default=64, help="kernel evaluations per shape")
    ap.add_argument("--out", default="", help="write the table as JSON here")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--merge", default="", help="an existing table (JSON): its entries are kept, except where this run "
                    "tuned the same kernel and shape again; its general configurations are kept for the kernels this run "
                    "did not tune")
    ap.add_argument("--keep-general", action="store_true", help="with --merge: keep the existing general configurations "
                    "of the kernels tuned in this run as well (for a run over shapes only some stages can serve)")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("tuning needs a CUDA device")
    table, report = tune(parse_shapes(args.shapes), budget=args.budget, seed=args.seed, verbose=True)
    if args.merge:
        with open(args.merge) as f:
            table = merge_tables(B.SpecTable.from_json(json.load(f)), table, args.keep_general)
    if args.out:
        with open(args.out, "w") as f:
            json.dump(table.to_json(), f, indent=1)
    print(json.dumps(report))


if __name__ == "__main__":
    main()
