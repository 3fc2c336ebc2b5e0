#!/usr/bin/env python
"""Benchmark of the fused residual-add + RMSNorm hot path: HBM GB/s of the search-chosen configuration.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME]

One "step" is one pass of the whole operator (one launch of the tuner's chosen theta) over one batch of
seeded synthetic input.  The workload is the prefill configuration (bf16, 16384 x 8192): the case the
bandwidth metric is quoted on.  Before the timed region the tuner runs once (not timed): the guided search,
and the exhaustive sweep it is compared with.  Rank 0 prints one JSON line.

N > 1 (torchrun): every rank owns its own block of rows of an N-times larger job (weak scaling); there is
no data-path collective, only a barrier and the max over ranks of the measured time.

--impl reference times the CPU oracle (the deliberately plain checker) on the host cores, on a bounded
sample of the same workload.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "fused_add_rmsnorm_hbm_gbs"
METRICS = {"add_rmsnorm": METRIC, "silu_and_mul": "silu_and_mul_hbm_gbs", "merge_attn_states": "merge_attn_states_hbm_gbs",
           "add_rmsnorm_fp8": "fused_add_rmsnorm_fp8out_hbm_gbs",
           "add_rmsnorm_allreduce": "fused_allreduce_add_rmsnorm_hbm_gbs"}
BYTES_LABEL = {"add_rmsnorm": "algorithmic: 2 reads + 2 writes per element + w once",
               "silu_and_mul": "algorithmic: 2 reads + 1 write per output element",
               "merge_attn_states": "algorithmic: 2 reads + 1 write per element + 3 binary32 per (token, head)",
               "add_rmsnorm_fp8": "algorithmic: 2 reads + 1 write per element + 1 byte of q per element + w once + a scale per token",
               "add_rmsnorm_allreduce": "algorithmic: n_parts + 1 reads + 2 writes per element + w once (all parts and the one "
                                        "destination in this GPU's memory)"}
KERNEL_NAME = {"add_rmsnorm": "add_rmsnorm_kernel", "silu_and_mul": "silu_and_mul_kernel",
               "merge_attn_states": "merge_attn_states_kernel", "add_rmsnorm_fp8": "add_rmsnorm_fp8_kernel",
               "add_rmsnorm_allreduce": "add_rmsnorm_allreduce_kernel"}
UNIT = "GB/s"
DEFAULT_WORKLOAD = "c3_prefill_bf16_16384x8192"
FALLBACK_HBM_GBS = 6650.0  # used only when MEASURED_PEAKS.json is absent
NOMINAL_HBM_GBS = 8000.0

# DRAM traffic of one launch of the top kernel from an ncu capture (dram__bytes_read.sum +
# dram__bytes_write.sum), valid only for the kernel source and theta it was taken on.
NCU_TRAFFIC = {
    "kernel_sha256_16": "ca1f28704284bed6",
    # workload -> (threads_per_row, rows_per_cta, vec_bytes, unroll, stage, reduce, cluster_size) -> DRAM bytes per launch
    "bytes_per_launch": {
        "c3_prefill_bf16_16384x8192": {
            (256, 1, 32, 2, 0, 0, 1): 1020995584,  # 536.94 MB read + 484.06 MB written (--set full capture)
            (256, 1, 16, 1, 2, 0, 1): 1020571136,  # 536.91 MB read + 483.67 MB written (--set full capture)
            # the other configurations the search has returned on this shape (dram__bytes metrics only, first of two launches)
            (256, 2, 32, 2, 0, 0, 1): 1020452352,
            (256, 1, 32, 2, 0, 1, 1): 1019887104,
            (512, 1, 32, 1, 0, 0, 1): 1026409216,
            (256, 1, 32, 1, 2, 0, 1): 1022494720,
            (256, 2, 32, 2, 2, 0, 1): 1022360832,
            (256, 1, 16, 4, 0, 0, 1): 1019570944,
            (512, 1, 16, 2, 0, 0, 1): 1019498752,
            (256, 1, 16, 2, 2, 0, 1): 1019478272,
        },
        # the ragged-row stage; 201.42 MB read + 153.50 MB written (a quarter of the output is still dirty in L2 at the end)
        "c4x_fp16_8192x6145": {(256, 1, 16, 4, 3, 0, 1): 354928640},
    },
}


def kernel_source_hash() -> str:
    path = os.path.join(ROOT, "paper_2601_12698_b200", "csrc", "add_rmsnorm_kernel.cuh")
    return hashlib.sha256(open(path, "rb").read()).hexdigest()[:16]


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting"}

    def __init__(self, torch_device, period_s: float = 0.002):
        self.period = period_s
        self.samples: list[int] = []
        self.reason_bits = 0
        self.max_mhz = None
        self.handle = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            import torch
            self.nv = pynvml
            pynvml.nvmlInit()
            props = torch.cuda.get_device_properties(torch_device)
            try:
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(props.uuid)).encode())
            except Exception:
                self.handle = pynvml.nvmlDeviceGetHandleByIndex(torch_device.index or 0)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.handle = None

    def _loop(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM)))
                try:
                    bits = nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle)
                except Exception:
                    bits = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle)
                self.reason_bits |= int(bits)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.handle is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self) -> dict:
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz, "samples": len(s),
                "reasons": sorted(name for bit, name in self.REASONS.items() if self.reason_bits & bit)}


def measured_hbm_peak() -> tuple[float, str]:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(path))["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def theta_dict(th) -> dict:
    return th.as_dict()


# ---- the reference arm: the CPU oracle on the host cores --------------------------------------------------

def run_reference(args) -> None:
    from paper_2601_12698_b200 import dp, synth
    rank, world, _ = dp.env_world()
    if rank != 0:
        return  # rank 0 alone runs the oracle
    import oracle
    wl = synth.workloads()[args.workload]
    cores = os.cpu_count() or 1
    is_silu = wl.op == "silu_and_mul"

    is_merge = wl.op == "merge_attn_states"

    def sample(n_rows):
        if is_merge:
            va, sa, vb, sb = synth.make_merge_inputs(0, n_rows, wl.hidden // wl.head_dim, wl.head_dim, wl.dtype, wl.seed)
            return lambda: oracle.merge_attn_states(va, sa, vb, sb)
        if wl.op == "add_rmsnorm_fp8":
            w = synth.make_weight(wl.hidden, wl.dtype, wl.seed, wl.dist)
            xs = synth.make_rows(synth.TENSOR_X, 0, n_rows, wl.hidden, wl.dtype, wl.seed, wl.dist).contiguous()
            rs = synth.make_rows(synth.TENSOR_R, 0, n_rows, wl.hidden, wl.dtype, wl.seed, wl.dist).contiguous()
            return lambda: oracle.add_rmsnorm_fp8(xs, rs, w, wl.eps)
        if is_silu:
            xs = synth.make_gate_up(0, n_rows, wl.hidden, wl.dtype, wl.seed, wl.dist)
            return lambda: oracle.silu_and_mul(xs, threads=cores)
        if wl.op == "add_rmsnorm_allreduce":
            w = synth.make_weight(wl.hidden, wl.dtype, wl.seed, wl.dist)
            ps = synth.make_parts(0, n_rows, wl.hidden, wl.dtype, wl.seed, wl.n_parts, wl.dist)
            rs = synth.make_rows(synth.TENSOR_R, 0, n_rows, wl.hidden, wl.dtype, wl.seed, wl.dist).contiguous()
            return lambda: oracle.allreduce_add_rmsnorm(ps, rs, w, wl.eps, threads=cores)
        w = synth.make_weight(wl.hidden, wl.dtype, wl.seed, wl.dist)
        xs = synth.make_rows(synth.TENSOR_X, 0, n_rows, wl.hidden, wl.dtype, wl.seed, wl.dist).contiguous()
        rs = synth.make_rows(synth.TENSOR_R, 0, n_rows, wl.hidden, wl.dtype, wl.seed, wl.dist).contiguous()
        return lambda: oracle.add_rmsnorm(xs, rs, w, wl.eps, threads=cores)

    probe_rows = min(wl.n_tokens, 256)
    run = sample(probe_rows)
    t0 = time.perf_counter()
    run()
    per_row = (time.perf_counter() - t0) / probe_rows
    budget_s = 120.0
    rows = int(max(8, min(wl.n_tokens, budget_s / max(1, args.steps + args.warmup) / max(per_row, 1e-9))))
    run = sample(rows)
    for _ in range(args.warmup):
        run()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        run()
    elapsed = time.perf_counter() - t0
    b = synth.DTYPE_BYTES[wl.dtype]
    if wl.op == "add_rmsnorm_fp8":
        cores = 1  # this oracle is single-threaded
        step_bytes = (3 * b + 1) * rows * wl.hidden + b * wl.hidden + 4 * rows
    elif is_merge:
        cores = 1  # this oracle is single-threaded
        step_bytes = 3 * b * rows * wl.hidden + 12 * rows * (wl.hidden // wl.head_dim)
    elif wl.op == "add_rmsnorm_allreduce":
        step_bytes = (wl.n_parts + 3) * b * rows * wl.hidden + b * wl.hidden
    else:
        step_bytes = 3 * b * rows * wl.hidden if is_silu else 4 * b * rows * wl.hidden + b * wl.hidden
    value = step_bytes * args.steps / elapsed / 1e9
    sample = f"first {rows} of {wl.n_tokens} rows of {wl.name} per step, {cores} threads"
    line = {
        "impl": "reference", "metric": METRICS[wl.op], "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": elapsed * 1e3 / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
        "config": {"workload": wl.name, "n_tokens": wl.n_tokens, "hidden": wl.hidden, "sample_rows_per_step": rows,
                   "bytes": BYTES_LABEL[wl.op]},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---- our arm ----------------------------------------------------------------------------------------------------

def run_ours(args) -> None:
    import torch
    from paper_2601_12698_b200 import binding as B  # raises when the CUDA library is missing: no fall-back
    from paper_2601_12698_b200 import dp, synth

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU path)")
    rank, world, local_rank = dp.env_world()
    device = torch.device("cuda", local_rank)
    torch.cuda.set_device(device)
    dp.init(device=device)
    wl = synth.workloads()[args.workload]
    shard = dp.weak_shard(wl.n_tokens, rank, world)
    b = synth.DTYPE_BYTES[wl.dtype]
    T, H = wl.n_tokens, wl.hidden

    is_silu = wl.op == "silu_and_mul"
    is_merge = wl.op == "merge_attn_states"
    is_fp8 = wl.op == "add_rmsnorm_fp8"
    is_allreduce = wl.op == "add_rmsnorm_allreduce"  # all parts and the one destination on this GPU (one-shot form)
    op_code = {"add_rmsnorm": B.RT_OP_ADD_RMSNORM, "silu_and_mul": B.RT_OP_SILU_AND_MUL,
               "merge_attn_states": B.RT_OP_MERGE_ATTN_STATES, "add_rmsnorm_fp8": B.RT_OP_ADD_RMSNORM_FP8,
               "add_rmsnorm_allreduce": B.RT_OP_ADD_RMSNORM_ALLREDUCE}[wl.op]
    scale_ref = None
    heads = H // wl.head_dim if is_merge else 0
    sa = sb = None

    # Inputs: this rank's rows of the N-times larger job; w replicated.
    if is_merge:
        va, sa, vb, sb = synth.make_merge_inputs(shard.row_begin, shard.row_end, heads, wl.head_dim, wl.dtype, wl.seed)
        x, r, w = va.view(T, H), vb.view(T, H), None
    elif is_silu:
        x = synth.make_gate_up(shard.row_begin, shard.row_end, H, wl.dtype, wl.seed, wl.dist)
        r = w = None
    elif is_allreduce:
        x = synth.make_parts(shard.row_begin, shard.row_end, H, wl.dtype, wl.seed, wl.n_parts, wl.dist)  # [N, T, H]
        r = synth.make_rows(synth.TENSOR_R, shard.row_begin, shard.row_end, H, wl.dtype, wl.seed, wl.dist).contiguous()
        w = synth.make_weight(H, wl.dtype, wl.seed, wl.dist)
    else:
        x = synth.make_rows(synth.TENSOR_X, shard.row_begin, shard.row_end, H, wl.dtype, wl.seed, wl.dist).contiguous()
        r = synth.make_rows(synth.TENSOR_R, shard.row_begin, shard.row_end, H, wl.dtype, wl.seed, wl.dist).contiguous()
        w = synth.make_weight(H, wl.dtype, wl.seed, wl.dist)

    # The oracle's outputs for the correctness gate; on rank 0 of a 1-GPU run this call is also the timed
    # CPU baseline (the oracle as it stands, all host cores).
    import oracle
    cores = os.cpu_count() or 1
    oracle.build()
    t0 = time.perf_counter()
    if is_fp8:
        cores = 1  # this oracle is single-threaded
        y_ref, scale_ref, r_ref = oracle.add_rmsnorm_fp8(x, r, w, wl.eps)  # y_ref holds the e4m3 codes
    elif is_merge:
        cores = 1  # this oracle is single-threaded
        v_ref, r_ref = oracle.merge_attn_states(va, sa, vb, sb)  # r_ref holds the merged log-sum-exps
        y_ref = v_ref.view(T, H)
    elif is_silu:
        y_ref, r_ref = oracle.silu_and_mul(x, threads=cores), None
    elif is_allreduce:
        y_ref, r_ref = oracle.allreduce_add_rmsnorm(x, r, w, wl.eps, threads=cores)
    else:
        y_ref, r_ref = oracle.add_rmsnorm(x, r, w, wl.eps, threads=cores)
    oracle_s = time.perf_counter() - t0
    cpu_baseline = None
    if world == 1:
        cpu_baseline = {"value": wl.algorithmic_bytes / oracle_s / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
                        "sample": f"one pass over all {T} rows of {wl.name}, {cores} threads, {oracle_s:.2f} s"}

    stream = torch.cuda.Stream(device=device)
    limits = B.rt_query_limits()
    # A workload that fits in L2 is timed over a ring of identical input/output sets larger than L2, so that
    # every timed launch reads from DRAM; the large workloads exceed L2 on their own.
    resident = wl.algorithmic_bytes <= 2 * limits.l2_bytes
    sets = 1 if not resident else int(min(4096, -(-3 * limits.l2_bytes // wl.algorithmic_bytes)))
    ring = lambda t: t.to(device).unsqueeze(0).repeat(sets, *([1] * t.dim())).contiguous()
    xd = ring(x)
    rd = ring(r) if r is not None else None
    wd = w.to(device) if w is not None else None
    yd = torch.empty((sets, T, H), dtype=torch.uint8 if is_fp8 else xd.dtype, device=device)
    scaled = torch.empty((sets, T), dtype=torch.float32, device=device) if is_fp8 else None
    scale_ref_d = scale_ref.to(device) if is_fp8 else None
    od = torch.empty((sets, T, H), dtype=xd.dtype, device=device) if not (is_silu or is_merge) else None
    sad = sbd = None
    if is_merge:
        sad, sbd = ring(sa), ring(sb)
        od = torch.empty_like(sad)  # s_out
    y_ref_d = y_ref.to(device)
    r_ref_d = r_ref.to(device) if r_ref is not None else None
    set_bytes = T * H * b  # one output-sized set; silu_and_mul's input sets are twice as long
    live = [t for t in (xd, rd, wd, od if is_fp8 else yd, od) if t is not None]
    align = B._ptr_align(*live)
    shape = B.shape_of(T, H, wl.dtype, align if set_bytes % 256 == 0 else min(align, set_bytes & -set_bytes), op=op_code,
                       head_dim=wl.head_dim, n_parts=wl.n_parts)
    # warm: the paper's protocol (the same buffers every launch); cold: rotating over the ring
    w_or_sa = sad if is_merge else wd
    ws = B.make_workspace(xd, rd, w_or_sa, yd, od, y_ref_d, r_ref_d, wl.eps, n_ref_tokens=T, stream=stream, aux=sbd,
                          aux_out=scaled, aux_ref=scale_ref_d)
    ws_cold = B.make_workspace(xd, rd, w_or_sa, yd, od, y_ref_d, r_ref_d, wl.eps, n_ref_tokens=T, ring_sets=sets,
                               ring_stride_bytes=set_bytes, stream=stream, aux=sbd, aux_out=scaled, aux_ref=scale_ref_d)
    use_graph = resident  # launch gaps would otherwise dominate kernels of a few microseconds

    # The tuner (not timed): exhaustive sweep as ground truth, then the guided search with a stated budget.
    tuner = {}
    if args.theta:
        # a fixed theta (profiling runs): the tuner is skipped
        key = [int(v) for v in args.theta.split(",")]
        if len(key) != 7:
            raise SystemExit("--theta takes tpr,rpc,vec,unroll,stage,reduce,cluster")
        tuner = {"skipped": "theta given on the command line"}
    elif rank == 0:
        counts = B.tuner_derive_counts(shape)
        t0 = time.perf_counter()
        sweep, sweep_log = B.tuner_search(shape, B.make_budget(max_evals=counts["feasible"] + args.top_k, warmup=10,
                                                               iters=50, repeats=2, top_k=args.top_k,
                                                               strategy=B.RT_SEARCH_EXHAUSTIVE, use_graph=use_graph), ws)
        sweep_s = time.perf_counter() - t0
        t0 = time.perf_counter()
        guided, guided_log = B.tuner_search(shape, B.make_budget(max_evals=args.search_budget, warmup=20, iters=100,
                                                                 repeats=3, top_k=args.top_k, use_graph=use_graph), ws)
        guided_s = time.perf_counter() - t0
        # head-to-head re-timing of the two winners with the paper's protocol (20 warm-up, 100 timed)
        proto = B.make_budget(warmup=20, iters=100, repeats=5, use_graph=use_graph)
        t_guided = B.tuner_evaluate(shape, guided.best, proto, ws)
        t_sweep = B.tuner_evaluate(shape, sweep.best, proto, ws)
        t_cold = B.tuner_evaluate(shape, guided.best, proto, ws_cold)
        floor_us = B.tuner_launch_floor(proto, stream=stream)
        theta = guided.best
        tuner = {
            "feasible": counts["feasible"], "raw_grid": counts["raw"], "pruned": {k: v for k, v in counts.items()
                                                                                 if k not in ("feasible", "raw") and v},
            "search_budget_evals": args.search_budget, "search_evals_used": guided.evals_used,
            "search_best": theta_dict(guided.best), "search_best_us": round(t_guided.us, 3),
            "exhaustive_best": theta_dict(sweep.best), "exhaustive_best_us": round(t_sweep.us, 3),
            "exhaustive_evals": sweep.evals_used, "failed_gate": guided.n_failed_gate + sweep.n_failed_gate,
            "search_vs_exhaustive": round(t_guided.us / t_sweep.us, 4),
            "timing": ("CUDA graph of 100 launches, same buffers (L2-warm)" if use_graph else
                       "100 back-to-back launches, same buffers (exceed L2)"),
            "search_best_cold_us": round(t_cold.us, 3), "ring_sets": sets, "empty_kernel_us": round(floor_us, 3),
            "search_seconds": round(guided_s, 2), "exhaustive_seconds": round(sweep_s, 2),
            "occupancy_blocks_per_sm": t_guided.occupancy_blocks_per_sm, "regs_per_thread": t_guided.regs_per_thread,
        }
        if args.seed_thetas:
            # Cross-shape transfer: the same small budget, cold and seeded with configurations found on other
            # shapes; "evaluations to within 3%" counts evaluations until one scores within 3% of the
            # exhaustive-sweep optimum.
            seeds = [B.rt_params(*[int(v) for v in item.split(",")]) for item in args.seed_thetas.split(";") if item]
            threshold = 1.03 * t_sweep.us

            def first_within(log):
                for rec in log:
                    if rec.status == 0 and rec.us <= threshold:
                        return rec.eval_index + 1
                return None
            tb = args.transfer_budget
            cold, cold_log = B.tuner_search(shape, B.make_budget(max_evals=tb, warmup=20, iters=100, repeats=3,
                                                                 top_k=2, use_graph=use_graph), ws)
            warm, warm_log = B.tuner_search(shape, B.make_budget(max_evals=tb, warmup=20, iters=100, repeats=3,
                                                                 top_k=2, use_graph=use_graph, seeds=seeds), ws)
            tuner["transfer"] = {
                "budget_evals": tb, "n_seeds": len(seeds), "threshold_us": round(threshold, 3),
                "cold_best_us": round(cold.best_us, 3), "cold_evals_to_within_3pct": first_within(cold_log),
                "seeded_best_us": round(warm.best_us, 3), "seeded_evals_to_within_3pct": first_within(warm_log),
                "seeded_best": theta_dict(warm.best), "cold_best": theta_dict(cold.best),
            }
        if args.log:
            os.makedirs(os.path.dirname(os.path.abspath(args.log)) or ".", exist_ok=True)
            with open(args.log, "w") as f:
                for name, log in (("exhaustive", sweep_log), ("guided", guided_log)):
                    for rec in log:
                        f.write(json.dumps({"search": name, "workload": wl.name, **rec.as_dict()}) + "\n")
        key = list(theta.key())
    else:
        key = [0] * 7
    key = dp.broadcast_ints(key, device)
    theta = B.rt_params(*key)

    # The timed region: W warm-up steps, then exactly K steps between two events on the launch stream.
    # Step k works on set k mod sets (one set when the workload exceeds L2 by itself).
    theta_ref = B.byref(theta)
    dtype_code, stream_ptr, eps = B.DTYPE_CODES[wl.dtype], stream.cuda_stream, wl.eps
    if is_fp8:
        launch = B.lib.rmsnorm_fp8_template_launch
        ptrs = [(xd[k].data_ptr(), rd[k].data_ptr(), yd[k].data_ptr(), scaled[k].data_ptr(), od[k].data_ptr())
                for k in range(sets)]
        w_ptr = wd.data_ptr()

        def step(k):
            px, pr, pq, ps, po = ptrs[k % sets]
            st = launch(theta_ref, px, pr, w_ptr, pq, ps, po, T, H, eps, dtype_code, stream_ptr)
            if st != 0:
                raise B.TunerError(st, "rmsnorm_fp8_template_launch")
    elif is_merge:
        launch = B.lib.merge_attn_states_template_launch
        ptrs = [(xd[k].data_ptr(), sad[k].data_ptr(), rd[k].data_ptr(), sbd[k].data_ptr(), yd[k].data_ptr(),
                 od[k].data_ptr()) for k in range(sets)]
        head_dim = wl.head_dim

        def step(k):
            pa, psa, pb, psb, po, pso = ptrs[k % sets]
            st = launch(theta_ref, pa, psa, pb, psb, po, pso, T, heads, head_dim, dtype_code, stream_ptr)
            if st != 0:
                raise B.TunerError(st, "merge_attn_states_template_launch")
    elif is_allreduce:
        launch = B.lib.rmsnorm_allreduce_template_launch
        vp, n_parts = B.c_void_p, wl.n_parts
        ptrs = [((vp * n_parts)(*[xd[k, j].data_ptr() for j in range(n_parts)]), rd[k].data_ptr(),
                 (vp * 1)(yd[k].data_ptr()), (vp * 1)(od[k].data_ptr())) for k in range(sets)]
        w_ptr = wd.data_ptr()

        def step(k):
            px, pr, py, po = ptrs[k % sets]
            st = launch(theta_ref, px, n_parts, pr, w_ptr, py, 1, po, 1, 0, T, H, eps, dtype_code, stream_ptr)
            if st != 0:
                raise B.TunerError(st, "rmsnorm_allreduce_template_launch")
    elif is_silu:
        launch = B.lib.silu_and_mul_template_launch
        ptrs = [(xd[k].data_ptr(), yd[k].data_ptr()) for k in range(sets)]

        def step(k):
            px, py = ptrs[k % sets]
            st = launch(theta_ref, px, py, T, H, dtype_code, stream_ptr)
            if st != 0:
                raise B.TunerError(st, "silu_and_mul_template_launch")
    else:
        launch = B.lib.rmsnorm_template_launch
        ptrs = [(xd[k].data_ptr(), rd[k].data_ptr(), yd[k].data_ptr(), od[k].data_ptr()) for k in range(sets)]
        w_ptr = wd.data_ptr()

        def step(k):
            px, pr, py, po = ptrs[k % sets]
            st = launch(theta_ref, px, pr, w_ptr, py, po, T, H, eps, dtype_code, stream_ptr)
            if st != 0:
                raise B.TunerError(st, "rmsnorm_template_launch")

    for k in range(args.warmup):
        step(k)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    dp.barrier(device)
    launches_before = B.rt_launch_count()
    with ClockSampler(device) as clocks:
        with torch.cuda.stream(stream):
            e0.record(stream)
            for k in range(args.steps):
                step(k)
            e1.record(stream)
        e1.synchronize()
        dp.barrier(device)
    gpu_launches = B.rt_launch_count() - launches_before
    ms_local = e0.elapsed_time(e1)
    ms = dp.max_over_ranks(ms_local, device)
    value = dp.whole_job_rate(wl.algorithmic_bytes, args.steps, world, ms) / 1e9

    # Parity of what was just timed, against the oracle (all rows; r' bit-exact, y within tolerance).
    last = (args.steps - 1) % sets  # the set the last timed step wrote
    if is_fp8:
        r_bad = B.tuner_compare(od[last], r_ref_d, B.RT_CMP_BITS, stream=stream)[1]
        y_worst, y_bad = B.tuner_compare_e4m3(yd[last], y_ref_d, 1, stream=stream)
        y_bad += B.tuner_compare(scaled[last], scale_ref_d, B.RT_CMP_REL32, 1e-5, stream=stream)[1]
    elif is_merge:
        r_bad = B.tuner_compare_mixed(od[last], r_ref_d, 1e-5, 1e-5, stream=stream)[1]
        y_worst, y_bad = B.tuner_compare_mixed(yd[last], y_ref_d, 1e-5 if wl.dtype == "fp32" else 2.0, 1e-5, stream=stream)
    else:
        r_bad = 0 if is_silu else B.tuner_compare(od[last], r_ref_d, B.RT_CMP_BITS, stream=stream)[1]
    if is_merge or is_fp8:
        pass
    elif wl.dtype == "fp32":
        y_worst, y_bad = B.tuner_compare(yd[last], y_ref_d, B.RT_CMP_REL32, 1e-5, stream=stream)
    else:
        y_worst, y_bad = B.tuner_compare(yd[last], y_ref_d, B.RT_CMP_ULP16, 2.0, stream=stream)
    parity_ok = (r_bad == 0 and y_bad == 0 and B.rt_device_status() == 0)
    if not parity_ok:
        raise RuntimeError(f"timed configuration fails parity: r_bad={r_bad} y_bad={y_bad} worst={y_worst}")

    # End to end: host buffers, copies inside the timed region.  add_rmsnorm goes through the C ABI's host-buffer
    # entry point (chunked, copies overlapped with the kernel); silu_and_mul has no such entry point, so its
    # end-to-end step is copy in, launch, copy out on the launch stream.
    e2e_steps = max(3, min(args.steps, args.e2e_steps))
    if is_fp8:
        xp, rp, wp = x.pin_memory(), r.pin_memory(), w.pin_memory()
        yp, op, sp = torch.empty((T, H), dtype=torch.uint8).pin_memory(), torch.empty_like(xp).pin_memory(), torch.empty(T).pin_memory()
        h2d_bytes, d2h_bytes = 2 * T * H * b + H * b, T * H * b + T * H + 4 * T

        def e2e_step():
            with torch.cuda.stream(stream):
                xd[0].copy_(xp, non_blocking=True); rd[0].copy_(rp, non_blocking=True); wd.copy_(wp, non_blocking=True)
                step(0)
                yp.copy_(yd[0], non_blocking=True); op.copy_(od[0], non_blocking=True); sp.copy_(scaled[0], non_blocking=True)
            stream.synchronize()
    elif is_merge:
        xp, rp, sap, sbp = x.pin_memory(), r.pin_memory(), sa.pin_memory(), sb.pin_memory()
        yp, sop = torch.empty((T, H), dtype=x.dtype).pin_memory(), torch.empty((T, heads)).pin_memory()
        h2d_bytes, d2h_bytes = 2 * T * H * b + 8 * T * heads, T * H * b + 4 * T * heads

        def e2e_step():
            with torch.cuda.stream(stream):
                xd[0].copy_(xp, non_blocking=True); rd[0].copy_(rp, non_blocking=True)
                sad[0].copy_(sap, non_blocking=True); sbd[0].copy_(sbp, non_blocking=True)
                step(0)
                yp.copy_(yd[0], non_blocking=True); sop.copy_(od[0], non_blocking=True)
            stream.synchronize()
    elif is_allreduce:
        xp, rp, wp = x.pin_memory(), r.pin_memory(), w.pin_memory()
        yp, op = torch.empty_like(rp).pin_memory(), torch.empty_like(rp).pin_memory()
        h2d_bytes, d2h_bytes = (wl.n_parts + 1) * T * H * b + H * b, 2 * T * H * b

        def e2e_step():
            with torch.cuda.stream(stream):
                xd[0].copy_(xp, non_blocking=True); rd[0].copy_(rp, non_blocking=True); wd.copy_(wp, non_blocking=True)
                step(0)
                yp.copy_(yd[0], non_blocking=True); op.copy_(od[0], non_blocking=True)
            stream.synchronize()
    elif is_silu:
        xp = x.pin_memory()
        yp = torch.empty((T, H), dtype=x.dtype).pin_memory()
        h2d_bytes, d2h_bytes = 2 * T * H * b, T * H * b

        def e2e_step():
            with torch.cuda.stream(stream):
                xd[0].copy_(xp, non_blocking=True)
                step(0)
                yp.copy_(yd[0], non_blocking=True)
            stream.synchronize()
    else:
        xp, rp, wp = x.pin_memory(), r.pin_memory(), w.pin_memory()
        yp, op = torch.empty_like(xp).pin_memory(), torch.empty_like(xp).pin_memory()
        host_ws = torch.empty(B.rmsnorm_host_workspace_bytes(T, H, wl.dtype, 0), dtype=torch.uint8, device=device)
        h2d_bytes, d2h_bytes = 2 * T * H * b + H * b, 2 * T * H * b

        def e2e_step():
            B.rmsnorm_template_run_host(theta, xp, rp, wp, yp, op, wl.eps, host_ws, stream=stream)
    e2e_step()  # warm-up
    dp.barrier(device)
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    torch.cuda.synchronize(device)
    e2e_ms = dp.max_over_ranks((time.perf_counter() - t0) * 1e3, device)
    dp.barrier(device)
    e2e_value = dp.whole_job_rate(wl.algorithmic_bytes, e2e_steps, world, e2e_ms) / 1e9
    if is_fp8:
        e2e_bad = (oracle.compare_e4m3(yp[-64:], y_ref[-64:], tol_steps=1)[1] or oracle.bit_mismatches(op[:64], r_ref[:64])
                   or oracle.compare_y(sp, scale_ref, tol_rel=1e-5)[1])
    elif is_merge:
        e2e_bad = (oracle.compare_mixed(yp[-64:], y_ref[-64:], tol=1e-5 if wl.dtype == "fp32" else 2.0, tol_abs=1e-5)[1]
                   or oracle.compare_mixed(sop[:64], r_ref[:64], tol=1e-5, tol_abs=1e-5)[1])
    else:
        e2e_bad = (oracle.compare_y(yp[-64:], y_ref[-64:], tol_rel=1e-5)[1]
                   or (not is_silu and oracle.bit_mismatches(op[:64], r_ref[:64])))
    if e2e_bad:
        raise RuntimeError("end-to-end path fails parity")

    if rank == 0:
        peak, peak_kind = measured_hbm_peak()
        per_launch_ms = ms_local / args.steps
        achieved = wl.algorithmic_bytes / (per_launch_ms * 1e-3) / 1e9
        traffic = None
        if NCU_TRAFFIC["kernel_sha256_16"] == kernel_source_hash():
            traffic = NCU_TRAFFIC["bytes_per_launch"].get(wl.name, {}).get(tuple(theta_dict(theta).values()))
        line = {
            "metric": METRICS[wl.op], "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
            "config": {"workload": wl.name, "n_tokens_per_gpu": T, "hidden": H, "eps": wl.eps,
                       "l2": ("inputs_exceed_l2" if not resident else
                              f"ring of {sets} input/output sets ({sets * wl.algorithmic_bytes >> 20} MiB) exceeds L2"),
                       "bytes": BYTES_LABEL[wl.op],
                       "parallelism": f"rows x{world}, no collective", "theta": theta_dict(theta)},
            "value_nominal_5_access_gbs": value * wl.nominal_bytes / wl.algorithmic_bytes,
            "frac_of_8TBs": value / world / NOMINAL_HBM_GBS,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": UNIT, "frac": achieved / peak,
                         "traffic": traffic, "peak_kind": f"of {peak_kind}", "kernel": KERNEL_NAME[wl.op],
                         "algorithmic_bytes_per_launch": wl.algorithmic_bytes},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d_bytes,
                    "d2h_bytes_per_step": d2h_bytes, "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps},
            "gpu_launches": int(gpu_launches),
            "clocks": clocks.summary(),
            "parity": {"r_out_bit_mismatches": int(r_bad), "y_beyond_tolerance": int(y_bad), "y_worst": y_worst,
                       "rows_checked": T},
            "tuner": tuner,
        }
        if cpu_baseline is not None:
            line["cpu_baseline"] = cpu_baseline
        print(json.dumps(line), flush=True)
    dp.shutdown()


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--search-budget", type=int, default=64, help="guided search budget in kernel evaluations")
    ap.add_argument("--top-k", type=int, default=5)
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--theta", default="", help="skip the tuner and time this theta: tpr,rpc,vec,unroll,stage,reduce,cluster")
    ap.add_argument("--seed-thetas", default="", help="';'-separated thetas found on other shapes: also run the "
                    "cold-versus-seeded transfer experiment")
    ap.add_argument("--transfer-budget", type=int, default=24)
    ap.add_argument("--log", default="", help="write every evaluated theta of both searches to this JSONL file")
    args = ap.parse_args()
    if args.steps < 1 or args.warmup < 0:
        raise SystemExit("--steps must be >= 1 and --warmup >= 0")
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
