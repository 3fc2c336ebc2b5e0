#!/usr/bin/env python
"""Benchmark of the fused residual-add + RMSNorm hot path: HBM GB/s of the search-chosen configuration.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME]

One "step" is one pass of the whole operator (one launch of the tuner's chosen theta) over one batch of
seeded synthetic input.  The workload is the prefill configuration (bf16, 16384 x 8192): the case the
bandwidth metric is quoted on.  Before the timed region the tuner runs once (not timed): the guided search,
and the exhaustive sweep it is compared with.  Rank 0 prints one JSON line.

N > 1: one process per GPU.  Under a launcher (RANK / WORLD_SIZE in the environment, e.g. torchrun) this process
is one rank; started plainly with --gpus N > 1 it starts the N ranks itself.  Every rank owns its own block of rows
of an N-times larger job (weak scaling); there is no data-path collective, only a barrier and the max over ranks of
the measured time.  The c3ar* workloads (the tensor-parallel form of the norm) are the exception: with N equal to
their group size they run the all-reduce-fused kernel over the ranks' peer-mapped buffers.

--impl reference times the CPU oracle (the deliberately plain checker) on the host cores, on a bounded
sample of the same workload.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import socket
import subprocess
import sys
import tempfile
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

# DRAM traffic of one launch of the top kernel from ncu captures (dram__bytes_read.sum + dram__bytes_write.sum),
# keyed by workload and theta (tpr, rpc, vec, unroll, stage, reduce, cluster).  Each entry names the hash of the kernel
# header it was captured on: the bench prints the figure as `traffic` only while that hash is the current one, and
# prints the capture with both hashes beside it either way (`traffic_capture`).
NCU_TRAFFIC = {
    # One capture each (dram__bytes_read.sum + dram__bytes_write.sum of the first captured launch).  Reads equal the
    # algorithmic reads; of the writes, the 50-55 MB that are still dirty in L2 when the kernel ends are not counted,
    # so the figures sit a little below the algorithmic bytes (0.95 of them on c3, 0.85 on the smallest c4 shape).
    "c3_prefill_bf16_16384x8192": {
        (512, 1, 32, 1, 0, 0, 1): (1021497088, "b88197c58880f0a9"),  # 536.92 MB read + 484.58 MB written (--set full)
        (256, 1, 32, 2, 0, 0, 1): (1020529664, "b88197c58880f0a9"),
        (256, 2, 32, 2, 0, 0, 1): (1020083968, "b88197c58880f0a9"),
        (256, 1, 16, 4, 0, 0, 1): (1019405568, "b88197c58880f0a9"),
        (512, 1, 16, 2, 0, 0, 1): (1019772672, "b88197c58880f0a9"),
        (256, 1, 16, 1, 2, 0, 1): (1019693056, "b88197c58880f0a9"),
        (256, 1, 32, 1, 2, 0, 1): (1022521600, "b88197c58880f0a9"),
    },
    "c4_fp16_8192x5120": {(256, 1, 32, 2, 0, 0, 1): (283748096, "b88197c58880f0a9")},
    "c4_fp16_8192x7168": {(256, 1, 32, 2, 0, 0, 1): (416248320, "b88197c58880f0a9"),
                          (512, 1, 32, 1, 0, 0, 1): (416799744, "b88197c58880f0a9")},
    "c4_fp16_8192x6152": {(256, 1, 16, 4, 0, 0, 1): (350612992, "b88197c58880f0a9")},
    # the ragged-row stage with 32-byte chunks; 6145: 201.58 MB read + 152.15 MB written (--set full)
    "c4x_fp16_8192x6145": {(256, 1, 32, 2, 3, 0, 1): (353729280, "b88197c58880f0a9")},
    "c4x_fp16_8192x6146": {(256, 1, 32, 2, 3, 0, 1): (352781568, "b88197c58880f0a9")},
    "c4x_fp16_8192x6148": {(256, 1, 32, 2, 3, 0, 1): (352771584, "b88197c58880f0a9")},
}


def kernel_source_hash() -> str:
    path = os.path.join(ROOT, "paper_2601_12698_b200", "csrc", "add_rmsnorm_kernel.cuh")
    return hashlib.sha256(open(path, "rb").read()).hexdigest()[:16]


def ncu_traffic(workload: str, theta_key: tuple):
    """(traffic or None, description of the capture or None) for the roofline object."""
    hit = NCU_TRAFFIC.get(workload, {}).get(tuple(theta_key))
    if hit is None:
        return None, None
    nbytes, captured_on = hit
    current = kernel_source_hash()
    info = {"bytes_per_launch": nbytes, "kernel_sha256_16_at_capture": captured_on, "kernel_sha256_16_now": current,
            "current": captured_on == current}
    return (nbytes if captured_on == current else None), info


_SAMPLER_SOURCE = r"""
import sys, time
import pynvml as nv
nv.nvmlInit()
uuid, index, period = sys.argv[1], int(sys.argv[2]), float(sys.argv[3])
try:
    h = nv.nvmlDeviceGetHandleByUUID(uuid.encode()) if uuid else nv.nvmlDeviceGetHandleByIndex(index)
except Exception:
    h = nv.nvmlDeviceGetHandleByIndex(index)
sys.stdout.write("max %d\n" % nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM))
sys.stdout.flush()
while True:
    t = time.monotonic()
    mhz = nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)
    try:
        bits = nv.nvmlDeviceGetCurrentClocksEventReasons(h)
    except Exception:
        bits = nv.nvmlDeviceGetCurrentClocksThrottleReasons(h)
    sys.stdout.write("%.6f %d %d\n" % (t, mhz, bits))
    sys.stdout.flush()
    time.sleep(period)
"""


class ClockSampler:
    """SM clock and clock-event reasons of one GPU, read through NVML (reading only) by a child process while the
    measurements run.  A child process, not a thread: the timed loop holds the interpreter, and a sampling thread
    would get a turn every few milliseconds at best.  Samples carry CLOCK_MONOTONIC times, so any interval of this
    process's own clock can be looked up afterwards."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting"}

    def __init__(self, torch_device, period_s: float = 0.0005):
        self.proc = None
        self.max_mhz = None
        self.samples: list[tuple[float, int, int]] = []
        self._parsed = 0
        try:
            import torch
            props = torch.cuda.get_device_properties(torch_device)
            uuid = "GPU-" + str(props.uuid) if getattr(props, "uuid", None) is not None else ""
            self.out = tempfile.NamedTemporaryFile("w+", prefix="clocks_", suffix=".txt", delete=True)
            self.proc = subprocess.Popen([sys.executable, "-c", _SAMPLER_SOURCE, uuid, str(torch_device.index or 0),
                                          str(period_s)], stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def wait_ready(self, timeout_s: float = 20.0) -> None:
        """Returns once the child has delivered its first sample (or has died, or the time is up)."""
        t0 = time.monotonic()
        while self.proc is not None and self.proc.poll() is None and time.monotonic() - t0 < timeout_s:
            if len(self._read()) > 0:
                return
            time.sleep(0.01)

    def _read(self):
        if self.proc is None:
            return self.samples
        with open(self.out.name) as f:
            f.seek(self._parsed)
            text = f.read()
        done = text.rfind("\n") + 1  # whole lines only: a line cut off in mid-write comes again complete
        for line in text[:done].splitlines():
            parts = line.split()
            if len(parts) == 2 and parts[0] == "max":
                self.max_mhz = int(parts[1])
            elif len(parts) == 3:
                self.samples.append((float(parts[0]), int(parts[1]), int(parts[2])))
        self._parsed += done
        return self.samples

    def stop(self) -> None:
        if self.proc is not None:
            self._read()
            self.proc.terminate()  # this very child, by its handle
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
            self._read()
            self.proc = None

    def window(self, t_begin: float, t_end: float, widen_to: int = 3) -> dict:
        """Median SM clock and the union of the reasons over [t_begin, t_end] (time.monotonic() values).  A window
        with fewer than `widen_to` samples is widened to its nearest samples on either side, and says so."""
        samples = self._read()
        inside = [s for s in samples if t_begin <= s[0] <= t_end]
        widened = False
        if len(inside) < widen_to and samples:
            mid = 0.5 * (t_begin + t_end)
            inside = sorted(samples, key=lambda s: abs(s[0] - mid))[:widen_to]
            widened = True
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        mhz = sorted(s[1] for s in inside)
        bits = 0
        for s in inside:
            bits |= s[2]
        out = {"sm_mhz": mhz[len(mhz) // 2], "sm_min_mhz": mhz[0], "sm_max_mhz": self.max_mhz, "samples": len(inside),
               "reasons": sorted(name for bit, name in self.REASONS.items() if bits & bit)}
        if widened:
            out["window"] = "widened to the nearest samples around the timed region"
        return out

    def median_mhz(self, t_begin: float, t_end: float):
        w = self.window(t_begin, t_end, widen_to=1)
        return w["sm_mhz"]


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
    wl = workload_of(args.workload)
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
        "config": {"workload": wl.name, "n_tokens_per_gpu": wl.n_tokens, "hidden": wl.hidden, "eps": wl.eps,
                   "sample_rows_per_step": rows, "bytes": BYTES_LABEL[wl.op]},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_of(name: str):
    """A named workload of synth.workloads(), or an ad-hoc shape of the norm written dtype:TOKENSxHIDDEN (N(0, 1) inputs,
    seed 9) - e.g. bf16:5000x6144, for timing shapes the shipped table has no entry for."""
    from paper_2601_12698_b200 import synth
    table = synth.workloads()
    if name in table:
        return table[name]
    try:
        dtype, dims = name.split(":")
        tokens, hidden = (int(v) for v in dims.lower().split("x"))
        if dtype not in synth.DTYPE_BYTES or tokens < 1 or hidden < 1:
            raise ValueError(name)
    except ValueError:
        raise SystemExit(f"unknown workload {name!r}: one of {', '.join(table)} or dtype:TOKENSxHIDDEN")
    return synth.Workload(f"adhoc_{dtype}_{tokens}x{hidden}", dtype, tokens, hidden, seed=9)


def fastest_of(log, k: int) -> list:
    """The k fastest distinct thetas of a search log that passed their gate (a theta's last record counts)."""
    last = {}
    for rec in log:
        last[rec.params.key()] = rec
    good = sorted((rec for rec in last.values() if rec.status == 0), key=lambda rec: rec.us)
    return [rec.params for rec in good[:k]]


def resume_seeds(path: str, workload: str, k: int = 8) -> list:
    """Resume: the fastest thetas of an earlier search log (the JSONL file --log writes) become the seeds of this
    search, so it starts where that one stopped.  Records of other workloads in the file are seeds as well, after
    this workload's own (configurations found on other shapes; the tuner skips those that are infeasible here)."""
    from paper_2601_12698_b200 import binding as B
    own, other = {}, {}
    with open(path) as f:
        for line in f:
            line = line.strip()
            if not line:
                continue
            rec = json.loads(line)
            if rec.get("status") != 0 or not rec.get("us"):
                continue
            th = rec["params"]
            key = tuple(int(th[name]) for name, _ in B.rt_params._fields_)
            table = own if rec.get("workload") == workload else other
            table[key] = min(float(rec["us"]), table.get(key, float("inf")))
    ranked = sorted(own, key=own.get)[:k] + sorted(other, key=other.get)[:k]
    return [B.rt_params(*key) for key in ranked]


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
    wl = workload_of(args.workload)
    if wl.op == "add_rmsnorm_allreduce" and world > 1:
        return run_tensor_parallel(args, wl, rank, world, device)
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
        if wl.op == "add_rmsnorm":
            # the same oracle on one thread, on the first rows of the workload (about two seconds of work)
            rows1 = int(max(1, min(T, T * 2.0 / max(oracle_s * cores, 1e-6))))
            t0 = time.perf_counter()
            oracle.add_rmsnorm(x[:rows1], r[:rows1], w, wl.eps, threads=1)
            one_s = time.perf_counter() - t0
            cpu_baseline["single_thread"] = {
                "value": (4 * b * rows1 * H + b * H) / one_s / 1e9, "unit": UNIT, "cores": 1,
                "sample": f"first {rows1} of {T} rows, 1 thread, {one_s:.2f} s"}

    stream = torch.cuda.Stream(device=device)
    clock_sampler = ClockSampler(device)  # a child process that only reads NVML; stopped before the line is printed
    clock_sampler.wait_ready()
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
    # Three regimes.  Small (up to half of L2): the tuner times a CUDA graph of 100 launches on the same buffers, L2-warm
    # as in the paper's protocol - launch gaps would otherwise dominate kernels of a few microseconds.  Middle (up to
    # twice L2): the same buffers would be partly L2-resident from one launch to the next, which measures the cache
    # state more than the kernel (block-to-block spread of 10%), so the tuner rotates over the ring of buffer sets like
    # the timed region does.  Large: the same buffers, which exceed L2 on their own.
    small = wl.algorithmic_bytes <= limits.l2_bytes // 2
    use_graph = small
    ws_tune = ws if (small or not resident) else ws_cold

    # The tuner (not timed): exhaustive sweep as ground truth, then the guided search with a stated budget.
    tuner = {}
    if args.theta:
        # a fixed theta (profiling runs): the tuner is skipped
        key = [int(v) for v in args.theta.split(",")]
        if len(key) != 7:
            raise SystemExit("--theta takes tpr,rpc,vec,unroll,stage,reduce,cluster")
        tuner = {"skipped": "theta given on the command line"}
    elif rank == 0:
        # --include-pipeline puts the persistent TMA pipeline stage, which the default candidate set leaves out, into
        # both searches (and so into the per-stage table below)
        mask = B.RT_PRUNE_DEFAULT & ~B.RT_PRUNE_PIPELINE_STAGE if args.include_pipeline else B.RT_PRUNE_DEFAULT
        counts = B.tuner_derive_counts(shape, heuristics=mask)
        # --sweep-heuristics widens (or narrows) the exhaustive sweep alone: with 0 it covers every hard-feasible theta,
        # and the re-test below then shows what the heuristic rules cost on this shape, if anything
        sweep_mask = mask if args.sweep_heuristics < 0 else args.sweep_heuristics
        sweep_evals = B.tuner_derive_counts(shape, heuristics=sweep_mask)["feasible"]
        # bandwidth-bound workloads are compared on a loaded device: the tuner keeps the GPU busy this long before its
        # first timing and before every side-by-side re-test (the latency-bound ones never reach the power limit)
        heat = 0 if small else args.preheat_ms
        # Both searches time every candidate with the paper's protocol (20 warm-up launches, blocks of 100).
        t0 = time.perf_counter()
        sweep, sweep_log = B.tuner_search(shape, B.make_budget(max_evals=sweep_evals, warmup=20, iters=100, repeats=2,
                                                               top_k=0, strategy=B.RT_SEARCH_EXHAUSTIVE,
                                                               use_graph=use_graph, heuristics=sweep_mask, preheat_ms=heat), ws_tune)
        sweep_s = time.perf_counter() - t0
        seeds = resume_seeds(args.resume, wl.name) if args.resume else None
        t0 = time.perf_counter()
        guided, guided_log = B.tuner_search(shape, B.make_budget(max_evals=args.search_budget, warmup=20, iters=100,
                                                                 repeats=3, top_k=args.top_k, use_graph=use_graph,
                                                                 seeds=seeds, heuristics=mask, preheat_ms=heat), ws_tune)
        guided_s = time.perf_counter() - t0
        # Search-best against exhaustive-best, measured side by side: the sweep's fastest --retest-top points, the
        # guided winner and its two runners-up are re-timed together, block by block in rotation (20 warm-up + 100 timed
        # launches per block), so that every candidate meets the same clocks.  exhaustive_best is the fastest of
        # that set (the guided winner belongs to the feasible set the sweep covers, so it is a member by right).
        finalists = []
        for th in (fastest_of(sweep_log, args.retest_top) + [guided.best] + fastest_of(guided_log, 2)):
            if th.key() not in [f.key() for f in finalists]:
                finalists.append(th)
        # what the shipped table would launch on this shape without any search (its entry for the shape, else the
        # nearest entry's theta, else the general configuration), and the general configuration itself: timed in the
        # same re-test, so that the cost of a table miss and of the one-size-fits-all choice is on record
        shipped = B.SpecTable.default()
        table_theta, table_source = shipped.lookup(shape)
        general_theta = shipped.generals.get(op_code)
        extras = {"table": table_theta}
        if general_theta is not None and B.tuner_check_params(shape, general_theta) == B.RT_OK:
            extras["general"] = general_theta
        for th in extras.values():
            if th.key() not in [f.key() for f in finalists]:
                finalists.append(th)
        proto = B.make_budget(warmup=20, iters=100, repeats=1, use_graph=use_graph, preheat_ms=heat)
        recs, blocks = B.tuner_retest_interleaved(shape, finalists, proto, ws_tune, args.retest_rounds)
        i_guided = [f.key() for f in finalists].index(guided.best.key())
        ok = [i for i, rec in enumerate(recs) if rec.status == 0]
        if i_guided not in ok:
            raise RuntimeError(f"the guided winner failed its re-test: status {recs[i_guided].status}")
        i_best = min(ok, key=lambda i: recs[i].us)
        per = {i: [blk for blk in blocks if blk.theta_index == i] for i in ok}
        mhz = {i: [clock_sampler.median_mhz(blk.t_begin_s, blk.t_end_s) for blk in per[i]] for i in ok}

        def normalised(i):  # median over blocks of (time x SM clock): cycles per launch, in us x MHz
            vals = sorted(blk.us * m for blk, m in zip(per[i], mhz[i]) if m)
            return vals[len(vals) // 2] if vals else None
        round_ratio = sorted(per[i_guided][k].us / min(per[i][k].us for i in ok) for k in range(args.retest_rounds))
        norm_guided, norm_best = normalised(i_guided), min((normalised(i) for i in ok if normalised(i)), default=None)
        t_guided, t_sweep = recs[i_guided], recs[i_best]
        t_cold = B.tuner_evaluate(shape, guided.best, B.make_budget(warmup=20, iters=100, repeats=5, use_graph=use_graph), ws_cold)
        floor_us = B.tuner_launch_floor(B.make_budget(warmup=20, iters=100, repeats=5, use_graph=use_graph), stream=stream)
        theta = guided.best
        tuner = {
            "feasible": counts["feasible"], "raw_grid": counts["raw"], "pruned": {k: v for k, v in counts.items()
                                                                                 if k not in ("feasible", "raw") and v},
            "search_budget_evals": args.search_budget, "search_evals_used": guided.evals_used,
            "search_best": theta_dict(guided.best), "search_best_us": round(t_guided.us, 3),
            "exhaustive_best": theta_dict(finalists[i_best]), "exhaustive_best_us": round(t_sweep.us, 3),
            "exhaustive_evals": sweep.evals_used, "sweep_heuristics": sweep_mask, "failed_gate": guided.n_failed_gate + sweep.n_failed_gate,
            "search_vs_exhaustive": round(t_guided.us / t_sweep.us, 4),
            "search_vs_exhaustive_clock_normalised": (round(norm_guided / norm_best, 4) if norm_guided and norm_best else None),
            "retest": {
                "rule": ("sweep top-%d + guided winner + its two runners-up + the shipped table's and the general theta "
                         "re-timed together, %d rounds in rotation, 20 warm-up + 100 timed launches per block, after %d ms "
                         "of load; score = median block; exhaustive_best = fastest of the set"
                         % (args.retest_top, args.retest_rounds, heat)),
                "per_round_ratio_min_median_max": [round(round_ratio[0], 4), round(round_ratio[len(round_ratio) // 2], 4),
                                                   round(round_ratio[-1], 4)],
                "candidates": [{"theta": list(finalists[i].key()), "us": round(recs[i].us, 3),
                                "us_min": round(recs[i].us_min_block, 3),
                                "spread": round((max(blk.us for blk in per[i]) - recs[i].us_min_block) / recs[i].us, 4),
                                "sm_mhz": sorted(m for m in mhz[i] if m)[len([m for m in mhz[i] if m]) // 2] if any(mhz[i]) else None,
                                "us_x_mhz": round(normalised(i), 1) if normalised(i) else None,
                                "from": ("guided" if i == i_guided else "sweep" if i < args.retest_top else
                                         "shipped table / general" if finalists[i].key() in [e.key() for e in extras.values()]
                                         else "guided runner-up")}
                               for i in ok],
            },
            "timing": ("CUDA graph of 100 launches, same buffers (L2-warm)" if use_graph else
                       "100 back-to-back launches rotating over the ring of buffer sets" if ws_tune is ws_cold else
                       "100 back-to-back launches, same buffers (exceed L2)"),
            "search_best_cold_us": round(t_cold.us, 3), "ring_sets": sets, "empty_kernel_us": round(floor_us, 3),
            "search_seconds": round(guided_s, 2), "exhaustive_seconds": round(sweep_s, 2),
            "occupancy_blocks_per_sm": t_guided.occupancy_blocks_per_sm, "regs_per_thread": t_guided.regs_per_thread,
        }
        if seeds:
            tuner["resumed_seeds"] = len(seeds)
        for name, th in extras.items():
            i = [f.key() for f in finalists].index(th.key())
            tuner["shipped_" + name] = {"theta": list(th.key()), "us": round(recs[i].us, 3) if recs[i].status == 0 else None,
                                        "vs_exhaustive": round(recs[i].us / t_sweep.us, 4) if recs[i].status == 0 else None}
        tuner["shipped_table"]["source"] = table_source
        # the sweep's fastest point of every stage (first measurement, us): which organisation of the row wins here
        by_stage = {}
        for rec in sweep_log:
            name = B.STAGE_NAMES.get(rec.params.stage, str(rec.params.stage))
            if rec.status == 0 and (name not in by_stage or rec.us < by_stage[name][0]):
                by_stage[name] = (rec.us, list(rec.params.key()))
        tuner["sweep_best_per_stage"] = {name: {"us": round(us, 3), "theta": th} for name, (us, th) in sorted(by_stage.items())}
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
                                                                 top_k=2, use_graph=use_graph, preheat_ms=heat), ws_tune)
            warm, warm_log = B.tuner_search(shape, B.make_budget(max_evals=tb, warmup=20, iters=100, repeats=3,
                                                                 top_k=2, use_graph=use_graph, seeds=seeds, preheat_ms=heat), ws_tune)
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

    t_warm = time.monotonic()
    for k in range(args.warmup):
        step(k)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    dp.barrier(device)
    launches_before = B.rt_launch_count()
    t_begin = time.monotonic()
    with torch.cuda.stream(stream):
        e0.record(stream)
        for k in range(args.steps):
            step(k)
        e1.record(stream)
    e1.synchronize()
    t_end = time.monotonic()
    dp.barrier(device)
    gpu_launches = B.rt_launch_count() - launches_before
    clocks = clock_sampler.window(t_begin, t_end)
    clocks["warmup_and_timed"] = clock_sampler.window(t_warm, t_end)
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
        traffic, traffic_capture = ncu_traffic(wl.name, theta.key())
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
                         "traffic": traffic, "traffic_capture": traffic_capture, "peak_kind": f"of {peak_kind}",
                         "kernel": KERNEL_NAME[wl.op],
                         "algorithmic_bytes_per_launch": wl.algorithmic_bytes},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d_bytes,
                    "d2h_bytes_per_step": d2h_bytes, "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps},
            "gpu_launches": int(gpu_launches),
            "clocks": clocks,
            "parity": {"r_out_bit_mismatches": int(r_bad), "y_beyond_tolerance": int(y_bad), "y_worst": y_worst,
                       "rows_checked": T},
            "tuner": tuner,
        }
        if cpu_baseline is not None:
            line["cpu_baseline"] = cpu_baseline
        clock_sampler.stop()
        print(json.dumps(line), flush=True)
    clock_sampler.stop()
    dp.shutdown()


NVLINK_PEER_GBS = 770.0  # measured peer copy per direction on this kind of machine (nominal 900)


def run_tensor_parallel(args, wl, rank: int, world: int, device) -> None:
    """The c3ar* workloads on a real group: world == the workload's group size, one rank per GPU, every rank's partial
    x, y and r_out in symmetric memory.  A step is dp.FusedAllreduceNorm: the group meets, each rank's launch reads
    its block of rows of every rank's partial through plain peer loads and stores its rows of y into every rank's
    tensor, the group meets again.  No TMA and no multicast of any kind is involved."""
    import torch
    from paper_2601_12698_b200 import binding as B
    from paper_2601_12698_b200 import dp, synth
    import oracle
    if world != wl.n_parts:
        raise SystemExit(f"{wl.name} is a group of {wl.n_parts}: start it with --gpus {wl.n_parts} (got {world} ranks)")
    T, H, b = wl.n_tokens, wl.hidden, synth.DTYPE_BYTES[wl.dtype]
    tdtype = synth.TORCH_DTYPES[wl.dtype]
    stream = torch.cuda.Stream(device=device)
    group = dp.fused_allreduce_norm(T, H, tdtype, device)
    shard = group.shard
    parts = synth.make_parts(0, T, H, wl.dtype, wl.seed, world, wl.dist)       # every rank draws all parts: the oracle needs them
    r = synth.make_rows(synth.TENSOR_R, 0, T, H, wl.dtype, wl.seed, wl.dist).contiguous()
    w = synth.make_weight(H, wl.dtype, wl.seed, wl.dist)
    y_ref, r_ref = oracle.allreduce_add_rmsnorm(parts, r, w, wl.eps, threads=os.cpu_count() or 1)
    mine_host = parts[rank].contiguous().pin_memory()
    group.x_parts[rank].copy_(mine_host)
    rd, wd = r.to(device), w.to(device)
    # theta: the shipped table's entry for (rows of one block, hidden, parts); rank 0 decides for the group
    shape = B.shape_of(max(1, shard.rows), H, wl.dtype, op=B.RT_OP_ADD_RMSNORM_ALLREDUCE, n_parts=world)
    key = list(B.SpecTable.default().lookup(shape)[0].key()) if rank == 0 else [0] * 7
    theta = B.rt_params(*dp.broadcast_ints(key, device))
    clock_sampler = ClockSampler(device)
    clock_sampler.wait_ready()

    def step():
        group(theta, rd, wd, wl.eps, stream=stream)
    for _ in range(args.warmup):
        step()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    dp.barrier(device)
    launches_before = B.rt_launch_count()
    t_begin = time.monotonic()
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    e1.synchronize()
    t_end = time.monotonic()
    dp.barrier(device)
    gpu_launches = B.rt_launch_count() - launches_before
    ms = dp.max_over_ranks(e0.elapsed_time(e1), device)
    # parity: this rank's copy of every row of y, and the residual of its own block
    y_worst, y_bad = B.tuner_compare(group.y_outs[rank], y_ref.to(device), B.RT_CMP_REL32 if wl.dtype == "fp32" else B.RT_CMP_ULP16,
                                     1e-5 if wl.dtype == "fp32" else 2.0, stream=stream)
    rows = slice(shard.row_begin, shard.row_end)
    r_bad = B.tuner_compare(group.r_outs[rank][rows], r_ref[rows].to(device), B.RT_CMP_BITS, stream=stream)[1] if shard.rows else 0
    bad = dp.sum_over_ranks(float(y_bad + r_bad), device)
    if bad or B.rt_device_status() != 0:
        raise RuntimeError(f"rank {rank}: the group's outputs differ from the oracle (y_bad={y_bad}, r_bad={r_bad})")
    # end to end: this rank's partial comes from pinned host memory and its y goes back, inside the timed region
    y_host = torch.empty((T, H), dtype=tdtype).pin_memory()
    e2e_steps = max(3, min(args.steps, args.e2e_steps))

    def e2e_step():
        with torch.cuda.stream(stream):
            group.x_parts[rank].copy_(mine_host, non_blocking=True)
        step()
        with torch.cuda.stream(stream):
            y_host.copy_(group.y_outs[rank], non_blocking=True)
        stream.synchronize()
    e2e_step()
    dp.barrier(device)
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    e2e_ms = dp.max_over_ranks((time.perf_counter() - t0) * 1e3, device)
    dp.barrier(device)
    if oracle.compare_y(y_host[-64:], y_ref[-64:], tol_rel=1e-5)[1]:
        raise RuntimeError("end-to-end path fails parity")
    if rank == 0:
        step_s = ms * 1e-3 / args.steps
        link_bytes = 2.0 * (world - 1) / world * T * H * b   # per GPU and direction: peers' parts in, y out
        hbm_bytes = (3 + 2.0 / world) * T * H * b + H * b     # per GPU: parts and y of all rows, r and r' of its block
        hbm_peak, peak_kind = measured_hbm_peak()
        bound_s = max(link_bytes / (NVLINK_PEER_GBS * 1e9), hbm_bytes / (hbm_peak * 1e9))
        line = {
            "metric": METRICS[wl.op], "value": wl.algorithmic_bytes / step_s / 1e9, "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
            "config": {"workload": wl.name, "n_tokens": T, "hidden": H, "eps": wl.eps, "l2": "inputs_exceed_l2",
                       "bytes": "per element: one partial per rank and r read, y and r' written once (what the group must move)",
                       "parallelism": f"tensor-parallel group of {world}: all-reduce fused into the norm over peer-mapped memory",
                       "theta": theta_dict(theta)},
            "roofline": {"bound": "nvlink" if link_bytes / NVLINK_PEER_GBS > hbm_bytes / hbm_peak else "hbm",
                         "achieved": link_bytes / step_s / 1e9, "peak": NVLINK_PEER_GBS, "unit": UNIT,
                         "frac": bound_s / step_s, "traffic": None, "peak_kind": f"slower of link bytes / {NVLINK_PEER_GBS:.0f} GB/s "
                         f"per direction and HBM bytes / copy peak (of {peak_kind}); includes the two group meetings per step",
                         "kernel": KERNEL_NAME[wl.op], "link_bytes_per_direction_per_gpu": link_bytes,
                         "hbm_bytes_per_gpu": hbm_bytes},
            "e2e": {"value": wl.algorithmic_bytes * e2e_steps / (e2e_ms * 1e-3) / 1e9, "unit": UNIT,
                    "h2d_bytes_per_step": T * H * b, "d2h_bytes_per_step": T * H * b, "steps": e2e_steps,
                    "ms_per_step": e2e_ms / e2e_steps},
            "gpu_launches": int(gpu_launches), "clocks": clock_sampler.window(t_begin, t_end),
            "parity": {"r_out_bit_mismatches": 0, "y_beyond_tolerance": 0, "y_worst": y_worst, "rows_checked": T,
                       "ranks_checked": world},
            "tuner": {"theta_from": "shipped table (nearest entry for this block of rows)"},
        }
        clock_sampler.stop()
        print(json.dumps(line), flush=True)
    clock_sampler.stop()
    dp.shutdown()


def spawn_ranks(n: int, argv: list, script: str | None = None, extra_env: dict | None = None, timeout_s: float | None = None) -> int:
    """Start `n` ranks of `script` (this file by default), one process per GPU: RANK = LOCAL_RANK = 0..n-1, WORLD_SIZE = n,
    rendezvous on 127.0.0.1 at a port that is free now.  The ranks inherit stdout and stderr (rank 0 prints the JSON
    line; NCCL's own messages stay at their default).  Returns the largest exit code; when one rank fails the others
    are ended, each by its own handle."""
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    procs = []
    for rank in range(n):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(n), LOCAL_WORLD_SIZE=str(n),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        env.update(extra_env or {})
        procs.append(subprocess.Popen([sys.executable, script or os.path.abspath(__file__), *argv], env=env))
    worst, t0 = 0, time.monotonic()
    pending = list(procs)
    while pending:
        for pr in list(pending):
            rc = pr.poll()
            if rc is None:
                continue
            pending.remove(pr)
            worst = max(worst, abs(rc))
        if pending and (worst != 0 or (timeout_s is not None and time.monotonic() - t0 > timeout_s)):
            for pr in pending:
                pr.terminate()
            for pr in pending:
                try:
                    pr.wait(timeout=10)
                except subprocess.TimeoutExpired:
                    pr.kill()
            return worst or 124
        time.sleep(0.05)
    return worst


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
    ap.add_argument("--include-pipeline", action="store_true", help="search the persistent TMA pipeline stage as well")
    ap.add_argument("--sweep-heuristics", type=int, default=-1, help="RT_PRUNE_* mask of the exhaustive sweep alone "
                    "(0: every hard-feasible theta; default: the mask of the guided search)")
    ap.add_argument("--resume", default="", help="a JSONL file written by --log: its fastest thetas seed the guided search")
    ap.add_argument("--preheat-ms", type=int, default=300, help="how long the tuner loads the device before it compares "
                    "candidates of a bandwidth-bound workload")
    ap.add_argument("--retest-top", type=int, default=8, help="points of the sweep re-timed beside the guided winner")
    ap.add_argument("--retest-rounds", type=int, default=7, help="rounds of the side-by-side re-test")
    args = ap.parse_args()
    if args.steps < 1 or args.warmup < 0:
        raise SystemExit("--steps must be >= 1 and --warmup >= 0")
    if args.gpus > 1 and "RANK" not in os.environ:
        # started plainly: be the launcher - one process per GPU, this same command line in each
        raise SystemExit(spawn_ranks(args.gpus, sys.argv[1:]))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
