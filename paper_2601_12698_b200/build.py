"""Builds librmsnorm_tuner.so for sm_100a with nvcc (in-tree, no JIT cache).

The kernel template is instantiated in the units listed in ``csrc/instance_units.inc``; each unit is
``csrc/instantiate.cu`` compiled with the -D flags derived from the unit's name
(``<dtype>_v<vec bytes>_<group>[_r<reduce>]``).  Units compile in parallel; objects whose inputs are
older than the object are reused.

Two stages.  The instantiation units are compiled first, with ``-Xptxas -v``; the registers and static
shared memory ptxas reports for every instance are written to ``_build/instance_resources.inc``, which
``launch.cu`` includes: the feasible-region deriver can then reason about this very build's kernels even on a
machine without a GPU (with a GPU it asks the runtime instead).

    python -m paper_2601_12698_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import os
import re
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
OBJ_DIR = os.path.join(HERE, "_build")
LIB_PATH = os.path.join(HERE, "librmsnorm_tuner.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-std=c++17", "-O3", "-lineinfo",
              "-Xcompiler", "-fPIC", "-I", CSRC, "-I", INCLUDE]
HOST_UNITS = ["launch.cu", "feasible.cu", "search.cu", "host_run.cu", "table.cu", "trace.cu"]
ELEMENT_TYPES = {"bf16": ("__nv_bfloat16", 0), "fp16": ("__half", 1), "fp32": ("float", 2)}
GROUPS = {"reg": 0, "smem": 1, "narrow": 2, "silu": 3, "merge": 4, "fp8out": 5, "allreduce": 6, "realign": 7}


def instance_units() -> list[str]:
    text = open(os.path.join(CSRC, "instance_units.inc")).read()
    return re.findall(r"^RT_DECLARE_SLICE\((\w+)\)", text, flags=re.M)


def unit_flags(name: str) -> list[str]:
    m = re.fullmatch(r"(bf16|fp16|fp32)_v(\d+)_(reg|smem|narrow|silu|merge|fp8out|allreduce|realign)(?:_r(\d))?", name)
    if not m:
        raise ValueError(f"cannot parse instantiation unit name {name!r}")
    ctype, code = ELEMENT_TYPES[m.group(1)]
    flags = [f"-DRT_UNIT_NAME={name}", f"-DRT_UNIT_T={ctype}", f"-DRT_UNIT_DTYPE={code}",
             f"-DRT_UNIT_VB={m.group(2)}", f"-DRT_UNIT_GROUP={GROUPS[m.group(3)]}"]
    if m.group(4) is not None:
        flags.append(f"-DRT_UNIT_REDUCE={m.group(4)}")
    return flags


# (the plain instances: TRACE = false, mangled Lb0E; the instrumented ones of trace.cu are not part of the table)
_ENTRY = re.compile(r"Compiling entry function '_ZN2rt18add_rmsnorm_kernelI(\w+?)Li(\d+)ELi(\d+)ELi(\d+)ELi(\d+)ELi(\d+)ELb0E"
                    r"EEvNS_10KernelArgsE'.*?(\d+) bytes spill stores.*?Used (\d+) registers.*?(\d+) bytes smem", re.S)
_MANGLED_DTYPE = {"13__nv_bfloat16": 0, "6__half": 1, "f": 2}


_SILU_ENTRY = re.compile(r"Compiling entry function '_ZN2rt19silu_and_mul_kernelI(\w+?)Li(\d+)ELi(\d+)ELi(\d+)E"
                         r"EEvNS_8SiluArgsE'.*?(\d+) bytes spill stores.*?Used (\d+) registers(?:.*?(\d+) bytes smem)?", re.S)


_MERGE_ENTRY = re.compile(r"Compiling entry function '_ZN2rt24merge_attn_states_kernelI(\w+?)Li(\d+)ELi(\d+)ELi(\d+)E"
                          r"EEvNS_9MergeArgsE'.*?(\d+) bytes spill stores.*?Used (\d+) registers(?:.*?(\d+) bytes smem)?", re.S)


_FP8_ENTRY = re.compile(r"Compiling entry function '_ZN2rt22add_rmsnorm_fp8_kernelI(\w+?)Li(\d+)ELi(\d+)ELi(\d+)ELi(\d+)E"
                        r"EEvNS_7Fp8ArgsE'.*?(\d+) bytes spill stores.*?Used (\d+) registers(?:.*?(\d+) bytes smem)?", re.S)


_ALLREDUCE_ENTRY = re.compile(r"Compiling entry function '_ZN2rt28add_rmsnorm_allreduce_kernelI(\w+?)Li(\d+)ELi(\d+)ELi(\d+)ELi(\d+)E"
                              r"EEvNS_13AllreduceArgsE'.*?(\d+) bytes spill stores.*?Used (\d+) registers(?:.*?(\d+) bytes smem)?", re.S)


def parse_ptxas(log: str) -> list[tuple]:
    """(op, dtype, vec, stage, reduce, unroll, cap, registers, static smem, spill bytes, parts) per entry function."""
    rows = []
    for m in _ENTRY.finditer(log):
        t, vb, st, rd, u, cap, spill, regs, smem = m.groups()
        rows.append((0, _MANGLED_DTYPE[t], int(vb), int(st), int(rd), int(u), int(cap) if int(st) in (0, 3) else 0,
                     int(regs), int(smem), int(spill), 0))
    for block in log.split("ptxas info    : Compiling entry function")[1:]:
        for op, pattern in ((1, _SILU_ENTRY), (2, _MERGE_ENTRY)):
            m = pattern.search("Compiling entry function" + block)
            if m:
                t, vb, st, u, spill, regs, smem = m.groups()
                rows.append((op, _MANGLED_DTYPE[t], int(vb), int(st), 0, int(u), 0, int(regs), int(smem or 0), int(spill), 0))
    for block in log.split("ptxas info    : Compiling entry function")[1:]:
        m = _FP8_ENTRY.search("Compiling entry function" + block)
        if m:
            t, vb, st, u, cap, spill, regs, smem = m.groups()
            rows.append((3, _MANGLED_DTYPE[t], int(vb), int(st), 0, int(u), int(cap) if int(st) == 0 else 0, int(regs),
                         int(smem or 0), int(spill), 0))
        m = _ALLREDUCE_ENTRY.search("Compiling entry function" + block)
        if m:
            t, vb, parts, u, cap, spill, regs, smem = m.groups()
            rows.append((4, _MANGLED_DTYPE[t], int(vb), 0, 0, int(u), int(cap), int(regs), int(smem or 0), int(spill), int(parts)))
    return rows


def write_resource_table(rows: list[tuple]) -> str:
    path = os.path.join(OBJ_DIR, "instance_resources.inc")
    lines = ["// Generated by build.py from the ptxas reports of the instantiation units: per instance\n"
             "// {op, dtype, vec_bytes, stage, reduce, unroll, cap, registers per thread, static smem, spill bytes, parts}.\n"]
    lines += ["{%d, %d, %d, %d, %d, %d, %d, %d, %d, %d, %d},\n" % r for r in sorted(set(rows))]
    text = "".join(lines)
    if not os.path.exists(path) or open(path).read() != text:
        with open(path, "w") as f:
            f.write(text)
    return path


def _newest_input() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(INCLUDE, "rmsnorm_tuner.h"), __file__]
    return max(os.path.getmtime(p) for p in paths)


def _compile(job):
    src, obj, flags, verbose = job
    cmd = ["nvcc", "-Xptxas=-v", *NVCC_FLAGS, "-I", OBJ_DIR, *flags, "-c", src, "-o", obj]
    proc = subprocess.run(cmd, capture_output=True, text=True)
    if proc.returncode != 0:
        raise RuntimeError(f"nvcc failed for {os.path.basename(obj)}:\n{proc.stdout}\n{proc.stderr}")
    with open(obj + ".ptxas.txt", "w") as f:
        f.write(proc.stderr)
    return obj, proc.stderr


def build(force: bool = False, verbose: bool = False, jobs: int | None = None) -> str:
    os.makedirs(OBJ_DIR, exist_ok=True)
    newest = _newest_input()
    pool_size = jobs or os.cpu_count() or 4

    def stale(obj: str) -> bool:
        return force or not os.path.exists(obj) or os.path.getmtime(obj) < newest or not os.path.exists(obj + ".ptxas.txt")

    # stage 1: the instantiation units
    inst_objs, work = [], []
    for name in instance_units():
        obj = os.path.join(OBJ_DIR, f"inst_{name}.o")
        inst_objs.append(obj)
        if stale(obj):
            work.append((os.path.join(CSRC, "instantiate.cu"), obj, unit_flags(name), verbose))
    rebuilt = bool(work)
    if work:
        with ThreadPoolExecutor(max_workers=pool_size) as pool:
            list(pool.map(_compile, work))
    rows = []
    for obj in inst_objs:
        rows += parse_ptxas(open(obj + ".ptxas.txt").read())
    table = write_resource_table(rows)

    # stage 2: the host units (launch.cu includes the resource table)
    host_objs, work = [], []
    for src in HOST_UNITS:
        obj = os.path.join(OBJ_DIR, src.replace(".cu", ".o"))
        host_objs.append(obj)
        if stale(obj) or (src == "launch.cu" and os.path.getmtime(obj) < os.path.getmtime(table)):
            work.append((os.path.join(CSRC, src), obj, [], verbose))
    if work:
        rebuilt = True
        with ThreadPoolExecutor(max_workers=pool_size) as pool:
            list(pool.map(_compile, work))
    if rebuilt or not os.path.exists(LIB_PATH):
        tmp = LIB_PATH + f".tmp{os.getpid()}"
        cmd = ["nvcc", "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp, *inst_objs, *host_objs]
        proc = subprocess.run(cmd, capture_output=True, text=True)
        if proc.returncode != 0:
            raise RuntimeError(f"link failed:\n{proc.stdout}\n{proc.stderr}")
        os.replace(tmp, LIB_PATH)
    if verbose:
        print(f"{len(rows)} instances, resource table {table}")
    return LIB_PATH


if __name__ == "__main__":
    path = build(force="--force" in sys.argv, verbose="--verbose" in sys.argv)
    print(path)
