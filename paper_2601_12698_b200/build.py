"""Builds librmsnorm_tuner.so for sm_100a with nvcc (in-tree, no JIT cache).

The kernel template is instantiated in the units listed in ``csrc/instance_units.inc``; each unit is
``csrc/instantiate.cu`` compiled with the -D flags derived from the unit's name
(``<dtype>_v<vec bytes>_<group>[_r<reduce>]``).  Units compile in parallel; objects whose inputs are
older than the object are reused.

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
HOST_UNITS = ["launch.cu", "feasible.cu", "search.cu", "host_run.cu", "table.cu"]
ELEMENT_TYPES = {"bf16": ("__nv_bfloat16", 0), "fp16": ("__half", 1), "fp32": ("float", 2)}
GROUPS = {"reg": 0, "smem": 1, "narrow": 2}


def instance_units() -> list[str]:
    text = open(os.path.join(CSRC, "instance_units.inc")).read()
    return re.findall(r"^RT_DECLARE_SLICE\((\w+)\)", text, flags=re.M)


def unit_flags(name: str) -> list[str]:
    m = re.fullmatch(r"(bf16|fp16|fp32)_v(\d+)_(reg|smem|narrow)(?:_r(\d))?", name)
    if not m:
        raise ValueError(f"cannot parse instantiation unit name {name!r}")
    ctype, code = ELEMENT_TYPES[m.group(1)]
    flags = [f"-DRT_UNIT_NAME={name}", f"-DRT_UNIT_T={ctype}", f"-DRT_UNIT_DTYPE={code}",
             f"-DRT_UNIT_VB={m.group(2)}", f"-DRT_UNIT_GROUP={GROUPS[m.group(3)]}"]
    if m.group(4) is not None:
        flags.append(f"-DRT_UNIT_REDUCE={m.group(4)}")
    return flags


def _newest_input() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(INCLUDE, "rmsnorm_tuner.h"), __file__]
    return max(os.path.getmtime(p) for p in paths)


def _compile(job):
    src, obj, flags, verbose = job
    cmd = ["nvcc", *NVCC_FLAGS, *flags, "-c", src, "-o", obj]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    proc = subprocess.run(cmd, capture_output=True, text=True)
    if proc.returncode != 0:
        raise RuntimeError(f"nvcc failed for {os.path.basename(obj)}:\n{proc.stdout}\n{proc.stderr}")
    return obj, proc.stderr


def build(force: bool = False, verbose: bool = False, jobs: int | None = None) -> str:
    os.makedirs(OBJ_DIR, exist_ok=True)
    newest = _newest_input()
    work, objs = [], []
    for name in instance_units():
        obj = os.path.join(OBJ_DIR, f"inst_{name}.o")
        objs.append(obj)
        if force or not os.path.exists(obj) or os.path.getmtime(obj) < newest:
            work.append((os.path.join(CSRC, "instantiate.cu"), obj, unit_flags(name), verbose))
    for src in HOST_UNITS:
        obj = os.path.join(OBJ_DIR, src.replace(".cu", ".o"))
        objs.append(obj)
        if force or not os.path.exists(obj) or os.path.getmtime(obj) < newest:
            work.append((os.path.join(CSRC, src), obj, [], verbose))
    if work:
        with ThreadPoolExecutor(max_workers=jobs or os.cpu_count() or 4) as pool:
            for obj, log in pool.map(_compile, work):
                if verbose and log:
                    with open(obj + ".ptxas.txt", "w") as f:
                        f.write(log)
    if work or not os.path.exists(LIB_PATH):
        tmp = LIB_PATH + f".tmp{os.getpid()}"
        cmd = ["nvcc", "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp, *objs]
        proc = subprocess.run(cmd, capture_output=True, text=True)
        if proc.returncode != 0:
            raise RuntimeError(f"link failed:\n{proc.stdout}\n{proc.stderr}")
        os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    path = build(force="--force" in sys.argv, verbose="--verbose" in sys.argv)
    print(path)
