"""Writes tests/golden/oracle_regression.txt: bit patterns the oracle produces on small seeded cases.

Calls only the input generator and ``oracle/``; never the CUDA path.  The stored values are a
regression record (they catch an accidental change of the generator or of the oracle), not a pin of
the oracle's correctness - the pins are the closed-form, exact-arithmetic and library tests.

Run from the repository root:  python tests/golden/make_golden.py
"""
import hashlib
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2601_12698_b200 import synth  # noqa: E402

CASES = [("bf16", 3, 40, 0), ("fp16", 2, 6152, 3), ("fp32", 2, 24, 4)]


def digest(t) -> str:
    s, _ = oracle.as_storage(t)
    return hashlib.sha256(s.tobytes()).hexdigest()[:32]


def lines():
    yield "# dtype n_tokens hidden seed | sha256/32 of x, r, w, y, r_out storage | first 4 y words, first 4 r_out words (hex)"
    for dtype, T, H, seed in CASES:
        x, r, w = synth.make_inputs(T, H, dtype, seed)
        y, ro = oracle.add_rmsnorm(x, r, w, 1e-6)
        ys, _ = oracle.as_storage(y)
        rs, _ = oracle.as_storage(ro)
        word = (lambda a: a.view(np.uint32)) if dtype == "fp32" else (lambda a: a)
        heads = " ".join(f"{int(v):x}" for v in list(word(ys).ravel()[:4]) + list(word(rs).ravel()[:4]))
        yield f"{dtype} {T} {H} {seed} | {digest(x)} {digest(r)} {digest(w)} {digest(y)} {digest(ro)} | {heads}"


if __name__ == "__main__":
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_regression.txt")
    with open(out, "w") as f:
        f.write("\n".join(lines()) + "\n")
    print(open(out).read())
