"""CPU oracle for the general-configuration choice (test infrastructure only).

SelectGeneral of the paper's Algorithm 1 with the scoring of "Performance Measurement and Evaluation":
the speedup of a configuration on an input is a ratio of run times and speedups are aggregated over the
test set by their geometric mean.  With no external baseline kernel, the reference time on each shape is
the best time any candidate reached there, T*(x), so a score of 1 means "best everywhere".

Plain Python floats (fp64), written from the definition; shares nothing with the CUDA library.
Pins (tests/test_selection.py): hand-computed tables, invariance of the ranking under rescaling of one
shape's times (which an arithmetic mean of times would not have), exclusion of candidates that cannot run
on some shape.
"""
from __future__ import annotations

import math


def _ran(t: float) -> bool:
    return t is not None and t > 0.0 and math.isfinite(t)


def select_general(times_us):
    """times_us[c][x]: time of candidate c on shape x (<= 0, None, NaN, inf: did not run).

    Returns (best_index, best_score, scores).  best_index is None when no candidate ran everywhere."""
    n_c, n_x = len(times_us), len(times_us[0])
    best_time = []
    for x in range(n_x):
        ran = [times_us[c][x] for c in range(n_c) if _ran(times_us[c][x])]
        best_time.append(min(ran) if ran else math.inf)
    scores = []
    for c in range(n_c):
        if all(_ran(times_us[c][x]) for x in range(n_x)):
            product = 1.0
            for x in range(n_x):
                product *= best_time[x] / times_us[c][x]
            scores.append(product ** (1.0 / n_x))
        else:
            scores.append(0.0)
    eligible = [c for c in range(n_c) if scores[c] > 0.0]
    if not eligible:
        return None, 0.0, scores
    best = max(eligible, key=lambda c: (scores[c], -c))
    return best, scores[best], scores
