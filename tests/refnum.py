"""Independent number-format helpers for pinning the oracle.

Nothing here comes from the oracle or from the CUDA path.  The tables of
representable values are decoded by torch's own conversion to float64, and
rounding is done by bracketing a value between two adjacent table entries and
comparing against their exact midpoint (every quantity involved is exactly a
float64, or a Fraction / Decimal where stated).
"""
from __future__ import annotations

import bisect
from decimal import Decimal, getcontext
from fractions import Fraction
from functools import lru_cache

import numpy as np
import torch

getcontext().prec = 80
TORCH_16 = {0: torch.bfloat16, 1: torch.float16}


@lru_cache(maxsize=None)
def finite_table(dtype: int):
    """(values ascending float64, bit patterns) of all finite, non-negative-zero-deduplicated values.

    -0 is dropped so that values are strictly increasing; +0 keeps pattern 0."""
    bits = np.arange(65536, dtype=np.int64).astype(np.uint16)
    vals = torch.from_numpy(bits.view(np.int16)).view(TORCH_16[dtype]).to(torch.float64).numpy()
    ok = np.isfinite(vals) & (bits != 0x8000)
    vals, bits = vals[ok], bits[ok]
    order = np.argsort(vals, kind="stable")
    return vals[order], bits[order]


def max_finite(dtype: int) -> float:
    return float(finite_table(dtype)[0][-1])


def round_array(v: np.ndarray, dtype: int) -> np.ndarray:
    """Round float64 values to the 16-bit format: nearest, ties to even, overflow to infinity.

    Exact: neighbours a <= v <= b are adjacent table entries, and (a + b) / 2 is exactly
    representable in float64, so the comparisons below involve no rounding."""
    vals, bits = finite_table(dtype)
    v = np.asarray(v, dtype=np.float64)
    out = np.empty(v.shape, dtype=np.uint16)
    flat, o = v.ravel(), out.ravel()
    hi = np.searchsorted(vals, flat, side="left")  # first index with vals >= v
    n = len(vals)
    inf_bits = 0x7F80 if dtype == 0 else 0x7C00
    top = vals[-1]
    ulp_top = vals[-1] - vals[-2]
    for i in range(flat.size):
        x = flat[i]
        if np.isnan(x):
            o[i] = inf_bits | 1
            continue
        if x >= top + ulp_top / 2:
            o[i] = inf_bits
            continue
        if x <= -(top + ulp_top / 2):
            o[i] = 0x8000 | inf_bits
            continue
        h = min(int(hi[i]), n - 1)
        if vals[h] == x:
            pick = h
        else:
            l = max(h - 1, 0)
            if x > vals[h]:  # beyond the largest finite but below the overflow threshold
                pick = h
            elif x < vals[l]:
                pick = l
            else:
                mid = (vals[l] + vals[h]) / 2
                if x < mid:
                    pick = l
                elif x > mid:
                    pick = h
                else:
                    pick = l if (int(bits[l]) & 1) == 0 else h
        b = int(bits[pick])
        if b == 0 and np.signbit(x):
            b = 0x8000
        o[i] = b
    return out


def round_exact(value, dtype: int) -> int:
    """Round an exact Fraction / Decimal / float to the 16-bit format (bit pattern)."""
    vals, bits = finite_table(dtype)
    if isinstance(value, Decimal):
        cmp_val = value
        conv = lambda f: Decimal(float(f))  # exact: Decimal(float) is exact
    else:
        cmp_val = Fraction(value)
        conv = lambda f: Fraction(float(f))
    neg = cmp_val < 0
    top = conv(vals[-1])
    half_top = (conv(vals[-1]) - conv(vals[-2])) / 2
    inf_bits = 0x7F80 if dtype == 0 else 0x7C00
    if cmp_val >= top + half_top:
        return inf_bits
    if cmp_val <= -(top + half_top):
        return 0x8000 | inf_bits
    # bisect on floats is safe for locating the bracket; the decision uses exact values
    approx = float(cmp_val)
    h = min(bisect.bisect_left(vals.tolist(), approx), len(vals) - 1)
    cands = range(max(h - 2, 0), min(h + 3, len(vals)))
    best, best_d = None, None
    for k in cands:
        d = abs(cmp_val - conv(vals[k]))
        if best is None or d < best_d or (d == best_d and (int(bits[k]) & 1) == 0 and (int(bits[best]) & 1) == 1):
            best, best_d = k, d
    b = int(bits[best])
    if b == 0 and neg:
        b = 0x8000
    return b


def decode_bits(bits, dtype: int) -> np.ndarray:
    """Bit patterns -> float64 through torch's conversion (library decode)."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return torch.from_numpy(b.view(np.int16)).view(TORCH_16[dtype]).to(torch.float64).numpy()
