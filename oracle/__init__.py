"""CPU oracles of the tuned kernels (test infrastructure only).

Thin ctypes wrapper over ``add_rmsnorm_oracle.c``, ``silu_and_mul_oracle.c`` and
``merge_attn_states_oracle.c`` / ``add_rmsnorm_fp8_oracle.c``;
all arithmetic is in the C files (``selection.py`` holds the plain-Python oracle
of the general-configuration choice).  Only the tests, the smoke check and the benchmark's CPU-baseline leg may
import this package.  It imports nothing from the CUDA package and shares no
code with it.

Arrays cross this boundary as raw element storage: ``numpy.uint16`` bit
patterns for bf16 / fp16, ``numpy.float32`` for fp32.  ``torch`` CPU tensors
are accepted as a convenience and converted by reinterpreting their storage.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

BF16, FP16, FP32 = 0, 1, 2
DTYPE_NAMES = {BF16: "bf16", FP16: "fp16", FP32: "fp32"}

_HERE = os.path.dirname(os.path.abspath(__file__))
SOURCES = ("add_rmsnorm_oracle.c", "silu_and_mul_oracle.c", "merge_attn_states_oracle.c",
           "add_rmsnorm_fp8_oracle.c", "allreduce_add_rmsnorm_oracle.c")
HEADERS = ("number_formats.h",)
_LIB = os.path.join(_HERE, "liboracle.so")
_lock = threading.Lock()
_lib = None


def compile_sources(src_dir: str, out_path: str) -> str:
    """gcc the oracle's C files found in `src_dir` into one shared library."""
    cmd = ["gcc", "-O2", "-fno-fast-math", "-ffp-contract=off", "-std=c99", "-shared", "-fPIC", "-pthread",
           "-I", src_dir, *[os.path.join(src_dir, f) for f in SOURCES], "-o", out_path, "-lm"]
    subprocess.run(cmd, check=True)
    return out_path


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no-op when the library is up to date)."""
    with _lock:
        newest = max(os.path.getmtime(os.path.join(_HERE, f)) for f in SOURCES + HEADERS)
        if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= newest:
            return _LIB
        tmp = _LIB + f".tmp{os.getpid()}"
        compile_sources(_HERE, tmp)
        os.replace(tmp, _LIB)
        return _LIB


def _bind(path: str):
    """Load one build of the C oracle and declare its signatures."""
    lib = ctypes.CDLL(path)
    vp, i64, i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32
    lib.oracle_add_rmsnorm.argtypes = [vp, vp, vp, vp, vp, i64, i64, ctypes.c_float,
                                       ctypes.c_int, ctypes.c_int, ctypes.c_int]
    lib.oracle_add_rmsnorm.restype = ctypes.c_int
    lib.oracle_decode16.argtypes = [vp, vp, i64, ctypes.c_int]
    lib.oracle_decode16.restype = None
    lib.oracle_encode16_from_f64.argtypes = [vp, vp, i64, ctypes.c_int]
    lib.oracle_encode16_from_f64.restype = None
    lib.oracle_encode16_from_f32.argtypes = [vp, vp, i64, ctypes.c_int]
    lib.oracle_encode16_from_f32.restype = None
    lib.oracle_ulp_compare16.argtypes = [vp, vp, i64, ctypes.c_int, i32,
                                         ctypes.POINTER(i32), ctypes.POINTER(i64)]
    lib.oracle_ulp_compare16.restype = None
    lib.oracle_rel_compare32.argtypes = [vp, vp, i64, ctypes.c_double, ctypes.c_double,
                                         ctypes.POINTER(ctypes.c_double), ctypes.POINTER(i64)]
    lib.oracle_rel_compare32.restype = None
    lib.oracle_silu_and_mul.argtypes = [vp, vp, i64, i64, ctypes.c_int, ctypes.c_int]
    lib.oracle_silu_and_mul.restype = ctypes.c_int
    lib.oracle_merge_attn_states.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, ctypes.c_int]
    lib.oracle_merge_attn_states.restype = ctypes.c_int
    lib.oracle_mixed_compare.argtypes = [vp, vp, i64, ctypes.c_int, ctypes.c_double, ctypes.c_double,
                                         ctypes.POINTER(ctypes.c_double), ctypes.POINTER(i64)]
    lib.oracle_mixed_compare.restype = None
    lib.oracle_decode_e4m3.argtypes = [vp, vp, i64]
    lib.oracle_decode_e4m3.restype = None
    lib.oracle_encode_e4m3.argtypes = [vp, vp, i64]
    lib.oracle_encode_e4m3.restype = None
    lib.oracle_add_rmsnorm_fp8.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, ctypes.c_float, ctypes.c_int]
    lib.oracle_add_rmsnorm_fp8.restype = ctypes.c_int
    lib.oracle_allreduce_add_rmsnorm.argtypes = [vp, ctypes.c_int, vp, vp, vp, vp, i64, i64, ctypes.c_float,
                                                 ctypes.c_int, ctypes.c_int]
    lib.oracle_allreduce_add_rmsnorm.restype = ctypes.c_int
    lib.oracle_e4m3_compare.argtypes = [vp, vp, i64, i32, ctypes.POINTER(i32), ctypes.POINTER(i64)]
    lib.oracle_e4m3_compare.restype = None
    return lib


def _load():
    global _lib
    if _lib is None:
        _lib = _bind(build())
    return _lib


def _storage_dtype(dtype: int):
    return np.float32 if dtype == FP32 else np.uint16


def as_storage(a, dtype: int | None = None):
    """Return (contiguous numpy storage array, dtype code) for a numpy array or torch tensor."""
    if hasattr(a, "detach"):  # torch tensor, reinterpret without arithmetic
        import torch
        t = a.detach().cpu().contiguous()
        if t.dtype == torch.bfloat16:
            return t.view(torch.int16).numpy().view(np.uint16), BF16
        if t.dtype == torch.float16:
            return t.view(torch.int16).numpy().view(np.uint16), FP16
        if t.dtype == torch.float32:
            return t.numpy(), FP32
        raise TypeError(f"unsupported tensor dtype {t.dtype}")
    a = np.ascontiguousarray(a)
    if dtype is None:
        if a.dtype == np.float32:
            return a, FP32
        if a.dtype == np.float16:
            return a.view(np.uint16), FP16
        raise TypeError("dtype code required for raw uint16 storage")
    if a.dtype != _storage_dtype(dtype):
        if dtype == FP16 and a.dtype == np.float16:
            return a.view(np.uint16), FP16
        raise TypeError(f"storage dtype {a.dtype} does not match dtype code {dtype}")
    return a, dtype


def to_torch(storage: np.ndarray, dtype: int):
    """Reinterpret oracle storage as a torch CPU tensor of the matching dtype."""
    import torch
    if dtype == FP32:
        return torch.from_numpy(storage)
    t = torch.from_numpy(storage.view(np.int16))
    return t.view(torch.bfloat16 if dtype == BF16 else torch.float16)


def add_rmsnorm(x, r, w, eps: float, dtype: int | None = None, *, norm_from_rounded: bool = False,
                threads: int = 1):
    """y, r_out = oracle(x, r, w).  x, r: [T, H]; w: [H].  Returns storage arrays
    (uint16 / float32) when given numpy input, torch tensors when given torch input."""
    want_torch = hasattr(x, "detach")
    xs, dt = as_storage(x, dtype)
    rs, dt_r = as_storage(r, dtype)
    ws, dt_w = as_storage(w, dtype)
    if not (dt == dt_r == dt_w):
        raise TypeError("x, r and w must share one dtype")
    if xs.ndim != 2 or rs.shape != xs.shape or ws.shape != (xs.shape[1],):
        raise ValueError("expected x, r of shape [T, H] and w of shape [H]")
    T, H = xs.shape
    y = np.empty_like(xs)
    r_out = np.empty_like(xs)
    rc = _load().oracle_add_rmsnorm(xs.ctypes.data, rs.ctypes.data, ws.ctypes.data,
                                    y.ctypes.data, r_out.ctypes.data, T, H, float(eps), dt,
                                    int(bool(norm_from_rounded)), int(threads))
    if rc != 0:
        raise RuntimeError(f"oracle_add_rmsnorm failed with status {rc}")
    if want_torch:
        return to_torch(y, dt), to_torch(r_out, dt)
    return y, r_out


def silu_and_mul(x, dtype: int | None = None, *, threads: int = 1):
    """out = silu(x[:, :d]) * x[:, d:] for x of shape [T, 2*d]; storage array or torch tensor like the input."""
    want_torch = hasattr(x, "detach")
    xs, dt = as_storage(x, dtype)
    if xs.ndim != 2 or xs.shape[1] % 2:
        raise ValueError("expected x of shape [T, 2*d]")
    T, d = xs.shape[0], xs.shape[1] // 2
    out = np.empty((T, d), dtype=xs.dtype)
    rc = _load().oracle_silu_and_mul(xs.ctypes.data, out.ctypes.data, T, d, dt, int(threads))
    if rc != 0:
        raise RuntimeError(f"oracle_silu_and_mul failed with status {rc}")
    return to_torch(out, dt) if want_torch else out


def merge_attn_states(v_a, s_a, v_b, s_b, dtype: int | None = None):
    """(v_out, s_out) for v_a, v_b of shape [n, h, d] and float32 log-sum-exps s_a, s_b of shape [n, h]."""
    want_torch = hasattr(v_a, "detach")
    va, dt = as_storage(v_a, dtype)
    vb, dt_b = as_storage(v_b, dtype)
    sa, _ = as_storage(s_a, FP32)
    sb, _ = as_storage(s_b, FP32)
    if dt != dt_b or va.ndim != 3 or vb.shape != va.shape or sa.shape != va.shape[:2] or sb.shape != sa.shape:
        raise ValueError("expected v_a, v_b of shape [n, h, d] and s_a, s_b of shape [n, h]")
    if sa.dtype != np.float32 or sb.dtype != np.float32:
        raise TypeError("s_a and s_b must be float32")
    n, h, d = va.shape
    v_out = np.empty_like(va)
    s_out = np.empty((n, h), dtype=np.float32)
    rc = _load().oracle_merge_attn_states(va.ctypes.data, sa.ctypes.data, vb.ctypes.data, sb.ctypes.data,
                                          v_out.ctypes.data, s_out.ctypes.data, n, h, d, dt)
    if rc != 0:
        raise RuntimeError(f"oracle_merge_attn_states failed with status {rc}")
    if want_torch:
        return to_torch(v_out, dt), to_torch(s_out, FP32)
    return v_out, s_out


def compare_mixed(got, ref, dtype: int | None = None, *, tol: float = 2.0, tol_abs: float = 1e-5):
    """(largest absolute difference, count failing) where an element passes within `tol` (ulps for 16-bit
    types, relative for fp32) OR within `tol_abs` absolutely."""
    g, dt = as_storage(got, dtype)
    q, dt2 = as_storage(ref, dtype)
    if dt != dt2 or g.shape != q.shape:
        raise ValueError("got and ref must match in dtype and shape")
    worst, bad = ctypes.c_double(0.0), ctypes.c_int64(0)
    _load().oracle_mixed_compare(g.ctypes.data, q.ctypes.data, g.size, dt, tol, tol_abs, ctypes.byref(worst),
                                 ctypes.byref(bad))
    return worst.value, bad.value


def add_rmsnorm_fp8(x, r, w, eps: float, dtype: int | None = None):
    """(q, scale, r_out): e4m3 codes as uint8 [T, H], float32 per-token scales [T], the rounded residual."""
    want_torch = hasattr(x, "detach")
    xs, dt = as_storage(x, dtype)
    rs, dt_r = as_storage(r, dtype)
    ws, dt_w = as_storage(w, dtype)
    if not (dt == dt_r == dt_w):
        raise TypeError("x, r and w must share one dtype")
    if xs.ndim != 2 or rs.shape != xs.shape or ws.shape != (xs.shape[1],):
        raise ValueError("expected x, r of shape [T, H] and w of shape [H]")
    T, H = xs.shape
    q = np.empty((T, H), dtype=np.uint8)
    scale = np.empty((T,), dtype=np.float32)
    r_out = np.empty_like(xs)
    rc = _load().oracle_add_rmsnorm_fp8(xs.ctypes.data, rs.ctypes.data, ws.ctypes.data, q.ctypes.data,
                                        scale.ctypes.data, r_out.ctypes.data, T, H, float(eps), dt)
    if rc != 0:
        raise RuntimeError(f"oracle_add_rmsnorm_fp8 failed with status {rc}")
    if want_torch:
        import torch
        return torch.from_numpy(q), torch.from_numpy(scale), to_torch(r_out, dt)
    return q, scale, r_out


def allreduce_add_rmsnorm(x_parts, r, w, eps: float, dtype: int | None = None, *, threads: int = 1):
    """y, r_out for x given as parts: x_parts [N, T, H] summed in binary32 in rank order, then the residual, then
    the norm.  Storage arrays for numpy input, torch tensors for torch input."""
    want_torch = hasattr(x_parts, "detach")
    xs, dt = as_storage(x_parts, dtype)
    rs, dt_r = as_storage(r, dtype)
    ws, dt_w = as_storage(w, dtype)
    if not (dt == dt_r == dt_w):
        raise TypeError("x_parts, r and w must share one dtype")
    if xs.ndim != 3 or xs.shape[0] < 1 or rs.shape != xs.shape[1:] or ws.shape != (xs.shape[2],):
        raise ValueError("expected x_parts of shape [N, T, H], r of shape [T, H] and w of shape [H]")
    N, T, H = xs.shape
    y = np.empty_like(rs)
    r_out = np.empty_like(rs)
    rc = _load().oracle_allreduce_add_rmsnorm(xs.ctypes.data, N, rs.ctypes.data, ws.ctypes.data, y.ctypes.data,
                                              r_out.ctypes.data, T, H, float(eps), dt, int(threads))
    if rc != 0:
        raise RuntimeError(f"oracle_allreduce_add_rmsnorm failed with status {rc}")
    if want_torch:
        return to_torch(y, dt), to_torch(r_out, dt)
    return y, r_out


def decode_e4m3(bits) -> np.ndarray:
    b = np.ascontiguousarray(bits, dtype=np.uint8)
    out = np.empty(b.shape, dtype=np.float64)
    _load().oracle_decode_e4m3(b.ctypes.data, out.ctypes.data, b.size)
    return out


def encode_e4m3(v) -> np.ndarray:
    a = np.ascontiguousarray(v, dtype=np.float64)
    out = np.empty(a.shape, dtype=np.uint8)
    _load().oracle_encode_e4m3(a.ctypes.data, out.ctypes.data, a.size)
    return out


def compare_e4m3(got, ref, tol_steps: int = 1):
    """(largest distance in e4m3 code steps, count beyond tol_steps) between two uint8 code arrays."""
    g = np.ascontiguousarray(got.numpy() if hasattr(got, "numpy") else got, dtype=np.uint8)
    q = np.ascontiguousarray(ref.numpy() if hasattr(ref, "numpy") else ref, dtype=np.uint8)
    if g.shape != q.shape:
        raise ValueError("got and ref must match in shape")
    worst, bad = ctypes.c_int32(0), ctypes.c_int64(0)
    _load().oracle_e4m3_compare(g.ctypes.data, q.ctypes.data, g.size, tol_steps, ctypes.byref(worst), ctypes.byref(bad))
    return worst.value, bad.value


def decode16(bits, dtype: int) -> np.ndarray:
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(b.shape, dtype=np.float64)
    _load().oracle_decode16(b.ctypes.data, out.ctypes.data, b.size, dtype)
    return out


def encode16_from_f64(v, dtype: int) -> np.ndarray:
    a = np.ascontiguousarray(v, dtype=np.float64)
    out = np.empty(a.shape, dtype=np.uint16)
    _load().oracle_encode16_from_f64(a.ctypes.data, out.ctypes.data, a.size, dtype)
    return out


def encode16_from_f32(v, dtype: int) -> np.ndarray:
    a = np.ascontiguousarray(v, dtype=np.float32)
    out = np.empty(a.shape, dtype=np.uint16)
    _load().oracle_encode16_from_f32(a.ctypes.data, out.ctypes.data, a.size, dtype)
    return out


def compare_y(got, ref, dtype: int | None = None, *, tol_ulp: int = 2, tol_rel: float = 1e-5,
              abs_floor: float = 1e-30):
    """Distance between a candidate y and the oracle's y.

    16-bit dtypes: (max ulp distance, count beyond tol_ulp).
    fp32: (max relative error, count beyond tol_rel)."""
    g, dt = as_storage(got, dtype)
    q, dt2 = as_storage(ref, dtype)
    if dt != dt2 or g.shape != q.shape:
        raise ValueError("got and ref must match in dtype and shape")
    bad = ctypes.c_int64(0)
    if dt == FP32:
        worst = ctypes.c_double(0.0)
        _load().oracle_rel_compare32(g.ctypes.data, q.ctypes.data, g.size, tol_rel, abs_floor,
                                     ctypes.byref(worst), ctypes.byref(bad))
        return worst.value, bad.value
    worst = ctypes.c_int32(0)
    _load().oracle_ulp_compare16(g.ctypes.data, q.ctypes.data, g.size, dt, tol_ulp,
                                 ctypes.byref(worst), ctypes.byref(bad))
    return worst.value, bad.value


def bit_mismatches(got, ref, dtype: int | None = None) -> int:
    """Number of elements whose bit patterns differ (the r' contract)."""
    g, dt = as_storage(got, dtype)
    q, _ = as_storage(ref, dtype)
    if dt == FP32:
        g, q = g.view(np.uint32), q.view(np.uint32)
    return int(np.count_nonzero(g != q))
