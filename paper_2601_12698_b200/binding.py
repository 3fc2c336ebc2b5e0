"""ctypes binding of librmsnorm_tuner.so: the same names as the C ABI, argument marshalling only.

Every step of the operator, of the feasible-region derivation and of the search runs inside the shared
library.  torch is used here for device memory, streams and dtype bookkeeping; there is no CPU or
PyTorch fall-back: if the library is missing, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, byref, c_char_p, c_double, c_float, c_int, c_int32, c_int64, c_void_p

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librmsnorm_tuner.so")
HEADER_PATH = os.path.join(os.path.dirname(_HERE), "include", "rmsnorm_tuner.h")

RT_BF16, RT_FP16, RT_FP32 = 0, 1, 2
RT_OP_ADD_RMSNORM, RT_OP_SILU_AND_MUL, RT_OP_MERGE_ATTN_STATES, RT_OP_ADD_RMSNORM_FP8 = 0, 1, 2, 3
RT_OP_ADD_RMSNORM_ALLREDUCE = 4
RT_MAX_PARTS = 8
RT_OPTION_PROGRAMMATIC_LAUNCH, RT_OPTION_TMA_WAIT_POLL_LIMIT, RT_OPTION_DEBUG_DROP_TMA_COPIES = 0, 1, 2
RT_STAGE_REG, RT_STAGE_SMEM_LDG, RT_STAGE_SMEM_TMA, RT_STAGE_REG_REALIGN, RT_STAGE_TMA_PIPELINE = 0, 1, 2, 3, 4
RT_REDUCE_SHFL, RT_REDUCE_SMEM, RT_REDUCE_CLUSTER = 0, 1, 2
RT_PRUNE_IDLE_THREADS, RT_PRUNE_DUPLICATES, RT_PRUNE_CLUSTER_WAVES, RT_PRUNE_IDLE_ROWS = 1, 2, 4, 8
RT_PRUNE_PIPELINE_STAGE = 16
RT_PRUNE_BYTES_IN_FLIGHT = 32
RT_PRUNE_DEFAULT = 63
RT_SEARCH_GUIDED, RT_SEARCH_EXHAUSTIVE = 0, 1
RT_CMP_BITS, RT_CMP_ULP16, RT_CMP_REL32 = 0, 1, 2
(RT_OK, RT_ERR_NULL, RT_ERR_DTYPE, RT_ERR_SHAPE, RT_ERR_ALIGN, RT_ERR_INFEASIBLE, RT_ERR_CUDA, RT_ERR_MISMATCH,
 RT_ERR_BUDGET, RT_ERR_DEVICE_TIMEOUT, RT_ERR_CAPACITY, RT_ERR_NO_DEVICE) = range(12)
PHASE_NAMES = {0: "seed", 1: "grid", 2: "climb", 3: "topk", 4: "sweep"}
STAGE_NAMES = {0: "reg", 1: "smem_ldg", 2: "smem_tma", 3: "reg_realign", 4: "tma_pipeline"}
REDUCE_NAMES = {0: "shfl", 1: "smem", 2: "cluster"}
DTYPE_CODES = {"bf16": RT_BF16, "fp16": RT_FP16, "fp32": RT_FP32}


class rt_params(Structure):
    _fields_ = [("threads_per_row", c_int32), ("rows_per_cta", c_int32), ("vec_bytes", c_int32),
                ("unroll", c_int32), ("stage", c_int32), ("reduce", c_int32), ("cluster_size", c_int32)]

    def as_dict(self) -> dict:
        return {k: int(getattr(self, k)) for k, _ in self._fields_}

    def key(self) -> tuple:
        return tuple(int(getattr(self, k)) for k, _ in self._fields_)

    def __repr__(self):
        return (f"theta(tpr={self.threads_per_row}, rpc={self.rows_per_cta}, vec={self.vec_bytes}, "
                f"unroll={self.unroll}, stage={STAGE_NAMES.get(self.stage, self.stage)}, "
                f"reduce={REDUCE_NAMES.get(self.reduce, self.reduce)}, cluster={self.cluster_size})")


def make_params(threads_per_row=256, rows_per_cta=1, vec_bytes=16, unroll=1, stage=RT_STAGE_REG,
                reduce=RT_REDUCE_SHFL, cluster_size=1) -> rt_params:
    return rt_params(threads_per_row, rows_per_cta, vec_bytes, unroll, stage, reduce, cluster_size)


class rt_shape(Structure):
    _fields_ = [("n_tokens", c_int64), ("hidden", c_int64), ("dtype", c_int32), ("min_ptr_align", c_int32),
                ("op", c_int32), ("head_dim", c_int32), ("n_parts", c_int32), ("reserved", c_int32)]


class rt_limits(Structure):
    _fields_ = [("sm_count", c_int32), ("warp_size", c_int32), ("max_threads_per_block", c_int32),
                ("max_threads_per_sm", c_int32), ("max_blocks_per_sm", c_int32), ("regs_per_block", c_int32),
                ("regs_per_sm", c_int32), ("max_regs_per_thread", c_int32), ("max_cluster_size", c_int32),
                ("have_device", c_int32), ("smem_per_block_optin", c_int64), ("smem_per_sm", c_int64),
                ("smem_reserved_per_block", c_int64), ("l2_bytes", c_int64)]


class rt_budget(Structure):
    _fields_ = [("max_evals", c_int32), ("warmup", c_int32), ("iters", c_int32), ("repeats", c_int32),
                ("top_k", c_int32), ("strategy", c_int32), ("heuristics", c_int32), ("use_graph", c_int32),
                ("seeds", POINTER(rt_params)), ("n_seeds", c_int32), ("preheat_ms", c_int32)]


class rt_workspace(Structure):
    _fields_ = [("x", c_void_p), ("r", c_void_p), ("w", c_void_p), ("y", c_void_p), ("r_out", c_void_p),
                ("y_ref", c_void_p), ("r_ref", c_void_p), ("n_ref_tokens", c_int64),
                ("ring_stride_bytes", c_int64), ("ring_sets", c_int32), ("eps", c_float), ("stream", c_void_p),
                ("aux", c_void_p), ("aux_out", c_void_p), ("aux_ref", c_void_p)]


class rt_eval_record(Structure):
    _fields_ = [("params", rt_params), ("phase", c_int32), ("eval_index", c_int32), ("status", c_int32),
                ("y_max_ulp", c_int32), ("y_bad", c_int64), ("r_bad", c_int64), ("y_max_rel", c_float),
                ("us", c_float), ("us_min_block", c_float), ("us_mean", c_float),
                ("occupancy_blocks_per_sm", c_int32), ("regs_per_thread", c_int32)]

    def as_dict(self) -> dict:
        d = {k: getattr(self, k) for k, _ in self._fields_ if k != "params"}
        d["params"] = self.params.as_dict()
        d["phase"] = PHASE_NAMES.get(self.phase, self.phase)
        return d


class rt_block_record(Structure):
    _fields_ = [("theta_index", c_int32), ("round", c_int32), ("us", c_float), ("reserved", c_int32),
                ("t_begin_s", c_double), ("t_end_s", c_double)]


class rt_result(Structure):
    _fields_ = [("best", rt_params), ("best_us", c_float), ("evals_used", c_int32), ("n_candidates", c_int32),
                ("n_log", c_int32), ("n_failed_gate", c_int32)]


class rt_spec_entry(Structure):
    _fields_ = [("shape", rt_shape), ("best", rt_params), ("best_us", c_float), ("reserved", c_int32)]


SOURCE_NAMES = {0: "table_exact", 1: "table_nearest", 2: "general", 3: "feasible_set"}

rt_evaluate_fn = ctypes.CFUNCTYPE(c_double, POINTER(rt_params), c_void_p)

_SIGNATURES = {
    "rmsnorm_template_launch": (c_int, [POINTER(rt_params), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                        c_int64, c_int64, c_float, c_int, c_void_p]),
    "silu_and_mul_template_launch": (c_int, [POINTER(rt_params), c_void_p, c_void_p, c_int64, c_int64, c_int, c_void_p]),
    "rmsnorm_fp8_template_launch": (c_int, [POINTER(rt_params), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                            c_int64, c_int64, c_float, c_int, c_void_p]),
    "rmsnorm_allreduce_template_launch": (c_int, [POINTER(rt_params), POINTER(c_void_p), c_int32, c_void_p, c_void_p,
                                                  POINTER(c_void_p), c_int32, POINTER(c_void_p), c_int32, c_int64,
                                                  c_int64, c_int64, c_float, c_int, c_void_p]),
    "rt_kernel_instance_parts": (c_int32, [c_int32]),
    "rt_set_option": (c_int, [c_int32, c_int32]),
    "rt_get_option": (c_int32, [c_int32]),
    "merge_attn_states_template_launch": (c_int, [POINTER(rt_params), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                                  c_void_p, c_int64, c_int64, c_int64, c_int, c_void_p]),
    "rmsnorm_template_launch_traced": (c_int, [POINTER(rt_params), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                               c_int64, c_int64, c_float, c_int, c_void_p, c_int64, c_void_p]),
    "rmsnorm_trace_words": (c_int64, [POINTER(rt_params), c_int64, c_int64, c_int]),
    "rmsnorm_template_run_host": (c_int, [POINTER(rt_params), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                          c_int64, c_int64, c_float, c_int, c_void_p, c_int64, c_int64, c_void_p]),
    "rmsnorm_host_workspace_bytes": (c_int64, [c_int64, c_int64, c_int, c_int64]),
    "rt_query_limits": (c_int, [POINTER(rt_limits)]),
    "rt_limits_sm100_nominal": (None, [POINTER(rt_limits)]),
    "tuner_derive_feasible": (c_int, [POINTER(rt_shape), POINTER(rt_params), c_int32, POINTER(c_int32)]),
    "tuner_derive_feasible_ex": (c_int, [POINTER(rt_shape), POINTER(rt_limits), c_int32, POINTER(rt_params),
                                         c_int32, POINTER(c_int32)]),
    "tuner_check_params": (c_int, [POINTER(rt_shape), POINTER(rt_limits), POINTER(rt_params)]),
    "tuner_raw_grid": (c_int, [POINTER(rt_shape), POINTER(rt_params), c_int32, POINTER(c_int32)]),
    "tuner_derive_counts": (c_int, [POINTER(rt_shape), POINTER(rt_limits), c_int32, POINTER(c_int32), c_int32]),
    "tuner_search": (c_int, [POINTER(rt_shape), POINTER(rt_budget), POINTER(rt_workspace), POINTER(rt_result),
                             POINTER(rt_eval_record), c_int32]),
    "tuner_search_with": (c_int, [POINTER(rt_shape), POINTER(rt_limits), POINTER(rt_budget), rt_evaluate_fn, c_void_p,
                                  POINTER(rt_result), POINTER(rt_eval_record), c_int32]),
    "tuner_evaluate": (c_int, [POINTER(rt_shape), POINTER(rt_params), POINTER(rt_budget), POINTER(rt_workspace),
                               POINTER(rt_eval_record)]),
    "tuner_retest_interleaved": (c_int, [POINTER(rt_shape), POINTER(rt_params), c_int32, POINTER(rt_budget),
                                         POINTER(rt_workspace), c_int32, POINTER(rt_eval_record),
                                         POINTER(rt_block_record), POINTER(c_int32)]),
    "tuner_select_general": (c_int, [POINTER(c_float), c_int32, c_int32, POINTER(c_int32), POINTER(c_float),
                                     POINTER(c_float)]),
    "tuner_table_lookup": (c_int, [POINTER(rt_spec_entry), c_int32, POINTER(rt_params), POINTER(rt_shape),
                                   POINTER(rt_limits), POINTER(rt_params), POINTER(c_int32)]),
    "rmsnorm_launch_auto": (c_int, [POINTER(rt_spec_entry), c_int32, POINTER(rt_params), c_void_p, c_void_p, c_void_p,
                                    c_void_p, c_void_p, c_int64, c_int64, c_float, c_int, c_void_p, POINTER(rt_params)]),
    "tuner_launch_floor": (c_int, [POINTER(rt_budget), c_void_p, POINTER(c_float)]),
    "tuner_compare": (c_int, [c_void_p, c_void_p, c_int64, c_int, c_int, c_double, POINTER(c_double),
                              POINTER(c_int64), c_void_p]),
    "tuner_compare_e4m3": (c_int, [c_void_p, c_void_p, c_int64, c_int32, POINTER(c_int32), POINTER(c_int64), c_void_p]),
    "tuner_compare_mixed": (c_int, [c_void_p, c_void_p, c_int64, c_int, c_double, c_double, POINTER(c_double),
                                    POINTER(c_int64), c_void_p]),
    "tuner_compare_static": (c_int, [c_void_p, c_void_p, c_int64, c_int, c_int, c_double, POINTER(c_double),
                                     POINTER(c_int64), c_void_p]),
    "rt_status_string": (c_char_p, [c_int]),
    "rt_last_error": (c_char_p, []),
    "rt_device_status": (c_int, []),
    "rt_num_kernel_instances": (c_int32, []),
    "rt_kernel_instance": (c_int, [c_int32] + [POINTER(c_int32)] * 6),
    "rt_kernel_instance_op": (c_int32, [c_int32]),
    "rt_launch_count": (c_int64, []),
    "rt_shutdown": (None, []),
}
EXPORTED = tuple(_SIGNATURES)

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2601_12698_b200.build` "
                      "(there is no fall-back path)")
lib = ctypes.CDLL(LIB_PATH)
for _name, (_res, _args) in _SIGNATURES.items():
    _fn = getattr(lib, _name)
    _fn.restype = _res
    _fn.argtypes = _args


class TunerError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        text = lib.rt_status_string(status).decode()
        detail = lib.rt_last_error().decode()
        super().__init__(f"{where}: status {status} ({text}){': ' + detail if detail else ''}")


def _check(status: int, where: str):
    if status != RT_OK:
        raise TunerError(status, where)


def _dtype_code(t) -> int:
    import torch
    if isinstance(t, int):
        return t
    return {torch.bfloat16: RT_BF16, torch.float16: RT_FP16, torch.float32: RT_FP32}[t.dtype]


def _stream_ptr(stream=None) -> int:
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def _ptr_align(*tensors) -> int:
    bits = 256
    for t in tensors:
        bits |= t.data_ptr()
    return bits & -bits


def shape_of(n_tokens: int, hidden: int, dtype, min_ptr_align: int = 256, op: int = RT_OP_ADD_RMSNORM,
             head_dim: int = 0, n_parts: int = 0) -> rt_shape:
    """hidden is the output row width (d for silu_and_mul, heads * head_dim for merge_attn_states); n_parts is the
    number of partial inputs of the all-reduce-fused norm."""
    code = DTYPE_CODES[dtype] if isinstance(dtype, str) else int(dtype)
    return rt_shape(n_tokens, hidden, code, min_ptr_align, op, head_dim, n_parts, 0)


def sm100_nominal_limits() -> rt_limits:
    L = rt_limits()
    lib.rt_limits_sm100_nominal(byref(L))
    return L


def rt_query_limits() -> rt_limits:
    L = rt_limits()
    _check(lib.rt_query_limits(byref(L)), "rt_query_limits")
    return L


# ---- 1. the template kernel -----------------------------------------------------------------------------

def rmsnorm_template_launch(params: rt_params, x, r, w, y, r_out, eps: float, stream=None) -> None:
    """Launch theta on device tensors (asynchronous on the stream).  y may be x, r_out may be r."""
    if not (x.is_cuda and r.is_cuda and w.is_cuda and y.is_cuda and r_out.is_cuda):
        raise ValueError("rmsnorm_template_launch takes CUDA tensors")
    for t in (x, r, y, r_out):
        if not t.is_contiguous() or t.shape != x.shape or t.dtype != x.dtype:
            raise ValueError("x, r, y, r_out must be contiguous and alike")
    n_tokens, hidden = x.shape
    if w.shape != (hidden,) or w.dtype != x.dtype or not w.is_contiguous():
        raise ValueError("w must be a contiguous [hidden] tensor of the same dtype")
    _check(lib.rmsnorm_template_launch(byref(params), x.data_ptr(), r.data_ptr(), w.data_ptr(), y.data_ptr(),
                                       r_out.data_ptr(), n_tokens, hidden, eps, _dtype_code(x), _stream_ptr(stream)),
           "rmsnorm_template_launch")


RT_TRACE_WORDS = 8


def rmsnorm_template_launch_traced(params: rt_params, x, r, w, y, r_out, eps: float, trace, stream=None) -> None:
    """rmsnorm_template_launch through an instrumented instance; `trace` is an int64 device tensor of at least
    rmsnorm_trace_words(...) elements that receives RT_TRACE_WORDS words per CTA."""
    n_tokens, hidden = x.shape
    _check(lib.rmsnorm_template_launch_traced(byref(params), x.data_ptr(), r.data_ptr(), w.data_ptr(), y.data_ptr(),
                                              r_out.data_ptr(), n_tokens, hidden, eps, _dtype_code(x), trace.data_ptr(),
                                              trace.numel(), _stream_ptr(stream)), "rmsnorm_template_launch_traced")


def rmsnorm_trace_words(params: rt_params, n_tokens: int, hidden: int, dtype) -> int:
    code = DTYPE_CODES[dtype] if isinstance(dtype, str) else int(dtype)
    return int(lib.rmsnorm_trace_words(byref(params), n_tokens, hidden, code))


def silu_and_mul_template_launch(params: rt_params, x, out, stream=None) -> None:
    """out[t, j] = silu(x[t, j]) * x[t, d + j] on device tensors x [T, 2d] and out [T, d] (asynchronous)."""
    if not (x.is_cuda and out.is_cuda and x.is_contiguous() and out.is_contiguous()):
        raise ValueError("silu_and_mul_template_launch takes contiguous CUDA tensors")
    n_tokens, d = out.shape
    if x.shape != (n_tokens, 2 * d) or x.dtype != out.dtype:
        raise ValueError("x must be [n_tokens, 2*d] of the output's dtype")
    _check(lib.silu_and_mul_template_launch(byref(params), x.data_ptr(), out.data_ptr(), n_tokens, d, _dtype_code(x),
                                            _stream_ptr(stream)), "silu_and_mul_template_launch")


def rmsnorm_fp8_template_launch(params: rt_params, x, r, w, q, scale, r_out, eps: float, stream=None) -> None:
    """add_rmsnorm with e4m3 output: q uint8 [T, H], scale float32 [T], r_out like x (device tensors; asynchronous)."""
    import torch
    n_tokens, hidden = x.shape
    ok = (all(t.is_cuda and t.is_contiguous() for t in (x, r, w, q, scale, r_out)) and r.shape == x.shape
          and r_out.shape == x.shape and q.shape == x.shape and q.dtype == torch.uint8 and scale.shape == (n_tokens,)
          and scale.dtype == torch.float32 and w.shape == (hidden,) and r.dtype == x.dtype == w.dtype == r_out.dtype)
    if not ok:
        raise ValueError("rmsnorm_fp8_template_launch: tensors of the wrong device, layout, shape or dtype")
    _check(lib.rmsnorm_fp8_template_launch(byref(params), x.data_ptr(), r.data_ptr(), w.data_ptr(), q.data_ptr(),
                                           scale.data_ptr(), r_out.data_ptr(), n_tokens, hidden, eps, _dtype_code(x),
                                           _stream_ptr(stream)), "rmsnorm_fp8_template_launch")


def rmsnorm_allreduce_template_launch(params: rt_params, x_parts, r, w, y_outs, r_outs, row_begin: int, row_count: int,
                                      eps: float, stream=None) -> None:
    """The tensor-parallel form of add_rmsnorm on rows [row_begin, row_begin + row_count): x_parts is a list of 2, 4
    or 8 device tensors [T, H] (one partial x per rank, each addressable from the current device); y_outs and r_outs
    are lists of 1..8 destination tensors [T, H]: every y destination receives those rows of y, every r_out
    destination those rows of the new residual.  Asynchronous."""
    n_rows, hidden = r.shape
    tensors = list(x_parts) + [r] + list(y_outs) + list(r_outs)
    ok = (all(t.is_cuda and t.is_contiguous() and t.shape == (n_rows, hidden) and t.dtype == r.dtype for t in tensors)
          and w.is_cuda and w.is_contiguous() and w.shape == (hidden,) and w.dtype == r.dtype
          and 0 <= row_begin and row_begin + row_count <= n_rows)
    if not ok:
        raise ValueError("rmsnorm_allreduce_template_launch: tensors of the wrong device, layout, shape or dtype, "
                         "or rows out of range")
    xp = (c_void_p * len(x_parts))(*[t.data_ptr() for t in x_parts])
    yo = (c_void_p * len(y_outs))(*[t.data_ptr() for t in y_outs])
    ro = (c_void_p * len(r_outs))(*[t.data_ptr() for t in r_outs])
    _check(lib.rmsnorm_allreduce_template_launch(byref(params), xp, len(x_parts), r.data_ptr(), w.data_ptr(), yo,
                                                 len(y_outs), ro, len(r_outs), row_begin, row_count, hidden, eps,
                                                 _dtype_code(r), _stream_ptr(stream)), "rmsnorm_allreduce_template_launch")


def merge_attn_states_template_launch(params: rt_params, v_a, s_a, v_b, s_b, v_out, s_out, stream=None) -> None:
    """Merge two partial attention results (device tensors; v: [n, h, d], s: float32 [n, h]); asynchronous."""
    import torch
    n, h, d = v_a.shape
    for t in (v_a, v_b, v_out):
        if not (t.is_cuda and t.is_contiguous() and t.shape == (n, h, d) and t.dtype == v_a.dtype):
            raise ValueError("v_a, v_b, v_out must be contiguous CUDA tensors of one shape [n, h, d] and dtype")
    for t in (s_a, s_b, s_out):
        if not (t.is_cuda and t.is_contiguous() and t.shape == (n, h) and t.dtype == torch.float32):
            raise ValueError("s_a, s_b, s_out must be contiguous float32 CUDA tensors of shape [n, h]")
    _check(lib.merge_attn_states_template_launch(byref(params), v_a.data_ptr(), s_a.data_ptr(), v_b.data_ptr(),
                                                 s_b.data_ptr(), v_out.data_ptr(), s_out.data_ptr(), n, h, d,
                                                 _dtype_code(v_a), _stream_ptr(stream)),
           "merge_attn_states_template_launch")


def rmsnorm_host_workspace_bytes(n_tokens: int, hidden: int, dtype, chunk_tokens: int = 0) -> int:
    code = DTYPE_CODES[dtype] if isinstance(dtype, str) else int(dtype)
    return int(lib.rmsnorm_host_workspace_bytes(n_tokens, hidden, code, chunk_tokens))


def rmsnorm_template_run_host(params: rt_params, x, r, w, y, r_out, eps: float, workspace, chunk_tokens: int = 0,
                              stream=None) -> None:
    """The operator on host (ideally pinned) tensors through a device workspace; returns when y and r_out
    are complete in host memory."""
    for t in (x, r, w, y, r_out):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("rmsnorm_template_run_host takes contiguous host tensors")
    n_tokens, hidden = x.shape
    _check(lib.rmsnorm_template_run_host(byref(params), x.data_ptr(), r.data_ptr(), w.data_ptr(), y.data_ptr(),
                                         r_out.data_ptr(), n_tokens, hidden, eps, _dtype_code(x),
                                         workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                         chunk_tokens, _stream_ptr(stream)),
           "rmsnorm_template_run_host")


# ---- 2. the feasible region ---------------------------------------------------------------------------------

def _collect(call, where: str) -> list[rt_params]:
    n = c_int32(0)
    _check(call(None, 0, byref(n)), where)
    while True:
        cap = max(1, n.value)
        arr = (rt_params * cap)()
        _check(call(arr, cap, byref(n)), where)
        if n.value <= cap:
            return [rt_params.from_buffer_copy(arr[i]) for i in range(n.value)]


def tuner_derive_feasible(shape: rt_shape, limits: rt_limits | None = None,
                          heuristics: int = RT_PRUNE_DEFAULT) -> list[rt_params]:
    """Theta_feasible for a shape.  limits=None asks the current device."""
    lim = byref(limits) if limits is not None else None
    return _collect(lambda out, cap, n: lib.tuner_derive_feasible_ex(byref(shape), lim, heuristics, out, cap, n),
                    "tuner_derive_feasible")


def tuner_raw_grid(shape: rt_shape) -> list[rt_params]:
    return _collect(lambda out, cap, n: lib.tuner_raw_grid(byref(shape), out, cap, n), "tuner_raw_grid")


def tuner_derive_counts(shape: rt_shape, limits: rt_limits | None = None, heuristics: int = RT_PRUNE_DEFAULT) -> dict:
    counts = (c_int32 * 11)()
    lim = byref(limits) if limits is not None else None
    _check(lib.tuner_derive_counts(byref(shape), lim, heuristics, counts, 11), "tuner_derive_counts")
    names = ["unused", "arguments", "threads_per_cta", "alignment", "registers", "shared_memory", "cluster",
             "grid", "heuristics", "feasible", "raw"]
    return {k: int(v) for k, v in zip(names, counts) if k != "unused"}


def tuner_check_params(shape: rt_shape, params: rt_params, limits: rt_limits | None = None) -> int:
    lim = byref(limits) if limits is not None else None
    return int(lib.tuner_check_params(byref(shape), lim, byref(params)))


# ---- 3. search ------------------------------------------------------------------------------------------------

def make_budget(max_evals=64, warmup=20, iters=100, repeats=3, top_k=5, strategy=RT_SEARCH_GUIDED,
                heuristics=RT_PRUNE_DEFAULT, use_graph=False, seeds=None, preheat_ms=0) -> rt_budget:
    b = rt_budget(max_evals, warmup, iters, repeats, top_k, strategy, heuristics, int(use_graph), None, 0, int(preheat_ms))
    if seeds:
        arr = (rt_params * len(seeds))(*seeds)
        b._seed_storage = arr  # keep alive
        b.seeds = ctypes.cast(arr, POINTER(rt_params))
        b.n_seeds = len(seeds)
    return b


def make_workspace(x, r, w, y, r_out, y_ref, r_ref, eps: float, n_ref_tokens: int | None = None, ring_sets: int = 1,
                   ring_stride_bytes: int = 0, stream=None, aux=None, aux_out=None, aux_ref=None) -> rt_workspace:
    """Device tensors for the tuner.  With ring_sets > 1, x, r, y, r_out are [ring_sets, T, H] and the
    references cover set 0.  For silu_and_mul pass r = w = r_out = r_ref = None; for merge_attn_states
    x = v_a, r = v_b, w = s_a, aux = s_b, y = v_out, r_out = s_out; for the fp8-output norm y = q (uint8),
    aux_out = scale, aux_ref its reference."""
    T = x.shape[-2]
    ptr = lambda t: t.data_ptr() if t is not None else None
    return rt_workspace(ptr(x), ptr(r), ptr(w), ptr(y), ptr(r_out), ptr(y_ref), ptr(r_ref),
                        n_ref_tokens if n_ref_tokens is not None else T, ring_stride_bytes,
                        ring_sets, eps, _stream_ptr(stream), ptr(aux), ptr(aux_out), ptr(aux_ref))


def tuner_search(shape: rt_shape, budget: rt_budget, ws: rt_workspace, log_cap: int = 4096):
    """Returns (rt_result, [rt_eval_record...])."""
    res = rt_result()
    log = (rt_eval_record * log_cap)()
    st = lib.tuner_search(byref(shape), byref(budget), byref(ws), byref(res), log, log_cap)
    _check(st, "tuner_search")
    return res, [rt_eval_record.from_buffer_copy(log[i]) for i in range(res.n_log)]


def tuner_search_with(shape: rt_shape, limits: rt_limits, budget: rt_budget, evaluate, log_cap: int = 4096):
    """The search over a Python cost function evaluate(theta) -> microseconds (negative: gate failed)."""
    res = rt_result()
    log = (rt_eval_record * log_cap)()
    cb = rt_evaluate_fn(lambda p, _user: float(evaluate(p.contents)))
    st = lib.tuner_search_with(byref(shape), byref(limits), byref(budget), cb, None, byref(res), log, log_cap)
    _check(st, "tuner_search_with")
    return res, [rt_eval_record.from_buffer_copy(log[i]) for i in range(res.n_log)]


def tuner_evaluate(shape: rt_shape, params: rt_params, budget: rt_budget, ws: rt_workspace) -> rt_eval_record:
    rec = rt_eval_record()
    _check(lib.tuner_evaluate(byref(shape), byref(params), byref(budget), byref(ws), byref(rec)), "tuner_evaluate")
    return rec


def tuner_retest_interleaved(shape: rt_shape, thetas, budget: rt_budget, ws: rt_workspace, rounds: int):
    """Several thetas re-timed side by side, round-robin block by block.  Returns ([rt_eval_record per theta],
    [rt_block_record per block, in the order the blocks ran])."""
    n = len(thetas)
    arr = (rt_params * n)(*thetas)
    recs = (rt_eval_record * n)()
    blocks = (rt_block_record * (n * rounds))()
    ran = c_int32(0)
    _check(lib.tuner_retest_interleaved(byref(shape), arr, n, byref(budget), byref(ws), rounds, recs, blocks, byref(ran)),
           "tuner_retest_interleaved")
    return ([rt_eval_record.from_buffer_copy(recs[i]) for i in range(n)],
            [rt_block_record.from_buffer_copy(blocks[i]) for i in range(ran.value)])


def tuner_launch_floor(budget: rt_budget, stream=None) -> float:
    """Microseconds per launch of an empty kernel under the budget's timing protocol."""
    us = c_float(0.0)
    _check(lib.tuner_launch_floor(byref(budget), _stream_ptr(stream), byref(us)), "tuner_launch_floor")
    return us.value


def tuner_compare(got, ref, mode: int, tol: float = 0.0, stream=None):
    """(max_err, n_bad) between two device tensors of one dtype."""
    if got.shape != ref.shape or got.dtype != ref.dtype:
        raise ValueError("got and ref must match")
    worst, bad = c_double(0.0), c_int64(0)
    _check(lib.tuner_compare(got.data_ptr(), ref.data_ptr(), got.numel(), _dtype_code(got), mode, tol, byref(worst),
                             byref(bad), _stream_ptr(stream)), "tuner_compare")
    return worst.value, bad.value


def tuner_compare_e4m3(got, ref, tol_steps: int = 1, stream=None):
    """(largest distance in e4m3 code steps, elements beyond tol_steps) between two uint8 device tensors."""
    if got.shape != ref.shape:
        raise ValueError("got and ref must match")
    worst, bad = c_int32(0), c_int64(0)
    _check(lib.tuner_compare_e4m3(got.data_ptr(), ref.data_ptr(), got.numel(), tol_steps, byref(worst), byref(bad),
                                  _stream_ptr(stream)), "tuner_compare_e4m3")
    return worst.value, bad.value


def tuner_compare_mixed(got, ref, tol: float, tol_abs: float, stream=None):
    """(largest absolute difference, failing elements): pass within tol (ulps / relative) OR tol_abs absolutely."""
    if got.shape != ref.shape or got.dtype != ref.dtype:
        raise ValueError("got and ref must match")
    worst, bad = c_double(0.0), c_int64(0)
    _check(lib.tuner_compare_mixed(got.data_ptr(), ref.data_ptr(), got.numel(), _dtype_code(got), tol, tol_abs,
                                   byref(worst), byref(bad), _stream_ptr(stream)), "tuner_compare_mixed")
    return worst.value, bad.value


def tuner_compare_static(got, ref, mode: int, tol: float = 0.0, stream=None):
    """tuner_compare for callers that must not allocate: same result, accumulator in a fixed device array
    (shared by all calls on the device, so calls must not overlap on the GPU)."""
    if got.shape != ref.shape or got.dtype != ref.dtype:
        raise ValueError("got and ref must match")
    worst, bad = c_double(0.0), c_int64(0)
    _check(lib.tuner_compare_static(got.data_ptr(), ref.data_ptr(), got.numel(), _dtype_code(got), mode, tol,
                                    byref(worst), byref(bad), _stream_ptr(stream)), "tuner_compare_static")
    return worst.value, bad.value


# ---- 4. general configuration and specialised table -------------------------------------------------------------

def tuner_select_general(times_us) -> tuple[int, float, list[float]]:
    """times_us[c][x] -> (index of theta_gen, its geometric-mean score, every candidate's score)."""
    n_c, n_x = len(times_us), len(times_us[0])
    flat = (c_float * (n_c * n_x))(*[float(v) for row in times_us for v in row])
    best, score, scores = c_int32(-1), c_float(0.0), (c_float * n_c)()
    _check(lib.tuner_select_general(flat, n_c, n_x, byref(best), byref(score), scores), "tuner_select_general")
    return best.value, score.value, list(scores)


class SpecTable:
    """D_spec and theta_gen as the C arrays the library consumes, with JSON persistence (marshalling only).

    Entries of every kernel (rt_shape.op) live in one table; there is one general configuration per kernel."""

    def __init__(self, entries=(), general: rt_params | None = None, device_name: str = "", generals: dict | None = None):
        self.entries = list(entries)  # [(rt_shape, rt_params, best_us)]
        self.generals = dict(generals or {})  # rt_op -> rt_params
        if general is not None:
            self.generals[RT_OP_ADD_RMSNORM] = general
        self.device_name = device_name
        self._pack()

    @property
    def general(self) -> rt_params | None:
        return self.generals.get(RT_OP_ADD_RMSNORM)

    def _pack(self):
        self._arr = (rt_spec_entry * max(1, len(self.entries)))()
        for i, (shape, theta, us) in enumerate(self.entries):
            self._arr[i] = rt_spec_entry(shape, theta, us, 0)

    def add(self, shape: rt_shape, theta: rt_params, best_us: float):
        self.entries.append((shape, theta, best_us))
        self._pack()

    def lookup(self, shape: rt_shape, limits: rt_limits | None = None):
        out, src = rt_params(), c_int32(-1)
        general = self.generals.get(int(shape.op))
        _check(lib.tuner_table_lookup(self._arr, len(self.entries), byref(general) if general else None,
                                      byref(shape), byref(limits) if limits is not None else None, byref(out),
                                      byref(src)), "tuner_table_lookup")
        return out, SOURCE_NAMES[src.value]

    def launch(self, x, r, w, y, r_out, eps: float, stream=None) -> rt_params:
        """rmsnorm_launch_auto on device tensors; returns the theta that was launched."""
        n_tokens, hidden = x.shape
        used = rt_params()
        general = self.general
        _check(lib.rmsnorm_launch_auto(self._arr, len(self.entries), byref(general) if general else None,
                                       x.data_ptr(), r.data_ptr(), w.data_ptr(), y.data_ptr(), r_out.data_ptr(),
                                       n_tokens, hidden, eps, _dtype_code(x), _stream_ptr(stream), byref(used)),
               "rmsnorm_launch_auto")
        return used

    def launch_silu_and_mul(self, x, out, stream=None) -> rt_params:
        """Table lookup (in the library) for this shape, then silu_and_mul_template_launch."""
        n_tokens, d = out.shape
        theta, _ = self.lookup(shape_of(n_tokens, d, _dtype_code(out), _ptr_align(x, out), op=RT_OP_SILU_AND_MUL))
        silu_and_mul_template_launch(theta, x, out, stream)
        return theta

    def launch_merge_attn_states(self, v_a, s_a, v_b, s_b, v_out, s_out, stream=None) -> rt_params:
        n, h, d = v_a.shape
        theta, _ = self.lookup(shape_of(n, h * d, _dtype_code(v_a), _ptr_align(v_a, v_b, v_out),
                                        op=RT_OP_MERGE_ATTN_STATES, head_dim=d))
        merge_attn_states_template_launch(theta, v_a, s_a, v_b, s_b, v_out, s_out, stream)
        return theta

    def launch_rmsnorm_fp8(self, x, r, w, q, scale, r_out, eps: float, stream=None) -> rt_params:
        n_tokens, hidden = x.shape
        theta, _ = self.lookup(shape_of(n_tokens, hidden, _dtype_code(x), _ptr_align(x, r, w, r_out), op=RT_OP_ADD_RMSNORM_FP8))
        rmsnorm_fp8_template_launch(theta, x, r, w, q, scale, r_out, eps, stream)
        return theta

    def launch_rmsnorm_allreduce(self, x_parts, r, w, y_outs, r_outs, row_begin: int, row_count: int, eps: float,
                                 stream=None) -> rt_params:
        """The tensor-parallel form of the norm with the table's theta for (row_count, hidden, parts)."""
        n_rows, hidden = r.shape
        shape = shape_of(max(1, row_count), hidden, _dtype_code(r), _ptr_align(*x_parts, r, w, *y_outs, *r_outs),
                         op=RT_OP_ADD_RMSNORM_ALLREDUCE, n_parts=len(x_parts))
        theta, _ = self.lookup(shape)
        rmsnorm_allreduce_template_launch(theta, x_parts, r, w, y_outs, r_outs, row_begin, row_count, eps, stream)
        return theta

    def to_json(self) -> dict:
        names = {v: k for k, v in DTYPE_CODES.items()}
        return {"device": self.device_name, "general": self.general.as_dict() if self.general else None,
                "generals": {str(op): th.as_dict() for op, th in sorted(self.generals.items())},
                "specialised": [{"dtype": names[s.dtype], "n_tokens": int(s.n_tokens), "hidden": int(s.hidden),
                                 "op": int(s.op), "head_dim": int(s.head_dim), "n_parts": int(s.n_parts), "theta": t.as_dict(), "us": round(float(us), 3)}
                                for s, t, us in self.entries]}

    @classmethod
    def default(cls) -> "SpecTable":
        """The table shipped with the package (tuned on a B200 with ``python -m paper_2601_12698_b200.tune``)."""
        import json
        with open(os.path.join(_HERE, "tables", "b200_default.json")) as f:
            return cls.from_json(json.load(f))

    @classmethod
    def from_json(cls, d: dict) -> "SpecTable":
        fields = [k for k, _ in rt_params._fields_]
        mk = lambda t: rt_params(*[int(t[k]) for k in fields])
        entries = [(shape_of(e["n_tokens"], e["hidden"], e["dtype"], op=int(e.get("op", 0)),
                             head_dim=int(e.get("head_dim", 0)), n_parts=int(e.get("n_parts", 0))), mk(e["theta"]), float(e["us"]))
                   for e in d.get("specialised", [])]
        generals = {int(op): mk(th) for op, th in (d.get("generals") or {}).items()}
        return cls(entries, mk(d["general"]) if d.get("general") else None, d.get("device", ""), generals)


def rt_device_status() -> int:
    return int(lib.rt_device_status())


def rt_launch_count() -> int:
    return int(lib.rt_launch_count())


def kernel_instances() -> list[dict]:
    out = []
    vals = [c_int32() for _ in range(6)]
    for i in range(lib.rt_num_kernel_instances()):
        _check(lib.rt_kernel_instance(i, *[byref(v) for v in vals]), "rt_kernel_instance")
        out.append(dict(zip(("dtype", "vec_bytes", "stage", "reduce", "unroll", "reg_vectors"), (v.value for v in vals))))
        out[-1]["op"] = int(lib.rt_kernel_instance_op(i))
        out[-1]["parts"] = int(lib.rt_kernel_instance_parts(i))
    return out


def rt_shutdown() -> None:
    lib.rt_shutdown()
