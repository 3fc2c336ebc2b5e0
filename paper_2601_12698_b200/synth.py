"""Seeded synthetic inputs for the fused residual-add + RMSNorm workloads.

This module only draws random numbers and converts them to the storage type.
It holds none of the operator's arithmetic, so both the CPU oracle's tests and
the CUDA path's tests feed from it without sharing anything else.

Generator.  Counter-based Philox-4x64 (numpy's ``Philox`` bit generator).  The
key is ``(seed, tensor_id)`` and the third counter word is the index of a block
of ``ROWS_PER_BLOCK`` rows, so any row block can be regenerated on its own:
the first rows of a tensor do not depend on how many rows follow, and a sample
of rows of a very large workload can be re-drawn for a row-by-row check.

Distributions.  ``x`` and ``r``: N(0, sigma) element-wise; with probability
``outlier_p`` an element is *replaced* by a draw from N(0, outlier_sigma).
``w``: N(w_mean, w_sigma).  The second argument of every normal is a standard
deviation.  Values are drawn in float32 and converted to the storage dtype by
``torch.Tensor.to`` (round to nearest even).

The workload table mirrors the shapes of the paper's Experimental Setup
("Kernels": hidden sizes typical of LLaMA-class models, fp32 and fp16/bf16) as
five named configurations; no dataset is involved.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field

import numpy as np
import torch

ROWS_PER_BLOCK = 64
TENSOR_X, TENSOR_R, TENSOR_W, TENSOR_GATE_UP, TENSOR_LSE_A, TENSOR_LSE_B = 0, 1, 2, 3, 4, 5
TENSOR_PART0 = 16  # partial inputs of the tensor-parallel norm: tensor ids 16, 17, ...

TORCH_DTYPES = {"bf16": torch.bfloat16, "fp16": torch.float16, "fp32": torch.float32}
DTYPE_CODES = {"bf16": 0, "fp16": 1, "fp32": 2}
DTYPE_BYTES = {"bf16": 2, "fp16": 2, "fp32": 4}


@dataclass(frozen=True)
class Dist:
    sigma: float = 1.0
    outlier_p: float = 0.0
    outlier_sigma: float = 50.0
    w_mean: float = 1.0
    w_sigma: float = 0.1


@dataclass(frozen=True)
class Workload:
    name: str
    dtype: str
    n_tokens: int
    hidden: int
    seed: int
    dist: Dist = field(default_factory=Dist)
    eps: float = 1e-6
    op: str = "add_rmsnorm"  # "silu_and_mul": hidden is d, the output width; "merge_attn_states": hidden = heads * head_dim
    head_dim: int = 0
    n_parts: int = 0  # "add_rmsnorm_allreduce": partial inputs per element (the tensor-parallel group size)

    @property
    def elements(self) -> int:
        return self.n_tokens * self.hidden

    @property
    def algorithmic_bytes(self) -> int:
        """Bytes the operator must move.  add_rmsnorm: read x, read r, write r', write y, w once.
        silu_and_mul: read gate, read value, write out."""
        b = DTYPE_BYTES[self.dtype]
        if self.op == "silu_and_mul":
            return 3 * b * self.elements
        if self.op == "add_rmsnorm_fp8":  # read x, r; write r' and one byte of q per element; w once; a scale per token
            return (3 * b + 1) * self.elements + b * self.hidden + 4 * self.n_tokens
        if self.op == "merge_attn_states":  # v_a, v_b in, v_out out; s_a, s_b in, s_out out (binary32 per head)
            return 3 * b * self.elements + 3 * 4 * self.n_tokens * (self.hidden // self.head_dim)
        if self.op == "add_rmsnorm_allreduce":  # n_parts partial x, r; write r' and y once; w once
            return (self.n_parts + 3) * b * self.elements + b * self.hidden
        return 4 * b * self.elements + b * self.hidden

    @property
    def nominal_bytes(self) -> int:
        """add_rmsnorm: three reads and two writes per element (w counted as a full stream)."""
        if self.op != "add_rmsnorm":
            return self.algorithmic_bytes
        return 5 * DTYPE_BYTES[self.dtype] * self.elements


_PREFILL_DIST = Dist(sigma=2.0, outlier_p=0.01, outlier_sigma=50.0)


def workloads() -> dict[str, Workload]:
    """The five benchmark configurations, keyed by name."""
    out: dict[str, Workload] = {}

    def add(wl: Workload):
        out[wl.name] = wl

    add(Workload("c1_bf16_128x4096", "bf16", 128, 4096, seed=0))
    for t in (1, 4, 16, 64, 256):
        add(Workload(f"c2_decode_bf16_{t}x4096", "bf16", t, 4096, seed=1))
    add(Workload("c3_prefill_bf16_16384x8192", "bf16", 16384, 8192, seed=2, dist=_PREFILL_DIST))
    for h in (5120, 7168, 6152):
        add(Workload(f"c4_fp16_8192x{h}", "fp16", 8192, h, seed=3))
    add(Workload("c4x_fp16_8192x6148", "fp16", 8192, 6148, seed=3))
    # rows that are only 4- and 2-byte multiples: no 8-byte vector divides them (narrow fall-back or the ragged-row stage)
    add(Workload("c4x_fp16_8192x6146", "fp16", 8192, 6146, seed=3))
    add(Workload("c4x_fp16_8192x6145", "fp16", 8192, 6145, seed=3))
    add(Workload("c5_fp32_32768x12288", "fp32", 32768, 12288, seed=4))
    # mid-size batches: a few thousand rows, i.e. a few waves of CTAs with a ragged last one - between the
    # latency-bound and the bandwidth-bound configurations (where a persistent grid would have to pay, if anywhere)
    add(Workload("mid_bf16_2048x8192", "bf16", 2048, 8192, seed=5, dist=_PREFILL_DIST))
    add(Workload("mid_bf16_4096x4096", "bf16", 4096, 4096, seed=5, dist=_PREFILL_DIST))
    add(Workload("mid_bf16_3000x5120", "bf16", 3000, 5120, seed=5, dist=_PREFILL_DIST))
    # silu_and_mul: a bandwidth case (LLaMA-3-8B MLP width), and the paper's fp32 (m, n) shapes with n = d
    gate = Dist(sigma=2.5)
    add(Workload("silu_bf16_16384x14336", "bf16", 16384, 14336, seed=6, dist=gate, op="silu_and_mul"))
    add(Workload("silu_fp32_2048x8192", "fp32", 2048, 8192, seed=6, dist=gate, op="silu_and_mul"))
    add(Workload("silu_fp32_128x11008", "fp32", 128, 11008, seed=6, dist=gate, op="silu_and_mul"))
    add(Workload("silu_bf16_64x11008", "bf16", 64, 11008, seed=6, dist=gate, op="silu_and_mul"))
    # the fp8-output variant of the norm on the prefill shape
    add(Workload("c3q_prefill_bf16_16384x8192_fp8out", "bf16", 16384, 8192, seed=2, dist=_PREFILL_DIST, op="add_rmsnorm_fp8"))
    # the tensor-parallel form of the norm on the prefill shape cut to a quarter of its rows, and a decode shape
    for n in (2, 4, 8):
        add(Workload(f"c3ar{n}_prefill_bf16_4096x8192", "bf16", 4096, 8192, seed=2, dist=_PREFILL_DIST,
                     op="add_rmsnorm_allreduce", n_parts=n))
    add(Workload("c2ar8_decode_bf16_64x8192", "bf16", 64, 8192, seed=1, op="add_rmsnorm_allreduce", n_parts=8))
    # merge_attn_states: the paper's (n, h, d) shapes in bf16, and a bandwidth case
    for n, h, d in ((512, 32, 256), (512, 40, 128), (768, 32, 256), (768, 40, 128), (512, 64, 128)):
        add(Workload(f"merge_bf16_{n}x{h}x{d}", "bf16", n, h * d, seed=7, op="merge_attn_states", head_dim=d))
    add(Workload("merge_bf16_32768x32x128", "bf16", 32768, 32 * 128, seed=7, op="merge_attn_states", head_dim=128))
    return out


# Shapes (m, n) listed in the paper's Experimental Setup for its two row-wise kernels.
PAPER_SHAPES_FP32 = [(128, 4096), (256, 4096), (1024, 4096), (2048, 8192), (128, 11008),
                     (256, 13824), (512, 14336), (1024, 8192)]
PAPER_SHAPES_16BIT = [(16, 4096), (32, 5120), (32, 8192), (16, 12288), (64, 8192)]


def _rng(seed: int, tensor_id: int, block: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed, tensor_id], counter=[0, 0, block, 0]))


def _block_f32(seed: int, tensor_id: int, block: int, hidden: int, dist: Dist) -> np.ndarray:
    g = _rng(seed, tensor_id, block)
    n = ROWS_PER_BLOCK * hidden
    v = g.standard_normal(n, dtype=np.float32)
    v *= np.float32(dist.sigma)
    if dist.outlier_p > 0.0:
        u = g.random(n, dtype=np.float32)
        o = g.standard_normal(n, dtype=np.float32)
        o *= np.float32(dist.outlier_sigma)
        np.copyto(v, o, where=u < np.float32(dist.outlier_p))
    return v.reshape(ROWS_PER_BLOCK, hidden)


def make_rows(tensor_id: int, row_begin: int, row_end: int, hidden: int, dtype: str, seed: int,
              dist: Dist = Dist(), threads: int = 8) -> torch.Tensor:
    """Rows [row_begin, row_end) of tensor ``x`` (tensor_id 0) or ``r`` (1) as a CPU tensor."""
    if row_end <= row_begin:
        return torch.empty((0, hidden), dtype=TORCH_DTYPES[dtype])
    b0, b1 = row_begin // ROWS_PER_BLOCK, (row_end - 1) // ROWS_PER_BLOCK + 1
    out = torch.empty(((b1 - b0) * ROWS_PER_BLOCK, hidden), dtype=TORCH_DTYPES[dtype])

    def fill(b: int):
        blk = torch.from_numpy(_block_f32(seed, tensor_id, b, hidden, dist))
        lo = (b - b0) * ROWS_PER_BLOCK
        out[lo:lo + ROWS_PER_BLOCK].copy_(blk)  # dtype conversion, round to nearest even

    if b1 - b0 > 1 and threads > 1:
        with ThreadPoolExecutor(max_workers=threads) as pool:
            list(pool.map(fill, range(b0, b1)))
    else:
        for b in range(b0, b1):
            fill(b)
    lo = row_begin - b0 * ROWS_PER_BLOCK
    return out[lo:lo + (row_end - row_begin)]


def make_weight(hidden: int, dtype: str, seed: int, dist: Dist = Dist()) -> torch.Tensor:
    g = _rng(seed, TENSOR_W, 0)
    v = g.standard_normal(hidden, dtype=np.float32)
    v = v * np.float32(dist.w_sigma) + np.float32(dist.w_mean)
    return torch.from_numpy(v).to(TORCH_DTYPES[dtype])


def make_inputs(n_tokens: int, hidden: int, dtype: str, seed: int, dist: Dist = Dist(),
                threads: int = 8):
    """(x, r, w) as contiguous CPU tensors of the storage dtype."""
    x = make_rows(TENSOR_X, 0, n_tokens, hidden, dtype, seed, dist, threads).contiguous()
    r = make_rows(TENSOR_R, 0, n_tokens, hidden, dtype, seed, dist, threads).contiguous()
    w = make_weight(hidden, dtype, seed, dist)
    return x, r, w


def make_parts(row_begin: int, row_end: int, hidden: int, dtype: str, seed: int, n_parts: int, dist: Dist = Dist(),
               threads: int = 8) -> torch.Tensor:
    """Rows of the n_parts partial inputs of the tensor-parallel norm as one [n_parts, rows, hidden] tensor: part k
    is N(0, sigma / sqrt(n_parts)) with the same outlier mix, so that the sum over parts has the spread of x."""
    scaled = Dist(sigma=dist.sigma / float(np.sqrt(n_parts)), outlier_p=dist.outlier_p,
                  outlier_sigma=dist.outlier_sigma / float(np.sqrt(n_parts)), w_mean=dist.w_mean, w_sigma=dist.w_sigma)
    parts = [make_rows(TENSOR_PART0 + k, row_begin, row_end, hidden, dtype, seed, scaled, threads) for k in range(n_parts)]
    return torch.stack(parts).contiguous()


def make_gate_up(row_begin: int, row_end: int, d: int, dtype: str, seed: int, dist: Dist = Dist(sigma=2.5),
                 threads: int = 8) -> torch.Tensor:
    """Rows of the [T, 2*d] input of silu_and_mul: gate and value halves, N(0, sigma) each."""
    return make_rows(TENSOR_GATE_UP, row_begin, row_end, 2 * d, dtype, seed, dist, threads).contiguous()


def make_lse(tensor_id: int, row_begin: int, row_end: int, heads: int, seed: int, mean: float = 4.0,
             sigma: float = 2.0) -> torch.Tensor:
    """Rows of a float32 [T, heads] log-sum-exp tensor: N(mean, sigma), the spread two key blocks of unequal
    length typically show."""
    t = make_rows(tensor_id, row_begin, row_end, heads, "fp32", seed, Dist(sigma=sigma), threads=1).contiguous()
    return (t + mean).contiguous()


def make_merge_inputs(row_begin: int, row_end: int, heads: int, head_dim: int, dtype: str, seed: int, threads: int = 8):
    """(v_a, s_a, v_b, s_b): partial outputs N(0, 1) of shape [T, heads, head_dim], float32 log-sum-exps [T, heads]."""
    n = row_end - row_begin
    v_a = make_rows(TENSOR_X, row_begin, row_end, heads * head_dim, dtype, seed, Dist(), threads).contiguous()
    v_b = make_rows(TENSOR_R, row_begin, row_end, heads * head_dim, dtype, seed, Dist(), threads).contiguous()
    return (v_a.view(n, heads, head_dim), make_lse(TENSOR_LSE_A, row_begin, row_end, heads, seed),
            v_b.view(n, heads, head_dim), make_lse(TENSOR_LSE_B, row_begin, row_end, heads, seed))


def make_workload_inputs(wl: Workload, threads: int = 8):
    if wl.op == "merge_attn_states":
        return make_merge_inputs(0, wl.n_tokens, wl.hidden // wl.head_dim, wl.head_dim, wl.dtype, wl.seed, threads)
    if wl.op == "silu_and_mul":
        return (make_gate_up(0, wl.n_tokens, wl.hidden, wl.dtype, wl.seed, wl.dist, threads),)
    if wl.op == "add_rmsnorm_allreduce":
        _, r, w = make_inputs(wl.n_tokens, wl.hidden, wl.dtype, wl.seed, wl.dist, threads)
        return make_parts(0, wl.n_tokens, wl.hidden, wl.dtype, wl.seed, wl.n_parts, wl.dist, threads), r, w
    return make_inputs(wl.n_tokens, wl.hidden, wl.dtype, wl.seed, wl.dist, threads)


def sample_rows(wl: Workload, rows, threads: int = 1):
    """Regenerate the given rows of a workload: (x_rows, r_rows, w), each row drawn on its own."""
    xs = [make_rows(TENSOR_X, t, t + 1, wl.hidden, wl.dtype, wl.seed, wl.dist, threads) for t in rows]
    rs = [make_rows(TENSOR_R, t, t + 1, wl.hidden, wl.dtype, wl.seed, wl.dist, threads) for t in rows]
    w = make_weight(wl.hidden, wl.dtype, wl.seed, wl.dist)
    return torch.cat(xs).contiguous(), torch.cat(rs).contiguous(), w
