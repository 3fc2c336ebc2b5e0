"""The input generator: determinism, prefix property, distributions, workload table."""
import numpy as np
import torch

from paper_2601_12698_b200 import synth


def test_rows_are_a_prefix_and_blocks_regenerate():
    a = synth.make_rows(synth.TENSOR_X, 0, 200, 96, "bf16", seed=1)
    b = synth.make_rows(synth.TENSOR_X, 0, 70, 96, "bf16", seed=1)
    c = synth.make_rows(synth.TENSOR_X, 130, 131, 96, "bf16", seed=1, threads=1)
    assert torch.equal(a[:70], b) and torch.equal(a[130:131], c)
    assert not torch.equal(a, synth.make_rows(synth.TENSOR_R, 0, 200, 96, "bf16", seed=1))
    assert not torch.equal(a, synth.make_rows(synth.TENSOR_X, 0, 200, 96, "bf16", seed=2))


def test_distributions():
    wl = synth.workloads()["c3_prefill_bf16_16384x8192"]
    x = synth.make_rows(synth.TENSOR_X, 0, 256, wl.hidden, wl.dtype, wl.seed, wl.dist).float()
    frac_big = (x.abs() > 12).float().mean().item()   # 6 sigma of the bulk: essentially outliers only
    assert 0.006 < frac_big < 0.010                    # 1% replaced, ~81% of N(0,50) beyond 12
    bulk = x[x.abs() <= 12]
    assert abs(bulk.std().item() - 2.0) < 0.05
    w = synth.make_weight(8192, "bf16", 2).float()
    assert abs(w.mean().item() - 1.0) < 0.01 and abs(w.std().item() - 0.1) < 0.01
    x1 = synth.make_rows(synth.TENSOR_X, 0, 128, 4096, "fp32", 0)
    assert abs(x1.std().item() - 1.0) < 0.01 and abs(x1.mean().item()) < 0.01


def test_workload_table_and_byte_accounting():
    w = synth.workloads()
    c3 = w["c3_prefill_bf16_16384x8192"]
    assert c3.elements == 134_217_728
    assert c3.algorithmic_bytes == 4 * 2 * c3.elements + 2 * 8192
    assert c3.nominal_bytes == 1_342_177_280
    c5 = w["c5_fp32_32768x12288"]
    assert c5.algorithmic_bytes == 4 * 4 * 402_653_184 + 4 * 12288
    assert {k for k in w if k.startswith("c2_")} == {f"c2_decode_bf16_{t}x4096" for t in (1, 4, 16, 64, 256)}
    assert w["c4_fp16_8192x6152"].hidden * 2 % 16 == 0 and w["c4x_fp16_8192x6148"].hidden * 2 % 16 == 8


def test_sample_rows_match_full_generation():
    wl = synth.Workload("t", "fp16", 300, 200, seed=9)
    x, r, w = synth.make_workload_inputs(wl)
    xs, rs, ws = synth.sample_rows(wl, [0, 64, 299])
    assert torch.equal(xs, x[[0, 64, 299]]) and torch.equal(rs, r[[0, 64, 299]]) and torch.equal(ws, w)
