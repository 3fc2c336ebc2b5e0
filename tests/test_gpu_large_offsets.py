"""Tensors beyond 4 GiB: row offsets that do not fit 32 bits, in every staging level of the norm and in the comparison
kernels.  The tensors are zero except three bands of rows (the first block, a band astride the 4 GiB boundary, the last
rows), which are generated and checked against the oracle; a zero row must come back as zeros."""
import pytest
import torch

pytestmark = pytest.mark.gpu

EPS = 1e-6
HIDDEN = 8192                 # bf16: 16 KiB per row, so row 262 144 starts at byte 2^32
T = 262144 + 320
BANDS = [(0, 64), (262144 - 96, 262144 + 96), (T - 64, T)]


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2601_12698_b200 import binding
    torch.cuda.set_device(0)
    free, _ = torch.cuda.mem_get_info()
    if free < 24 << 30:
        pytest.skip("needs 24 GiB of free device memory")
    return binding


@pytest.fixture(scope="module")
def tensors(B, oracle_lib):
    from paper_2601_12698_b200 import synth
    x = torch.zeros((T, HIDDEN), dtype=torch.bfloat16, device="cuda")
    r = torch.zeros_like(x)
    w = synth.make_weight(HIDDEN, "bf16", seed=31)
    refs = []
    for lo, hi in BANDS:
        xb = synth.make_rows(synth.TENSOR_X, lo, hi, HIDDEN, "bf16", 31).contiguous()
        rb = synth.make_rows(synth.TENSOR_R, lo, hi, HIDDEN, "bf16", 31).contiguous()
        x[lo:hi].copy_(xb)
        r[lo:hi].copy_(rb)
        refs.append(oracle_lib.add_rmsnorm(xb, rb, w, EPS))
    assert x.numel() * x.element_size() > 1 << 32
    yield x, r, w.cuda(), refs
    del x, r
    torch.cuda.empty_cache()


THETAS = [dict(threads_per_row=512, vec_bytes=32),                                             # registers
          dict(threads_per_row=256, vec_bytes=16, unroll=4),
          dict(threads_per_row=256, rows_per_cta=2, vec_bytes=32, stage=1),                    # ld.global -> shared
          dict(threads_per_row=256, vec_bytes=16, stage=2),                                    # bulk copy, one row block per CTA
          dict(threads_per_row=256, vec_bytes=16, unroll=2, stage=4),                          # persistent pipeline
          dict(threads_per_row=128, vec_bytes=16, stage=1, reduce=2, cluster_size=2)]         # row split over a cluster


@pytest.mark.parametrize("theta", THETAS, ids=lambda t: "-".join(f"{k[0]}{v}" for k, v in t.items()))
def test_rows_beyond_4_gib_match_the_oracle(B, oracle_lib, tensors, theta):
    x, r, w, refs = tensors
    y = torch.full_like(x, 7.0)
    r_out = torch.full_like(x, 7.0)
    B.rmsnorm_template_launch(B.make_params(**theta), x, r, w, y, r_out, EPS)
    torch.cuda.synchronize()
    assert B.rt_device_status() == 0
    for (lo, hi), (y_ref, r_ref) in zip(BANDS, refs):
        assert oracle_lib.bit_mismatches(r_out[lo:hi].cpu().contiguous(), r_ref) == 0, (lo, hi)
        worst, bad = oracle_lib.compare_y(y[lo:hi].cpu().contiguous(), y_ref)
        assert bad == 0 and worst <= 2, (lo, hi, worst)
    # the rows between the bands are zero in, zero out (every row was written: the fill value is gone)
    for lo, hi in ((64, 4096), (262144 + 96, 262144 + 128), (T - 200, T - 64)):
        assert not bool(y[lo:hi].any()) and not bool(r_out[lo:hi].any()), (lo, hi)
    del y, r_out


def test_comparison_kernels_index_beyond_32_bits(B, tensors):
    """tuner_compare over 2.15e9 elements: one planted difference in the very last element, one just past 2^31."""
    x, r, w, _ = tensors
    other = x.clone()
    n = x.numel()
    assert n > 1 << 31
    flat = other.view(-1)
    flat[n - 1] = 3.0
    flat[(1 << 31) + 5] = -2.0
    worst, bad = B.tuner_compare(other, x, B.RT_CMP_ULP16, 2.0)
    assert bad == 2 and worst > 2
    assert B.tuner_compare(other, x, B.RT_CMP_BITS)[1] == 2 and B.tuner_compare(x, x, B.RT_CMP_BITS)[1] == 0
    del other


@pytest.mark.parametrize("theta", [dict(threads_per_row=512, vec_bytes=32), dict(threads_per_row=256, vec_bytes=16, stage=2)],
                         ids=["registers", "bulk-copy"])
def test_silu_and_mul_rows_beyond_4_gib(B, oracle_lib, theta):
    """silu_and_mul on [T, 2 x 8192] bf16: the input passes 4 GiB at row 131 072, the output at row 262 144."""
    from paper_2601_12698_b200 import synth
    x = torch.zeros((T, 2 * HIDDEN), dtype=torch.bfloat16, device="cuda")
    bands = [(0, 64), (131072 - 64, 131072 + 64), (262144 - 64, 262144 + 64), (T - 64, T)]
    refs = []
    for lo, hi in bands:
        xb = synth.make_gate_up(lo, hi, HIDDEN, "bf16", seed=33).contiguous()
        x[lo:hi].copy_(xb)
        refs.append(oracle_lib.silu_and_mul(xb))
    out = torch.full((T, HIDDEN), 7.0, dtype=torch.bfloat16, device="cuda")
    B.silu_and_mul_template_launch(B.make_params(**theta), x, out)
    torch.cuda.synchronize()
    assert B.rt_device_status() == 0
    for (lo, hi), ref in zip(bands, refs):
        worst, bad = oracle_lib.compare_y(out[lo:hi].cpu().contiguous(), ref)
        assert bad == 0 and worst <= 2, (lo, hi, worst)
    assert not bool(out[64:4096].any()) and not bool(out[262144 + 64:T - 64].any())   # silu(0) x 0 = 0 everywhere else
    del x, out
    torch.cuda.empty_cache()
