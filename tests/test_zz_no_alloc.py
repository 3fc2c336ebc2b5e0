"""The allocation-free comparison entry point gives what tuner_compare gives.

Kept in a file that pytest collects last.  It is for callers that cannot allocate device memory (a process
whose memory pool owns the whole GPU, or a latency path that cannot afford the device-wide synchronisation
of cudaMalloc): its accumulator is a fixed array inside the library, shared by every call on the device.
The test calls it twice in a row on different data, so a result left over from the first call would show
in the second, and compares each answer with the allocating entry point's.
"""
import ctypes

import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2601_12698_b200 import binding
    torch.cuda.set_device(0)
    return binding


def _pair(dtype, n, n_perturbed, seed):
    g = torch.Generator().manual_seed(seed)
    ref = torch.randn(n, generator=g).to(dtype)
    got = ref.clone()
    idx = torch.randperm(n, generator=g)[:n_perturbed]
    if dtype == torch.float32:
        got[idx] = got[idx] * (1 + 4e-5 * torch.randn(n_perturbed, generator=g))
    else:
        bits = got.view(torch.int16)
        bits[idx] = bits[idx] + torch.randint(-5, 6, (n_perturbed,), generator=g).to(torch.int16)
    return got.cuda(), ref.cuda()


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16, torch.float32])
def test_static_compare_matches_allocating_compare_twice_in_a_row(B, oracle_lib, dtype):
    y_mode, tol = (B.RT_CMP_REL32, 1e-5) if dtype == torch.float32 else (B.RT_CMP_ULP16, 2.0)
    first = _pair(dtype, 1_000_003 if dtype != torch.float32 else 1_000_000, 700, seed=1)
    second = _pair(dtype, 4097, 3, seed=2)  # far fewer differences: leftovers from the first call would show
    for k, (got, ref) in enumerate((first, second)):
        for mode, t in ((y_mode, tol), (B.RT_CMP_BITS, 0.0)):
            want = B.tuner_compare(got, ref, mode, t)
            have = B.tuner_compare_static(got, ref, mode, t)
            assert have[1] == want[1]
            assert have[0] == want[0]  # integer distances, and the same float maximum, bit for bit
            if k == 0:
                assert have[1] > 100  # the first pair really differs, so a stale record would be visible next
        # and against the CPU oracle's own comparison of the same pair, so that the check does not rest on the
        # library agreeing with itself
        have = B.tuner_compare_static(got, ref, y_mode, tol)
        if dtype == torch.float32:
            worst, bad = oracle_lib.compare_y(got.cpu(), ref.cpu(), tol_rel=tol)
            assert have[1] == bad and abs(have[0] - worst) <= 1e-6 * worst
        else:
            assert (int(have[0]), have[1]) == oracle_lib.compare_y(got.cpu(), ref.cpu(), tol_ulp=int(tol))
        assert B.tuner_compare_static(got, ref, B.RT_CMP_BITS, 0.0)[1] == oracle_lib.bit_mismatches(got.cpu(), ref.cpu())
    # identical buffers: zero after a call that found differences
    assert B.tuner_compare_static(first[1], first[1].clone(), y_mode, tol) == (0.0, 0)


def test_static_compare_rejects_what_it_cannot_do(B):
    a = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    worst, bad = ctypes.c_double(0.0), ctypes.c_int64(0)
    call = B.lib.tuner_compare_static
    too_many = (1 << 40) + 1
    assert call(a.data_ptr(), a.data_ptr(), too_many, B.RT_BF16, B.RT_CMP_BITS, 0.0, ctypes.byref(worst),
                ctypes.byref(bad), None) == B.RT_ERR_CAPACITY
    assert b"limit" in B.lib.rt_last_error()
    assert call(None, a.data_ptr(), 64, B.RT_BF16, B.RT_CMP_BITS, 0.0, ctypes.byref(worst), ctypes.byref(bad),
                None) == B.RT_ERR_NULL
    assert call(a.data_ptr(), a.data_ptr(), 64, B.RT_BF16, B.RT_CMP_REL32, 0.0, ctypes.byref(worst),
                ctypes.byref(bad), None) == B.RT_ERR_DTYPE
    assert call(a.data_ptr(), a.data_ptr(), 0, B.RT_BF16, B.RT_CMP_BITS, 0.0, ctypes.byref(worst),
                ctypes.byref(bad), None) == B.RT_OK
