"""The allocation-free split-K entry point against the workspace-taking one.

`atb_gemm_splitk_noalloc` is for callers that are not allowed to allocate device memory (an
operator living inside another framework's memory pool, a serving loop that must not hit the
allocator after start-up): its FP32 partial sums go to a 64 MiB array built into the library.
It has to produce exactly what `atb_gemm_splitk` produces with a caller workspace, on the first
call (which also resolves the array's device address) and on a second call that finds the
previous call's leftovers in the array.  This file is named so that pytest collects it last.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2511_16041_b200 as atb
from paper_2511_16041_b200 import inputs
import oracle
from tests.gpu_util import dev, planes_to_dev, bf16_bits_to_dev, bf16_dev_to_bits

pytestmark = pytest.mark.gpu


def _problem(M, N, K, kind, seed):
    A = inputs.make_A(kind, M, K, seed)
    Bb = inputs.make_B_bits(K, N, 1.0, seed)
    mant, exp = oracle.quantize_bfp16(A)
    md, ed = planes_to_dev(mant, exp)
    return mant, exp, Bb, md, ed, bf16_bits_to_dev(Bb)


def test_noalloc_matches_workspace_entry_on_two_calls_in_a_row():
    lib = atb.load_library()
    tiling = (128, 256, 64, 256)
    # two different problems back to back: the second one finds the first one's partial sums in the array
    for call, (M, N, K, splits, kind) in enumerate([(1024, 1024, 2048, 8, "laplace"), (520, 776, 1024, 4, "outlier")]):
        mant, exp, Bb, md, ed, Bd = _problem(M, N, K, kind, inputs.BASE_SEED + call)
        want = atb.atb_gemm_splitk(M, N, K, *tiling, md, ed, Bd, splits)          # caller workspace
        got = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=dev())
        rc = lib.atb_gemm_splitk_noalloc(M, N, K, *tiling, md.data_ptr(), ed.data_ptr(), Bd.data_ptr(), N,
                                         got.data_ptr(), N, splits, ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
        assert rc == 0, atb.atb_last_error_message()
        atb.atb_device_status()
        # same kernels, same order of additions: equal bit for bit ...
        assert torch.equal(got.view(torch.int16), want.view(torch.int16)), call
        # ... and inside the tolerance every GEMM test of this suite uses
        Cr, S = oracle.gemm(mant, exp, Bb)
        bad, ratio = oracle.check_tolerance(bf16_dev_to_bits(got), Cr, S)
        assert bad == 0 and ratio < 0.75, (call, bad, ratio)


def test_noalloc_rejects_what_does_not_fit_and_allocates_nothing():
    lib = atb.load_library()
    M = N = 4096
    K = 1024
    md = torch.zeros((M, K), dtype=torch.int8, device=dev())
    ed = torch.zeros(atb.atb_bfp16_exp_bytes(M, K), dtype=torch.uint8, device=dev())
    B = torch.zeros((K, N), dtype=torch.bfloat16, device=dev())
    C = torch.zeros((M, N), dtype=torch.bfloat16, device=dev())
    assert atb.atb_gemm_splitk_workspace_bytes(M, N, 256, 2) > atb.NOALLOC_SCRATCH_BYTES
    with pytest.raises(atb.AtbError) as e:
        atb.atb_gemm_splitk_noalloc(M, N, K, 128, 256, 64, 256, md, ed, B, 2, C)
    assert e.value.status == 7 and "scratch" in str(e.value)
    # the largest split count that still fits goes through, with no change in what CUDA has handed out
    atb.atb_gemm_splitk_noalloc(M, N, K, 128, 256, 64, 256, md, ed, B, 1, C)    # loads the kernels (lazy module loading)
    atb.atb_device_status()
    free_before, _ = torch.cuda.mem_get_info()
    atb.atb_gemm_splitk_noalloc(M, N, K, 128, 256, 64, 256, md, ed, B, 1, C)
    atb.atb_device_status()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    assert bool((C == 0).all())
