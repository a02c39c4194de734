"""The timeout path of the GEMM kernels, run once in the form that cannot hang a GPU.

Every mbarrier wait in the kernels is bounded: when it runs out, the CTA raises an abort flag, every
role leaves its loop, copies in flight get time to land, tensor memory is released, the kernel returns
and `atb_device_status` reports ATB_ERR_DEVICE_TIMEOUT.  The product build never takes that path on a
healthy run, so a separate diagnostic build of the same sources (never the product library) shortens
the limit to 2 ms and has one dequantiser warp of CTA 0 keep back its first arrival: on a one-tile,
one-CTA problem the UMMA issuer then waits for an operand that is never announced - no copy and no
UMMA depends on it - and gives up.  No trap, no unbounded loop, one CTA.
"""
import ctypes
import os

import numpy as np
import pytest
import torch

import oracle
import paper_2511_16041_b200 as atb
from paper_2511_16041_b200 import _build, inputs
from tests.gpu_util import bf16_dev_to_bits, dev, planes_to_dev, bf16_bits_to_dev

pytestmark = pytest.mark.gpu


def _diagnostic_library():
    path = _build.build_library(variant="timeout_test")       # built in-tree beside the product library
    lib = ctypes.CDLL(path)
    i64, vp, ci = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
    lib.atb_gemm.restype = ci
    lib.atb_gemm.argtypes = [i64, i64, i64, ci, ci, ci, ci, vp, vp, vp, i64, vp, i64, vp]
    lib.atb_device_status.restype = ci
    lib.atb_device_status.argtypes = [vp]
    lib.atb_last_error_message.restype = ctypes.c_char_p
    return lib


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    assert os.path.realpath(_build.variant_path("timeout_test")) != os.path.realpath(atb.LIB_PATH)
    diag = _diagnostic_library()
    M, N, K = 128, 128, 64                                   # one tile, one K-step, one CTA
    A = inputs.make_A("normal", M, K)
    Bb = inputs.make_B_bits(K, N)
    mant, exp = oracle.quantize_bfp16(A)
    md, ed = planes_to_dev(mant, exp)
    Bd = bf16_bits_to_dev(Bb)
    C = torch.zeros((M, N), dtype=torch.bfloat16, device=dev())
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    args = (M, N, K, 128, 128, 64, 128, md.data_ptr(), ed.data_ptr(), Bd.data_ptr(), N, C.data_ptr(), N, stream)

    assert diag.atb_device_status(stream) == atb.ATB_OK
    assert diag.atb_gemm(*args) == atb.ATB_OK                # the launch itself succeeds
    status = diag.atb_device_status(stream)                  # ... the kernel gave up a wait and returned
    assert status == 8, diag.atb_last_error_message()        # ATB_ERR_DEVICE_TIMEOUT
    assert b"bounded wait" in diag.atb_last_error_message()
    assert diag.atb_device_status(stream) == atb.ATB_OK      # reading the flag cleared it
    torch.cuda.synchronize()                                 # no sticky CUDA error: the context is intact

    # the product build on the same context right afterwards: a normal GEMM, checked against the oracle
    Cg = atb.atb_gemm(M, N, K, 128, 128, 64, 128, md, ed, Bd)
    atb.atb_device_status()
    Cr, S = oracle.gemm(mant, exp, Bb)
    bad, ratio = oracle.check_tolerance(bf16_dev_to_bits(Cg), Cr, S)
    assert bad == 0 and ratio < 0.75
    # and a multi-tile one, so that tensor memory released on the abort path is seen to be allocatable again
    M2, N2, K2 = 1024, 1024, 512
    A2 = inputs.make_A("laplace", M2, K2)
    B2 = inputs.make_B_bits(K2, N2)
    m2, e2 = oracle.quantize_bfp16(A2)
    md2, ed2 = planes_to_dev(m2, e2)
    Cg2 = atb.atb_gemm(M2, N2, K2, 128, 256, 64, 256, md2, ed2, bf16_bits_to_dev(B2))
    atb.atb_device_status()
    Cr2, S2 = oracle.gemm(m2, e2, B2)
    bad, ratio = oracle.check_tolerance(bf16_dev_to_bits(Cg2), Cr2, S2)
    assert bad == 0 and ratio < 0.75
