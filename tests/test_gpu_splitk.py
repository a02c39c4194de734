"""GPU parity of the split-K entry point against the FP64 oracle and against atb_gemm."""
import numpy as np
import pytest
import torch

import oracle
import paper_2511_16041_b200 as atb
from paper_2511_16041_b200 import inputs
from tests.gpu_util import dev, planes_to_dev, bf16_bits_to_dev, bf16_dev_to_bits

pytestmark = pytest.mark.gpu


def _operands(M, N, K, kind="normal"):
    A = inputs.make_A(kind, M, K)
    Bb = inputs.make_B_bits(K, N)
    mant, exp = oracle.quantize_bfp16(A)
    return mant, exp, Bb


@pytest.mark.parametrize("shape,tiling,splits", [
    ((256, 256, 1024), (128, 256, 64, 256), 4),
    ((300, 264, 1536), (64, 128, 64, 128), 3),          # ragged M and N, splits not a power of two
    ((1024, 1024, 4096), (128, 256, 64, 256), 8),
    ((129, 136, 448), (128, 128, 64, 256), 7),           # one K-step per split
    ((200, 136, 400), (64, 128, 64, 128), 7),            # K not a multiple of 64: a ragged last K-step
    ((512, 512, 512), (64, 256, 64, 128), 1),
])
def test_splitk_against_oracle(shape, tiling, splits):
    M, N, K = shape
    mant, exp, Bb = _operands(M, N, K, "laplace")
    md, ed = planes_to_dev(mant, exp)
    Bd = bf16_bits_to_dev(Bb)
    C = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=dev())
    atb.atb_gemm_splitk(M, N, K, *tiling, md, ed, Bd, splits, C=C)
    atb.atb_device_status()
    Cr, S = oracle.gemm(mant, exp, Bb)
    bad, ratio = oracle.check_tolerance(bf16_dev_to_bits(C), Cr, S)
    assert bad == 0 and ratio < 0.75, (shape, tiling, splits, bad, ratio)


def test_splitk_exact_on_integer_matrices_and_one_split_equals_gemm():
    rng = np.random.default_rng(4)
    M, N, K = 256, 256, 512
    a = rng.integers(-1, 2, size=(M, K)).astype(np.float32)
    a[:, ::8] = np.where(a[:, ::8] == 0, 1, a[:, ::8])
    b = rng.integers(-1, 2, size=(K, N)).astype(np.float32)
    mant, exp = oracle.quantize_bfp16(a)
    md, ed = planes_to_dev(mant, exp)
    Bd = bf16_bits_to_dev(inputs.to_bf16_bits(b))
    want = (a.astype(np.int64) @ b.astype(np.int64)).astype(np.float64)
    for splits in (1, 2, 8):
        C = atb.atb_gemm_splitk(M, N, K, 128, 256, 64, 256, md, ed, Bd, splits)
        assert np.array_equal(inputs.bf16_bits_to_f32(bf16_dev_to_bits(C)).astype(np.float64), want), splits
    # one split: same accumulation order as atb_gemm -> bitwise equal on real data
    mant, exp, Bb = _operands(384, 256, 640)
    md, ed = planes_to_dev(mant, exp)
    Bd = bf16_bits_to_dev(Bb)
    C1 = atb.atb_gemm_splitk(384, 256, 640, 128, 128, 64, 256, md, ed, Bd, 1)
    C0 = atb.atb_gemm(384, 256, 640, 128, 128, 64, 256, md, ed, Bd)
    atb.atb_device_status()
    assert torch.equal(C0.view(torch.int16), C1.view(torch.int16))


def test_splitk_argument_errors_and_workspace_size():
    lib = atb.load_library()
    assert atb.atb_gemm_splitk_workspace_bytes(300, 264, 128, 3) == 3 * 384 * 264 * 4
    M = N = 256
    K = 512
    md = torch.zeros((M, K), dtype=torch.int8, device=dev())
    ed = torch.zeros(atb.atb_bfp16_exp_bytes(M, K), dtype=torch.uint8, device=dev())
    B = torch.zeros((K, N), dtype=torch.bfloat16, device=dev())
    C = torch.zeros((M, N), dtype=torch.bfloat16, device=dev())
    ws = torch.zeros(4 * M * N, dtype=torch.float32, device=dev())

    def call(til=(128, 256, 64, 256), splits=4, wsb=ws.numel() * 4, wsp=ws.data_ptr()):
        return lib.atb_gemm_splitk(M, N, K, *til, md.data_ptr(), ed.data_ptr(), B.data_ptr(), N, C.data_ptr(), N,
                                   splits, wsp, wsb, None)
    assert call() == 0
    assert call(wsb=ws.numel() * 4 - 4) == 7            # workspace too small
    assert call(splits=9) == 2                           # more splits than K-steps
    assert call(splits=0) == 2
    assert call(til=(32, 256, 64, 256)) == 3 and call(til=(128, 256, 128, 128)) == 3
    assert call(wsp=None) == 1
    torch.cuda.synchronize()


def test_select_splits_heuristic():
    assert atb.atb_select_splits(8192, 8192, 8192, 256, 64, 256) == 1        # enough tiles already
    assert atb.atb_select_splits(1024, 1024, 16384, 256, 64, 256) >= 4       # 16 tiles for 148 SMs
    assert atb.atb_select_splits(1024, 1024, 256, 256, 64, 256) == 1         # too few K-steps to split
