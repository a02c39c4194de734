"""GPU parity: atb_quantize_bfp16 must equal the oracle's quantiser bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import paper_2511_16041_b200 as atb
from paper_2511_16041_b200 import inputs
from tests.gpu_util import dev

pytestmark = pytest.mark.gpu


def _compare(A: np.ndarray, lda=None):
    M, K = A.shape
    mant_o, exp_o = oracle.quantize_bfp16(A)
    if lda is None:
        Ad = torch.from_numpy(A).to(dev())
    else:
        full = torch.full((M, lda), 7.0, dtype=torch.float32, device=dev())
        full[:, :K] = torch.from_numpy(A).to(dev())
        Ad = full[:, :K]
    mant, plane = atb.atb_quantize_bfp16(Ad)
    torch.cuda.synchronize()
    assert plane.numel() == atb.atb_bfp16_exp_bytes(M, K)
    assert np.array_equal(mant.cpu().numpy(), mant_o)
    plane_h = plane.cpu().numpy()
    assert np.array_equal(atb.exp_plane_to_logical(plane_h, M, K), exp_o)
    # padding rows / blocks of the device plane are zero
    assert np.array_equal(plane_h, atb.logical_to_exp_plane(exp_o, M, K))


@pytest.mark.parametrize("kind", ["normal", "laplace", "outlier"])
@pytest.mark.parametrize("shape", [(256, 256), (1000, 520), (33, 8), (1, 64), (4096, 1024), (31, 72)])
def test_quantize_distributions(kind, shape):
    _compare(inputs.make_A(kind, *shape))


def test_quantize_leading_dimension():
    _compare(inputs.make_A("normal", 70, 136), lda=200)


def test_quantize_whole_range_ties_and_specials():
    rng = np.random.default_rng(2024)
    M, K = 512, 256
    a = rng.standard_normal((M, K)) * np.exp2(rng.integers(-149, 128, size=(M, K // 8)).repeat(8, axis=1))
    a = a.astype(np.float32)
    # exact ties and saturation candidates in some blocks
    a[:64] = (rng.integers(-255, 256, size=(64, K)) * 0.5).astype(np.float32)
    a[:64, ::8] = 100.0
    a[64:96] = (127.0 + rng.integers(-4, 5, size=(32, K)) * 0.25).astype(np.float32)
    # specials
    a[100, 0] = np.inf; a[100, 9] = -np.inf; a[101, 3] = np.nan; a[102, :8] = np.nan
    a[103, :] = 0.0; a[104, :8] = -0.0
    a[105, 0] = np.finfo(np.float32).max; a[105, 1] = -np.finfo(np.float32).max
    a[106, :8] = np.float32(2.0 ** -149); a[107, :8] = np.float32(2.0 ** -126)
    _compare(a)


def test_quantize_bf16_single_nonzero_exhaustive():
    bits = np.arange(1 << 16, dtype=np.uint16)
    a = np.zeros((1 << 16, 8), np.float32)
    a[:, 5] = inputs.bf16_bits_to_f32(bits)
    _compare(a)


def test_quantize_empty_and_errors():
    z = torch.empty((0, 64), dtype=torch.float32, device=dev())
    mant, plane = atb.atb_quantize_bfp16(z)
    assert mant.numel() == 0 and plane.numel() == 0
    bad = torch.zeros((4, 12), dtype=torch.float32, device=dev())
    with pytest.raises(atb.AtbError) as e:
        atb.atb_quantize_bfp16(bad)
    assert e.value.status == 2
    lib = atb.load_library()
    assert lib.atb_quantize_bfp16(None, 8, 8, 8, None, None, None) == 1          # NULL pointers
    a = torch.zeros((8, 16), dtype=torch.float32, device=dev())
    m = torch.zeros(8 * 16 + 16, dtype=torch.int8, device=dev())
    e8 = torch.zeros(atb.atb_bfp16_exp_bytes(8, 16), dtype=torch.uint8, device=dev())
    assert lib.atb_quantize_bfp16(a.data_ptr(), 8, 16, 16, m.data_ptr() + 1, e8.data_ptr(), None) == 4   # misaligned


def test_quantize_full_size_sampled():
    """8192 x 8192 Laplace (the headline operand): every block of 64 sampled rows."""
    M = K = 8192
    A = inputs.make_A("laplace", M, K)
    Ad = torch.from_numpy(A).to(dev())
    mant, plane = atb.atb_quantize_bfp16(Ad)
    torch.cuda.synchronize()
    rows = np.unique(np.concatenate([[0, 31, 32, M - 1], np.random.default_rng(1).integers(0, M, 60)]))
    mant_o, exp_o = oracle.quantize_bfp16(A[rows])
    assert np.array_equal(mant[torch.from_numpy(rows).to(dev())].cpu().numpy(), mant_o)
    assert np.array_equal(atb.exp_plane_to_logical(plane.cpu().numpy(), M, K)[rows], exp_o)
