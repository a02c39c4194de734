"""GPU parity of the quantising epilogue (atb_gemm_bfp16_out: C written as BFP16 planes).

Two pins.  (1) Integer work, bit-exact: the planes must equal the oracle's quantiser applied to the
kernel's own FP32 accumulators - those are read back from the split-K entry point with one split, which
runs the same K loop and stores the FP32 tile unrounded.  (2) Against the FP64 oracle GEMM: a BFP16
element is off by at most half a quantisation step 2^(E-133) of its block (a whole step where the
mantissa saturated at +-127: the block maximum may round up to 128) plus the accumulation error,
|C_q - C_ref| <= 2^(E-134) (or 2^(E-133)) + 2^-12 sum_k |a_ik b_kj|.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2511_16041_b200 as atb
from paper_2511_16041_b200 import inputs
from tests.gpu_util import dev, planes_to_dev, bf16_bits_to_dev

pytestmark = pytest.mark.gpu

TILINGS = [(64, 128, 64, 128), (128, 128, 64, 256), (64, 256, 64, 128), (128, 256, 64, 256), (64, 256, 64, 256)]
# The CTA-pair tilings have no split-K form to read their FP32 accumulators through.  Their UMMAs add the
# same products in the same order as the single-CTA 256 x 256 tiling, so their planes are compared with
# that tiling's bit for bit, and with the FP64 oracle like the others.  The same holds for the stacked pair
# (two 128 x 256 tiles on a CTA pair, B stages 128 rows deep) on shapes where no CTA has a second tile.
PAIR_TILINGS = [(64, 256, 64, 512), (128, 256, 64, 512), (64, 128, 128, 256), (128, 128, 128, 256)]


def fp32_accumulators(M, N, K, tiling, md, ed, Bd):
    ws = torch.zeros(atb.atb_gemm_splitk_workspace_bytes(M, N, tiling[1], 1) // 4, dtype=torch.float32, device=dev())
    atb.atb_gemm_splitk(M, N, K, *tiling, md, ed, Bd, 1, workspace=ws)
    atb.atb_device_status()
    m_pad = -(-M // tiling[1]) * tiling[1]
    return ws.view(m_pad, N)[:M].cpu().numpy()


def run_qout(M, N, K, tiling, md, ed, Bd):
    Cm = torch.full((M, N), 77, dtype=torch.int8, device=dev())
    Ce = torch.full((atb.atb_bfp16_exp_bytes(M, N),), 201, dtype=torch.uint8, device=dev())
    atb.atb_gemm_bfp16_out(M, N, K, *tiling, md, ed, Bd, Cm, Ce)
    atb.atb_device_status()
    return Cm.cpu().numpy(), Ce.cpu().numpy()


@pytest.mark.parametrize("shape", [(256, 256, 256), (300, 272, 448), (1000, 1040, 1104)])
def test_planes_equal_the_quantiser_on_the_fp32_accumulators(shape):
    M, N, K = shape
    A = inputs.make_A("laplace", M, K)
    Bb = inputs.make_B_bits(K, N)
    mant, exp = oracle.quantize_bfp16(A)
    md, ed = planes_to_dev(mant, exp)
    Bd = bf16_bits_to_dev(Bb)
    Cr, S = oracle.gemm(mant, exp, Bb)
    for tiling in TILINGS:
        acc = fp32_accumulators(M, N, K, tiling, md, ed, Bd)
        want_m, want_e = oracle.quantize_bfp16(np.ascontiguousarray(acc))
        got_m, plane = run_qout(M, N, K, tiling, md, ed, Bd)
        got_e = atb.exp_plane_to_logical(plane, M, N)
        assert np.array_equal(got_e, want_e), tiling
        assert np.array_equal(got_m, want_m), tiling
        # padding rows of the exponent plane are written as 0, nothing else is touched
        m_pad = -(-M // 32) * 32
        p3 = plane.reshape(-(-N // 64), m_pad, 8)
        assert np.all(p3[:, M:, :] == 0)
        # pin (2): against the FP64 oracle
        Cq = oracle.dequantize(got_m, got_e)
        half_step = np.repeat(np.ldexp(1.0, got_e.astype(np.int64) - 134), 8, axis=1)
        q_err = np.where(np.abs(got_m.astype(np.int64)) == 127, 2.0 * half_step, half_step)
        assert np.all(np.abs(Cq - Cr) <= q_err + S * 2.0 ** -12), tiling
    ref_m, ref_plane = run_qout(M, N, K, (128, 256, 64, 256), md, ed, Bd)
    for tiling in PAIR_TILINGS:
        got_m, plane = run_qout(M, N, K, tiling, md, ed, Bd)
        assert np.array_equal(got_m, ref_m) and np.array_equal(plane, ref_plane), tiling
        got_e = atb.exp_plane_to_logical(plane, M, N)
        Cq = oracle.dequantize(got_m, got_e)
        half_step = np.repeat(np.ldexp(1.0, got_e.astype(np.int64) - 134), 8, axis=1)
        q_err = np.where(np.abs(got_m.astype(np.int64)) == 127, 2.0 * half_step, half_step)
        assert np.all(np.abs(Cq - Cr) <= q_err + S * 2.0 ** -12), tiling


def test_stacked_tiling_with_one_tile_row():
    """(T_MA, 128, 128, 256) on M <= 128 runs on single CTAs (as in atb_gemm): planes equal those of the T_K = 64 form
    of the same tile, whose UMMAs add the same products in the same order."""
    M, N, K = 100, 528, 448
    A = inputs.make_A("laplace", M, K)
    Bb = inputs.make_B_bits(K, N)
    mant, exp = oracle.quantize_bfp16(A)
    md, ed = planes_to_dev(mant, exp)
    Bd = bf16_bits_to_dev(Bb)
    ref_m, ref_plane = run_qout(M, N, K, (128, 128, 64, 256), md, ed, Bd)
    for tiling in [(64, 128, 128, 256), (128, 128, 128, 256)]:
        got_m, plane = run_qout(M, N, K, tiling, md, ed, Bd)
        assert np.array_equal(got_m, ref_m) and np.array_equal(plane, ref_plane), tiling


def test_output_feeds_the_next_gemm():
    """C in BFP16 is a valid A operand: chain two products and compare with the oracle's chain."""
    M, K1, K2, N2 = 384, 256, 512, 264
    A = inputs.make_A("normal", M, K1)
    B1 = inputs.make_B_bits(K1, K2)
    B2 = inputs.make_B_bits(K2, N2)
    mant, exp = oracle.quantize_bfp16(A)
    md, ed = planes_to_dev(mant, exp)
    Cm, Ce = atb.atb_gemm_bfp16_out(M, K2, K1, 128, 256, 64, 256, md, ed, bf16_bits_to_dev(B1))
    C2 = atb.atb_gemm(M, N2, K2, 64, 128, 64, 128, Cm, Ce, bf16_bits_to_dev(B2))
    atb.atb_device_status()
    mid_m = Cm.cpu().numpy()
    mid_e = atb.exp_plane_to_logical(Ce.cpu().numpy(), M, K2)
    Cr, S = oracle.gemm(mid_m, mid_e, B2)
    bits = C2.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    bad, ratio = oracle.check_tolerance(bits, Cr, S)
    assert bad == 0 and ratio < 0.75


def test_special_values_in_the_accumulator():
    """Zero blocks give E = 0, m = 0; a block whose largest element is a power of two lands on m = 64."""
    M, N, K = 128, 128, 64
    mant = np.zeros((M, K), np.int8)
    exp = np.full((M, K // 8), 133, np.uint8)             # scale 2^0
    mant[0, 0] = 1                                         # row 0 of A = e_0
    Bf = np.zeros((K, N), np.float32)
    Bf[0, :8] = [64, -32, 1, 0, 0.5, -0.25, 3, -64]        # first block of C row 0
    Bf[0, 8:16] = 2.0 ** -100
    md, ed = planes_to_dev(mant, exp)
    Cm, Ce = atb.atb_gemm_bfp16_out(M, N, K, 64, 128, 64, 128, md, ed, bf16_bits_to_dev(inputs.to_bf16_bits(Bf)))
    atb.atb_device_status()
    got_m = Cm.cpu().numpy()
    got_e = atb.exp_plane_to_logical(Ce.cpu().numpy(), M, N)
    assert got_e[0, 0] == 133 and list(got_m[0, :8]) == [64, -32, 1, 0, 0, 0, 3, -64]   # 0.5 and -0.25 tie to even 0
    assert got_e[0, 1] == 27 and list(got_m[0, 8:16]) == [64] * 8
    assert np.all(got_e[1:] == 0) and np.all(got_m[1:] == 0) and np.all(got_e[0, 2:] == 0)


def test_argument_errors():
    lib = atb.load_library()
    t = torch.zeros(256 * 256, dtype=torch.int8, device=dev())
    p = t.data_ptr()
    assert lib.atb_gemm_bfp16_out(256, 264, 256, 64, 128, 64, 128, p, p, p, 264, p, p, None) == 2      # N % 16
    assert lib.atb_gemm_bfp16_out(256, 256, 256, 32, 128, 64, 128, p, p, p, 256, p, p, None) == 3      # tiling
    assert lib.atb_gemm_bfp16_out(256, 256, 256, 32, 128, 128, 256, p, p, p, 256, p, p, None) == 3     # 32-row slabs: none
    assert lib.atb_gemm_bfp16_out(256, 256, 256, 128, 256, 128, 256, p, p, p, 256, p, p, None) == 3    # T_K = 128 elsewhere
    assert lib.atb_gemm_bfp16_out(256, 256, 256, 64, 128, 64, 128, p, p, p, 256, None, p, None) == 1   # NULL
    assert lib.atb_gemm_bfp16_out(256, 256, 256, 64, 128, 64, 128, p, p, p, 256, p + 8, p, None) == 4  # alignment


def test_full_size_headline_shape_sampled_rows():
    """8192^3 in the benchmark's launch configuration: sampled rows of the BFP16 planes against the
    quantiser on the kernel's FP32 accumulators (bit exact) and against the FP64 oracle GEMM."""
    c = inputs.CONFIGS["cfg3_8192"]
    M, N, K = c["M"], c["N"], c["K"]
    A, Bb = inputs.make_config("cfg3_8192")
    mant_d, plane_d = atb.atb_quantize_bfp16(torch.from_numpy(A).to(dev()))
    Bd = bf16_bits_to_dev(Bb)
    tiling = (128, 256, 64, 256)
    rows = np.unique(np.concatenate([np.arange(0, M, 256), np.arange(255, M, 256),
                                     np.random.default_rng(5).integers(0, M, 32)])).astype(np.int64)
    rows_d = torch.from_numpy(rows).to(dev())
    ws = torch.empty(atb.atb_gemm_splitk_workspace_bytes(M, N, tiling[1], 1) // 4, dtype=torch.float32, device=dev())
    atb.atb_gemm_splitk(M, N, K, *tiling, mant_d, plane_d, Bd, 1, workspace=ws)
    acc = ws.view(M, N)[rows_d].cpu().numpy()
    del ws
    Cm, Ce = atb.atb_gemm_bfp16_out(M, N, K, *tiling, mant_d, plane_d, Bd)
    atb.atb_device_status()
    got_m = Cm[rows_d].cpu().numpy()
    got_e = atb.exp_plane_to_logical(Ce.cpu().numpy(), M, N)[rows]
    want_m, want_e = oracle.quantize_bfp16(np.ascontiguousarray(acc))
    assert np.array_equal(got_e, want_e) and np.array_equal(got_m, want_m)
    mant_o, exp_o = oracle.quantize_bfp16(A[rows])
    Cr, S = oracle.gemm(mant_o, exp_o, Bb)
    half_step = np.repeat(np.ldexp(1.0, got_e.astype(np.int64) - 134), 8, axis=1)
    q_err = np.where(np.abs(got_m.astype(np.int64)) == 127, 2.0 * half_step, half_step)
    assert np.all(np.abs(oracle.dequantize(got_m, got_e) - Cr) <= q_err + S * 2.0 ** -12)
