"""GPU parity of atb_gemm_config: the paper's precision configurations (Section 6.1) with the BFP16
operand on the B side.  The reference is the plain definition: the FP64 product of the operands as
given - bf16 A (config 1) or dequantised BFP16 A (config 2) times the dequantised BFP16 B - with the
acceptance rule of atb_gemm for a bf16 C and that of atb_gemm_bfp16_out for a BFP16 C."""
import numpy as np
import pytest
import torch

import oracle
import paper_2511_16041_b200 as atb
from paper_2511_16041_b200 import inputs
from tests.gpu_util import dev, planes_to_dev, bf16_bits_to_dev, bf16_dev_to_bits

pytestmark = pytest.mark.gpu


def make_Bt_planes(K, N, seed):
    """B (K x N, fp32) and the oracle's BFP16 planes of its transpose."""
    Bf = inputs.make_A("normal", N, K, seed=seed)
    mant, exp = oracle.quantize_bfp16(Bf)
    return mant, exp


def ref_product(A64, Bt_mant, Bt_exp):
    """FP64 C = A x dequant(Bt)^T and S = |A| x |dequant(Bt)|^T."""
    Bd = oracle.dequantize(Bt_mant, Bt_exp)            # N x K, float64, exact
    return A64 @ Bd.T, np.abs(A64) @ np.abs(Bd).T


@pytest.mark.parametrize("shape", [(256, 256, 256), (300, 272, 448), (1000, 528, 1104)])
def test_config1_bf16_A_bfp16_B(shape):
    M, N, K = shape
    A_bits = inputs.to_bf16_bits(inputs.make_A("laplace", M, K))
    A64 = inputs.bf16_bits_to_f32(A_bits).astype(np.float64)
    Bt_mant, Bt_exp = make_Bt_planes(K, N, 3)
    Cr, S = ref_product(A64, Bt_mant, Bt_exp)
    bm, be = planes_to_dev(Bt_mant, Bt_exp)
    Ad = bf16_bits_to_dev(A_bits)
    C = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=dev())
    atb.atb_gemm_config(1, M, N, K, Ad, None, bm, be, C)
    atb.atb_device_status()
    bad, ratio = oracle.check_tolerance(bf16_dev_to_bits(C), Cr, S)
    assert bad == 0 and ratio < 0.75, (shape, bad, ratio)


def test_config1_equals_atb_gemm_on_the_transposed_problem():
    """C = A x B computed with B in BFP16 (config 1) and C^T = B^T x A^T computed by atb_gemm with
    B^T as its BFP16 operand are the same numbers: both accumulate the same products in FP32."""
    M, N, K = 512, 384, 512
    A_bits = inputs.to_bf16_bits(inputs.make_A("normal", M, K))
    Bt_mant, Bt_exp = make_Bt_planes(K, N, 5)
    bm, be = planes_to_dev(Bt_mant, Bt_exp)
    Ad = bf16_bits_to_dev(A_bits)
    C1 = atb.atb_gemm_config(1, M, N, K, Ad, None, bm, be)
    At = Ad.t().contiguous()                                     # K x M, the bf16 operand of the transposed product
    Ct = atb.atb_gemm(N, M, K, 128, 256, 64, 256, bm, be, At)
    atb.atb_device_status()
    Cr, S = ref_product(inputs.bf16_bits_to_f32(A_bits).astype(np.float64), Bt_mant, Bt_exp)
    for bits in (bf16_dev_to_bits(C1), bf16_dev_to_bits(Ct.t().contiguous())):
        bad, ratio = oracle.check_tolerance(bits, Cr, S)
        assert bad == 0 and ratio < 0.75


@pytest.mark.parametrize("shape", [(256, 256, 256), (300, 272, 448), (1000, 528, 1104)])
def test_config2_all_bfp16(shape):
    M, N, K = shape
    A = inputs.make_A("laplace", M, K)
    am, ae = oracle.quantize_bfp16(A)
    Bt_mant, Bt_exp = make_Bt_planes(K, N, 7)
    Cr, S = ref_product(oracle.dequantize(am, ae), Bt_mant, Bt_exp)
    amd, aed = planes_to_dev(am, ae)
    bm, be = planes_to_dev(Bt_mant, Bt_exp)
    Cm = torch.full((M, N), 55, dtype=torch.int8, device=dev())
    Ce = torch.full((atb.atb_bfp16_exp_bytes(M, N),), 199, dtype=torch.uint8, device=dev())
    atb.atb_gemm_config(2, M, N, K, amd, aed, bm, be, Cm, Ce)
    atb.atb_device_status()
    got_m = Cm.cpu().numpy()
    got_e = atb.exp_plane_to_logical(Ce.cpu().numpy(), M, N)
    Cq = oracle.dequantize(got_m, got_e)
    half_step = np.repeat(np.ldexp(1.0, got_e.astype(np.int64) - 134), 8, axis=1)
    q_err = np.where(np.abs(got_m.astype(np.int64)) == 127, 2.0 * half_step, half_step)
    assert np.all(np.abs(Cq - Cr) <= q_err + S * 2.0 ** -12), shape
    # the block exponent is the exponent of the block's largest magnitude: never off by more than one
    # from the oracle's exponent of the exact product (FP32 accumulation moves a maximum across a
    # power of two at most)
    _, ref_e = oracle.quantize_bfp16(Cr.astype(np.float32))
    assert np.max(np.abs(got_e.astype(np.int64) - ref_e.astype(np.int64))) <= 1


def test_config2_matches_the_a_side_kernels_bit_for_bit_on_exact_data():
    """Small-integer operands make every product and sum exact in FP32, so the quantised C of config 2
    must equal the quantised C of atb_gemm_bfp16_out (BFP16 A x bf16 B) bit for bit."""
    M, N, K = 256, 256, 128
    rng = np.random.default_rng(11)
    am = rng.integers(-9, 10, size=(M, K)).astype(np.int8)
    ae = np.full((M, K // 8), 133, np.uint8)
    bm = rng.integers(-9, 10, size=(N, K)).astype(np.int8)
    be = np.full((N, K // 8), 133, np.uint8)
    amd, aed = planes_to_dev(am, ae)
    bmd, bed = planes_to_dev(bm, be)
    Cm2, Ce2 = atb.atb_gemm_config(2, M, N, K, amd, aed, bmd, bed)
    B_bits = inputs.to_bf16_bits(bm.T.astype(np.float32))
    Cm1, Ce1 = atb.atb_gemm_bfp16_out(M, N, K, 128, 256, 64, 256, amd, aed, bf16_bits_to_dev(B_bits))
    atb.atb_device_status()
    assert torch.equal(Cm1, Cm2) and torch.equal(Ce1, Ce2)
    want_m, want_e = oracle.quantize_bfp16((am.astype(np.float64) @ bm.T.astype(np.float64)).astype(np.float32))
    assert np.array_equal(Cm2.cpu().numpy(), want_m)
    assert np.array_equal(atb.exp_plane_to_logical(Ce2.cpu().numpy(), M, N), want_e)


def test_argument_errors():
    lib = atb.load_library()
    t = torch.zeros(256 * 256, dtype=torch.int8, device=dev())
    p = t.data_ptr()
    assert lib.atb_gemm_config(3, 256, 256, 256, p, p, 256, p, p, p, p, 256, None) == 3       # config
    assert lib.atb_gemm_config(1, 256, 264, 256, p, None, 256, p, p, p, None, 264, None) == 2  # N % 16
    assert lib.atb_gemm_config(2, 256, 256, 256, p, None, 256, p, p, p, p, 256, None) == 1     # config 2 needs A_exp
    assert lib.atb_gemm_config(1, 256, 256, 256, p, None, 250, p, p, p, None, 256, None) == 2  # lda


SLAB_HEIGHTS = (256, 128, 64, 32)            # T_MA: the symmetric form first, then rho = 2, 4, 8
FORMS = (256, 512)                           # T_MC: one SM, or a CTA pair that shares the converted B tile


@pytest.mark.parametrize("shape", [(512, 512, 512), (300, 272, 448), (1000, 528, 1104), (2048, 1040, 2064)])
def test_config1_every_slab_height_bitwise_and_against_the_definition(shape):
    """A streamed in slabs of T_MA rows through the resident BFP16 tile of B (the orientation of the
    paper's own experiment): only buffer lifetimes change with T_MA, and only who converts which half of
    the B tile changes between one SM and a CTA pair, so every slab height in either form gives the same
    bits, ragged edges included, and those bits pass the acceptance rule of the plain product."""
    M, N, K = shape
    A_bits = inputs.to_bf16_bits(inputs.make_A("laplace", M, K))
    A64 = inputs.bf16_bits_to_f32(A_bits).astype(np.float64)
    Bt_mant, Bt_exp = make_Bt_planes(K, N, 3)
    Cr, S = ref_product(A64, Bt_mant, Bt_exp)
    bm, be = planes_to_dev(Bt_mant, Bt_exp)
    Ad = bf16_bits_to_dev(A_bits)
    ref = None
    for mc in FORMS:
        for ma in SLAB_HEIGHTS:
            C = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=dev())
            atb.atb_gemm_config_tiled(1, M, N, K, ma, mc, 64, 256, Ad, None, bm, be, C)
            atb.atb_device_status()
            bits = bf16_dev_to_bits(C)
            if ref is None:
                ref = bits
                bad, ratio = oracle.check_tolerance(bits, Cr, S)
                assert bad == 0 and ratio < 0.75, (shape, ma, bad, ratio)
            assert np.array_equal(bits, ref), (shape, ma, mc)


@pytest.mark.parametrize("shape", [(512, 512, 512), (300, 272, 448), (1000, 528, 1104)])
def test_config2_every_slab_height_bitwise(shape):
    """All-BFP16 configuration: raw slabs of T_MA rows, each with its own buffer and barrier, converted
    in bundles (thin slabs) or as two operand units (256 rows).  The BFP16 planes of C are bit-identical
    for every slab height, and equal to those of the fixed-tiling entry point."""
    M, N, K = shape
    A = inputs.make_A("outlier", M, K)
    am, ae = oracle.quantize_bfp16(A)
    Bt_mant, Bt_exp = make_Bt_planes(K, N, 7)
    amd, aed = planes_to_dev(am, ae)
    bm, be = planes_to_dev(Bt_mant, Bt_exp)
    Cm0, Ce0 = atb.atb_gemm_config(2, M, N, K, amd, aed, bm, be)
    atb.atb_device_status()
    # the reference entry itself against the definition (half a quantisation step, a whole one where saturated)
    Cr, S = ref_product(oracle.dequantize(am, ae), Bt_mant, Bt_exp)
    got_e = atb.exp_plane_to_logical(Ce0.cpu().numpy(), M, N)
    got_m = Cm0.cpu().numpy()
    half_step = np.repeat(np.ldexp(1.0, got_e.astype(np.int64) - 134), 8, axis=1)
    q_err = np.where(np.abs(got_m.astype(np.int64)) == 127, 2.0 * half_step, half_step)
    assert np.all(np.abs(oracle.dequantize(got_m, got_e) - Cr) <= q_err + S * 2.0 ** -12), shape
    for mc in FORMS:
        for ma in SLAB_HEIGHTS:
            Cm = torch.full((M, N), 55, dtype=torch.int8, device=dev())
            Ce = torch.full((atb.atb_bfp16_exp_bytes(M, N),), 199, dtype=torch.uint8, device=dev())
            atb.atb_gemm_config_tiled(2, M, N, K, ma, mc, 64, 256, amd, aed, bm, be, Cm, Ce)
            atb.atb_device_status()
            assert torch.equal(Cm, Cm0) and torch.equal(Ce, Ce0), (shape, ma, mc)


def test_config_tiled_rejects_other_tilings():
    lib = atb.load_library()
    t = torch.zeros(256 * 256, dtype=torch.int8, device=dev())
    p = t.data_ptr()
    ok = lambda til: lib.atb_gemm_config_tiled(1, 256, 256, 256, *til, p, None, 256, p, p, p, None, 256, None)
    assert ok((128, 256, 64, 256)) == 0 and ok((32, 256, 64, 256)) == 0 and ok((128, 512, 64, 256)) == 0
    assert ok((128, 384, 64, 256)) == 3 and ok((128, 512, 64, 512)) == 3
    assert ok((128, 256, 64, 128)) == 3 and ok((128, 128, 64, 256)) == 3 and ok((48, 256, 64, 256)) == 3 and ok((128, 256, 128, 256)) == 3
    torch.cuda.synchronize()


@pytest.mark.parametrize("shape", [(8192, 4096, 1024), (4200, 4112, 2064)])
def test_pair_form_equals_single_cta_form_at_full_launch_size(shape):
    """Several waves of tiles over all 148 SMs (74 CTA pairs), ragged edges in the second shape: the planes
    / the bf16 C of the CTA-pair form equal those of the single-CTA form bit for bit, for both
    configurations, and sampled rows of config 1 pass the acceptance rule of the plain product."""
    M, N, K = shape
    g = torch.Generator(device=dev())
    g.manual_seed(5)
    A32 = torch.randn((M, K), device=dev(), generator=g)
    Bt32 = torch.randn((N, K), device=dev(), generator=g)
    A16 = A32.to(torch.bfloat16)
    am, ae = atb.atb_quantize_bfp16(A32)
    bm, be = atb.atb_quantize_bfp16(Bt32)
    C1 = {mc: atb.atb_gemm_config_tiled(1, M, N, K, 128, mc, 64, 256, A16, None, bm, be) for mc in FORMS}
    C2 = {mc: atb.atb_gemm_config_tiled(2, M, N, K, 64, mc, 64, 256, am, ae, bm, be) for mc in FORMS}
    atb.atb_device_status()
    assert torch.equal(C1[256].view(torch.int16), C1[512].view(torch.int16))
    assert torch.equal(C2[256][0], C2[512][0]) and torch.equal(C2[256][1], C2[512][1])
    rows = np.unique(np.concatenate([np.arange(0, M, 512), np.arange(255, M, 512), np.arange(256, M, 512), [M - 1],
                                     np.random.default_rng(1).integers(0, M, 48)]))
    rows_d = torch.from_numpy(rows).to(dev())
    A64 = inputs.bf16_bits_to_f32(A16[rows_d].view(torch.int16).cpu().numpy().view(np.uint16)).astype(np.float64)
    Bt_mant = bm.cpu().numpy()
    Bt_exp = atb.exp_plane_to_logical(be.cpu().numpy(), N, K)
    Cr, S = ref_product(A64, Bt_mant, Bt_exp)
    bad, ratio = oracle.check_tolerance(C1[512][rows_d].view(torch.int16).cpu().numpy().view(np.uint16), Cr, S)
    assert bad == 0 and ratio < 0.75, (shape, bad, ratio)
