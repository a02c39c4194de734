"""Pins for the oracle's FP64 GEMM, S = sum|a b| and the acceptance test.

The GEMM is the plain definition C = A x B (Section 1); asymmetric tile
buffering (Section 3) re-tiles it without changing the result.
"""
from fractions import Fraction

import numpy as np

import oracle
from paper_2511_16041_b200 import inputs
from tests import exact_ref


def _bf16_fraction(bits):
    return Fraction(float(inputs.bf16_bits_to_f32(np.array([bits], np.uint16))[0]))


def test_brute_force_tiny_exact_rational():
    rng = np.random.default_rng(11)
    for (M, N, K) in [(3, 5, 8), (16, 7, 16), (5, 16, 24), (1, 1, 8)]:
        mant = rng.integers(-127, 128, size=(M, K)).astype(np.int8)
        exp = rng.integers(100, 150, size=(M, K // 8)).astype(np.uint8)
        B = inputs.to_bf16_bits(rng.standard_normal((K, N)).astype(np.float32) * 3)
        C, S = oracle.gemm(mant, exp, B)
        for i in range(M):
            for j in range(N):
                acc, sabs = Fraction(0), Fraction(0)
                for k in range(K):
                    a = exact_ref.dequant(int(exp[i, k // 8]), int(mant[i, k]))
                    b = _bf16_fraction(B[k, j])
                    acc += a * b
                    sabs += abs(a * b)
                # FP64 accumulation of exact products: error <= K ulps of the running sums
                assert abs(Fraction(C[i, j]) - acc) <= Fraction(K, 2 ** 52) * sabs
                assert abs(Fraction(S[i, j]) - sabs) <= Fraction(K, 2 ** 52) * sabs


def _int_operands(rng, M, N, K):
    a = rng.integers(-1, 2, size=(M, K)).astype(np.float32)
    a[:, ::8] = np.where(a[:, ::8] == 0, 1, a[:, ::8])     # every block holds a +-1 -> exact
    b = rng.integers(-1, 2, size=(K, N)).astype(np.float32)
    return a, b


def test_small_integer_matrices_are_exact():
    rng = np.random.default_rng(5)
    a, b = _int_operands(rng, 40, 24, 256)
    mant, exp = oracle.quantize_bfp16(a)
    assert np.array_equal(oracle.dequantize(mant, exp), a.astype(np.float64))
    C, S = oracle.gemm(mant, exp, inputs.to_bf16_bits(b))
    assert np.array_equal(C, (a.astype(np.int64) @ b.astype(np.int64)).astype(np.float64))
    assert np.array_equal(S, (np.abs(a).astype(np.int64) @ np.abs(b).astype(np.int64)).astype(np.float64))


def test_identity_and_permutation_A():
    rng = np.random.default_rng(6)
    K = N = 64
    Bf = rng.standard_normal((K, N)).astype(np.float32)
    Bb = inputs.to_bf16_bits(Bf)
    Bv = inputs.bf16_bits_to_f32(Bb).astype(np.float64)
    eye = np.eye(K, dtype=np.float32)
    mant, exp = oracle.quantize_bfp16(eye)
    C, S = oracle.gemm(mant, exp, Bb)
    assert np.array_equal(C, Bv) and np.array_equal(S, np.abs(Bv))
    perm = rng.permutation(K)
    mant, exp = oracle.quantize_bfp16(eye[perm])
    C, _ = oracle.gemm(mant, exp, Bb)
    assert np.array_equal(C, Bv[perm])
    # a transposed-operand mistake would show here: A = shift matrix, not symmetric
    shift = np.roll(eye, 1, axis=1)
    mant, exp = oracle.quantize_bfp16(shift)
    C, _ = oracle.gemm(mant, exp, Bb)
    assert np.array_equal(C, np.roll(Bv, -1, axis=0))


def test_identity_B_returns_dequantised_A():
    a = inputs.make_A("laplace", 48, 64)
    mant, exp = oracle.quantize_bfp16(a)
    eye = inputs.to_bf16_bits(np.eye(64, dtype=np.float32))
    C, S = oracle.gemm(mant, exp, eye)
    d = oracle.dequantize(mant, exp)
    assert np.array_equal(C, d) and np.array_equal(S, np.abs(d))


def test_matches_library_matmul():
    a = inputs.make_A("normal", 33, 512)
    Bb = inputs.make_B_bits(512, 65)
    mant, exp = oracle.quantize_bfp16(a)
    C, S = oracle.gemm(mant, exp, Bb)
    d = oracle.dequantize(mant, exp)
    Bv = inputs.bf16_bits_to_f32(Bb).astype(np.float64)
    ref = d @ Bv
    sref = np.abs(d) @ np.abs(Bv)
    assert np.allclose(C, ref, rtol=0, atol=1e-12 * sref.max())
    assert np.allclose(S, sref, rtol=1e-13, atol=0)


def test_power_of_two_scaling_is_exact():
    a = inputs.make_A("normal", 8, 128)
    Bb = inputs.make_B_bits(128, 16)
    mant, exp = oracle.quantize_bfp16(a)
    C, S = oracle.gemm(mant, exp, Bb)
    C2, S2 = oracle.gemm(mant, (exp.astype(int) + 9).astype(np.uint8), Bb)
    assert np.array_equal(C2, C * 512.0) and np.array_equal(S2, S * 512.0)


def test_row_subset_matches_full():
    a = inputs.make_A("outlier", 64, 128)
    Bb = inputs.make_B_bits(128, 40, None)
    mant, exp = oracle.quantize_bfp16(a)
    C, S = oracle.gemm(mant, exp, Bb)
    rows = np.array([63, 0, 17, 17, 5], np.int64)
    Cr, Sr = oracle.gemm(mant, exp, Bb, rows=rows)
    assert np.array_equal(Cr, C[rows]) and np.array_equal(Sr, S[rows])
    Ce, Se = oracle.gemm(mant, exp, Bb, rows=np.zeros(0, np.int64))
    assert Ce.shape == (0, 40) and Se.shape == (0, 40)


def test_equal_exponents_reduce_to_integer_gemm():
    rng = np.random.default_rng(9)
    M, N, K = 12, 10, 64
    mant = rng.integers(-127, 128, size=(M, K)).astype(np.int8)
    exp = np.full((M, K // 8), 140, np.uint8)
    bi = rng.integers(-100, 101, size=(K, N))
    C, _ = oracle.gemm(mant, exp, inputs.to_bf16_bits(bi.astype(np.float32)))
    assert np.array_equal(C, (mant.astype(np.int64) @ bi) * 2.0 ** 7)


def test_tolerance_check_semantics():
    C_ref = np.array([[1.0, -2.0, 0.0, 100.0]])
    S = np.array([[4.0, 2.0, 0.0, 100.0]])
    bound = np.abs(C_ref) * 2.0 ** -7 + S * 2.0 ** -12

    def bits(v):
        return inputs.to_bf16_bits(np.asarray(v, np.float32))
    # exact values pass with ratio 0
    assert oracle.check_tolerance(bits(C_ref), C_ref, S) == (0, 0.0)
    # an error of one bf16 ulp of 1.0 (2^-7) on the first element: bound is 2^-7 + 2^-10
    bad, ratio = oracle.check_tolerance(bits([[1.0078125, -2.0, 0.0, 100.0]]), C_ref, S)
    assert bad == 0 and abs(ratio - 2.0 ** -7 / bound[0, 0]) < 1e-12
    # two ulps fail
    bad, ratio = oracle.check_tolerance(bits([[1.015625, -2.0, 0.0, 100.0]]), C_ref, S)
    assert bad == 1 and ratio > 1
    # sign error fails; zero reference with zero S demands exact zero
    assert oracle.check_tolerance(bits([[1.0, 2.0, 0.0, 100.0]]), C_ref, S)[0] == 1
    assert oracle.check_tolerance(bits([[1.0, -2.0, 1e-30, 100.0]]), C_ref, S)[0] == 1
    # non-finite output fails
    assert oracle.check_tolerance(bits([[np.inf, -2.0, 0.0, 100.0]]), C_ref, S)[0] == 1
    assert oracle.check_tolerance(bits([[np.nan, -2.0, 0.0, 100.0]]), C_ref, S)[0] == 1


def test_fp32_accumulate_bf16_round_model_sits_well_inside_tolerance():
    """A plain fp32-accumulate, single-RNE-to-bf16 evaluation of the same GEMM
    must pass the acceptance test with margin (the bound allows one bf16 ulp)."""
    a = inputs.make_A("laplace", 32, 1024)
    Bb = inputs.make_B_bits(1024, 48)
    mant, exp = oracle.quantize_bfp16(a)
    C, S = oracle.gemm(mant, exp, Bb)
    d32 = oracle.dequantize(mant, exp).astype(np.float32)
    b32 = inputs.bf16_bits_to_f32(Bb)
    acc = np.zeros((32, 48), np.float32)
    for k0 in range(0, 1024, 16):
        acc += d32[:, k0:k0 + 16] @ b32[k0:k0 + 16]
    bad, ratio = oracle.check_tolerance(inputs.to_bf16_bits(acc), C, S)
    assert bad == 0 and ratio < 0.6
