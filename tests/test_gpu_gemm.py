"""GPU parity: atb_gemm against the FP64 oracle.

Acceptance per element: |C_gpu - C_ref| <= 2^-7 |C_ref| + 2^-12 sum_k |a_ik b_kj| (evaluated by the
oracle's checker); exact equality where the result is exactly representable; bitwise equality
across T_MA for fixed (T_MC, T_K, T_N), because asymmetric tile buffering (Section 3) only changes
buffer lifetimes.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2511_16041_b200 as atb
from paper_2511_16041_b200 import inputs
from tests.gpu_util import run_gemm, dev, planes_to_dev, bf16_bits_to_dev, bf16_dev_to_bits

pytestmark = pytest.mark.gpu

ALL_TILINGS = [(ma, mc, k, n) for mc in (128, 256, 384) for n in (64, 128, 256, 512) for k in (64, 128)
               for ma in (32, 64, 128, 256) if ma <= mc and mc % ma == 0]


def supported():
    return [t for t in ALL_TILINGS if atb.atb_tiling_supported(*t)]


def _check(mant, exp, Bb, tiling, max_ratio=0.75):
    Cg = run_gemm(mant, exp, Bb, tiling)
    Cr, S = oracle.gemm(mant, exp, Bb)
    bad, ratio = oracle.check_tolerance(Cg, Cr, S)
    assert bad == 0, (tiling, bad, ratio)
    assert ratio <= max_ratio, (tiling, ratio)     # one RNE to bf16 sits near 0.25-0.5 of the bound
    return Cg


def test_config1_256_cubed():
    A, Bb = inputs.make_config("cfg1_256")
    mant, exp = oracle.quantize_bfp16(A)
    _check(mant, exp, Bb, (64, 128, 64, 128))


def test_every_supported_tiling_ragged_shape():
    """Shape that is a multiple of no tile extent: several tiles plus ragged tails in M and N,
    K not a multiple of 128."""
    M, N, K = 600, 328, 448
    A = inputs.make_A("laplace", M, K)
    Bb = inputs.make_B_bits(K, N)
    mant, exp = oracle.quantize_bfp16(A)
    Cr, S = oracle.gemm(mant, exp, Bb)
    tl = supported()
    assert len(tl) >= 20
    for t in tl:
        Cg = run_gemm(mant, exp, Bb, t)
        bad, ratio = oracle.check_tolerance(Cg, Cr, S)
        assert bad == 0 and ratio < 0.75, (t, bad, ratio)


def test_atb_invariance_bitwise_across_T_MA():
    M, N, K = 512, 512, 1024
    A = inputs.make_A("outlier", M, K)
    Bb = inputs.make_B_bits(K, N, None)
    mant, exp = oracle.quantize_bfp16(A)
    for (mc, k, n) in [(256, 64, 256), (256, 128, 128), (128, 64, 128), (256, 64, 512), (128, 128, 256)]:
        ref = None
        for ma in (32, 64, 128, 256):
            if ma > mc or not atb.atb_tiling_supported(ma, mc, k, n):
                continue
            Cg = run_gemm(mant, exp, Bb, (ma, mc, k, n))
            if ref is None:
                ref = Cg
            assert np.array_equal(Cg, ref), (ma, mc, k, n)


def test_cta_pair_equals_the_single_cta_tiling_bitwise():
    """The CTA-pair kernel (T_N = 512) adds the same products in the same order as the single-CTA 256 x 256
    tiling with the same T_K wherever no CTA computes more than one tile (a CTA's second tile walks K
    downwards): every element of C is bit-identical, ragged edges included."""
    for (M, N, K) in [(512, 1024, 1024), (1000, 1544, 1104)]:
        A = inputs.make_A("outlier", M, K)
        Bb = inputs.make_B_bits(K, N, None)
        mant, exp = oracle.quantize_bfp16(A)
        ref = run_gemm(mant, exp, Bb, (128, 256, 64, 256))
        for ma in (32, 64, 128):
            assert np.array_equal(run_gemm(mant, exp, Bb, (ma, 256, 64, 512)), ref), (M, N, K, ma)


def test_rho_that_is_not_a_power_of_two():
    """T_MC = 384 (three 128-row groups): rho = 3, 6 and 12 (the paper's Table 2 uses rho = 6).  Several
    tiles and ragged tails; bitwise equal across T_MA like every other (T_MC, T_K, T_N)."""
    M, N, K = 1000, 392, 1104
    A = inputs.make_A("normal", M, K)
    Bb = inputs.make_B_bits(K, N)
    mant, exp = oracle.quantize_bfp16(A)
    for (tk, tn) in [(64, 128), (64, 64), (128, 128)]:
        ref = None
        for ma in (128, 64, 32):
            if not atb.atb_tiling_supported(ma, 384, tk, tn):
                continue
            Cg = _check(mant, exp, Bb, (ma, 384, tk, tn))
            ref = Cg if ref is None else ref
            assert np.array_equal(Cg, ref), (ma, tk, tn)
        assert ref is not None


def test_small_integer_matrices_exact():
    rng = np.random.default_rng(5)
    M, N, K = 384, 256, 256
    a = rng.integers(-1, 2, size=(M, K)).astype(np.float32)
    a[:, ::8] = np.where(a[:, ::8] == 0, 1, a[:, ::8])
    b = rng.integers(-1, 2, size=(K, N)).astype(np.float32)
    mant, exp = oracle.quantize_bfp16(a)
    Cr, _ = oracle.gemm(mant, exp, inputs.to_bf16_bits(b))
    for t in [(128, 128, 64, 128), (64, 256, 64, 256), (64, 256, 128, 64), (128, 256, 64, 512), (128, 128, 64, 512)]:
        Cg = run_gemm(mant, exp, inputs.to_bf16_bits(b), t)
        assert np.array_equal(inputs.bf16_bits_to_f32(Cg).astype(np.float64), Cr), t


def test_identity_B_returns_dequantised_A_bitwise():
    """B = I isolates the dequantiser: C must be m * 2^(E-133) exactly (it is a bf16 value)."""
    M, K = 256, 256
    A = inputs.make_A("laplace", M, K)
    mant, exp = oracle.quantize_bfp16(A)
    eye = inputs.to_bf16_bits(np.eye(K, dtype=np.float32))
    want = oracle.dequantize(mant, exp)
    for t in [(64, 128, 64, 128), (128, 256, 128, 256), (32, 256, 64, 64), (64, 256, 64, 512)]:
        if not atb.atb_tiling_supported(*t):
            continue
        Cg = run_gemm(mant, exp, eye, t)
        assert np.array_equal(inputs.bf16_bits_to_f32(Cg).astype(np.float64), want), t


def test_permutation_A_returns_permuted_B_bitwise():
    K = N = 256
    rng = np.random.default_rng(8)
    perm = rng.permutation(K)
    a = np.eye(K, dtype=np.float32)[perm]
    Bb = inputs.make_B_bits(K, N)
    mant, exp = oracle.quantize_bfp16(a)
    Cg = run_gemm(mant, exp, Bb, (128, 256, 64, 128))
    assert np.array_equal(Cg, Bb[perm])


def test_largest_exponents_among_ordinary_blocks_every_tiling():
    """Blocks with E = 253 and 254 (the dequantiser converts a thread's share of a slab a second time,
    in another form, when it meets E >= 254) and blocks with bf16-subnormal scales, sprinkled among
    ordinary ones so that some threads of a slab take that path and others do not.  B = 2^j I makes every
    product a single term: the result must be the dequantised element, exactly, wherever it is a normal
    bf16 number."""
    M, K = 520, 256
    rng = np.random.default_rng(254)
    mant = rng.integers(-127, 128, (M, K), dtype=np.int8)
    exp = rng.integers(118, 136, (M, K // 8)).astype(np.uint8)
    pick = rng.random((M, K // 8))
    exp[pick < 0.04] = 254
    exp[(pick >= 0.04) & (pick < 0.07)] = 253
    exp[(pick >= 0.07) & (pick < 0.10)] = rng.integers(0, 7, int(((pick >= 0.07) & (pick < 0.10)).sum())).astype(np.uint8)
    exp[300:428] = rng.integers(120, 130, (128, K // 8)).astype(np.uint8)      # a 128-row group without any
    assert (exp == 254).sum() > 100
    deq = oracle.dequantize(mant, exp)
    for shift in (0, 60):
        Bb = inputs.to_bf16_bits(np.eye(K, dtype=np.float32) * np.float32(2.0 ** shift))
        want = deq * 2.0 ** shift
        normal = ((np.abs(want) >= 2.0 ** -126) & (np.abs(want) < 2.0 ** 127)) | (want == 0)
        assert normal.mean() > 0.85
        assert shift != 0 or (normal & (want != 0) & (exp.repeat(8, axis=1) == 254)).sum() > 1000
        for t in supported():
            got = inputs.bf16_bits_to_f32(run_gemm(mant, exp, Bb, t)).astype(np.float64)
            assert np.array_equal(got[normal], want[normal]), (t, shift)


def test_dequant_every_exponent_through_the_kernel():
    """All 255 block exponents (incl. bf16-subnormal results and the E >= 238 branch) times all
    mantissas, read back through B = 2^j I so that the product stays a normal fp32 / bf16 value."""
    K = 256
    mvals = np.arange(-127, 128, dtype=np.int8)
    for lo, hi, shift in [(0, 85, 100), (85, 170, 20), (170, 255, -60)]:
        Es = np.arange(lo, hi, dtype=np.uint8)
        M = len(Es) * 8                       # 8 rows per exponent, 255 mantissas spread over them
        mant = np.zeros((M, K), np.int8)
        exp = np.zeros((M, K // 8), np.uint8)
        for i, E in enumerate(Es):
            block = np.resize(mvals, 8 * K).reshape(8, K)
            mant[i * 8:(i + 1) * 8] = block
            exp[i * 8:(i + 1) * 8] = E
        Bb = inputs.to_bf16_bits(np.eye(K, dtype=np.float32) * np.float32(2.0 ** shift))
        Cg = run_gemm(mant, exp, Bb, (128, 128, 64, 128))
        want = oracle.dequantize(mant, exp) * 2.0 ** shift
        got = inputs.bf16_bits_to_f32(Cg).astype(np.float64)
        normal = (np.abs(want) >= 2.0 ** -126) | (want == 0)
        assert normal.mean() > 0.9
        assert np.array_equal(got[normal], want[normal]), (lo, hi)


def test_leading_dimensions_and_untouched_padding():
    M, N, K = 256, 136, 128
    A = inputs.make_A("normal", M, K)
    Bb = inputs.make_B_bits(K, N)
    mant, exp = oracle.quantize_bfp16(A)
    md, ed = planes_to_dev(mant, exp)
    ldb, ldc = 200, 160
    Bfull = torch.zeros((K, ldb), dtype=torch.bfloat16, device=dev())
    Bfull[:, :N] = bf16_bits_to_dev(Bb)
    Bfull[:, N:] = 3.0                                   # must not leak into C
    Cfull = torch.full((M, ldc), -5.0, dtype=torch.bfloat16, device=dev())
    atb.atb_gemm(M, N, K, 64, 128, 64, 64, md, ed, Bfull, Cfull, ldb=ldb, ldc=ldc)
    atb.atb_device_status()
    Cr, S = oracle.gemm(mant, exp, Bb)
    bad, ratio = oracle.check_tolerance(bf16_dev_to_bits(Cfull[:, :N]), Cr, S)
    assert bad == 0
    assert torch.all(Cfull[:, N:] == -5.0)


def test_leading_dimensions_ragged_edges_every_epilogue():
    """The two ways C leaves a kernel - TMA stores clipped by the tensor map (single-CTA tilings, the CTA pair
    under 32-row slabs) and plain 16-byte stores guarded row by row and chunk by chunk (the CTA pair under
    64- and 128-row slabs) - on a shape whose last tiles are ragged in M and N (N ends 8 columns into a
    64-column box), with ldb > N and ldc > N: C is right, and not a byte of the padding is touched."""
    M, N, K = 300, 584, 192
    A = inputs.make_A("normal", M, K)
    Bb = inputs.make_B_bits(K, N)
    mant, exp = oracle.quantize_bfp16(A)
    md, ed = planes_to_dev(mant, exp)
    Cr, S = oracle.gemm(mant, exp, Bb)
    ldb, ldc = 600, 640
    Bfull = torch.full((K, ldb), 3.0, dtype=torch.bfloat16, device=dev())          # padding must not leak into C
    Bfull[:, :N] = bf16_bits_to_dev(Bb)
    for t in [(128, 256, 64, 256), (128, 256, 64, 512), (64, 256, 64, 512), (32, 256, 64, 512), (128, 128, 64, 128),
              (128, 128, 128, 256), (32, 128, 128, 256)]:
        Cfull = torch.full((M + 3, ldc), -5.0, dtype=torch.bfloat16, device=dev())  # three guard rows below C
        atb.atb_gemm(M, N, K, *t, md, ed, Bfull, Cfull, ldb=ldb, ldc=ldc)
        atb.atb_device_status()
        bad, ratio = oracle.check_tolerance(bf16_dev_to_bits(Cfull[:M, :N].contiguous()), Cr, S)
        assert bad == 0 and ratio < 0.75, (t, bad, ratio)
        assert torch.all(Cfull[:M, N:] == -5.0) and torch.all(Cfull[M:] == -5.0), t


def test_tiny_and_degenerate_shapes():
    for (M, N, K) in [(1, 8, 64), (7, 24, 64), (129, 72, 192), (5, 16, 16), (130, 264, 80), (300, 40, 464)]:
        A = inputs.make_A("normal", M, K)
        Bb = inputs.make_B_bits(K, N)
        mant, exp = oracle.quantize_bfp16(A)
        _check(mant, exp, Bb, (128, 128, 64, 64))
        _check(mant, exp, Bb, (32, 256, 128, 128))
        _check(mant, exp, Bb, (128, 256, 64, 512))       # CTA-pair kernel on a single partial tile
        _check(mant, exp, Bb, (64, 128, 128, 256))       # stacked pair of tiles (single CTAs where M <= 128)


def test_argument_errors():
    lib = atb.load_library()
    M = N = K = 256
    md = torch.zeros((M, K), dtype=torch.int8, device=dev())
    ed = torch.zeros(atb.atb_bfp16_exp_bytes(M, K), dtype=torch.uint8, device=dev())
    B = torch.zeros((K, N), dtype=torch.bfloat16, device=dev())
    C = torch.zeros((M, N), dtype=torch.bfloat16, device=dev())

    def call(M=M, N=N, K=K, til=(64, 128, 64, 128), a=md.data_ptr(), e=ed.data_ptr(), b=B.data_ptr(),
             c=C.data_ptr(), ldb=N, ldc=N):
        return lib.atb_gemm(M, N, K, *til, a, e, b, ldb, c, ldc, None)

    assert call() == 0
    assert call(a=None) == 1
    assert call(K=100) == 2 and call(K=72) == 2 and call(N=12) == 2 and call(M=0) == 2 and call(ldb=N - 8) == 2
    assert call(til=(64, 128, 64, 96)) == 3          # unsupported T_N
    assert call(til=(256, 128, 64, 128)) == 3        # T_MA > T_MC
    assert call(til=(256, 256, 128, 256)) == 3       # shared-memory rings do not fit
    assert call(b=B.data_ptr() + 2) == 4
    assert "T_MA" in atb.atb_last_error_message() or atb.atb_last_error_message() != ""
    torch.cuda.synchronize()


def _sampled_rows(M, T_MC, n_random, seed):
    edges = np.concatenate([np.arange(0, M, T_MC), np.arange(T_MC - 1, M, T_MC)])
    rnd = np.random.default_rng(seed).integers(0, M, n_random)
    return np.unique(np.concatenate([edges, rnd])).astype(np.int64)


@pytest.mark.parametrize("name,tilings", [
    ("cfg2_4096", [(32, 256, 64, 256), (64, 256, 64, 256), (128, 256, 64, 256), (256, 256, 64, 256)]),
    ("cfg3_8192", ["selected", (128, 256, 64, 256), (256, 256, 64, 256), (128, 256, 64, 512)]),
    ("cfg4_ffn_up", ["selected"]),
    ("cfg4_ffn_down", ["selected"]),
])
def test_full_size_configs_sampled_rows(name, tilings):
    """The benchmark's launch configuration at full size; the oracle evaluates the first and last
    row of every T_MC tile plus random rows (all N columns)."""
    c = inputs.CONFIGS[name]
    M, N, K = c["M"], c["N"], c["K"]
    A, Bb = inputs.make_config(name)
    Ad = torch.from_numpy(A).to(dev())
    mant_d, plane_d = atb.atb_quantize_bfp16(Ad)        # the device quantiser feeds the device GEMM
    del Ad
    Bd = bf16_bits_to_dev(Bb)
    n_rand = 512 if name.startswith("cfg4") else 96
    rows = _sampled_rows(M, 256, n_rand, 17)
    mant_o, exp_o = oracle.quantize_bfp16(A[rows])
    del A
    # the device planes must equal the oracle's on the sampled rows (bit exact)
    rows_d = torch.from_numpy(rows).to(dev())
    assert np.array_equal(mant_d[rows_d].cpu().numpy(), mant_o)
    assert np.array_equal(atb.exp_plane_to_logical(plane_d.cpu().numpy(), M, K)[rows], exp_o)
    Cr, S = oracle.gemm(mant_o, exp_o, Bb)
    first = None
    for t in tilings:
        if t == "selected":
            t, _ = atb.atb_select_tiling(M, N, K)
        C = atb.atb_gemm(M, N, K, *t, mant_d, plane_d, Bd)
        atb.atb_device_status()
        Cg = bf16_dev_to_bits(C[rows_d])
        bad, ratio = oracle.check_tolerance(Cg, Cr, S)
        assert bad == 0 and ratio < 0.75, (name, t, bad, ratio)
        assert bool(torch.isfinite(C.float()).all())
        if name == "cfg2_4096":                      # same (T_MC, T_K, T_N): bitwise equal across T_MA
            full = bf16_dev_to_bits(C)
            if first is None:
                first = full
            assert np.array_equal(full, first), t
