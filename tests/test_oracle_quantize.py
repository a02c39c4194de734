"""Pins for the oracle's BFP16 quantiser / dequantiser (Section 2.4 format)."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2511_16041_b200 import inputs
from tests import exact_ref

HERE = os.path.dirname(os.path.abspath(__file__))


def f32(v):
    return np.asarray(v, dtype=np.float32)


def q1(block):
    m, e = oracle.quantize_bfp16(f32(block).reshape(1, 8))
    return int(e[0, 0]), [int(v) for v in m[0]]


def _parse(tok):
    return float.fromhex(tok) if "0x" in tok else float(tok)


def golden_blocks():
    out = []
    with open(os.path.join(HERE, "golden", "bfp16_blocks.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            xs, E, ms = line.split("|")
            out.append(([_parse(t) for t in xs.split()], int(E), [int(t) for t in ms.split()]))
    return out


@pytest.mark.parametrize("xs,E,ms", golden_blocks())
def test_hand_worked_blocks(xs, E, ms):
    x32 = [float(v) for v in f32(xs)]
    assert exact_ref.quantize_block(x32) == (E, ms)      # the fixture itself is right
    assert q1(xs) == (E, ms)


def _random_blocks(rng, n):
    """Blocks mixing magnitudes over the whole fp32 range, ties, zeros, specials."""
    kind = rng.integers(0, 6, size=n)
    out = np.empty((n, 8), np.float32)
    for i in range(n):
        k = kind[i]
        if k == 0:
            b = rng.standard_normal(8)
        elif k == 1:
            b = rng.standard_normal(8) * 2.0 ** rng.integers(-140, 120)
        elif k == 2:     # exact half-integers relative to the scale -> ties
            e = int(rng.integers(-100, 100))
            b = (rng.integers(-255, 256, size=8) * 0.5) * 2.0 ** e
            b[rng.integers(0, 8)] = 100.0 * 2.0 ** e
        elif k == 3:     # wide dynamic range inside the block
            b = rng.standard_normal(8) * 2.0 ** rng.integers(-30, 5, size=8)
        elif k == 4:     # subnormal / tiny
            b = rng.integers(-2 ** 23, 2 ** 23, size=8) * 2.0 ** -149 * rng.integers(0, 3)
        else:            # near the saturation boundary
            e = int(rng.integers(-20, 20))
            b = (127.0 + rng.integers(-4, 5, size=8) * 0.25) * 2.0 ** e * rng.choice([-1, 1], 8)
        with np.errstate(over="ignore"):
            out[i] = b.astype(np.float32)
    return out


def test_against_exact_rational_random():
    rng = np.random.default_rng(1234)
    blocks = _random_blocks(rng, 6000)
    m, e = oracle.quantize_bfp16(blocks)
    for i in range(blocks.shape[0]):
        E, ms = exact_ref.quantize_block([float(v) for v in blocks[i]])
        assert int(e[i, 0]) == E, (i, blocks[i])
        assert [int(v) for v in m[i]] == ms, (i, blocks[i])


def test_specials():
    nan, inf = float("nan"), float("inf")
    assert q1([nan] * 8) == (0, [0] * 8)
    assert q1([nan, 1, 0, 0, 0, 0, 0, 0]) == (127, [0, 64, 0, 0, 0, 0, 0, 0])
    assert q1([inf, -inf, 1e38, nan, 0, 0, 0, 0]) == (254, [127, -127, 38, 0, 0, 0, 0, 0])
    E, ms = exact_ref.quantize_block([inf, -inf, float(np.float32(1e38)), nan, 0, 0, 0, 0])
    assert (E, ms) == (254, [127, -127, 38, 0, 0, 0, 0, 0])
    # largest finite fp32: exponent field 254
    big = float(np.finfo(np.float32).max)
    assert q1([big, -big, 0, 0, 0, 0, 0, 0]) == (254, [127, -127, 0, 0, 0, 0, 0, 0])
    # -0.0 behaves like 0
    assert q1([-0.0] * 8) == (0, [0] * 8)
    # smallest normal and largest subnormal
    assert q1([2.0 ** -126] + [0] * 7)[0] == 1
    assert q1([2.0 ** -126 - 2.0 ** -149] + [0] * 7)[0] == 0


def test_single_nonzero_all_bf16_values():
    """Every bf16 bit pattern as the only non-zero element of a block."""
    bits = np.arange(1 << 16, dtype=np.uint16)
    vals = inputs.bf16_bits_to_f32(bits)
    blocks = np.zeros((1 << 16, 8), np.float32)
    blocks[:, 3] = vals
    m, e = oracle.quantize_bfp16(blocks)
    expf = (bits >> 7) & 0xFF
    frac = bits & 0x7F
    sign = np.where(bits >> 15, -1, 1)
    normal = (expf >= 1) & (expf <= 254)
    # normal bf16 value = (128+frac) * 2^(expf-134): E = expf, m = (128+frac)/2 rounded to even
    mm = 128 + frac.astype(np.int64)
    half = mm // 2 + ((mm % 2 == 1) & ((mm // 2) % 2 == 1))
    half = np.minimum(half, 127)
    assert np.array_equal(e[normal, 0], expf[normal].astype(np.uint8))
    assert np.array_equal(m[normal, 3].astype(np.int64), (sign * half)[normal])
    sub = expf == 0          # value = frac * 2^-133 -> E = 0, m = frac
    assert np.all(e[sub, 0] == 0)
    assert np.array_equal(m[sub, 3].astype(np.int64), (sign * frac)[sub])
    isinf = (expf == 255) & (frac == 0)
    assert np.all(e[isinf, 0] == 254)
    assert np.array_equal(m[isinf, 3].astype(np.int64), (sign * 127)[isinf])
    isnan = (expf == 255) & (frac != 0)
    assert np.all(e[isnan, 0] == 0) and np.all(m[isnan, 3] == 0)
    others = np.delete(np.arange(8), 3)
    assert np.all(m[:, others] == 0)


def test_block_max_sweep_with_integer_bit_reference():
    """All 2^23 fractions of one binade as block maximum with a fixed partner grid,
    against a vectorised integer-bit re-statement (different from the oracle's ldexp)."""
    n = 1 << 18                       # every 32nd fraction of the binade [2^3, 2^4)
    frac = (np.arange(n, dtype=np.uint32) << np.uint32(5))
    amax = ((np.uint32(130) << np.uint32(23)) | frac).view(np.float32)
    grid = np.array([1.0, -0.5, 0.03125, 7.96875, -15.9375, 0.0625 * 3, 1e-3], np.float32)
    blocks = np.empty((n, 8), np.float32)
    blocks[:, 0] = amax
    blocks[:, 1:] = grid[None, :]
    blocks[:, 5] = np.minimum(np.abs(blocks[:, 5]), amax) * -1.0
    m, e = oracle.quantize_bfp16(blocks)
    assert np.all(e[:, 0] == 130)
    # scale 2^-3: q = x*8 exactly representable in fp64; RNE by integer arithmetic on x*2^30
    fixed = np.round(blocks.astype(np.float64) * 2.0 ** 30).astype(np.int64)   # exact: x has <= 24 bits above 2^-27
    sh = 27                                                                    # x/2^-3 = fixed / 2^27
    fl = fixed >> sh
    rem = fixed - (fl << sh)
    half = 1 << (sh - 1)
    up = (rem > half) | ((rem == half) & ((fl & 1) == 1))
    ref = np.clip(fl + up, -127, 127)
    # only elements that are exact on the 2^-30 grid take part (1e-3 is not)
    exact = fixed.astype(np.float64) * 2.0 ** -30 == blocks.astype(np.float64)
    assert exact[:, :7].all()
    assert np.array_equal(m[:, :7].astype(np.int64), ref[:, :7])


def test_invariants():
    rng = np.random.default_rng(7)
    x = (rng.standard_normal((512, 64)) * 2.0 ** rng.integers(-20, 20, size=(512, 1))).astype(np.float32)
    m, e = oracle.quantize_bfp16(x)
    d = oracle.dequantize(m, e)
    # I-1 idempotence
    m2, e2 = oracle.quantize_bfp16(d.astype(np.float32))
    assert np.array_equal(m, m2) and np.array_equal(e, e2)
    # I-2 error bound: <= s/2 unsaturated, < s saturated
    s = np.repeat(2.0 ** (e.astype(np.float64) - 133), 8, axis=1)
    err = np.abs(x.astype(np.float64) - d)
    sat = np.abs(x.astype(np.float64) / s) >= 127.5
    assert np.all(err[~sat] <= s[~sat] / 2)
    assert np.all(err[sat] < s[sat])
    # I-3 sign symmetry
    m3, e3 = oracle.quantize_bfp16(-x)
    assert np.array_equal(e3, e) and np.array_equal(m3, -m)
    # I-4 power-of-two equivariance
    for j in (-9, 5, 31):
        m4, e4 = oracle.quantize_bfp16((x.astype(np.float64) * 2.0 ** j).astype(np.float32))
        assert np.array_equal(m4, m) and np.array_equal(e4.astype(int), e.astype(int) + j)
    # I-5 the largest element lands in [64, 127]
    mx = np.abs(m.reshape(512, 8, 8)).max(axis=2)
    assert mx.min() >= 64 and mx.max() <= 127
    # never -128
    assert m.min() >= -127


def test_integer_blocks_are_exact():
    rng = np.random.default_rng(3)
    x = rng.integers(-127, 128, size=(256, 32)).astype(np.float32)
    x[:, ::8] = np.where(rng.random((256, 4)) < 0.5, 64, -127)      # force max in [64,127]
    m, e = oracle.quantize_bfp16(x)
    assert np.all(e == 133)
    assert np.array_equal(m.astype(np.float32), x)


def test_dequantize_exhaustive_exact_and_bf16_representable():
    E = np.repeat(np.arange(255, dtype=np.uint8), 255)
    mvals = np.tile(np.arange(-127, 128, dtype=np.int8), 255)
    n = E.size
    pad = (-n) % 8
    mant = np.concatenate([mvals, np.zeros(pad, np.int8)]).reshape(-1, 8)
    # one element per block so that each (E, m) pair gets its own exponent
    mant8 = np.zeros((n, 8), np.int8)
    mant8[:, 0] = mvals
    exp = E.reshape(n, 1)
    d = oracle.dequantize(mant8, exp)
    for idx in range(0, n, 997):                      # exact rational spot checks
        assert Fraction(d[idx, 0]) == exact_ref.dequant(int(E[idx]), int(mvals[idx]))
    expect = mvals.astype(np.float64) * np.exp2(E.astype(np.float64) - 133)
    assert np.array_equal(d[:, 0], expect)
    # exactly representable in bf16 (hence the in-kernel conversion is lossless)
    f = d[:, 0].astype(np.float32)
    assert np.array_equal(f.astype(np.float64), d[:, 0])
    back = inputs.bf16_bits_to_f32(inputs.to_bf16_bits(f))
    assert np.array_equal(back, f)
    assert mant.shape[1] == 8


def test_rejects_bad_k():
    with pytest.raises(ValueError):
        oracle.quantize_bfp16(np.zeros((2, 12), np.float32))


def test_input_distributions_have_expected_exponents():
    a = inputs.make_A("normal", 64, 512)
    m, e = oracle.quantize_bfp16(a)
    assert np.isin(e, [125, 126, 127, 128, 129]).mean() > 0.999
    assert ((e == 127) | (e == 128)).mean() > 0.8
    o = inputs.make_A("outlier", 64, 512)
    _, eo = oracle.quantize_bfp16(o)
    assert (eo >= 130).mean() > 0.03          # ~8% of blocks hold a x20 outlier
