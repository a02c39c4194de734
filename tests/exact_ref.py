"""Exact-rational re-statement of BFP16 quantisation, used only to pin the oracle.

Deliberately written differently from ``oracle/atb_oracle.cpp``: Python
``Fraction`` arithmetic, exponent found by comparing against powers of two,
rounding by floor/compare.  Slow; for small cases.
"""
from fractions import Fraction
import math


def quantize_block(xs):
    """xs: 8 Python floats holding fp32 values -> (E, [m0..m7])."""
    assert len(xs) == 8
    mags = [abs(x) for x in xs if not math.isnan(x)]
    amax = max(mags) if mags else 0.0
    if amax == 0.0:
        E = 0
    elif math.isinf(amax):
        E = 254
    else:
        fa = Fraction(amax)
        e = -160
        while Fraction(2) ** (e + 1) <= fa:       # largest e with 2^e <= amax
            e += 1
        E = e + 127
        if E < 1:
            E = 0
        if E > 254:
            E = 254
    s = Fraction(2) ** (E - 133)
    ms = []
    for x in xs:
        if math.isnan(x):
            ms.append(0)
            continue
        if math.isinf(x):
            ms.append(127 if x > 0 else -127)
            continue
        q = Fraction(x) / s
        lo = math.floor(q)
        rem = q - lo
        if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and lo % 2 == 1):
            lo += 1
        ms.append(max(-127, min(127, lo)))
    return E, ms


def dequant(E, m):
    return Fraction(m) * Fraction(2) ** (E - 133)
