"""Host-side checks of the arithmetic identities the CUDA quantizer's division-free arithmetic
relies on, against the plain definition (Appendix A.3: SINT4, fp16 scale, RTN)."""
from fractions import Fraction

import numpy as np

from oracle import lq_oracle as O


def test_scale_by_reciprocal_equals_division_for_every_fp16_maximum():
    """The kernel forms the group scale as fp16(a * fl32(1/7)); the definition is fp16(a /fl32 7).
    Every finite non-negative fp16 value can be a group maximum: check them all through the
    oracle's quantizer (a one-element group has maximum a)."""
    a16 = np.arange(0, 0x7C00, dtype=np.uint16).view(np.float16)
    _, s_def = O.qgrp(a16.astype(np.float32)[:, None], group=64)
    s_fast = (a16.astype(np.float32) * np.float32(1.0 / 7.0)).astype(np.float16)
    s_fast = np.maximum(s_fast, O.SCALE_FLOOR)
    assert np.array_equal(s_def[:, 0].view(np.uint16), s_fast.view(np.uint16))


def _rn32(v: Fraction) -> Fraction:
    """v rounded to the nearest binary32 number, ties to even (normal range), in exact rational arithmetic."""
    if v == 0:
        return Fraction(0)
    sign, a = (-1 if v < 0 else 1), abs(v)
    e = a.numerator.bit_length() - a.denominator.bit_length() - 23
    while a / Fraction(2) ** e >= 2 ** 24:
        e += 1
    while a / Fraction(2) ** e < 2 ** 23:
        e -= 1
    t = a / Fraction(2) ** e
    n = t.numerator // t.denominator
    rem = t - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1):
        n += 1
    return sign * n * Fraction(2) ** e


def test_fma_corrected_quotient_is_the_correctly_rounded_division():
    """The kernel never divides: with y = fl32(1/b) it forms q0 = fl32(a y), r = a - b q0 (exact in an FMA) and
    q1 = fl32(q0 + r y).  q1 must be fl32(a / b), the definition's quotient (Appendix A.3: RTN of the scaled value),
    for fp16 numerators over fp16 scales (main branch) and over fp32 per-token scales (low-rank branch), including
    quotients that sit exactly on k + 1/2.  Everything here is exact rational arithmetic."""
    rng = np.random.default_rng(0)
    cases = []
    x16 = rng.standard_normal(6000).astype(np.float16)
    s16 = (np.abs(rng.standard_normal(6000)) * 0.3 + 2.0 ** -10).astype(np.float16)
    cases += [(Fraction(float(a)), Fraction(float(b))) for a, b in zip(x16, s16)]
    for k in range(0, 8):                                    # exact ties x = (k + 1/2) s
        for b in s16[:60]:
            a = np.float16((k + 0.5) * float(b))
            cases.append((Fraction(float(a)), Fraction(float(b))))
    xb = (rng.standard_normal(6000) * 3).astype(np.float16)
    rowmax = np.abs(xb).max()
    for qm in (127.0, 31.0, 7.0):
        sb = np.float32(np.float32(rowmax) / np.float32(qm))
        cases += [(Fraction(float(a)), Fraction(float(sb))) for a in xb[:2000]]
    ties = 0
    for a, b in cases:
        y = _rn32(1 / b)
        q0 = _rn32(a * y)
        r = a - b * q0
        assert _rn32(r) == r, "the remainder must be a binary32 number (exact FMA)"
        q1 = _rn32(q0 + r * y)
        assert q1 == _rn32(a / b), (float(a), float(b))
        ties += (2 * a / b).denominator == 1 and (a / b).denominator == 2
    assert ties > 100
