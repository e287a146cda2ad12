"""Host-side checks of the arithmetic identities the CUDA quantizer's division-free fast path
relies on, against the oracle's plain definition (Appendix A.3: SINT4, fp16 scale, RTN)."""
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


def test_exact_remainder_flags_exactly_the_ties():
    """Main-branch fast path: q' = rint(x * r) with r ~ 1/s, remainder e = x - q' s; the code is
    q' unless |e| == s/2.  Emulated in fl32 on random fp16 rows plus planted ties; the flagged
    elements re-done with true division must give the oracle's codes everywhere."""
    rng = np.random.default_rng(0)
    X = rng.standard_normal((64, 1024)).astype(np.float16)
    X[:8] = (rng.integers(-14, 15, size=(8, 1024)) * 0.5).astype(np.float16); X[:8, ::64] = 7   # ties k + 1/2, s = 1
    codes, scales = O.qgrp(X.astype(np.float32))
    s = np.repeat(scales.astype(np.float32), 64, axis=1)
    x = X.astype(np.float32)
    r = (np.float32(1.0) / s).astype(np.float32) * np.float32(1.0 + 2.0 ** -22)          # a reciprocal 2 ulp off
    q = np.rint((x * r).astype(np.float32)).astype(np.float32)
    e = (x.astype(np.float64) - q.astype(np.float64) * s.astype(np.float64)).astype(np.float32)  # exact in fl32
    tie = np.abs(e) == np.float32(0.5) * s
    q_exact = np.clip(np.rint(x / s), -7, 7)
    q = np.where(tie, q_exact, q)
    assert tie.any()
    assert np.array_equal(q.astype(np.int8), codes)
