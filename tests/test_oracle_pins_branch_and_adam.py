"""Pins for two parts of the oracle that the other pin files leave free:
the fp16 rounding of the rank-r intermediate T in the full-precision reference branch (Section 4.2 / Table 2 keep the
branch's activations at full precision; T = fp16(X L1) is this build's reading), and the Adam update of the data-free
calibration (Appendix A "Optimization": Adam, learning rate 1e-4, 1000 steps).  Expected values are worked out in exact
rational arithmetic or by hand, never by the code under test."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import lq_oracle as O


def _rn16(v: Fraction) -> Fraction:
    """v rounded to the nearest fp16 number (normal range), ties to even, in exact arithmetic."""
    if v == 0:
        return Fraction(0)
    sign, a = (-1 if v < 0 else 1), abs(v)
    e = -24
    while a / Fraction(2) ** e >= 2048:
        e += 1
    t = a / Fraction(2) ** e
    if e > -24:
        assert t >= 1024
    n = t.numerator // t.denominator
    rem = t - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1):
        n += 1
    return sign * n * Fraction(2) ** e


def test_rn16_helper_on_hand_values():
    assert _rn16(Fraction(2049)) == 2048          # midpoint of 2048 and 2050 -> even mantissa 1024
    assert _rn16(Fraction(2051)) == 2052          # midpoint of 2050 and 2052 -> even mantissa 1026
    assert _rn16(Fraction(2049) + Fraction(1, 1000)) == 2050
    assert _rn16(Fraction(1, 3)) == Fraction(float(np.float16(1.0 / 3.0)))
    assert _rn16(Fraction(-4097, 2)) == -2048     # -2048.5 -> -2048 (step 2 there: nearest)


def _w16a16_case(main: str):
    """K = 40 (one short group / two MX blocks), r = 2, three tokens.  Row 0: T[0,0] = 2049 and T[0,1] = 2051, exact fp16
    midpoints; row 1: sums that need ordinary rounding; row 2: zeros."""
    K, N, r = 40, 8, 2
    X = np.zeros((3, K), dtype=np.float16)
    L1 = np.zeros((K, r), dtype=np.float16)
    X[0, 0], X[0, 1], X[0, 2] = 2048, 1, 3
    L1[0, :] = 1
    L1[1, 0] = 1
    L1[2, 1] = 1                                   # T[0] = (2048 + 1, 2048 + 3)
    rng = np.random.default_rng(5)
    X[1, :] = (rng.standard_normal(K) * 3).astype(np.float16)
    L1[3:, :] = (rng.standard_normal((K - 3, r)) * 0.37).astype(np.float16)
    X[1, :3] = 0
    L2 = (rng.standard_normal((r, N)) * 0.5).astype(np.float16)
    W = (rng.standard_normal((K, N)) * 0.02).astype(np.float16).astype(np.float64)
    layer = {"branch": "w16a16", "rank": r, "K": K, "N": N, "bias": None, "main": main, "L1h": L1, "L2h": L2}
    if main == "mxint4":
        layer["Wq"], layer["ew"] = O.q_weight_main_mx(W)
    else:
        layer["Wq"], layer["sw"] = O.q_weight_main(W)
    return X, layer


@pytest.mark.parametrize("main", ["sint4", "mxint4"])
def test_w16a16_intermediate_is_rounded_once_to_fp16(main):
    X, layer = _w16a16_case(main)
    out = O.forward(X, layer)
    M, K = X.shape
    N, r = layer["N"], layer["rank"]
    fx = [[Fraction(float(v)) for v in row] for row in X]
    T16 = [[_rn16(sum(fx[m][k] * Fraction(float(layer["L1h"][k, j])) for k in range(K))) for j in range(r)] for m in range(M)]
    assert T16[0][0] == 2048 and T16[0][1] == 2052            # the two midpoints, ties to even
    assert any(T16[1][j] != sum(fx[1][k] * Fraction(float(layer["L1h"][k, j])) for k in range(K)) for j in range(r))
    # main part from the oracle's own codes (pinned elsewhere), low-rank part from the hand-rounded T
    if main == "mxint4":
        def main_term(m, n):
            return sum(Fraction(2) ** int(out["ex"][m, k // 32]) * Fraction(2) ** int(layer["ew"][k // 32, n]) *
                       int(out["qx"][m, k]) * int(layer["Wq"][k, n]) for k in range(K))
    else:
        def main_term(m, n):
            return sum(Fraction(float(out["sx"][m, k // 64])) * Fraction(float(layer["sw"][k // 64, n])) *
                       int(out["qx"][m, k]) * int(layer["Wq"][k, n]) for k in range(K))
    for m in range(M):
        for n in range(N):
            expect = main_term(m, n) + sum(T16[m][j] * Fraction(float(layer["L2h"][j, n])) for j in range(r))
            assert abs(Fraction(float(out["Y"][m, n])) - expect) <= abs(expect) * Fraction(1, 10 ** 12) + Fraction(1, 10 ** 15), (m, n)
    # an unrounded (or late-rounded) T would move Y[0, :] by L2[0, :] - 1 * L2[1, :], far above that bound
    assert np.array_equal(out["T16"].astype(np.float64), np.array([[float(v) for v in row] for row in T16]))


def test_adam_first_step_closed_form():
    """From zero moments, with bias correction, step 1 moves every entry by exactly lr * g / (|g| + eps)."""
    g = np.array([3e-9, -2.5e-7, 0.0, 4.0, -1e-12])
    x0 = np.array([0.1, -0.2, 0.3, 0.4, 0.5])
    lr, eps = 1e-4, 1e-8
    x1, m1, v1 = O.adam_update(x0, g, np.zeros(5), np.zeros(5), 1, lr, 0.9, 0.999, eps)
    assert np.allclose(x1, x0 - lr * g / (np.abs(g) + eps), rtol=1e-13, atol=0)
    assert np.allclose(m1, 0.1 * g, rtol=1e-15) and np.allclose(v1, 0.001 * g * g, rtol=1e-12)
    # eps inside the root, swapped betas or no bias correction all change the small-gradient entries by > 1 %
    assert abs((x0[0] - x1[0]) / lr - 3e-9 / (3e-9 + 1e-8)) < 1e-12


def test_adam_two_steps_by_hand():
    """g1 = 0.5, g2 = -0.25, lr = 0.1, betas (0.9, 0.999), eps = 1e-8, worked by hand:
    m1 = 0.05, v1 = 0.00025, step 1 = 0.1 * 0.5 / (0.5 + eps);
    m2 = 0.02, v2 = 0.00031225, m2 / (1 - 0.81) = 0.10526315789..., v2 / (1 - 0.998001) = 0.15620310155...,
    step 2 = 0.1 * 0.10526315789 / (0.39522538070 + eps)."""
    x, m, v = O.adam_update(np.array([1.0]), np.array([0.5]), np.zeros(1), np.zeros(1), 1, 0.1, 0.9, 0.999, 1e-8)
    assert abs(x[0] - (1.0 - 0.1 * 0.5 / (0.5 + 1e-8))) < 1e-15
    x2, m2, v2 = O.adam_update(x, np.array([-0.25]), m, v, 2, 0.1, 0.9, 0.999, 1e-8)
    assert abs(m2[0] - 0.02) < 1e-15 and abs(v2[0] - 0.00031225) < 1e-15
    mhat, vhat = 0.02 / 0.19, 0.00031225 / 0.001999
    assert abs(vhat - 0.15620310155) < 1e-10
    assert abs((x[0] - x2[0]) - 0.1 * mhat / (vhat ** 0.5 + 1e-8)) < 1e-15
    assert abs((x[0] - x2[0]) - 0.026633703) < 1e-8


def test_calibrate_takes_exactly_that_step():
    """The trace's entry 1 is the objective at (L, R) moved by the closed-form first step from the SVD start."""
    rng = np.random.default_rng(2)
    W = (rng.standard_normal((64, 24)) * 0.02).astype(np.float16)
    Wd = W.astype(np.float64)
    r, lr, eps = 3, 1e-4, 1e-8
    _, trace = O.calibrate(W, r, "w8a8", steps=1, lr=lr, eps=eps)
    L0, R0 = O.svd_init(Wd, r)
    L, R = -L0, R0
    loss0, gL, gR = O.gradients(Wd, L, R)
    assert abs(trace[0] - loss0) <= 1e-15 * loss0
    L1 = L - lr * gL / (np.abs(gL) + eps)
    R1 = R - lr * gR / (np.abs(gR) + eps)
    assert abs(trace[1] - O.objective(Wd, L1, R1)) <= 1e-12 * loss0
    # the gradients here are ~1e-9 .. 1e-7, so eps = 1e-8 matters: a step without it is a different point
    assert abs(O.objective(Wd, L - lr * np.sign(gL), R - lr * np.sign(gR)) - trace[1]) > 1e-6 * loss0
