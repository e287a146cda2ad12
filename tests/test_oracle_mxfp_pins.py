"""Pins of the MXFP oracle (oracle/lq_oracle_mxfp.py) against what the format definitions and the mathematics fix:
the element grids enumerated from their bit patterns, hand-worked blocks (tests/golden/mxfp_hand_examples.txt),
idempotence, the exponent rule's range guarantees, exact equivariance under powers of two, the half-step error bound,
brute-force forwards on tiny shapes in Python scalars, and the calibration's invariants (Sections 3.2-3.3)."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import lq_oracle_mxfp as F


def _decode(bits: int, ebits: int, mbits: int, bias: int) -> float:
    """Value of a sign-less minifloat bit pattern per the OCP element definitions."""
    e, m = bits >> mbits, bits & ((1 << mbits) - 1)
    if e == 0:
        return m / 2 ** mbits * 2.0 ** (1 - bias)
    return (1 + m / 2 ** mbits) * 2.0 ** (e - bias)


def test_element_grids_match_the_bit_patterns():
    e2m1 = sorted({_decode(b, 2, 1, 1) for b in range(8)})
    assert e2m1 == [0, 0.5, 1, 1.5, 2, 3, 4, 6] and list(F.element_values("e2m1")) == e2m1
    e2m3 = sorted({_decode(b, 2, 3, 1) for b in range(32)})
    assert len(e2m3) == 32 and e2m3[-1] == 7.5 and list(F.element_values("e2m3")) == e2m3
    e4m3 = sorted({_decode(b, 4, 3, 7) for b in range(127)})          # pattern 0x7F is NaN in e4m3
    assert e4m3[-1] == 448 and e4m3[1] == 2.0 ** -9 and list(F.element_values("e4m3")) == e4m3


@pytest.mark.parametrize("fmt", ["e2m1", "e2m3", "e4m3"])
def test_round_to_element_is_nearest_with_ties_to_even(fmt):
    """Against a brute-force search over the enumerated grid, on a dense sweep that contains every midpoint."""
    grid = F.element_values(fmt)
    mids = (grid[1:] + grid[:-1]) / 2
    rng = np.random.default_rng(0)
    v = np.concatenate([grid, mids, mids * (1 + 1e-9), mids * (1 - 1e-9), rng.uniform(0, grid[-1] * 1.2, 4000)])
    v = np.concatenate([v, -v])
    got = F.round_to_element(v, fmt)
    mant = F.FORMATS[fmt][0]
    for x, g in zip(v, got):
        a = abs(x)
        d = np.abs(grid - a)
        near = grid[d == d.min()]
        if len(near) == 2:                       # a tie: the candidate whose mantissa is even
            idx = [int(np.where(grid == n)[0][0]) for n in near]
            want = near[0] if idx[0] % 2 == 0 else near[1]   # grid index parity = mantissa parity (2^mant values per binade)
        else:
            want = near[0]
        assert g == np.sign(x) * want, (fmt, x, g, want)
    assert mant in (1, 3)


def test_mxfp_hand_examples(golden_dir):
    cases, cur = [], {}
    for line in open(os.path.join(golden_dir, "mxfp_hand_examples.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, val = line.split(":", 1)
        cur[key] = val.split()
        if key == "q":
            cases.append(cur)
            cur = {}
    assert len(cases) == 8
    for c in cases:
        v = np.array([float(x) for x in c["v"]])
        el, ex = F.qmxfp(v[None, :], c["f"][0])
        assert int(ex[0, 0]) == int(c["e"][0]), c
        assert np.array_equal(el[0], np.array([float(x) for x in c["q"]], dtype=np.float32)), (c, el[0])


@pytest.mark.parametrize("fmt", ["e2m1", "e2m3", "e4m3"])
def test_quantizer_invariants(fmt):
    rng = np.random.default_rng(1)
    v = rng.standard_normal((64, 200)) * np.exp2(rng.integers(-12, 12, size=(64, 1)))
    v[3, :] = 0                                                   # an all-zero row
    v[4, 40:] = 0                                                 # all-zero blocks behind a live one
    el, ex = F.qmxfp(v, fmt)
    mant, emin, emax, vmax = F.FORMATS[fmt]
    grid = F.element_values(fmt)
    assert np.isin(np.abs(el), grid.astype(np.float32)).all()
    assert ex.shape == (64, 7) and (ex[3] == -127).all() and (el[3] == 0).all() and (ex[4, 2:] == -127).all()
    # the exponent rule: the block maximum lands in the top binade [2^emax, 2^(emax+1)) before rounding
    a = np.abs(np.pad(v, ((0, 0), (0, 24))).reshape(64, 7, 32)).max(-1)
    live = a > 0
    scaled = a[live] / np.exp2(ex[live].astype(np.float64))
    assert (scaled >= 2.0 ** emax).all() and (scaled < 2.0 ** (emax + 1)).all()
    # idempotence (Section 3.2: Q is idempotent on its image)
    deq = F.deq_mxfp(el, ex)
    el2, ex2 = F.qmxfp(deq, fmt)
    assert np.array_equal(F.deq_mxfp(el2, ex2), deq)
    # error: at most half a step of the element's binade, except where the top binade clamps
    step = np.exp2(np.clip(np.floor(np.log2(np.maximum(np.abs(el), 2.0 ** emin))), emin, emax) - mant)
    err = np.abs(deq - v) / np.repeat(np.exp2(ex.astype(np.float64)), 32, axis=1)[:, :200]
    unclamped = np.abs(v) / np.repeat(np.exp2(ex.astype(np.float64)), 32, axis=1)[:, :200] <= vmax
    assert (err[unclamped] <= 0.5 * step[unclamped] + 1e-12).all()
    assert (err[~unclamped] <= 2.0 ** (emax + 1) - vmax).all()
    # exact equivariance under powers of two, sign symmetry
    el3, ex3 = F.qmxfp(v * 8.0, fmt)
    assert np.array_equal(el3, el) and np.array_equal(ex3[live], ex[live] + 3)
    el4, _ = F.qmxfp(-v, fmt)
    assert np.array_equal(el4, -el)


def test_blocks_run_along_the_contraction_axis():
    rng = np.random.default_rng(2)
    P = rng.standard_normal((70, 5))
    el, ex = F.q_columns(P, "e2m1")
    assert el.shape == (70, 5) and ex.shape == (3, 5)
    P2 = P.copy(); P2[0:32, 1] *= 64.0                              # only block 0 of column 1 changes
    el2, ex2 = F.q_columns(P2, "e2m1")
    assert ex2[0, 1] == ex[0, 1] + 6 and np.array_equal(np.delete(ex2, 1, axis=1), np.delete(ex, 1, axis=1))
    assert np.array_equal(el2[32:], el[32:]) and np.array_equal(el2[:32, 1], el[:32, 1])


def _tiny_layer(rng, K, N, r, branch):
    layer = {"main": "mxfp4", "branch": branch, "rank": r, "K": K, "N": N, "bias": (rng.standard_normal(N) * 0.1).astype(np.float16)}
    layer["Wv"], layer["ew"] = F.q_columns(rng.standard_normal((K, N)) * 0.05, "e2m1")
    if r:
        fmt = F.BRANCH_FORMAT[branch]
        layer["L1v"], layer["e1"] = F.q_columns(rng.standard_normal((K, r)) * 0.2, fmt)
        layer["L2v"], layer["e2"] = F.q_columns(rng.standard_normal((r, N)) * 0.2, fmt)
    return layer


@pytest.mark.parametrize("branch,r,act", [("mxfp8", 5, "e4m3"), ("mxfp6", 40, "e4m3"), ("mxfp4", 33, "e4m3"), ("none", 0, "e4m3"),
                                          ("mxfp6", 40, "e2m3"), ("none", 0, "e2m3")])
def test_forward_against_python_scalars(branch, r, act):
    """Tiny ragged shapes (K = 72: two full blocks and a short one), every sum in exact rational arithmetic from the
    oracle's own element values and exponents of X and T (their quantizer is pinned above)."""
    rng = np.random.default_rng(3)
    M, K, N = 3, 72, 4
    layer = _tiny_layer(rng, K, N, r, branch)
    if act != "e4m3":
        layer["act"] = act                      # Table 4: activations in the branch's 6-bit format
    X = (rng.standard_normal((M, K)) * 2).astype(np.float16)
    out = F.forward(X, layer)
    # the activations' images are the pinned quantizer's, in the format asked for (the 6-bit grid is coarser: it must show)
    xa_ref, ex_ref = F.qmxfp(X.astype(np.float64), act)
    assert np.array_equal(out["xa"], xa_ref) and np.array_equal(out["ex"], ex_ref)
    assert np.isin(np.abs(out["xa"]), F.element_values(act).astype(np.float32)).all()
    if act == "e2m3":
        assert not np.array_equal(F.deq_mxfp(out["xa"], out["ex"]), F.deq_mxfp(*F.qmxfp(X.astype(np.float64), "e4m3")))
    fr = lambda x: Fraction(float(x))
    p2 = lambda e: Fraction(2) ** int(e)
    for m in range(M):
        # T from the definition, then its MXFP8e4 image through the oracle's quantizer on the exact value
        if r:
            T = [sum(p2(out["ex"][m, k // 32]) * p2(layer["e1"][k // 32, j]) * fr(out["xa"][m, k]) * fr(layer["L1v"][k, j])
                     for k in range(K)) for j in range(r)]
            assert all(abs(float(T[j]) - out["T"][m, j]) <= 1e-12 * (abs(float(T[j])) + 1e-30) for j in range(r))
        for n in range(N):
            y = sum(p2(out["ex"][m, k // 32]) * p2(layer["ew"][k // 32, n]) * fr(out["xa"][m, k]) * fr(layer["Wv"][k, n]) for k in range(K))
            if r:
                y += sum(p2(out["et"][m, j // 32]) * p2(layer["e2"][j // 32, n]) * fr(out["tq"][m, j]) * fr(layer["L2v"][j, n]) for j in range(r))
            y += fr(layer["bias"][n])
            assert abs(Fraction(float(out["Y"][m, n])) - y) <= abs(y) * Fraction(1, 10 ** 12) + Fraction(1, 10 ** 14)
    if r:
        tq2, et2 = F.qmxfp(out["T"], act)
        assert np.array_equal(tq2, out["tq"]) and np.array_equal(et2, out["et"])


def test_forward_special_cases():
    rng = np.random.default_rng(4)
    M, K, N = 8, 96, 16
    # inputs already on the MXFP8e4 grid and weights on the MXFP4 grid: the main branch is an exact matrix product
    X = (rng.integers(-8, 9, size=(M, K)) * 16.0).astype(np.float16)     # multiples of 16 up to 128: e4m3 values at e = -1..0
    Wgrid = rng.choice([0, 0.5, 1, 1.5, 2, 3, 4, 6], size=(K, N)) * rng.choice([-1, 1], size=(K, N))
    layer = {"main": "mxfp4", "branch": "none", "rank": 0, "K": K, "N": N, "bias": None}
    layer["Wv"], layer["ew"] = F.q_columns(Wgrid, "e2m1")
    assert np.array_equal(F.deq_columns(layer["Wv"], layer["ew"]), Wgrid)
    out = F.forward(X, layer)
    assert np.array_equal(out["Y"], X.astype(np.float64) @ Wgrid)
    # rows are independent
    out2 = F.forward(X[2:5], layer)
    assert np.array_equal(out2["Y"], out["Y"][2:5])


def test_calibration_invariants():
    rng = np.random.default_rng(5)
    W = (rng.standard_normal((96, 40)) * 0.02).astype(np.float16)
    W64 = W.astype(np.float64)
    layer, trace = F.calibrate(W, 8, "mxfp8", steps=60)
    # iterate 0 is the SVD start: objective = mean((Q1(W - L0 R0) - (W - L0 R0))^2)
    from oracle import lq_oracle as O
    L0, R0 = O.svd_init(W64, 8)
    E0 = F.q1_dequant(W64 - L0 @ R0) - (W64 - L0 @ R0)
    assert abs(trace[0] - np.mean(E0 * E0)) <= 1e-15
    assert np.minimum.accumulate(trace)[-1] < trace[0]
    # Figure 1: the stored residual is Q1 of P = W - Q2(L1) Q2(L2)
    D = F.deq_columns(layer["L1v"], layer["e1"]) @ F.deq_columns(layer["L2v"], layer["e2"])
    Wv, ew = F.q_columns(W64 - D, "e2m1")
    assert np.array_equal(Wv, layer["Wv"]) and np.array_equal(ew, layer["ew"])
    # the calibrated layer is closer to W than plain MXFP4 rounding
    assert np.linalg.norm(F.effective_weight(layer) - W64) < np.linalg.norm(F.q1_dequant(W64) - W64)
    # a weight already on the MXFP4 grid: rank 0 reproduces it with zero loss
    Wg = F.q1_dequant(W64)
    l0, t0 = F.calibrate(Wg.astype(np.float16), 0, "none")
    assert t0[0] == 0.0 or np.array_equal(F.effective_weight(l0), Wg.astype(np.float16).astype(np.float64))
