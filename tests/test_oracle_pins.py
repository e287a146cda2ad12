"""Pins of the CPU oracle against what the paper and the mathematics fix.

Every check here uses something other than the oracle's own formula: hand-worked
values, closed forms (Eckart-Young, the Frobenius bound of Section 3.1), brute
force with Python scalars, special cases that collapse to an integer matmul, and
finite differences.  None of them needs a GPU.
"""
import itertools
import os

import numpy as np
import pytest

from oracle import lq_oracle as O
from paper_2604_18117_b200 import inputs as I


# ---------------------------------------------------------------------------------------
# Quantizers (Appendix A.3 "Blockwise Formats"; idempotence: Section 3.2)
# ---------------------------------------------------------------------------------------
def _read_cases(path):
    cases, cur = [], {}
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tag, vals = line.split(":")
        cur[tag] = [float(t) for t in vals.split()]
        if tag == "q":
            cases.append(cur)
            cur = {}
    return cases


def test_sint4_hand_examples(golden_dir):
    cases = _read_cases(os.path.join(golden_dir, "sint4_hand_examples.txt"))
    assert len(cases) == 5
    for c in cases:
        v = np.array([c["v"]], dtype=np.float32)
        q, s = O.qgrp(v)
        assert float(s[0, 0]) == c["s"][0]
        assert q[0].tolist() == [int(t) for t in c["q"]]


def test_sint4_groups_are_independent_and_ragged():
    # two full groups and a short one: each group's scale depends on that group only
    rng = np.random.default_rng(1)
    v = rng.standard_normal((3, 64 * 2 + 32)).astype(np.float16).astype(np.float32)
    q, s = O.qgrp(v)
    assert s.shape == (3, 3)
    for g, (a, b) in enumerate([(0, 64), (64, 128), (128, 160)]):
        q1, s1 = O.qgrp(v[:, a:b])
        assert np.array_equal(q1, q[:, a:b]) and np.array_equal(s1[:, 0], s[:, g])
    # scaling one group by 4 changes only that group's scale (x4) and leaves every code alone
    v2 = v.copy(); v2[:, 64:128] *= 4
    q2, s2 = O.qgrp(v2)
    assert np.array_equal(q2, q)
    assert np.array_equal(s2[:, 1].astype(np.float32), s[:, 1].astype(np.float32) * 4)
    assert np.array_equal(s2[:, [0, 2]], s[:, [0, 2]])


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_sint4_properties(seed):
    rng = np.random.default_rng(seed)
    v = (rng.standard_normal((37, 200)) * rng.lognormal(0, 2, size=(37, 1))).astype(np.float16).astype(np.float32)
    q, s = O.qgrp(v)
    assert q.min() >= -7 and q.max() <= 7
    d = O.deq_grp(q, s)
    sfull = np.repeat(s.astype(np.float64), 64, axis=1)[:, :200]
    amax = np.repeat(np.stack([np.abs(v[:, g * 64:(g + 1) * 64]).max(1) for g in range(4)], 1), 64, 1)[:, :200]
    # rounding error at most half a step (plus the fp16 rounding of the scale at the clamp)
    assert np.all(np.abs(v - d) <= sfull / 2 + amax * 2.0 ** -10)
    # the group maximum always maps to code +-7
    for g in range(4):
        blk = slice(g * 64, min(200, (g + 1) * 64))
        assert np.all(np.abs(q[:, blk]).max(1) == 7)
    # idempotence: Q(deq(Q(v))) reproduces codes and scales
    q2, s2 = O.qgrp(d.astype(np.float32))
    assert np.array_equal(q, q2) and np.array_equal(s, s2)
    # sign symmetry
    qn, sn = O.qgrp(-v)
    assert np.array_equal(qn, -q) and np.array_equal(sn, s)


def test_sint4_zero_and_subnormal_groups():
    v = np.zeros((2, 128), dtype=np.float32)
    v[1, 64:] = np.float32(2.0 ** -24)          # smallest fp16 subnormal everywhere in one group
    q, s = O.qgrp(v)
    assert np.all(q[0] == 0) and np.all(s[0] == np.float16(2.0 ** -24))
    assert np.all(q[1, :64] == 0)
    # a = 2^-24, a/7 rounds to 0 in fp16, floor lifts it to 2^-24 -> code 1
    assert np.all(s[1, 1] == np.float16(2.0 ** -24)) and np.all(q[1, 64:] == 1)
    big = np.full((1, 64), 65504.0, dtype=np.float32); big[0, 1] = -65504.0
    qb, sb = O.qgrp(big)
    assert np.isfinite(float(sb[0, 0])) and qb[0, 0] == 7 and qb[0, 1] == -7


@pytest.mark.parametrize("bits", [4, 6, 8])
def test_qtok_hand_and_properties(bits):
    qm = {4: 7, 6: 31, 8: 127}[bits]
    assert O.qmax(bits) == qm
    # absmax = qmax -> scale exactly 1 -> codes are rint-to-even of the inputs
    v = np.array([[qm, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.25, -qm, 0]], dtype=np.float32)
    q, s = O.qtok(v, bits)
    assert s[0] == 1.0 and q[0].tolist() == [qm, 0, 2, 2, 0, -2, -2, 3, -qm, 0]
    # zero row: scale 1, codes 0
    q0, s0 = O.qtok(np.zeros((1, 5), np.float32), bits)
    assert s0[0] == 1.0 and not q0.any()
    rng = np.random.default_rng(bits)
    v = (rng.standard_normal((50, 300)) * 3).astype(np.float16).astype(np.float32)
    q, s = O.qtok(v, bits)
    assert np.abs(q).max() <= qm and np.all(np.abs(q).max(1) == qm)
    d = O.deq_tok(q, s)
    assert np.all(np.abs(v - d) <= s[:, None].astype(np.float64) * (0.5 + 1e-6))
    q2, s2 = O.qtok(d.astype(np.float32), bits)
    assert np.array_equal(q, q2)                      # idempotent codes
    assert np.allclose(s, s2, rtol=2e-7, atol=0)      # scale reproduced to fp32 rounding


def test_weight_quantizer_groups_along_K_per_output_column():
    rng = np.random.default_rng(3)
    P = rng.standard_normal((160, 5)) * 0.02
    Wq, sw = O.q_weight_main(P)
    assert Wq.shape == (160, 5) and sw.shape == (3, 5)
    for n in range(5):
        q, s = O.qgrp(P[:, n].astype(np.float32)[None, :])
        assert np.array_equal(q[0], Wq[:, n]) and np.array_equal(s[0], sw[:, n])
    # a column scaled by 8 keeps its codes, scales x8; the other columns are untouched
    P2 = P.copy(); P2[:, 2] *= 8
    Wq2, sw2 = O.q_weight_main(P2)
    assert np.array_equal(Wq2, Wq)
    assert np.array_equal(sw2[:, 2].astype(np.float32), sw[:, 2].astype(np.float32) * 8)


def test_factor_quantizer_is_per_column():
    rng = np.random.default_rng(4)
    F = rng.standard_normal((40, 6))
    Fq, s = O.q_factor(F, 8)
    assert Fq.shape == F.shape and s.shape == (6,)
    for j in range(6):
        assert s[j] == np.float32(np.float32(np.abs(F[:, j].astype(np.float32)).max()) / np.float32(127))
        assert np.abs(Fq[:, j]).max() == 127
    Fh, none = O.q_factor(F, None)
    assert none is None and Fh.dtype == np.float16


# ---------------------------------------------------------------------------------------
# Section 3.1: error upper bound holds for the oracle's quantizers
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("seed", [0, 1])
def test_error_upper_bound(seed):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((48, 192)).astype(np.float16)
    X[:, 5] *= 20
    W = (rng.standard_normal((192, 40)) * 0.02).astype(np.float16)
    qx, sx = O.qgrp(X.astype(np.float32))
    QX = O.deq_grp(qx, sx)
    QW = O.q1_dequant(W.astype(np.float64))
    X64, W64 = X.astype(np.float64), W.astype(np.float64)
    lhs = np.linalg.norm(X64 @ W64 - QX @ QW)
    rhs = np.linalg.norm(X64 - QX) * np.linalg.norm(W64) + np.linalg.norm(QX) * np.linalg.norm(W64 - QW)
    assert lhs <= rhs * (1 + 1e-12)
    assert lhs > 0


# ---------------------------------------------------------------------------------------
# Forward (Figure 1; Appendix A.2)
# ---------------------------------------------------------------------------------------
def _tiny_layer(rng, K, N, r, branch):
    W = (rng.standard_normal((K, N)) * 0.05)
    layer = {"branch": branch, "rank": r, "K": K, "N": N, "bias": None}
    layer["Wq"], layer["sw"] = O.q_weight_main(W)
    if branch == "none":
        layer["rank"] = 0
    elif branch == "w16a16":
        layer["L1h"] = (rng.standard_normal((K, r)) * 0.1).astype(np.float16)
        layer["L2h"] = (rng.standard_normal((r, N)) * 0.1).astype(np.float16)
    else:
        bw, _ = O.BRANCH_BITS[branch]
        layer["L1q"], layer["sL1"] = O.q_factor(rng.standard_normal((K, r)) * 0.1, bw)
        layer["L2q"], layer["sL2"] = O.q_factor(rng.standard_normal((r, N)) * 0.1, bw)
    return layer


@pytest.mark.parametrize("branch", ["w8a8", "w6a6", "w4a8"])
def test_forward_brute_force_tiny(branch):
    """Python-scalar evaluation of Y[m,n] = sum_k (sx qx)(sw Wq) + sum_j (sT tq)(sL2 L2q),
    with the branch intermediate rebuilt element by element from the definition."""
    rng = np.random.default_rng(7)
    M, K, N, r = 2, 64 + 64 + 32, 3, 2
    X = rng.standard_normal((M, K)).astype(np.float16)
    X[:, 3] *= 20
    layer = _tiny_layer(rng, K, N, r, branch)
    layer["bias"] = (rng.standard_normal(N) * 0.1).astype(np.float16)
    out = O.forward(X, layer)
    bw, ba = O.BRANCH_BITS[branch]
    qm = (1 << (ba - 1)) - 1
    for m in range(M):
        # per-token branch codes from the definition
        a = max(abs(float(x)) for x in X[m])
        s = np.float32(a) / np.float32(qm)
        qb = [int(np.clip(np.rint(np.float32(x) / s), -qm, qm)) for x in X[m]]
        assert qb == out["qb"][m].tolist() and s == out["sXb"][m]
        I1 = [sum(qb[k] * int(layer["L1q"][k, j]) for k in range(K)) for j in range(r)]
        t = [np.float32(np.float32(I1[j]) * np.float32(s * layer["sL1"][j])) for j in range(r)]
        at = max(abs(float(x)) for x in t)
        sT = np.float32(at) / np.float32(qm)
        tq = [int(np.clip(np.rint(x / sT), -qm, qm)) for x in t]
        assert tq == out["tq"][m].tolist() and sT == out["sT"][m]
        for n in range(N):
            y = 0.0
            for k in range(K):
                g = k // 64
                y += (float(out["sx"][m, g]) * int(out["qx"][m, k])) * (float(layer["sw"][g, n]) * int(layer["Wq"][k, n]))
            for j in range(r):
                y += (float(sT) * tq[j]) * (float(layer["sL2"][n]) * int(layer["L2q"][j, n]))
            y += float(layer["bias"][n])
            assert abs(y - out["Y"][m, n]) <= 1e-12 * max(1.0, abs(y))


def test_forward_rank0_is_plain_w4a4_dequant_matmul():
    rng = np.random.default_rng(8)
    M, K, N = 9, 200, 11
    X = rng.standard_normal((M, K)).astype(np.float16)
    layer = _tiny_layer(rng, K, N, 0, "none")
    out = O.forward(X, layer)
    qx, sx = O.qgrp(X.astype(np.float32))
    Y2 = O.deq_grp(qx, sx) @ O.deq_weight_main(layer["Wq"], layer["sw"])   # dequantize, then one matmul
    assert np.allclose(out["Y"], Y2, rtol=1e-12, atol=1e-12)
    assert "qb" not in out
    # a layer with a branch whose second factor is all zero gives the same output
    layer2 = _tiny_layer(rng, K, N, 4, "w8a8")
    layer2["Wq"], layer2["sw"] = layer["Wq"], layer["sw"]
    layer2["L2q"][:] = 0
    assert np.allclose(O.forward(X, layer2)["Y"], out["Y"], rtol=0, atol=0)


def test_forward_exact_integer_case_w8a8():
    """Inputs chosen so that every quantizer on the branch is exact: X holds integers with
    row maximum 127 (per-token scale 1), L1q selects channels (scale 1) including the
    maximum, so T = X[:, sel] with row maximum 127 (scale 1).  The branch output must then
    equal the plain integer product X[:, sel] @ L2, and the main branch the dequantized
    product."""
    rng = np.random.default_rng(9)
    M, K, N, r = 5, 128, 7, 4
    X = rng.integers(-100, 101, size=(M, K)).astype(np.float16)
    X[:, 17] = 127
    sel = [17, 3, 70, 127]
    L1q = np.zeros((K, r), np.int8)
    for j, k in enumerate(sel):
        L1q[k, j] = 1
    L2q = rng.integers(-127, 128, size=(r, N)).astype(np.int8)
    layer = {"branch": "w8a8", "rank": r, "K": K, "N": N, "bias": None,
             "L1q": L1q, "sL1": np.ones(r, np.float32), "L2q": L2q,
             "sL2": np.full(N, 0.25, np.float32)}
    layer["Wq"], layer["sw"] = O.q_weight_main(rng.standard_normal((K, N)) * 0.02)
    out = O.forward(X, layer)
    assert np.all(out["sXb"] == 1) and np.array_equal(out["qb"], X.astype(np.int8))
    assert np.all(out["sT"] == 1) and np.array_equal(out["tq"], X[:, sel].astype(np.int8))
    Xi = X.astype(np.int64)
    branch = (Xi[:, sel] @ L2q.astype(np.int64)) * 0.25
    main = O.deq_grp(out["qx"], out["sx"]) @ O.deq_weight_main(layer["Wq"], layer["sw"])
    assert np.allclose(out["Y"], main + branch, rtol=1e-13, atol=1e-13)


def test_forward_exact_integer_case_w16a16():
    """Small-integer X (group maxima 7 -> SINT4 scale 1, codes = X), integer fp16 factors:
    everything is exact and Y = X @ (deq(Wq) + L1 L2) in integers."""
    rng = np.random.default_rng(10)
    M, K, N, r = 6, 128, 5, 3
    X = rng.integers(-7, 8, size=(M, K)).astype(np.float16)
    X[:, 0] = 7; X[:, 64] = -7
    Wint = rng.integers(-7, 8, size=(K, N)); Wint[0, :] = 7; Wint[64, :] = 7
    layer = {"branch": "w16a16", "rank": r, "K": K, "N": N, "bias": None,
             "L1h": rng.integers(-2, 3, size=(K, r)).astype(np.float16),
             "L2h": rng.integers(-3, 4, size=(r, N)).astype(np.float16)}
    layer["Wq"], layer["sw"] = O.q_weight_main(Wint.astype(np.float64))
    assert np.all(layer["sw"] == 1) and np.array_equal(layer["Wq"], Wint)
    out = O.forward(X, layer)
    assert np.all(out["sx"] == 1) and np.array_equal(out["qx"], X.astype(np.int8))
    Xi = X.astype(np.int64)
    expect = Xi @ (Wint + layer["L1h"].astype(np.int64) @ layer["L2h"].astype(np.int64))
    assert np.array_equal(out["Y"], expect.astype(np.float64))


def test_forward_rows_are_independent():
    rng = np.random.default_rng(11)
    X = rng.standard_normal((12, 192)).astype(np.float16)
    layer = _tiny_layer(rng, 192, 9, 4, "w4a8")
    full = O.forward(X, layer)
    part = O.forward(X[5:8], layer)
    for k in ("qx", "sx", "qb", "sXb", "tq", "sT", "Y"):
        assert np.array_equal(full[k][5:8], part[k])


# ---------------------------------------------------------------------------------------
# SVD initialisation (Section 3.2): Eckart-Young closed form
# ---------------------------------------------------------------------------------------
def test_svd_init_eckart_young_known_spectrum():
    rng = np.random.default_rng(12)
    K, N, r = 60, 40, 7
    U, _ = np.linalg.qr(rng.standard_normal((K, N)))
    V, _ = np.linalg.qr(rng.standard_normal((N, N)))
    sig = np.sort(rng.uniform(0.1, 5.0, N))[::-1]
    W = (U * sig[None, :]) @ V.T
    L0, R0 = O.svd_init(W, r)
    assert L0.shape == (K, r) and R0.shape == (r, N)
    err2 = np.linalg.norm(W - L0 @ R0) ** 2
    assert abs(err2 - np.sum(sig[r:] ** 2)) <= 1e-9 * np.sum(sig ** 2)
    assert np.allclose(L0 @ R0, (U[:, :r] * sig[None, :r]) @ V[:, :r].T, atol=1e-10)
    # even split of Sigma: both factors carry sqrt(sigma_i)
    assert np.allclose(np.linalg.norm(L0, axis=0), np.sqrt(sig[:r]), rtol=1e-10)
    assert np.allclose(np.linalg.norm(R0, axis=1), np.sqrt(sig[:r]), rtol=1e-10)
    # full rank reconstructs W
    Lf, Rf = O.svd_init(W, N)
    assert np.allclose(Lf @ Rf, W, atol=1e-10)


def test_svd_init_against_gram_eigenvalues():
    rng = np.random.default_rng(13)
    W = rng.standard_normal((50, 70)) * 0.02
    r = 5
    L0, R0 = O.svd_init(W, r)
    ev = np.sort(np.linalg.eigvalsh(W @ W.T))[::-1]        # sigma_i^2 from a different routine
    assert abs(np.linalg.norm(W - L0 @ R0) ** 2 - ev[r:].sum()) <= 1e-9 * ev.sum()


# ---------------------------------------------------------------------------------------
# Gradients (Appendix B.2) against central finite differences where no code flips
# ---------------------------------------------------------------------------------------
def test_gradients_match_finite_differences():
    rng = np.random.default_rng(14)
    K, N, r = 128, 6, 3
    W = (rng.standard_normal((K, N)) * 0.02).astype(np.float16).astype(np.float64)
    L = rng.standard_normal((K, r)) * 0.01
    R = rng.standard_normal((r, N)) * 0.01
    loss, gL, gR = O.gradients(W, L, R)
    assert abs(loss - O.objective(W, L, R)) <= 1e-18

    def codes(Lx, Rx):
        return O.q_weight_main(W + Lx @ Rx)

    h = 1e-7
    checked = 0
    for (which, idx) in itertools.chain((("L", (i, j)) for i in (0, 50, 127) for j in range(r)),
                                        (("R", (j, n)) for j in range(r) for n in (0, 5))):
        Lp, Lm, Rp, Rm = L.copy(), L.copy(), R.copy(), R.copy()
        if which == "L":
            Lp[idx] += h; Lm[idx] -= h
        else:
            Rp[idx] += h; Rm[idx] -= h
        cp, sp = codes(Lp, Rp); cm, sm = codes(Lm, Rm)
        if not (np.array_equal(cp, cm) and np.array_equal(sp, sm)):
            continue            # a code or a scale flipped: the objective is not smooth there
        fd = (O.objective(W, Lp, Rp) - O.objective(W, Lm, Rm)) / (2 * h)
        an = gL[idx] if which == "L" else gR[idx]
        assert abs(fd - an) <= 1e-6 * max(abs(an), 1e-9) + 1e-13
        checked += 1
    assert checked >= 8


# ---------------------------------------------------------------------------------------
# Calibration (Sections 3.2, 3.3; Appendix A)
# ---------------------------------------------------------------------------------------
@pytest.fixture(scope="module")
def small_calibration():
    W = I.make_weight(0, 0, "pin", 256, 192, 2)
    layer, trace = O.calibrate(W, 8, "w8a8", steps=150, lr=1e-4)
    return W, layer, trace


def test_calibration_objective(small_calibration):
    W16, layer, trace = small_calibration
    W = W16.astype(np.float64)
    # iterate 0 is the SVD initialisation with L = -L0: objective of the rank-deflated weight
    L0, R0 = O.svd_init(W, 8)
    Res = W - L0 @ R0
    e0 = O.deq_weight_main(*O.q_weight_main(Res)) - Res
    assert abs(trace[0] - np.mean(e0 * e0)) <= 1e-15
    best = np.minimum.accumulate(trace)
    assert np.all(np.diff(best) <= 0)
    assert best[-1] < trace[0] * 0.98            # Adam on (L, R) does lower the objective
    assert len(trace) == 151


def test_calibrated_layer_beats_rtn_and_svd_only(small_calibration):
    """Purpose of the method (Section 3.2): the decomposed layer approximates W better than
    round-to-nearest alone, and the optimised factors better than the SVD initialisation."""
    W16, layer, _ = small_calibration
    W = W16.astype(np.float64)
    err = np.linalg.norm(O.effective_weight(layer) - W)
    rtn = np.linalg.norm(O.q1_dequant(W) - W)
    svd_only, _ = O.calibrate(W16, 8, "w8a8", steps=0)
    err_svd = np.linalg.norm(O.effective_weight(svd_only) - W)
    assert err < err_svd < rtn
    # Figure 1: the stored residual codes are Q1 of P = W - Q2(L1) Q2(L2)
    D = O.deq_factor(layer["L1q"], layer["sL1"]) @ O.deq_factor(layer["L2q"], layer["sL2"])
    Wq, sw = O.q_weight_main(W - D)
    assert np.array_equal(Wq, layer["Wq"]) and np.array_equal(sw, layer["sw"])
    assert np.abs(layer["L1q"]).max() == 127 and np.abs(layer["L2q"]).max() == 127


def test_calibration_degenerate_cases():
    rng = np.random.default_rng(15)
    # W already in the image of Q1: objective 0 at rank 0
    Wq = rng.integers(-7, 8, size=(128, 10)); Wq[0] = 7; Wq[64] = -7
    W = (Wq * 0.03125).astype(np.float16)
    layer, trace = O.calibrate(W, 0, "none")
    assert trace[0] == 0.0 and layer["rank"] == 0
    assert np.array_equal(layer["Wq"], Wq) and np.all(layer["sw"] == np.float16(0.03125))
    assert O.objective(W.astype(np.float64), np.zeros((128, 2)), np.zeros((2, 10))) == 0.0
    # every branch format calibrates and keeps its code range
    W2 = I.make_weight(0, 0, "pin2", 128, 64, 1)
    for br, qm in (("w6a6", 31), ("w4a8", 7)):
        lay, tr = O.calibrate(W2, 4, br, steps=3)
        assert np.abs(lay["L1q"]).max() == qm and np.abs(lay["L2q"]).max() == qm
    lay, tr = O.calibrate(W2, 4, "w16a16", steps=3)
    assert lay["L1h"].dtype == np.float16 and lay["L2h"].shape == (4, 64)


def test_inputs_are_reproducible_and_shaped():
    wl = I.workload(1)
    X, W, b = I.layer_inputs(wl, wl.layers[3], M=64, with_bias=True)
    X2, W2, _ = I.layer_inputs(I.workload(2, branch="w6a6"), wl.layers[3], M=64)
    assert X.shape == (64, 4608) and W.shape == (4608, 1152) and b.shape == (1152,)
    assert np.array_equal(X, X2) and np.array_equal(W, W2)      # configs 1 and 2 share tensors
    assert X.dtype == np.float16 and np.isfinite(X.astype(np.float32)).all()
    assert np.mean(X.astype(np.float32)) > 0.1                   # GELU-shaped: positive skew
    chmax = np.abs(X.astype(np.float32)).max(0)
    assert np.sum(chmax > 25) == 8                               # eight outlier channels
    s3 = I.workload(3)
    assert s3.n_act_outliers(2240) == 22 and s3.n_w_outliers(5600) == 56


# --------------------------------------------------------------------------------------
# MXINT4 (Appendix A.3: signed int4, blocks of 32, E8M0 scale; Table 2 uses it for the residual branch)
# --------------------------------------------------------------------------------------
def test_mxint4_hand_examples(golden_dir):
    cases, cur = [], {}
    for line in open(os.path.join(golden_dir, "mxint4_hand_examples.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, vals = line.split(":")
        cur[key] = [float(t) for t in vals.split()]
        if key == "q":
            cases.append(cur); cur = {}
    assert len(cases) == 5
    for c in cases:
        v = np.zeros((1, 32)); v[0, :len(c["v"])] = c["v"]
        q, e = O.qmx(v)
        assert e[0, 0] == int(c["e"][0]), c
        assert list(q[0, :len(c["q"])]) == [int(t) for t in c["q"]], c
        assert not q[0, len(c["q"]):].any()


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_mxint4_properties(seed):
    """Minimal power-of-two scale without clipping, range, half-step error, idempotence (Section 3.2), sign symmetry,
    blocks independent; the exponent rule is re-derived with exact rational arithmetic."""
    from fractions import Fraction
    rng = np.random.default_rng(seed)
    v = (rng.standard_normal((40, 32 * 5 + 7)) * np.exp2(rng.integers(-12, 8, size=(40, 1)))).astype(np.float16).astype(np.float64)
    q, e = O.qmx(v)
    assert q.min() >= -7 and q.max() <= 7
    s = np.repeat(np.exp2(e.astype(np.float64)), 32, axis=1)[:, :v.shape[1]]
    assert np.all(np.abs(v - s * q) <= s / 2)                                  # RTN without clipping
    for r in range(0, 40, 7):
        for g in range(e.shape[1]):
            a = Fraction(float(np.abs(v[r, g * 32:(g + 1) * 32]).max()))
            if a == 0:
                assert e[r, g] == -127
                continue
            ee = int(e[r, g])
            assert 7 * Fraction(2) ** ee >= a > 7 * Fraction(2) ** (ee - 1)       # smallest admissible exponent
            assert np.abs(q[r, g * 32:(g + 1) * 32]).max() >= 4                  # so the top code is at least 4
    q2, e2 = O.qmx(O.deq_mx(q, e))
    assert np.array_equal(q2, q) and np.array_equal(e2, e)
    qn, en = O.qmx(-v)
    assert np.array_equal(qn, -q) and np.array_equal(en, e)
    w = v.copy(); w[:, 32:64] *= 16
    qw, ew = O.qmx(w)
    assert np.array_equal(np.delete(qw, np.s_[32:64], axis=1), np.delete(q, np.s_[32:64], axis=1))
    assert np.array_equal(ew[:, 1], np.where(e[:, 1] == -127, -127, e[:, 1] + 4)) and np.array_equal(qw[:, 32:64], q[:, 32:64])


def test_mxint4_weight_blocks_run_along_K():
    rng = np.random.default_rng(3)
    P = rng.standard_normal((96, 5)) * 0.02
    Wq, ew = O.q_weight_main_mx(P)
    assert Wq.shape == (96, 5) and ew.shape == (3, 5)
    for n in range(5):
        q, e = O.qmx(P[:, n][None, :])
        assert np.array_equal(q[0], Wq[:, n]) and np.array_equal(e[0], ew[:, n])


@pytest.mark.parametrize("branch", ["none", "w8a8", "w4a8"])
def test_forward_mxint4_brute_force_tiny(branch):
    """The MXINT4 forward against Python-scalar loops written from the definition: every block's integer dot product
    times 2^(ex + ew), plus the integer branch, in exact rational arithmetic."""
    from fractions import Fraction
    rng = np.random.default_rng(11)
    M, K, N, r = 3, 80, 4, (0 if branch == "none" else 3)                      # K = 2.5 blocks: a short last block
    X = rng.standard_normal((M, K)).astype(np.float16)
    X[:, 5] *= 20
    layer = {"main": "mxint4", "branch": branch if r else "none", "rank": r, "K": K, "N": N,
             "bias": (rng.standard_normal(N) * 0.1).astype(np.float16)}
    layer["Wq"], layer["ew"] = O.q_weight_main_mx(rng.standard_normal((K, N)) * 0.02)
    if r:
        bw, _ = O.BRANCH_BITS[branch]
        layer["L1q"], layer["sL1"] = O.q_factor(rng.standard_normal((K, r)) * 0.05, bw)
        layer["L2q"], layer["sL2"] = O.q_factor(rng.standard_normal((r, N)) * 0.05, bw)
    out = O.forward(X, layer)
    qx, ex = O.qmx(X.astype(np.float64))
    assert np.array_equal(out["qx"], qx) and np.array_equal(out["ex"], ex)
    for m in range(M):
        for n in range(N):
            y = Fraction(float(layer["bias"][n]))
            for g in range(3):
                dot = sum(int(qx[m, k]) * int(layer["Wq"][k, n]) for k in range(g * 32, min(K, g * 32 + 32)))
                y += Fraction(2) ** (int(ex[m, g]) + int(layer["ew"][g, n])) * dot
            if r:
                u = sum(int(out["tq"][m, j]) * int(layer["L2q"][j, n]) for j in range(r))
                y += Fraction(float(out["sT"][m])) * Fraction(float(layer["sL2"][n])) * u
            assert abs(float(y) - out["Y"][m, n]) <= 1e-12 * max(1.0, abs(float(y)))


def test_forward_mxint4_exact_integer_case():
    """Integer inputs in [-7, 7] whose block maxima are 7 quantize to themselves with exponent 0 on both sides: Y is the
    plain integer matrix product."""
    rng = np.random.default_rng(12)
    M, K, N = 5, 96, 6
    X = rng.integers(-7, 8, size=(M, K)).astype(np.float16); X[:, ::32] = 7
    Wi = rng.integers(-7, 8, size=(K, N)); Wi[::32, :] = 7
    layer = {"main": "mxint4", "branch": "none", "rank": 0, "K": K, "N": N, "bias": None}
    layer["Wq"], layer["ew"] = O.q_weight_main_mx(Wi.astype(np.float64))
    assert not layer["ew"].any() and np.array_equal(layer["Wq"], Wi)
    out = O.forward(X, layer)
    assert not out["ex"].any() and np.array_equal(out["Y"], (X.astype(np.int64) @ Wi).astype(np.float64))


# ----------------------------------------------------------------------------------------------
# Rotation-aware step (Section 3.3, Eq. "rotation-optimization" / "loss-rotation-aware")
def _rot_factors(seed, K=192, N=160, r=12):
    rng = np.random.default_rng(seed)
    L = rng.standard_normal((K, r)) * 0.1
    R = rng.standard_normal((r, N)) * 0.1
    L[:, 0] *= 6.0
    R[2, :] *= 5.0
    return L, R


@pytest.mark.parametrize("bits,lr", [(8, 0.5), (4, 0.5), (6, 0.1)])
def test_rotation_stays_orthogonal_and_keeps_the_product(bits, lr):
    L, R = _rot_factors(0)
    Om, trace = O.optimize_rotation(L, R, bits, steps=60, lr=lr)
    r = L.shape[1]
    assert np.abs(Om.T @ Om - np.eye(r)).max() < 1e-12 and abs(abs(np.linalg.det(Om)) - 1.0) < 1e-10
    assert np.abs((L @ Om) @ (Om.T @ R) - L @ R).max() < 1e-12 * np.abs(L @ R).max() + 1e-14
    # the returned rotation is the best iterate: its loss is the trace's minimum, not above the identity's
    loss_best, _, _ = O.rotation_loss(L, R, Om, bits)
    assert loss_best == trace.min() and trace.min() < trace[0]
    assert np.all(np.diff(np.minimum.accumulate(trace)) <= 0)


def test_rotation_loss_is_the_two_q2_errors_and_zero_steps_is_identity():
    L, R = _rot_factors(1)
    Om, trace = O.optimize_rotation(L, R, 8, steps=0, lr=0.5)
    assert np.array_equal(Om, np.eye(L.shape[1])) and trace.shape == (1,)
    q1, s1 = O.q_factor(L, 8); q2, s2 = O.q_factor(R, 8)
    e1 = O.deq_factor(q1, s1) - L; e2 = O.deq_factor(q2, s2) - R
    assert abs(trace[0] - (np.mean(e1 ** 2) + np.mean(e2 ** 2))) <= 1e-18 + 1e-12 * trace[0]


def test_rotation_gradient_matches_finite_differences_with_q2_frozen():
    """The derivative treats Q2's output as a constant: compare with central differences of that surrogate."""
    L, R = _rot_factors(2, K=40, N=36, r=5)
    rng = np.random.default_rng(3)
    A = rng.standard_normal((5, 5)); Om0, _ = np.linalg.qr(A)
    _, G = O.rotation_gradient(L, R, Om0, 6)
    Qa, Qb = O.q2_dequant(L @ Om0, 6), O.q2_dequant(Om0.T @ R, 6)

    def surrogate(Om):
        return float(np.mean((Qa - L @ Om) ** 2) + np.mean((Qb - Om.T @ R) ** 2))

    for _ in range(4):
        D = rng.standard_normal((5, 5))
        h = 1e-6
        fd = (surrogate(Om0 + h * D) - surrogate(Om0 - h * D)) / (2 * h)
        assert abs(fd - float(np.sum(G * D))) <= 1e-7 * max(1.0, abs(fd)) + 1e-12


def test_rotation_leaves_exactly_representable_factors_alone():
    """Factors already on Q2's grid have zero loss and zero gradient: the identity is kept."""
    rng = np.random.default_rng(4)
    L = rng.integers(-127, 128, size=(32, 4)).astype(np.float64); L[0, :] = 127
    R = rng.integers(-127, 128, size=(4, 24)).astype(np.float64); R[0, :] = 127
    Om, trace = O.optimize_rotation(L, R, 8, steps=5, lr=0.5)
    assert trace[0] == 0.0 and np.array_equal(Om, np.eye(4))


def test_calibrate_with_rotation_keeps_the_decomposition_consistent():
    W = I.make_weight(0, 0, "rot", 128, 96, 2)
    lay0, _ = O.calibrate(W, 8, "w4a8", steps=3)
    lay1, _ = O.calibrate(W, 8, "w4a8", steps=3, rot_steps=40, rot_lr=0.5)
    assert lay1["rot_trace"].shape == (41,) and lay1["rot_trace"].min() < lay1["rot_trace"][0]
    W64 = W.astype(np.float64)
    # stored residual codes are still Q1 of P = W - Q2(L1) Q2(L2)
    D1 = O.deq_factor(lay1["L1q"], lay1["sL1"]) @ O.deq_factor(lay1["L2q"], lay1["sL2"])
    Wq, sw = O.q_weight_main(W64 - D1)
    assert np.array_equal(Wq, lay1["Wq"]) and np.array_equal(sw, lay1["sw"])
    # both layers approximate the same product L1 L2: they differ by Q2's error only
    D0 = O.deq_factor(lay0["L1q"], lay0["sL1"]) @ O.deq_factor(lay0["L2q"], lay0["sL2"])
    assert np.linalg.norm(D1 - D0) <= 0.5 * np.linalg.norm(D0)
