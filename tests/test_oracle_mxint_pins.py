"""Pins for the oracle of the integer MX variant with 8-bit activations (oracle/lq_oracle_mxint.py): Appendix A.3's
MXINT8 / MXINT4 formats under the stated reading, and the decomposed forward / calibration of Figure 1 and
Sections 3.2-3.3 with the Table 3 integer rows' assignment of formats."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import lq_oracle as O
from oracle import lq_oracle_mxint as OI


def test_mxint8_hand_examples(golden_dir):
    cases, cur = [], {}
    for line in open(os.path.join(golden_dir, "mxint8_hand_examples.txt")):
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
        q, e = OI.qmxint(v, 8)
        assert e[0, 0] == int(c["e"][0]), c
        assert list(q[0, :len(c["q"])]) == [int(t) for t in c["q"]], c
        assert not q[0, len(c["q"]):].any()


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("seed", [0, 1])
def test_mxint_properties(bits, seed):
    """Minimal power-of-two scale without clipping (re-derived in exact rational arithmetic), range, half-step error,
    idempotence (Section 3.2), sign symmetry, exact equivariance under powers of two, blocks independent, short last
    block, zero block."""
    qmax = 2 ** (bits - 1) - 1
    rng = np.random.default_rng(seed)
    v = (rng.standard_normal((24, 32 * 4 + 9)) * np.exp2(rng.integers(-12, 8, size=(24, 1)))).astype(np.float16).astype(np.float64)
    v[3, 32:64] = 0.0
    q, e = OI.qmxint(v, bits)
    assert q.min() >= -qmax and q.max() <= qmax
    s = np.repeat(np.exp2(e.astype(np.float64)), 32, axis=1)[:, :v.shape[1]]
    assert np.all(np.abs(v - s * q) <= s / 2)                                  # RTN without clipping
    assert e[3, 1] == -127 and not q[3, 32:64].any()
    for r in range(0, 24, 5):
        for g in range(e.shape[1]):
            a = Fraction(float(np.abs(v[r, g * 32:(g + 1) * 32]).max()))
            if a == 0:
                continue
            ee = int(e[r, g])
            assert qmax * Fraction(2) ** ee >= a > qmax * Fraction(2) ** (ee - 1)   # the smallest exponent that does not clip
    q2, e2 = OI.qmxint(OI.deq_mxint(q, e), bits)                               # idempotent: Q(deq(Q(v))) = Q(v)
    # a block whose maximum rounded down may take a smaller exponent the second time; its VALUES must not change
    assert np.array_equal(OI.deq_mxint(q2, e2), OI.deq_mxint(q, e))
    qn, en = OI.qmxint(-v, bits)
    assert np.array_equal(qn, -q) and np.array_equal(en, e)
    qs, es = OI.qmxint(v * 2.0 ** -5, bits)
    assert np.array_equal(qs, q) and np.array_equal(es[e > -127], e[e > -127] - 5)
    w = v.copy(); w[:, 64:96] *= 3.0                                            # touching one block leaves the others alone
    qw, ew = OI.qmxint(w, bits)
    keep = np.r_[0:64, 96:v.shape[1]]
    assert np.array_equal(qw[:, keep], q[:, keep]) and np.array_equal(np.delete(ew, 2, axis=1), np.delete(e, 2, axis=1))


def test_four_bit_case_is_the_mxint4_quantizer():
    """bits = 4 must reproduce the MXINT4 quantizer that has its own hand-worked pins."""
    rng = np.random.default_rng(5)
    v = (rng.standard_normal((16, 200)) * np.exp2(rng.integers(-10, 6, size=(16, 1)))).astype(np.float16).astype(np.float64)
    q4, e4 = O.qmx(v)
    q, e = OI.qmxint(v, 4)
    assert np.array_equal(q, q4) and np.array_equal(e, e4)


def _scalar_forward(X, layer):
    """The forward written out with Python scalars from the definition: every operand dequantized to a float, plain
    triple loops, the intermediate re-quantized with the quantizer under test (its own pins are above)."""
    M, K = X.shape
    N = layer["Wq"].shape[1]
    r = layer["rank"]
    xa, ex = OI.qmxint(X, 8)
    xd = [[float(xa[m, k]) * 2.0 ** int(ex[m, k // 32]) for k in range(K)] for m in range(M)]
    wd = [[float(layer["Wq"][k, n]) * 2.0 ** int(layer["ew"][k // 32, n]) for n in range(N)] for k in range(K)]
    Y = [[sum(xd[m][k] * wd[k][n] for k in range(K)) for n in range(N)] for m in range(M)]
    if r:
        l1 = [[float(layer["L1q"][k, j]) * 2.0 ** int(layer["e1"][k // 32, j]) for j in range(r)] for k in range(K)]
        l2 = [[float(layer["L2q"][j, n]) * 2.0 ** int(layer["e2"][j // 32, n]) for n in range(N)] for j in range(r)]
        T = np.array([[sum(xd[m][k] * l1[k][j] for k in range(K)) for j in range(r)] for m in range(M)])
        tq, et = OI.qmxint(T, 8)
        for m in range(M):
            for n in range(N):
                Y[m][n] += sum(float(tq[m, j]) * 2.0 ** int(et[m, j // 32]) * l2[j][n] for j in range(r))
    if layer.get("bias") is not None:
        for m in range(M):
            for n in range(N):
                Y[m][n] += float(layer["bias"][n])
    return np.array(Y)


@pytest.mark.parametrize("branch,r", [("mxint8", 40), ("mxint4", 33), ("none", 0)])
def test_forward_against_scalar_loops(branch, r):
    rng = np.random.default_rng(11)
    M, K, N = 5, 70, 44                                                         # ragged: K and r are not multiples of 32
    W = (rng.standard_normal((K, N)) * 0.05).astype(np.float16)
    X = (rng.standard_normal((M, K)) * 1.5).astype(np.float16)
    layer, _ = OI.calibrate(W, r, branch, steps=2, bias=(rng.standard_normal(N) * 0.1).astype(np.float16))
    ref = _scalar_forward(X.astype(np.float64), layer)
    Y = OI.forward(X, layer)["Y"]
    assert np.max(np.abs(Y - ref)) <= 1e-12 * np.max(np.abs(ref))


def test_all_integer_case_is_an_integer_matrix_product():
    """Inputs on the grids (block maxima 127 for X, 7 for W, 127 for the factors and for T's blocks, all exponents 0):
    every quantizer is exact and Y = X W + (X L1) L2 as integer matrices - provided X L1 stays within [-127, 127]."""
    rng = np.random.default_rng(3)
    M, K, N, r = 6, 64, 10, 32
    X = rng.integers(-3, 4, size=(M, K)).astype(np.float64); X[:, 0] = 127; X[:, 32] = -127
    Wq = rng.integers(-7, 8, size=(K, N)); Wq[0, :] = 7; Wq[32, :] = -7
    L1 = np.zeros((K, r), dtype=np.int64); L1[1, :] = rng.integers(-20, 21, size=r); L1[1, 0] = 127   # T = X[:,1] * L1[1,:]
    X[:, 1] = 1.0
    L1[0, :] = 0
    L2 = rng.integers(-127, 128, size=(r, N)); L2[0, :] = 127
    layer = {"branch": "mxint8", "rank": r, "K": K, "N": N, "bias": None, "Wq": Wq, "ew": np.zeros((2, N), np.int16),
             "L1q": L1, "e1": np.zeros((2, r), np.int16), "L2q": L2, "e2": np.zeros((1, N), np.int16)}
    out = OI.forward(X.astype(np.float16), layer)
    assert np.array_equal(out["xa"], X.astype(np.int16)) and not out["ex"].any()
    T = X.astype(np.int64) @ L1
    assert np.abs(T).max() == 127 and np.array_equal(out["tq"], T) and not out["et"].any()
    assert np.array_equal(out["Y"], (X.astype(np.int64) @ Wq + T @ L2).astype(np.float64))


def test_calibration_invariants():
    rng = np.random.default_rng(2)
    K, N, r = 96, 48, 8
    W = (rng.standard_normal((K, N)) * 0.02).astype(np.float16)
    W[:, 3] *= 10
    layer, trace = OI.calibrate(W, r, "mxint8", steps=30, lr=1e-3)
    # the returned iterate is the best seen; it is at least as good as the SVD start
    assert trace.min() <= trace[0]
    # residual codes are Q1 of W - Q2(L1) Q2(L2) (Figure 1)
    D = OI.deq_columns(layer["L1q"], layer["e1"]) @ OI.deq_columns(layer["L2q"], layer["e2"])
    q, e = OI.q_columns(W.astype(np.float64) - D, 4)
    assert np.array_equal(q, layer["Wq"]) and np.array_equal(e, layer["ew"])
    # the decomposed layer is closer to W than plain MXINT4 rounding of W (Section 3.1)
    Wd = W.astype(np.float64)
    err_plain = np.linalg.norm(OI.q1_dequant(Wd) - Wd)
    err_layer = np.linalg.norm(OI.effective_weight(layer) - Wd)
    assert err_layer < err_plain
    # rank 0 / no branch: plain Q1
    l0, t0 = OI.calibrate(W, 0, "none")
    assert l0["rank"] == 0 and np.array_equal(OI.effective_weight(l0), OI.q1_dequant(Wd)) and t0.shape == (1,)
