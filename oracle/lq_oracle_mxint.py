"""CPU oracle for the integer MX variant of the LoRaQ layer with 8-bit activations.  TEST INFRASTRUCTURE ONLY (same
rules as lq_oracle.py: imported by the tests, the smoke check and the benchmark's CPU-baseline leg, never by the product).

What it follows
---------------
* MX formats (Appendix A.3 "MX Formats"): blocks of 32 values share one 8-bit power-of-two scale (E8M0); MXINT4 and
  MXINT8 quantize the scaled values to a signed 4-bit / 8-bit integer.
* Mixed-precision study, integer rows (Section 4.3, Table 3; its appendix figure states the setting): residual weights
  MXINT4, activations MXINT8 - forwarded to BOTH branches - and low-rank factors MXINT8 (rank 64) or MXINT4 (rank 128)
  at equal memory.
* Decomposed forward and calibration: as in lq_oracle.py (Figure 1, Sections 3.2-3.3, Appendix B.2), with
  Q1 = MXINT4 along K per output column and Q2 = the factors' format along each factor's contraction axis
  (L1 along K per column, L2 along r per column); learning rate 1e-4 for integer formats (Appendix A.2 "Optimization").

Readings taken where the paper is silent (the same as for MXINT4 in lq_oracle.py): symmetric codes in
[-qmax, qmax], qmax = 2^(bits-1) - 1 (the most negative code is unused); the block exponent is the smallest e with
qmax * 2^e >= max|v| so that nothing clips, limited to [-127, 127], -127 for an all-zero block; codes
rint_even(v / 2^e) (the division is exact); blocks run along the contraction axis, a short last block when the axis
is not a multiple of 32; the rank-r intermediate T = deq(Q(X)) deq(Q2(L1)) is re-quantized to the activations' format
(MXINT8) along r before the second factor.

Arithmetic: codes times powers of two are exact in float64; integer dot products over a block are exact; sums over
blocks are float64.
"""
from __future__ import annotations

import numpy as np

from oracle import lq_oracle as O

MX_BLOCK = 32
FACTOR_BITS = {"mxint8": 8, "mxint4": 4}
ACT_BITS = 8


def qmxint(v, bits: int, block: int = MX_BLOCK):
    """MX integer quantizer along the last axis.  Returns (codes int16 [.., n], exponents int16 [.., ceil(n / block)]);
    the real value is code * 2^exponent."""
    qmax = 2 ** (bits - 1) - 1
    v = np.asarray(v, dtype=np.float64)
    n = v.shape[-1]
    nb = -(-n // block)
    pad = nb * block - n
    vp = np.concatenate([v, np.zeros(v.shape[:-1] + (pad,))], axis=-1) if pad else v
    vb = vp.reshape(v.shape[:-1] + (nb, block))
    a = np.abs(vb).max(axis=-1)
    # a = m 2^x with m in [0.5, 1):  qmax 2^e >= a  <=>  2^(e - x) >= m / qmax;  qmax / 2^(bits-1) is just below 1
    m, x = np.frexp(np.where(a > 0, a, 1.0))
    e = np.where(m <= qmax / 2.0 ** (bits - 1), x - (bits - 1), x - (bits - 2)).astype(np.float64)
    e = np.where(a > 0, np.clip(e, -127, 127), -127.0)
    q = np.clip(np.rint(vb / np.exp2(e)[..., None]), -qmax, qmax)
    q = q.reshape(v.shape[:-1] + (nb * block,))[..., :n]
    return q.astype(np.int16), e.astype(np.int16)


def deq_mxint(codes, exps, block: int = MX_BLOCK):
    codes = np.asarray(codes, dtype=np.float64)
    return codes * np.repeat(np.exp2(np.asarray(exps, dtype=np.float64)), block, axis=-1)[..., :codes.shape[-1]]


def q_columns(F, bits: int):
    """Quantizer of a matrix whose blocks run down its columns (along axis 0, the contraction axis): returns
    (codes [rows, cols], exponents [ceil(rows / 32), cols])."""
    q, e = qmxint(np.asarray(F, dtype=np.float64).T.copy(), bits)
    return q.T.copy(), e.T.copy()


def deq_columns(q, e):
    return deq_mxint(np.asarray(q).T.copy(), np.asarray(e).T.copy()).T.copy()


def forward(X16, layer):
    """Reference forward of one layer with MXINT4 weights and MXINT8 activations.
    layer: Wq int [K, N] (codes in [-7, 7]), ew int16 [ceil(K/32), N]; branch "mxint8" | "mxint4" | "none"; rank;
    L1q [K, r], e1 [ceil(K/32), r]; L2q [r, N], e2 [ceil(r/32), N]; optional bias fp16 [N].
    Steps: (1) xa, ex = MXINT8 of X rows, shared by both branches; (2) main: sum over K blocks of
    2^(ex + ew) (xa_b Wq_b), exact integer block products; (3) T = sum over K blocks of 2^(ex + e1) (xa_b L1q_b);
    (4) tq, et = MXINT8 of T rows along r; (5) Y += sum over r blocks of 2^(et + e2) (tq_c L2q_c) (+ bias), float64."""
    X = np.asarray(X16, dtype=np.float16).astype(np.float64)
    M, K = X.shape
    Wq, ew = layer["Wq"].astype(np.float64), layer["ew"]
    N = Wq.shape[1]
    xa, ex = qmxint(X, ACT_BITS)
    out = {"xa": xa, "ex": ex}
    xa64 = xa.astype(np.float64)
    Y = np.zeros((M, N))
    nb = -(-K // MX_BLOCK)
    r = int(layer["rank"])
    has_branch = layer["branch"] != "none" and r > 0
    T = np.zeros((M, r)) if has_branch else None
    for b in range(nb):
        k0, k1 = b * MX_BLOCK, min(K, (b + 1) * MX_BLOCK)
        sa = np.exp2(ex[:, b].astype(np.float64))[:, None]
        Y += sa * np.exp2(ew[b, :].astype(np.float64))[None, :] * (xa64[:, k0:k1] @ Wq[k0:k1, :])
        if has_branch:
            T += sa * np.exp2(layer["e1"][b, :].astype(np.float64))[None, :] * (xa64[:, k0:k1] @ layer["L1q"][k0:k1, :].astype(np.float64))
    if has_branch:
        tq, et = qmxint(T, ACT_BITS)
        out.update(T=T, tq=tq, et=et)
        tq64 = tq.astype(np.float64)
        for c in range(-(-r // MX_BLOCK)):
            j0, j1 = c * MX_BLOCK, min(r, (c + 1) * MX_BLOCK)
            Y += (np.exp2(et[:, c].astype(np.float64))[:, None] * np.exp2(layer["e2"][c, :].astype(np.float64))[None, :] *
                  (tq64[:, j0:j1] @ layer["L2q"][j0:j1, :].astype(np.float64)))
    if layer.get("bias") is not None:
        Y += layer["bias"].astype(np.float64)[None, :]
    out["Y"] = Y
    return out


def q1_dequant(A):
    return deq_columns(*q_columns(A, 4))


def calibrate(W16, rank: int, branch: str = "mxint8", steps: int = 1000, lr: float = 1e-4, beta1: float = 0.9,
              beta2: float = 0.999, eps: float = 1e-8, bias=None):
    """Data-free calibration with Q1 = MXINT4 and Q2 = the factors' MX integer format (Sections 3.2-3.3; same
    procedure and readings as lq_oracle.calibrate).  Returns (layer dict, objective trace [steps + 1])."""
    W = np.asarray(W16, dtype=np.float16).astype(np.float64)
    K, N = W.shape
    layer = {"main": "mxint4a8", "branch": branch, "rank": int(rank), "K": K, "N": N,
             "bias": None if bias is None else np.asarray(bias, dtype=np.float16)}
    if branch == "none" or rank == 0:
        layer["branch"], layer["rank"] = "none", 0
        layer["Wq"], layer["ew"] = q_columns(W, 4)
        E = q1_dequant(W) - W
        return layer, np.array([float(np.mean(E * E))])
    L0, R0 = O.svd_init(W, rank)
    L, R = -L0, R0
    mL = np.zeros_like(L); vL = np.zeros_like(L)
    mR = np.zeros_like(R); vR = np.zeros_like(R)
    trace = np.zeros(steps + 1)
    best = (np.inf, None, None)
    for t in range(steps + 1):
        D = L @ R
        E = q1_dequant(W + D) - W - D                       # Eq. "low-rank-optimization"
        loss = float(np.mean(E * E))
        trace[t] = loss
        if loss < best[0]:
            best = (loss, L.copy(), R.copy())
        if t == steps:
            break
        c = -2.0 / E.size                                   # Appendix B.2, the quantizer's derivative taken as zero
        gL, gR = c * (E @ R.T), c * (L.T @ E)
        L, mL, vL = O.adam_update(L, gL, mL, vL, t + 1, lr, beta1, beta2, eps)
        R, mR, vR = O.adam_update(R, gR, mR, vR, t + 1, lr, beta1, beta2, eps)
    L1, L2 = -best[1], best[2]                              # Figure 1 sign: W ~ P + L1 L2
    bits = FACTOR_BITS[branch]
    layer["L1q"], layer["e1"] = q_columns(L1, bits)
    layer["L2q"], layer["e2"] = q_columns(L2, bits)
    D = deq_columns(layer["L1q"], layer["e1"]) @ deq_columns(layer["L2q"], layer["e2"])
    layer["Wq"], layer["ew"] = q_columns(W - D, 4)          # P = W - Q2(L1) Q2(L2), then Q1
    return layer, trace


def effective_weight(layer):
    Wd = deq_columns(layer["Wq"], layer["ew"])
    if layer["branch"] == "none" or layer["rank"] == 0:
        return Wd
    return Wd + deq_columns(layer["L1q"], layer["e1"]) @ deq_columns(layer["L2q"], layer["e2"])
