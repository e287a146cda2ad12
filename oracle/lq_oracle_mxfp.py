"""CPU oracle for the MXFP variants of the LoRaQ layer.  TEST INFRASTRUCTURE ONLY (same rules as lq_oracle.py:
imported by the tests, the smoke check and the benchmark's CPU-baseline leg, never by the product).

What it follows
---------------
* MX formats (Appendix A.3 "MX Formats"): blocks of 32 values share one 8-bit power-of-two scale (E8M0); the
  scaled values are rounded (round to nearest) to a small float: MXFP8e4 -> e4m3, MXFP6e2 -> e2m3, MXFP4e2 -> e2m1.
  The paper takes the formats from the OCP Microscaling specification it cites; that specification fixes the
  element grids and the conversion used here: shared exponent = floor(log2(max |v|)) - emax(element format), each
  element = v / 2^exponent rounded to the nearest element value, ties to even, clamped to the largest normal.
* Mixed-precision study (Section 4.3, Tables 3 and 4; Appendix A.2 "Quantization"): residual weights fixed to a
  4-bit MX format (MXFP4e2 here), activations forwarded to BOTH branches in one 8-bit MX format (MXFP8e4), low-rank
  factors in MXFP8e4 / MXFP6e2 / MXFP4e2 with rank 64 / 86 / 128 at equal memory.
* Rank study (Section 4.3, Table 4): activations and low-rank factors share ONE sub-16-bit format, MXFP8e4 or MXFP6e2;
  a layer's "act" entry names the activations' element format ("e4m3" when absent, "e2m3" for the MXFP6e2 rows) and
  applies to X and to the re-quantized intermediate alike.
* Decomposed forward and calibration: as in lq_oracle.py (Figure 1, Sections 3.2-3.3, Appendix B.2), with
  Q1 = MXFP4e2 along K per output column and Q2 = the branch format along each factor's contraction axis
  (L1 along K per column, L2 along r per column); learning rate 1e-3 for FP formats (Appendix A.2 "Optimization").

Readings taken where the paper is silent: blocks run along the contraction axis (K for X, W and L1; r for T and L2),
a short last block when the axis is not a multiple of 32; an all-zero block gets exponent -127 and zero elements;
the exponent is limited to the E8M0 range [-127, 127]; the rank-r intermediate T = deq(Q(X)) deq(Q2(L1)) is
re-quantized to the activations' format (MXFP8e4) along r before the second factor (the same reading as the integer
formats: the task's formula quantizes it; the paper lists it as future work).

Arithmetic: power-of-two scalings and element values are exact in float64; dot products of element values are
exact in float64 for every size used here (4-bit x 4-bit significands, at most 2^13 terms); sums over blocks are
float64.
"""
from __future__ import annotations

import numpy as np

from oracle import lq_oracle as O

MX_BLOCK = 32
# element format -> (mantissa bits, exponent of the smallest normal, exponent of the largest normal, largest normal)
FORMATS = {
    "e4m3": (3, -6, 8, 448.0),      # OCP FP8 E4M3: bias 7, no infinities, largest normal 1.75 * 2^8
    "e2m3": (3, 0, 2, 7.5),         # OCP FP6 E2M3: bias 1, largest 1.875 * 2^2
    "e2m1": (1, 0, 2, 6.0),         # OCP FP4 E2M1: bias 1, largest 1.5 * 2^2
}
BRANCH_FORMAT = {"mxfp8": "e4m3", "mxfp6": "e2m3", "mxfp4": "e2m1"}


def element_values(fmt: str) -> np.ndarray:
    """All non-negative values of an element format, ascending, from its definition: subnormals m / 2^mant * 2^emin,
    normals (1 + m / 2^mant) * 2^e for emin <= e <= emax, capped at the largest normal (e4m3 gives up its top
    mantissa pattern at the top exponent to NaN)."""
    mant, emin, emax, vmax = FORMATS[fmt]
    vals = [m / 2 ** mant * 2.0 ** emin for m in range(2 ** mant)]
    for e in range(emin, emax + 1):
        vals += [(1 + m / 2 ** mant) * 2.0 ** e for m in range(2 ** mant)]
    return np.array(sorted(v for v in set(vals) if v <= vmax))


def round_to_element(v, fmt: str):
    """v (float64, any shape) rounded to the nearest value of the element format, ties to the even mantissa,
    magnitudes above the largest normal clamped to it."""
    mant, emin, emax, vmax = FORMATS[fmt]
    v = np.asarray(v, dtype=np.float64)
    a = np.abs(v)
    e = np.frexp(np.where(a > 0, a, 1.0))[1] - 1.0          # floor(log2 a), exact: a = m 2^e with m in [0.5, 1)
    e = np.clip(e, emin, emax)
    quantum = np.exp2(e - mant)
    q = np.rint(a / quantum) * quantum        # numpy rint rounds half to even; a / quantum is exact (power of two)
    return np.sign(v) * np.minimum(q, vmax)


def qmxfp(v, fmt: str, block: int = MX_BLOCK):
    """MX quantizer along the last axis.  Returns (elements float32 [.., n] - the element VALUES, i.e. what the
    format's bit pattern decodes to - and exponents int16 [.., ceil(n / block)]); the real value is element * 2^exp."""
    mant, emin, emax, vmax = FORMATS[fmt]
    v = np.asarray(v, dtype=np.float64)
    n = v.shape[-1]
    nb = -(-n // block)
    pad = nb * block - n
    vp = np.concatenate([v, np.zeros(v.shape[:-1] + (pad,))], axis=-1) if pad else v
    vb = vp.reshape(v.shape[:-1] + (nb, block))
    a = np.abs(vb).max(axis=-1)
    ex = np.frexp(np.where(a > 0, a, 1.0))[1] - 1.0 - emax  # floor(log2 max) - emax
    ex = np.where(a > 0, np.clip(ex, -127, 127), -127.0)
    el = round_to_element(vb / np.exp2(ex)[..., None], fmt)
    el = np.where(a[..., None] > 0, el, 0.0)
    el = el.reshape(v.shape[:-1] + (nb * block,))[..., :n]
    return el.astype(np.float32), ex.astype(np.int16)


def deq_mxfp(el, ex, block: int = MX_BLOCK):
    el = np.asarray(el, dtype=np.float64)
    return el * np.repeat(np.exp2(np.asarray(ex, dtype=np.float64)), block, axis=-1)[..., :el.shape[-1]]


def q_columns(F, fmt: str):
    """Quantizer of a matrix whose blocks run down its columns (along axis 0, the contraction axis): returns
    (elements [rows, cols], exponents [ceil(rows / 32), cols])."""
    el, ex = qmxfp(np.asarray(F, dtype=np.float64).T.copy(), fmt)
    return el.T.copy(), ex.T.copy()


def deq_columns(el, ex):
    return deq_mxfp(np.asarray(el).T.copy(), np.asarray(ex).T.copy()).T.copy()


def forward(X16, layer):
    """Reference forward of one MXFP layer.
    layer: Wv float32 [K, N] (e2m1 element values), ew int16 [ceil(K/32), N]; branch "mxfp8" | "mxfp6" | "mxfp4" |
    "none"; rank; L1v [K, r], e1 [ceil(K/32), r]; L2v [r, N], e2 [ceil(r/32), N]; optional bias fp16 [N].
    layer["act"] (optional): element format of the activations, "e4m3" (default) or "e2m3"; written MXFP8e4 below.
    Steps: (1) xa, ex = MXFP8e4 of X rows, shared by both branches; (2) main: sum over K blocks of
    2^(ex + ew) (xa_b Wv_b), exact element products; (3) T = sum over K blocks of 2^(ex + e1) (xa_b L1v_b);
    (4) tq, et = MXFP8e4 of T rows along r; (5) Y += sum over r blocks of 2^(et + e2) (tq_c L2v_c) (+ bias), float64."""
    X = np.asarray(X16, dtype=np.float16).astype(np.float64)
    M, K = X.shape
    Wv, ew = layer["Wv"].astype(np.float64), layer["ew"]
    N = Wv.shape[1]
    act = layer.get("act", "e4m3")
    xa, ex = qmxfp(X, act)
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
        Y += sa * np.exp2(ew[b, :].astype(np.float64))[None, :] * (xa64[:, k0:k1] @ Wv[k0:k1, :])
        if has_branch:
            T += sa * np.exp2(layer["e1"][b, :].astype(np.float64))[None, :] * (xa64[:, k0:k1] @ layer["L1v"][k0:k1, :].astype(np.float64))
    if has_branch:
        tq, et = qmxfp(T, act)
        out.update(T=T, tq=tq, et=et)
        tq64 = tq.astype(np.float64)
        for c in range(-(-r // MX_BLOCK)):
            j0, j1 = c * MX_BLOCK, min(r, (c + 1) * MX_BLOCK)
            Y += (np.exp2(et[:, c].astype(np.float64))[:, None] * np.exp2(layer["e2"][c, :].astype(np.float64))[None, :] *
                  (tq64[:, j0:j1] @ layer["L2v"][j0:j1, :].astype(np.float64)))
    if layer.get("bias") is not None:
        Y += layer["bias"].astype(np.float64)[None, :]
    out["Y"] = Y
    return out


def q1_dequant(A):
    return deq_columns(*q_columns(A, "e2m1"))


def calibrate(W16, rank: int, branch: str = "mxfp8", steps: int = 1000, lr: float = 1e-3, beta1: float = 0.9,
              beta2: float = 0.999, eps: float = 1e-8, bias=None):
    """Data-free calibration with Q1 = MXFP4e2 and Q2 = the branch's MX format (Sections 3.2-3.3; same procedure and
    readings as lq_oracle.calibrate).  Returns (layer dict, objective trace [steps + 1])."""
    W = np.asarray(W16, dtype=np.float16).astype(np.float64)
    K, N = W.shape
    layer = {"main": "mxfp4", "branch": branch, "rank": int(rank), "K": K, "N": N,
             "bias": None if bias is None else np.asarray(bias, dtype=np.float16)}
    if branch == "none" or rank == 0:
        layer["branch"], layer["rank"] = "none", 0
        layer["Wv"], layer["ew"] = q_columns(W, "e2m1")
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
    fmt = BRANCH_FORMAT[branch]
    layer["L1v"], layer["e1"] = q_columns(L1, fmt)
    layer["L2v"], layer["e2"] = q_columns(L2, fmt)
    D = deq_columns(layer["L1v"], layer["e1"]) @ deq_columns(layer["L2v"], layer["e2"])
    layer["Wv"], layer["ew"] = q_columns(W - D, "e2m1")     # P = W - Q2(L1) Q2(L2), then Q1
    return layer, trace


def effective_weight(layer):
    Wd = deq_columns(layer["Wv"], layer["ew"])
    if layer["branch"] == "none" or layer["rank"] == 0:
        return Wd
    return Wd + deq_columns(layer["L1v"], layer["e1"]) @ deq_columns(layer["L2v"], layer["e2"])
