"""CPU oracle for the LoRaQ fully quantized linear layer.  TEST INFRASTRUCTURE ONLY.

This file is a plain, slow, obviously-correct numpy statement of what the hot
path computes.  It is imported only by the tests, by the smoke check and by the
benchmark's CPU-baseline leg; the product (the CUDA library and its binding)
never imports it and shares no code, table or constant generator with it.

What it follows
---------------
* Quantization error / upper bound: Section 3.1 (Eq. "error_upper_bound").
* Error absorption, idempotence of Q, the calibration objective
  ``min_{L,R} || Q(W + L R) - W - L R ||_F`` (MSE form): Section 3.2
  (Eq. "quantization-error", Eq. "low-rank-optimization").
* SVD initialisation ``L = -L0, R = R0``: Section 3.2, last paragraph.
* Gradients with dQ/d. = 0 almost everywhere: Appendix B.2
  (Eq. "low-rank-gradients", "low-rank-gradients-update", "...-R").
* Adam, 1000 steps, learning rate 1e-4 for integer formats: Appendix A.1/A.2 "Optimization".
* Two quantizers Q1 (residual branch) and Q2 (low-rank branch), residual
  ``P = W - Q2(L)Q2(R)``: Section 3.3 (Eq. "quantization-lr") and the Figure 1 caption.
* Decomposed forward ``Y = Q(X) Q1(P) + Q(X) Q2(L) Q2(R)`` with the activations of
  both branches quantized: Figure 1 caption and Appendix A.2 "Quantization".
* SINT4 format (signed int4, blocks of 64 values, one FP16 scale per block,
  round-to-nearest): Appendix A.3 "Blockwise Formats".
* MXINT4 format (signed int4, blocks of 32 values, one E8M0 power-of-two scale per
  block, round-to-nearest): Appendix A.3; used for the residual branch in Table 2.

Readings taken where the paper is silent (each is listed in the design notes):
symmetric range [-7, 7] with scale = absmax / 7 rounded to fp16; ties to even;
scale floor 2^-24; groups run along the contraction axis K; a short last group
when K is not a multiple of 64; the branch quantizers (W8A8 / W6A6 / W4A8) are
symmetric integers with one fp32 scale per token (activations, and the rank-r
intermediate) or per output column (the two factors); the intermediate
``T = Q(X) Q(L1)`` is re-quantized per token; Q2 is applied after the Adam loop
and P is recomputed from the quantized factors; Sigma is split evenly between
L0 and R0; the loss is the mean over K*N entries; Adam uses (0.9, 0.999, 1e-8)
with bias correction; the best iterate seen is returned.

MXINT4 reading (the paper gives neither range nor exponent rule): codes in [-7, 7],
scale 2^e with e the smallest integer such that 7 * 2^e >= absmax of the block (no
clipping), e limited to the E8M0 range [-127, 127], e = -127 for an all-zero block.

Parity unpinned (the paper prints no number for them): the Adam trajectory, the
split of Sigma between L0 and R0.

Arithmetic conventions: every "fl32" operation is IEEE binary32, round to nearest
even, true division, no fused multiply-add (numpy float32 scalars/arrays obey
this).  Integer products are exact (carried in float64, whose 53-bit significand
holds every sum that occurs).  Final sums are float64.
"""
from __future__ import annotations

import numpy as np

GROUP = 64                      # SINT4 block (Appendix A.3)
QMAX4 = 7                       # symmetric signed int4: codes in [-7, 7]
SCALE_FLOOR = np.float16(2.0 ** -24)   # smallest positive fp16

# branch format -> (weight bits, activation bits); None = fp16 (the W16A16 reference)
BRANCH_BITS = {"w8a8": (8, 8), "w6a6": (6, 6), "w4a8": (4, 8), "w16a16": (None, None), "none": (0, 0)}


def qmax(bits: int) -> int:
    return (1 << (bits - 1)) - 1


# --------------------------------------------------------------------------------------
# Quantizers (Appendix A.3; Section 3.2 for idempotence)
# --------------------------------------------------------------------------------------
def qgrp(v, group: int = GROUP):
    """SINT4 quantizer along the last axis of a 2-D array.

    v[i, :] is cut into consecutive groups of `group` values (the last may be
    short).  Per group: a = max|v| in fl32; s = fp16(a /fl32 7), floored at 2^-24;
    q = clamp(rint_even(v /fl32 s), -7, 7).
    Returns (codes int8 [R, L], scales fp16 [R, ceil(L/group)]).
    """
    v = np.asarray(v, dtype=np.float32)
    R, L = v.shape
    G = -(-L // group)
    codes = np.zeros((R, L), dtype=np.int8)
    scales = np.zeros((R, G), dtype=np.float16)
    for g in range(G):
        blk = v[:, g * group:(g + 1) * group]
        a = np.max(np.abs(blk), axis=1).astype(np.float32)
        s = (a / np.float32(QMAX4)).astype(np.float16)
        s = np.maximum(s, SCALE_FLOOR)
        q = np.rint(blk / s.astype(np.float32)[:, None])
        codes[:, g * group:(g + 1) * group] = np.clip(q, -QMAX4, QMAX4).astype(np.int8)
        scales[:, g] = s
    return codes, scales


MX_BLOCK = 32                   # MXINT4 block (Appendix A.3)


def qmx(v, block: int = MX_BLOCK):
    """MXINT4 quantizer along the last axis of a 2-D array.

    Per block of `block` consecutive values (the last may be short): a = max|v|;
    e = the smallest integer with 7 * 2^e >= a, clamped to [-127, 127] (-127 when a == 0);
    q = clamp(rint_even(v / 2^e), -7, 7) - the division by a power of two is exact.
    Returns (codes int8 [R, L], exponents int16 [R, ceil(L/block)]); the scale is 2.0**e.
    """
    v = np.asarray(v, dtype=np.float64)
    R, L = v.shape
    G = -(-L // block)
    codes = np.zeros((R, L), dtype=np.int8)
    exps = np.zeros((R, G), dtype=np.int16)
    for g in range(G):
        blk = v[:, g * block:(g + 1) * block]
        a = np.max(np.abs(blk), axis=1)
        e = np.full(R, -127, dtype=np.int64)
        nz = a > 0
        # frexp: a = m * 2^x with m in [0.5, 1); 7 * 2^e >= a  <=>  e >= x + log2(m / 7)
        m, x = np.frexp(a[nz])
        e[nz] = np.where(m <= 7.0 / 8.0, x - 3, x - 2)          # 7 * 2^(x-3) = (7/8) 2^x >= m 2^x  iff  m <= 7/8
        e = np.clip(e, -127, 127)
        q = np.rint(blk / np.exp2(e.astype(np.float64))[:, None])
        codes[:, g * block:(g + 1) * block] = np.clip(q, -QMAX4, QMAX4).astype(np.int8)
        exps[:, g] = e
    return codes, exps


def deq_mx(codes, exps, block: int = MX_BLOCK):
    """float64 values q * 2^e of a qmx() result."""
    R, L = codes.shape
    s = np.repeat(np.exp2(exps.astype(np.float64)), block, axis=1)[:, :L]
    return s * codes.astype(np.float64)


def q_weight_main_mx(P):
    """MXINT4 on the residual weight P [K, N]: blocks of 32 along K for each output column n.
    Returns (Wq int8 [K, N], ew int16 [K/32 blocks, N])."""
    c, e = qmx(np.asarray(P, dtype=np.float64).T.copy())
    return c.T.copy(), e.T.copy()


def deq_grp(codes, scales, group: int = GROUP):
    """float64 values s * q of a qgrp() result."""
    R, L = codes.shape
    s = np.repeat(scales.astype(np.float64), group, axis=1)[:, :L]
    return s * codes.astype(np.float64)


def qtok(v, bits: int):
    """Symmetric integer quantizer with ONE fp32 scale per row of a 2-D array.

    a = max|row| in fl32; s = a /fl32 qmax(bits), s = 1 when a == 0;
    q = clamp(rint_even(v /fl32 s), -qmax, qmax).  Returns (codes int8, scales fp32 [R]).
    """
    v = np.asarray(v, dtype=np.float32)
    qm = qmax(bits)
    a = np.max(np.abs(v), axis=1).astype(np.float32) if v.shape[1] else np.zeros(v.shape[0], np.float32)
    s = (a / np.float32(qm)).astype(np.float32)
    s = np.where(a == 0, np.float32(1.0), s).astype(np.float32)
    q = np.rint(v / s[:, None])
    return np.clip(q, -qm, qm).astype(np.int8), s


def deq_tok(codes, scales):
    return scales.astype(np.float64)[:, None] * codes.astype(np.float64)


def q_weight_main(P):
    """Q1 on the residual weight P [K, N]: SINT4 groups along K for each output column n.
    Returns (Wq int8 [K, N], sw fp16 [G, N])."""
    c, s = qgrp(np.asarray(P, dtype=np.float32).T.copy())
    return c.T.copy(), s.T.copy()


def deq_weight_main(Wq, sw):
    return deq_grp(Wq.T.copy(), sw.T.copy()).T.copy()


def q_factor(F, bits):
    """Q2 on a branch factor, one scale per COLUMN (L1: per column j over K; L2: per column n over r).
    bits None = fp16 cast (W16A16).  Returns (codes-or-fp16 array, scales fp32 or None)."""
    if bits is None:
        return np.asarray(F, dtype=np.float32).astype(np.float16), None
    c, s = qtok(np.asarray(F, dtype=np.float32).T.copy(), bits)
    return c.T.copy(), s


def deq_factor(Fq, s):
    if s is None:
        return Fq.astype(np.float64)
    return Fq.astype(np.float64) * s.astype(np.float64)[None, :]


# --------------------------------------------------------------------------------------
# Forward of the decomposed layer (Figure 1; Appendix A.2)
# --------------------------------------------------------------------------------------
def forward(X16, layer, group: int = GROUP):
    """All intermediates and the float64 output of one quantized linear layer.

    layer: dict with Wq int8 [K,N], sw fp16 [G,N], branch (str), rank, and for integer
    branches L1q int8 [K,r], sL1 f32 [r], L2q int8 [r,N], sL2 f32 [N]; for "w16a16"
    L1h fp16 [K,r], L2h fp16 [r,N]; optional bias fp16 [N].
    Steps: (1) qx,sx = SINT4 per token and group; (2) qb,sXb = per-token branch codes;
    (3) I1 = qb L1q exact; (4) t = fl32(fl32(I1) * fl32(sXb * sL1)); (5) tq,sT = per-token;
    (6) P_g = qx_g Wq_g exact; (7) U = tq L2q exact;
    (8) Y = sum_g sx sw P_g + sT sL2 U (+ bias), float64.
    """
    X16 = np.asarray(X16, dtype=np.float16)
    M, K = X16.shape
    Wq, sw = layer["Wq"], layer.get("sw")
    N = Wq.shape[1]
    G = -(-K // group)
    branch, r = layer["branch"], int(layer["rank"])
    out = {}
    Xf = X16.astype(np.float32)

    Y = np.zeros((M, N), dtype=np.float64)
    Wq64 = Wq.astype(np.float64)
    if layer.get("main", "sint4") == "mxint4":
        # MXINT4 main branch: blocks of 32, power-of-two scales 2^ex (activations) and 2^ew (weights)
        qx, ex = qmx(Xf)                                        # (1)
        out["qx"], out["ex"] = qx, ex
        qx64 = qx.astype(np.float64)
        ew = layer["ew"]
        for g in range(-(-K // MX_BLOCK)):                      # (6) + main part of (8)
            k0, k1 = g * MX_BLOCK, min(K, (g + 1) * MX_BLOCK)
            Pg = qx64[:, k0:k1] @ Wq64[k0:k1, :]                # exact integers
            Y += np.exp2(ex[:, g].astype(np.float64))[:, None] * np.exp2(ew[g, :].astype(np.float64))[None, :] * Pg
    else:
        qx, sx = qgrp(Xf, group)                                # (1)
        out["qx"], out["sx"] = qx, sx
        qx64 = qx.astype(np.float64)
        for g in range(G):                                      # (6) + main part of (8)
            k0, k1 = g * group, min(K, (g + 1) * group)
            Pg = qx64[:, k0:k1] @ Wq64[k0:k1, :]                # exact integers
            Y += (sx[:, g].astype(np.float64)[:, None] * sw[g, :].astype(np.float64)[None, :]) * Pg

    if branch != "none" and r > 0:
        if branch == "w16a16":
            # reference branch: fp16 operands, T rounded once to fp16, no scales
            T = (X16.astype(np.float64) @ layer["L1h"].astype(np.float64)).astype(np.float16)
            out["T16"] = T
            Y += T.astype(np.float64) @ layer["L2h"].astype(np.float64)
        else:
            bw, ba = BRANCH_BITS[branch]
            qb, sXb = qtok(Xf, ba)                              # (2)
            I1 = qb.astype(np.float64) @ layer["L1q"].astype(np.float64)   # (3) exact
            sc = (sXb[:, None] * layer["sL1"].astype(np.float32)[None, :]).astype(np.float32)
            t = (I1.astype(np.float32) * sc).astype(np.float32)            # (4)
            tq, sT = qtok(t, ba)                                # (5)
            U = tq.astype(np.float64) @ layer["L2q"].astype(np.float64)    # (7) exact
            Y += (sT.astype(np.float64)[:, None] * layer["sL2"].astype(np.float64)[None, :]) * U
            out.update(qb=qb, sXb=sXb, I1=I1, t=t, tq=tq, sT=sT)
    if layer.get("bias") is not None:
        Y += layer["bias"].astype(np.float64)[None, :]
    out["Y"] = Y
    return out


# --------------------------------------------------------------------------------------
# Data-free calibration (Sections 3.2, 3.3; Appendix A, B.2)
# --------------------------------------------------------------------------------------
def svd_init(W, r: int):
    """Best rank-r approximation M = L0 R0 of W (Eckart-Young), Sigma split evenly."""
    U, s, Vt = np.linalg.svd(np.asarray(W, dtype=np.float64), full_matrices=False)
    rs = np.sqrt(s[:r])
    return U[:, :r] * rs[None, :], rs[:, None] * Vt[:r, :]


def q1_dequant(A, main: str = "sint4"):
    """Q1(A) as real numbers: SINT4 (or MXINT4) along K (axis 0) per output column."""
    if main == "mxint4":
        c, e = q_weight_main_mx(A)
        return deq_mx(c.T.copy(), e.T.copy()).T.copy()
    c, s = q_weight_main(A)
    return deq_weight_main(c, s)


def residual_error(W, L, R, main: str = "sint4"):
    """E = Q1(W + L R) - W - L R  (Eq. "low-rank-optimization")."""
    D = L @ R
    return q1_dequant(W + D, main) - W - D


def objective(W, L, R, main: str = "sint4") -> float:
    """MSE form of the calibration objective: mean over K*N entries of E^2."""
    E = residual_error(W, L, R, main)
    return float(np.mean(E * E))


def gradients(W, L, R, main: str = "sint4"):
    """(loss, dL, dR) with the quantizer's derivative taken as zero (Appendix B.2):
    d/d(LR) = -2 E / (K N),  dL = d(LR) R^T,  dR = L^T d(LR)."""
    E = residual_error(W, L, R, main)
    c = -2.0 / E.size
    return float(np.mean(E * E)), c * (E @ R.T), c * (L.T @ E)


def q2_dequant(F, bits):
    """Q2(F) as real numbers (per-column integer quantizer; bits None = fp16 rounding)."""
    q, s = q_factor(F, bits)
    return deq_factor(q, s)


def rotation_loss(L, R, Om, bits):
    """Loss of the rotation-aware step (Eq. "loss-rotation-aware"), each term a mean of squares:
    mean((Q2(L Om) - L Om)^2) + mean((Q2(Om^T R) - Om^T R)^2).  Returns (loss, E1, E2)."""
    A, B = L @ Om, Om.T @ R
    E1, E2 = q2_dequant(A, bits) - A, q2_dequant(B, bits) - B
    return float(np.mean(E1 * E1) + np.mean(E2 * E2)), E1, E2


def rotation_gradient(L, R, Om, bits):
    """(loss, dLoss/dOm) with Q2's derivative taken as zero, as for Q1 in Appendix B.2:
    d/dOm mean((Q - L Om)^2) = -2 L^T E1 / (K r),  d/dOm mean((Q' - Om^T R)^2) = -2 R E2^T / (r N)."""
    loss, E1, E2 = rotation_loss(L, R, Om, bits)
    G = -2.0 * (L.T @ E1) / E1.size - 2.0 * (R @ E2.T) / E2.size
    return loss, G


def optimize_rotation(L, R, bits, steps: int = 500, lr: float = 0.5):
    """Rotation-aware step of Section 3.3: an orthogonal Om [r, r] that lowers the Q2 error of L Om and Om^T R while
    (L Om)(Om^T R) = L R.  The paper names Cayley SGD as its inspiration and gives the learning rate and the step count;
    the update taken here is the plain Cayley retraction of that method without momentum: with the skew-symmetric
    S = G Om^T - Om G^T,  Om <- (I + lr/2 S)^-1 (I - lr/2 S) Om, which keeps Om orthogonal to rounding.  Starts at the
    identity and returns the best iterate seen, with the trace [steps+1] of the loss."""
    r = L.shape[1]
    Om = np.eye(r)
    I = np.eye(r)
    trace = np.zeros(steps + 1)
    best = (np.inf, Om)
    for t in range(steps + 1):
        loss, G = rotation_gradient(L, R, Om, bits)
        trace[t] = loss
        if loss < best[0]:
            best = (loss, Om.copy())
        if t == steps:
            break
        S = G @ Om.T - Om @ G.T
        Om = np.linalg.solve(I + 0.5 * lr * S, (I - 0.5 * lr * S) @ Om)
    return best[1], trace


def adam_update(x, g, m, v, k: int, lr: float, beta1: float, beta2: float, eps: float):
    """One Adam step (Kingma & Ba, Algorithm 1; Appendix A "Optimization" names the optimiser and the learning rate):
    m <- b1 m + (1-b1) g,  v <- b2 v + (1-b2) g^2,  x <- x - lr (m / (1-b1^k)) / (sqrt(v / (1-b2^k)) + eps), k = 1, 2, ...
    Returns (x, m, v)."""
    m = beta1 * m + (1 - beta1) * g
    v = beta2 * v + (1 - beta2) * g * g
    x = x - lr * (m / (1 - beta1 ** k)) / (np.sqrt(v / (1 - beta2 ** k)) + eps)
    return x, m, v


def calibrate(W16, rank: int, branch: str = "w8a8", steps: int = 1000, lr: float = 1e-4,
              beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8, bias=None, main: str = "sint4",
              rot_steps: int = 0, rot_lr: float = 0.5):
    """Data-free calibration of one weight.  Returns (layer dict, trace [steps+1] of the
    objective at every iterate visited, iterate 0 = the SVD initialisation).  main selects Q1:
    "sint4" (blocks of 64, fp16 scale) or "mxint4" (blocks of 32, power-of-two scale; Table 2).
    rot_steps > 0 adds the rotation-aware step before the factors are quantized (its loss trace is
    stored as layer["rot_trace"])."""
    W = np.asarray(W16, dtype=np.float16).astype(np.float64)
    K, N = W.shape
    layer = {"branch": branch, "rank": int(rank), "K": K, "N": N, "main": main,
             "bias": None if bias is None else np.asarray(bias, dtype=np.float16)}

    def store_main(P):
        if main == "mxint4":
            layer["Wq"], layer["ew"] = q_weight_main_mx(P)
        else:
            layer["Wq"], layer["sw"] = q_weight_main(P)

    if branch == "none" or rank == 0:
        layer["branch"], layer["rank"] = "none", 0
        store_main(W)
        E = q1_dequant(W, main) - W
        return layer, np.array([float(np.mean(E * E))])

    L0, R0 = svd_init(W, rank)
    L, R = -L0, R0
    mL = np.zeros_like(L); vL = np.zeros_like(L)
    mR = np.zeros_like(R); vR = np.zeros_like(R)
    trace = np.zeros(steps + 1)
    best = (np.inf, None, None)
    for t in range(steps + 1):
        loss, gL, gR = gradients(W, L, R, main)
        trace[t] = loss
        if loss < best[0]:
            best = (loss, L.copy(), R.copy())
        if t == steps:
            break
        L, mL, vL = adam_update(L, gL, mL, vL, t + 1, lr, beta1, beta2, eps)
        R, mR, vR = adam_update(R, gR, mR, vR, t + 1, lr, beta1, beta2, eps)

    # Figure 1 sign: W ~ P + L1 L2 with L1 = -L*, L2 = R*
    L1, L2 = -best[1], best[2]
    bw, _ = BRANCH_BITS[branch]
    if rot_steps > 0:                                     # Section 3.3: Q2(L1 Om), Q2(Om^T L2); the product is unchanged
        Om, rot_trace = optimize_rotation(L1, L2, bw, rot_steps, rot_lr)
        L1, L2 = L1 @ Om, Om.T @ L2
        layer["rot_trace"] = rot_trace
    if branch == "w16a16":
        layer["L1h"], _ = q_factor(L1, None)
        layer["L2h"], _ = q_factor(L2, None)
        D = layer["L1h"].astype(np.float64) @ layer["L2h"].astype(np.float64)
    else:
        layer["L1q"], layer["sL1"] = q_factor(L1, bw)
        layer["L2q"], layer["sL2"] = q_factor(L2, bw)
        D = deq_factor(layer["L1q"], layer["sL1"]) @ deq_factor(layer["L2q"], layer["sL2"])
    store_main(W - D)                                     # P = W - Q2(L1) Q2(L2), then Q1
    return layer, trace


def effective_weight(layer):
    """float64 [K, N]: deq(Q1(P)) + deq(Q2(L1)) deq(Q2(L2)) - what the layer multiplies by
    when activations are exact."""
    if layer.get("main", "sint4") == "mxint4":
        Wd = deq_mx(layer["Wq"].T.copy(), layer["ew"].T.copy()).T.copy()
    else:
        Wd = deq_weight_main(layer["Wq"], layer["sw"])
    if layer["branch"] == "none" or layer["rank"] == 0:
        return Wd
    if layer["branch"] == "w16a16":
        return Wd + layer["L1h"].astype(np.float64) @ layer["L2h"].astype(np.float64)
    return Wd + deq_factor(layer["L1q"], layer["sL1"]) @ deq_factor(layer["L2q"], layer["sL2"])
