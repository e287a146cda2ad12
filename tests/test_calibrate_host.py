"""lq_calibrate (host-side C++ in the library) checked on the CPU against closed forms and
against the oracle's statement of the same procedure."""
import numpy as np
import pytest

from oracle import lq_oracle as O
from paper_2604_18117_b200 import binding as B
from paper_2604_18117_b200 import build as BUILD
from paper_2604_18117_b200 import inputs as I

BUILD.build()


def _export_as_oracle_layer(h):
    ex = B.lq_layer_export(h)
    layer = {"branch": ex["branch"], "rank": ex["rank"], "K": ex["K"], "N": ex["N"], "bias": None,
             "Wq": B.unpack_nibbles(ex["Wq_packed"]), "sw": ex["sw"]}
    if ex["branch"] == "w16a16":
        layer["L1h"], layer["L2h"] = ex["L1"], ex["L2"]
    elif ex["rank"] > 0:
        layer.update(L1q=ex["L1"], sL1=ex["sL1"], L2q=ex["L2"], sL2=ex["sL2"])
    return layer


def test_svd_init_eckart_young_known_spectrum():
    """steps = 0 with the fp16 branch exports L1 L2 = L0 R0 (rounded to fp16): its distance to W
    must equal the closed-form tail energy of a matrix built with a known spectrum."""
    rng = np.random.default_rng(0)
    K, N, r = 128, 96, 8
    U, _ = np.linalg.qr(rng.standard_normal((K, N)))
    V, _ = np.linalg.qr(rng.standard_normal((N, N)))
    sig = np.concatenate([np.linspace(4.0, 2.0, r), np.linspace(0.5, 0.05, N - r)])
    W = ((U * sig[None, :]) @ V.T).astype(np.float16)
    s_true = np.linalg.svd(W.astype(np.float64), compute_uv=False)
    cfg = B.lq_config_default(K, N, r, "w16a16"); cfg.steps = 0
    h, _ = B.lq_calibrate(cfg, W)
    ex = B.lq_layer_export(h)
    approx = ex["L1"].astype(np.float64) @ ex["L2"].astype(np.float64)
    err2 = np.linalg.norm(W.astype(np.float64) - approx) ** 2
    tail = np.sum(s_true[r:] ** 2)
    assert abs(err2 - tail) <= 2e-3 * tail + 1e-6 * np.sum(s_true ** 2)
    # even split of Sigma: column norms of L1 and row norms of L2 are sqrt(sigma_i)
    assert np.allclose(np.sort(np.linalg.norm(ex["L1"].astype(np.float64), axis=0))[::-1], np.sqrt(s_true[:r]), rtol=2e-3)
    assert np.allclose(np.sort(np.linalg.norm(ex["L2"].astype(np.float64), axis=1))[::-1], np.sqrt(s_true[:r]), rtol=2e-3)
    B.lq_layer_free(h)


def test_objective_trace_and_result():
    W = I.make_weight(0, 0, "pin", 256, 192, 2)
    cfg = B.lq_config_default(256, 192, 8, "w8a8"); cfg.steps = 150
    h, trace = B.lq_calibrate(cfg, W, want_trace=True)
    assert trace.shape == (151,)
    # iterate 0 = SVD initialisation: same objective as the oracle's closed statement of it
    _, tr_o = O.calibrate(W, 8, "w8a8", steps=0)
    assert abs(trace[0] - tr_o[0]) <= 1e-4 * tr_o[0]
    best = np.minimum.accumulate(trace)
    assert best[-1] < 0.98 * trace[0]
    layer = _export_as_oracle_layer(h)
    W64 = W.astype(np.float64)
    err = np.linalg.norm(O.effective_weight(layer) - W64)
    rtn = np.linalg.norm(O.q1_dequant(W64) - W64)
    assert err < rtn
    assert np.abs(layer["Wq"]).max() == 7 and np.abs(layer["L1q"]).max() == 127 and np.abs(layer["L2q"]).max() == 127
    # Figure 1: stored residual codes are Q1 of P = W - Q2(L1) Q2(L2)
    D = O.deq_factor(layer["L1q"], layer["sL1"]) @ O.deq_factor(layer["L2q"], layer["sL2"])
    Wq, sw = O.q_weight_main(W64 - D)
    assert np.mean(Wq == layer["Wq"]) > 0.9999 and np.mean(sw == layer["sw"]) > 0.999
    B.lq_layer_free(h)


def test_rank0_and_round_trip_of_import_export():
    rng = np.random.default_rng(1)
    Wq = rng.integers(-7, 8, size=(128, 16)); Wq[0] = 7; Wq[64] = -7
    W = (Wq * 0.03125).astype(np.float16)
    cfg = B.lq_config_default(128, 16, 0, "none"); cfg.steps = 0
    h, trace = B.lq_calibrate(cfg, W, want_trace=True)
    ex = B.lq_layer_export(h)
    assert trace[0] == 0.0 and np.array_equal(B.unpack_nibbles(ex["Wq_packed"]), Wq)
    assert np.all(ex["sw"] == np.float16(0.03125))
    B.lq_layer_free(h)
    lay, _ = O.calibrate(I.make_weight(0, 0, "rt", 128, 64, 1), 4, "w6a6", steps=2,
                         bias=(rng.standard_normal(64) * 0.1).astype(np.float16))
    c2 = B.lq_config_default(128, 64, 4, "w6a6")
    h2 = B.lq_layer_import(c2, B.pack_nibbles(lay["Wq"]), lay["sw"], lay["L1q"], lay["sL1"], lay["L2q"], lay["sL2"], lay["bias"])
    ex2 = B.lq_layer_export(h2)
    assert np.array_equal(B.unpack_nibbles(ex2["Wq_packed"]), lay["Wq"]) and np.array_equal(ex2["sw"], lay["sw"])
    assert np.array_equal(ex2["L1"], lay["L1q"]) and np.array_equal(ex2["L2"], lay["L2q"])
    assert np.array_equal(ex2["sL1"], lay["sL1"]) and np.array_equal(ex2["sL2"], lay["sL2"])
    assert np.array_equal(ex2["bias"], lay["bias"])
    B.lq_layer_free(h2)
    # codes outside the branch's range are rejected
    bad = lay["L1q"].copy(); bad[0, 0] = 100
    try:
        B.lq_layer_import(c2, B.pack_nibbles(lay["Wq"]), lay["sw"], bad, lay["sL1"], lay["L2q"], lay["sL2"], None)
        assert False
    except B.LqError as e:
        assert e.code == 1


def test_mxint4_main_calibration():
    """group = 32 selects the MXINT4 main branch (Table 2): exported scales are powers of two,
    the objective goes down, and the stored codes are MXINT4 of P = W - Q2(L1) Q2(L2)."""
    W = I.make_weight(0, 0, "pin-mx", 256, 192, 2)
    cfg = B.lq_config_default(256, 192, 8, "w8a8"); cfg.steps = 100; cfg.group = 32
    h, trace = B.lq_calibrate(cfg, W, want_trace=True)
    _, tr_o = O.calibrate(W, 8, "w8a8", steps=0, main="mxint4")
    assert abs(trace[0] - tr_o[0]) <= 1e-4 * tr_o[0]
    assert np.minimum.accumulate(trace)[-1] < 0.98 * trace[0]
    ex = B.lq_layer_export(h)
    sw = ex["sw"].astype(np.float64)
    assert sw.shape == (256 // 32, 192)
    ew = np.log2(sw)
    assert np.array_equal(ew, np.rint(ew))
    Wq = B.unpack_nibbles(ex["Wq_packed"])
    D = O.deq_factor(ex["L1"], ex["sL1"]) @ O.deq_factor(ex["L2"], ex["sL2"])
    Wq_o, ew_o = O.q_weight_main_mx(W.astype(np.float64) - D)
    assert np.mean(ew_o == ew) > 0.999 and np.mean(Wq_o == Wq) > 0.9999
    # the calibrated layer beats plain MXINT4 rounding of W
    layer = {"branch": "w8a8", "rank": 8, "K": 256, "N": 192, "bias": None, "main": "mxint4",
             "Wq": Wq, "ew": ew.astype(np.int16), "L1q": ex["L1"], "sL1": ex["sL1"], "L2q": ex["L2"], "sL2": ex["sL2"]}
    W64 = W.astype(np.float64)
    assert np.linalg.norm(O.effective_weight(layer) - W64) < np.linalg.norm(O.q1_dequant(W64, "mxint4") - W64)
    B.lq_layer_free(h)


def test_rotation_aware_step_on_the_host():
    """cfg.rot_steps > 0 (Section 3.3): the rotated factors multiply to the same product, so the layer still
    approximates W; the factors' quantization error - measured as the distance of Q2(L1) Q2(L2) to the fp16-branch product of
    the same seed, which is almost unquantized - goes down; the residual codes are still Q1 of W - Q2(L1) Q2(L2)."""
    W = I.make_weight(0, 0, "rot-host", 256, 192, 2)
    W64 = W.astype(np.float64)

    def run(branch, rot):
        cfg = B.lq_config_default(256, 192, 16, branch); cfg.steps = 3; cfg.rot_steps = rot; cfg.rot_lr = 0.5
        h, _ = B.lq_calibrate(cfg, W)
        ex = B.lq_layer_export(h)
        B.lq_layer_free(h)
        return ex

    ref = run("w16a16", 0)
    D_ref = ref["L1"].astype(np.float64) @ ref["L2"].astype(np.float64)
    ex0, ex1 = run("w4a8", 0), run("w4a8", 60)
    D0 = O.deq_factor(ex0["L1"], ex0["sL1"]) @ O.deq_factor(ex0["L2"], ex0["sL2"])
    D1 = O.deq_factor(ex1["L1"], ex1["sL1"]) @ O.deq_factor(ex1["L2"], ex1["sL2"])
    e0, e1 = np.linalg.norm(D0 - D_ref), np.linalg.norm(D1 - D_ref)
    assert e1 < e0, (e0, e1)
    assert not np.array_equal(ex0["L1"], ex1["L1"])                      # the factors really were rotated
    Wq, sw = O.q_weight_main(W64 - D1)
    assert np.mean(Wq == B.unpack_nibbles(ex1["Wq_packed"])) > 0.9999 and np.mean(sw == ex1["sw"]) > 0.999
    # same loss at the identity and a comparable gain as the oracle's statement of the step (trajectories are not bit-equal)
    L1 = ref["L1"].astype(np.float64); L2 = ref["L2"].astype(np.float64)
    _, tr = O.optimize_rotation(L1, L2, 4, steps=60, lr=0.5)
    loss_host_0 = np.mean((O.q2_dequant(L1, 4) - L1) ** 2) + np.mean((O.q2_dequant(L2, 4) - L2) ** 2)
    assert abs(loss_host_0 - tr[0]) <= 1e-12 * tr[0] and tr.min() < tr[0]


def test_first_adam_steps_match_the_oracle_trajectory():
    """Two Adam steps on a small weight with well separated singular values.  The SVD start is then unique up to the
    sign of each factor pair, a sign flip of (L_i, R_i) flips both gradients and leaves the product and the objective
    unchanged, and two steps are far from the chaotic regime: the library's objective trace must follow the oracle's
    (whose Adam step is pinned to its closed form in test_oracle_pins_branch_and_adam.py).  A library step without bias
    correction, with swapped betas or with eps under the root lands on a different point and fails this."""
    rng = np.random.default_rng(11)
    K, N, r = 64, 32, 3
    U, _ = np.linalg.qr(rng.standard_normal((K, N)))
    V, _ = np.linalg.qr(rng.standard_normal((N, N)))
    sig = np.concatenate([[0.9, 0.6, 0.35], np.linspace(0.05, 0.01, N - 3)])
    W = ((U * sig[None, :]) @ V.T).astype(np.float16)
    for main, group in (("sint4", 64), ("mxint4", 32)):
        cfg = B.lq_config_default(K, N, r, "w8a8")
        cfg.steps, cfg.group = 2, group
        h, trace = B.lq_calibrate(cfg, W, want_trace=True)
        _, tr_o = O.calibrate(W, r, "w8a8", steps=2, main=main)
        assert np.allclose(trace, tr_o, rtol=1e-7, atol=0), (main, trace, tr_o)
        assert abs(tr_o[1] - tr_o[0]) > 1e-4 * tr_o[0]     # the step is visible in the objective
        B.lq_layer_free(h)


def _export_mxfp_as_oracle_layer(h):
    from oracle import lq_oracle_mxfp as F
    cfg = B.lq_layer_info(h)
    ex = B.lq_layer_export(h)
    K, N, r = cfg.K, cfg.N, cfg.rank
    lo, hi = ex["Wq_packed"] & 0xF, ex["Wq_packed"] >> 4
    grid = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6, -0.0, -0.5, -1, -1.5, -2, -3, -4, -6], dtype=np.float32)
    Wv = np.empty((K, N), np.float32); Wv[:, 0::2] = grid[lo]; Wv[:, 1::2] = grid[hi]
    layer = {"main": "mxfp4", "branch": B.BRANCH_NAME[cfg.branch], "rank": r, "K": K, "N": N, "bias": None,
             "Wv": Wv, "ew": np.log2(ex["sw"].astype(np.float64)).astype(np.int16)}
    if r > 0:
        layer.update(L1v=B.e4m3_decode(ex["L1"]), e1=np.log2(ex["sL1"].astype(np.float64)).astype(np.int16),
                     L2v=B.e4m3_decode(ex["L2"]), e2=np.log2(ex["sL2"].astype(np.float64)).astype(np.int16))
    return layer


def test_mxfp_calibration_follows_the_oracle():
    """lq_calibrate with the MXFP4 residual and an MXFP8 / MXFP6 / MXFP4 branch: the first Adam steps follow the MXFP
    oracle's objective trace (same argument as for the integer formats: well separated singular values, two steps), the
    stored factors are on their format's grid, and the stored residual is Q1 of W - Q2(L1) Q2(L2) (Figure 1)."""
    from oracle import lq_oracle_mxfp as F
    rng = np.random.default_rng(12)
    K, N, r = 96, 32, 3
    U, _ = np.linalg.qr(rng.standard_normal((K, N)))
    V, _ = np.linalg.qr(rng.standard_normal((N, N)))
    sig = np.concatenate([[0.9, 0.6, 0.35], np.linspace(0.05, 0.01, N - 3)])
    W = ((U * sig[None, :]) @ V.T).astype(np.float16)
    for branch in ("mxfp8", "mxfp6", "mxfp4"):
        cfg = B.lq_config_default(K, N, r, branch)
        assert cfg.main_fmt == B.MAIN_MXFP4 and cfg.group == 32 and abs(cfg.lr - 1e-3) < 1e-9   # FP formats: 1e-3 (Appendix A.2)
        cfg.steps = 2
        h, trace = B.lq_calibrate(cfg, W, want_trace=True)
        _, tr_o = F.calibrate(W, r, branch, steps=2)
        assert np.allclose(trace, tr_o, rtol=1e-7, atol=0), (branch, trace, tr_o)
        layer = _export_mxfp_as_oracle_layer(h)
        fmt = F.BRANCH_FORMAT[branch]
        grid = F.element_values(fmt).astype(np.float32)
        assert np.isin(np.abs(layer["L1v"]), grid).all() and np.isin(np.abs(layer["L2v"]), grid).all()
        D = F.deq_columns(layer["L1v"], layer["e1"]) @ F.deq_columns(layer["L2v"], layer["e2"])
        Wv, ew = F.q_columns(W.astype(np.float64) - D, "e2m1")
        assert np.array_equal(F.deq_columns(Wv, ew), F.deq_columns(layer["Wv"], layer["ew"]))
        B.lq_layer_free(h)
    cfg = B.lq_config_default(K, N, 0, "none")
    cfg.group, cfg.main_fmt = 32, B.MAIN_MXFP4
    h, _ = B.lq_calibrate(cfg, W)
    layer = _export_mxfp_as_oracle_layer(h)
    assert np.array_equal(F.deq_columns(layer["Wv"], layer["ew"]), F.q1_dequant(W.astype(np.float64)))
    B.lq_layer_free(h)


def test_mxint8_activation_layers_calibration_follows_the_oracle():
    """lq_calibrate for MXINT4 weights with MXINT8 activations and an MXINT8 / MXINT4 branch (Table 3's integer rows):
    the first Adam steps follow the oracle's objective trace, the stored factors are within their format's range and
    on its grid, and the stored residual is Q1 of W - Q2(L1) Q2(L2)."""
    from oracle import lq_oracle_mxint as OI
    rng = np.random.default_rng(13)
    K, N, r = 96, 32, 3
    U, _ = np.linalg.qr(rng.standard_normal((K, N)))
    V, _ = np.linalg.qr(rng.standard_normal((N, N)))
    sig = np.concatenate([[0.9, 0.6, 0.35], np.linspace(0.05, 0.01, N - 3)])
    W = ((U * sig[None, :]) @ V.T).astype(np.float16)
    for branch in ("mxint8", "mxint4"):
        cfg = B.lq_config_default(K, N, r, branch)
        assert cfg.main_fmt == B.MAIN_MXINT4_A8 and cfg.group == 32 and abs(cfg.lr - 1e-4) < 1e-9   # integer formats: 1e-4
        cfg.steps = 2
        h, trace = B.lq_calibrate(cfg, W, want_trace=True)
        _, tr_o = OI.calibrate(W, r, branch, steps=2)
        assert np.allclose(trace, tr_o, rtol=1e-7, atol=0), (branch, trace, tr_o)
        ex = B.lq_layer_export(h)
        qm = 127 if branch == "mxint8" else 7
        assert np.abs(ex["L1"]).max() <= qm and np.abs(ex["L2"]).max() <= qm
        assert np.abs(ex["L1"]).max() > qm // 2                                  # the range is used: minimal exponents
        e1 = np.log2(ex["sL1"].astype(np.float64)).astype(np.int16)
        e2 = np.log2(ex["sL2"].astype(np.float64)).astype(np.int16)
        L1d, L2d = OI.deq_columns(ex["L1"], e1), OI.deq_columns(ex["L2"], e2)
        # idempotence pins the stored pair (codes, exponent): re-quantizing the dequantized factors changes nothing
        assert np.array_equal(OI.deq_columns(*OI.q_columns(L1d, OI.FACTOR_BITS[branch])), L1d)
        Wq = B.unpack_nibbles(ex["Wq_packed"])
        ew = np.log2(ex["sw"].astype(np.float64)).astype(np.int16)
        q, e = OI.q_columns(W.astype(np.float64) - L1d @ L2d, 4)
        assert np.array_equal(OI.deq_columns(q, e), OI.deq_columns(Wq, ew))
        B.lq_layer_free(h)
    # unsupported combinations are refused before any work
    cfg = B.lq_config_default(K, N, 96, "mxint8")
    cfg.steps = 0
    with pytest.raises(B.LqError):
        B.lq_calibrate(cfg, W)


def test_activation_format_option_is_checked():
    """MXFP6e2 activations (Table 4's 6-bit rows) exist for MXFP layers only; anything else is refused up front."""
    rng = np.random.default_rng(1)
    W = (rng.standard_normal((64, 32)) * 0.02).astype(np.float16)
    cfg = B.lq_config_default(64, 32, 4, "mxfp6")
    cfg.steps, cfg.act_fmt = 1, B.ACT_MXFP6
    h, _ = B.lq_calibrate(cfg, W)
    assert B.lq_layer_info(h).act_fmt == B.ACT_MXFP6
    B.lq_layer_free(h)
    for branch in ("w8a8", "mxint8"):
        cfg = B.lq_config_default(64, 32, 4, branch)
        cfg.steps, cfg.act_fmt = 1, B.ACT_MXFP6
        with pytest.raises(B.LqError):
            B.lq_calibrate(cfg, W)
