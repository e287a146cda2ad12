"""Glue used by the GPU parity tests: oracle layer -> library handle, one forward, comparisons."""
import numpy as np

from paper_2604_18117_b200 import binding as B


def import_oracle_layer(layer: dict):
    """Feeds a layer produced by the CPU oracle to lq_layer_import (the direction data flows in
    every parity test: oracle -> library, never the reverse)."""
    cfg = B.lq_config_default(layer["K"], layer["N"], layer["rank"], layer["branch"])
    mx = layer.get("main", "sint4") == "mxint4"
    if mx:
        cfg.group = 32                                     # MXINT4: blocks of 32, power-of-two scales (passed as halves 2^e)
    if layer["branch"] == "w16a16":
        L1, L2, s1, s2 = layer["L1h"], layer["L2h"], None, None
    elif layer["branch"] == "none" or layer["rank"] == 0:
        L1 = L2 = s1 = s2 = None
    else:
        L1, L2, s1, s2 = layer["L1q"], layer["L2q"], layer["sL1"], layer["sL2"]
    sw = np.exp2(layer["ew"].astype(np.float64)).astype(np.float16) if mx else layer["sw"]
    h = B.lq_layer_import(cfg, B.pack_nibbles(layer["Wq"]), sw, L1, s1, L2, s2, layer.get("bias"))
    return h, cfg


def import_oracle_mxfp_layer(layer: dict):
    """An MXFP layer of oracle/lq_oracle_mxfp.py -> library handle: element values become their bit patterns
    (e2m1 nibbles for the residual, e4m3 bytes for the factors), exponents become powers of two."""
    K, N, r = layer["K"], layer["N"], layer["rank"]
    branch = layer["branch"] if r > 0 else "none"
    cfg = B.lq_config_default(K, N, r, branch)
    cfg.group, cfg.main_fmt = 32, B.MAIN_MXFP4
    if layer.get("act", "e4m3") == "e2m3":
        cfg.act_fmt = B.ACT_MXFP6                                         # Table 4: activations in the 6-bit format too
    live = lambda e: np.where(e == -127, 0, e).astype(np.float64)       # an all-zero block: any scale does, its elements are zeros
    sw = np.exp2(live(layer["ew"])).astype(np.float16)
    if r > 0:
        L1, L2 = B.e4m3_encode(layer["L1v"]), B.e4m3_encode(layer["L2v"])
        s1 = np.exp2(live(layer["e1"])).astype(np.float32)
        s2 = np.exp2(live(layer["e2"])).astype(np.float32)
    else:
        L1 = L2 = s1 = s2 = None
    h = B.lq_layer_import(cfg, B.pack_e2m1(layer["Wv"]), sw, L1, s1, L2, s2, layer.get("bias"))
    return h, cfg


def import_oracle_mxint_layer(layer: dict):
    """A layer of oracle/lq_oracle_mxint.py (MXINT4 weights, MXINT8 activations, MX integer factors) -> library handle."""
    K, N, r = layer["K"], layer["N"], layer["rank"]
    branch = layer["branch"] if r > 0 else "none"
    cfg = B.lq_config_default(K, N, r, branch)
    cfg.group, cfg.main_fmt = 32, B.MAIN_MXINT4_A8
    live = lambda e: np.where(e == -127, 0, e).astype(np.float64)       # an all-zero block: any scale does, its codes are zeros
    sw = np.exp2(live(layer["ew"])).astype(np.float16)
    if r > 0:
        L1, L2 = layer["L1q"].astype(np.int8), layer["L2q"].astype(np.int8)
        s1 = np.exp2(live(layer["e1"])).astype(np.float32)
        s2 = np.exp2(live(layer["e2"])).astype(np.float32)
    else:
        L1 = L2 = s1 = s2 = None
    h = B.lq_layer_import(cfg, B.pack_nibbles(layer["Wq"].astype(np.int8)), sw, L1, s1, L2, s2, layer.get("bias"))
    return h, cfg


def gpu_forward(layer: dict, X16: np.ndarray, out_f32: bool = True, export: bool = True, device: int = 0,
                store_qb: bool = True):
    """Runs lq_quantize_act + lq_linear_forward through the C ABI; returns (Y, exported act dict).
    store_qb=True also writes the branch activation codes to HBM so that they can be compared
    (the benchmark configuration leaves them on chip)."""
    import torch
    B.lq_set_option("store_qb", 1 if store_qb else 0)
    h, cfg = (import_oracle_mxfp_layer(layer) if layer.get("main") == "mxfp4" else
              import_oracle_mxint_layer(layer) if layer.get("main") == "mxint4a8" else import_oracle_layer(layer))
    B.lq_layer_to_device(h, device)
    M = X16.shape[0]
    act = B.lq_act_create(h, M, device)
    try:
        Xd = torch.from_numpy(np.ascontiguousarray(X16)).to(f"cuda:{device}")
        Yd = torch.full((M, cfg.N), float("nan"), dtype=torch.float32 if out_f32 else torch.float16,
                        device=f"cuda:{device}")
        st = torch.cuda.current_stream().cuda_stream
        B.lq_quantize_act(h, Xd.data_ptr(), M, act, st)
        B.lq_linear_forward(h, act, Yd.data_ptr(), B.OUT_F32 if out_f32 else B.OUT_F16, st)
        torch.cuda.synchronize()
        code, stage = B.lq_get_device_status(device)
        assert code == 0, f"device status {code} at stage {stage}"
        ex = B.lq_act_export(act, M, cfg, st) if export else None
        return Yd.cpu().numpy(), ex
    finally:
        B.lq_set_option("store_qb", 0)
        B.lq_act_free(act)
        B.lq_layer_free(h)


def rel_fro(Y, Yref) -> float:
    Y = Y.astype(np.float64)
    return float(np.linalg.norm(Y - Yref) / max(np.linalg.norm(Yref), 1e-300))


def elementwise_excess(Y, Yref, out_f32: bool, tol: float = 1e-5) -> float:
    """Largest |Y - Yref| in units of the element-wise bound  tol * (|y| + row scale)  (+ 2^-10 |y| when the output was
    rounded to fp16), row scale = the largest magnitude in the reference row.  The Frobenius figure alone would hide one
    wrong element, a missing bias or a mis-scaled column pair among 10^5 good ones; this does not.  <= 1 passes.
    tol: 1e-5 for integer branches with SINT4 (a length-(G+1) fp32 sum of exact terms), larger where the tensor core
    sums thousands of exact products in its own order (MXINT4) or T is rounded to fp16 on the way (W16A16)."""
    Y = np.asarray(Y, dtype=np.float64)
    Yref = np.asarray(Yref, dtype=np.float64)
    scale = np.abs(Yref).max(axis=1, keepdims=True)
    bound = tol * (np.abs(Yref) + scale) + (0.0 if out_f32 else 2.0 ** -10 * np.abs(Yref) + 2.0 ** -24)
    return float((np.abs(Y - Yref) / np.maximum(bound, 1e-300)).max())


def assert_y_close(Y, Yref, out_f32: bool, tol: float = 1e-5, what: str = "Y"):
    ex = elementwise_excess(Y, Yref, out_f32, tol)
    assert ex <= 1.0, f"{what}: element-wise bound exceeded {ex:.2f}x (tol {tol}, {'fp32' if out_f32 else 'fp16'} output)"


def assert_codes_equal(ex: dict, ref: dict, branch: str, with_qb: bool = True):
    assert np.array_equal(ex["qx"], ref["qx"]), "qx differs"
    if "ex" in ref:                                        # MXINT4: the library exports the block exponents
        assert np.array_equal(ex["sx"], ref["ex"]), "block exponents differ"
    else:
        assert np.array_equal(ex["sx"].view(np.uint16), ref["sx"].view(np.uint16)), "sx differs"
    if branch in ("w8a8", "w6a6", "w4a8"):
        if with_qb:
            assert np.array_equal(ex["qb"], ref["qb"]), "qb differs"
        assert np.array_equal(ex["sXb"].view(np.uint32), ref["sXb"].view(np.uint32)), "sXb differs"
        assert np.array_equal(ex["tq"], ref["tq"]), "tq differs"
        assert np.array_equal(ex["sT"].view(np.uint32), ref["sT"].view(np.uint32)), "sT differs"
