"""GPU parity of the integer MX path with 8-bit activations (MXINT4 residual weights, MXINT8 activations for both
branches, MXINT8 / MXINT4 factors; Section 4.3, Table 3's integer rows, Appendix A.3) against oracle/lq_oracle_mxint.py,
through the C ABI.

Unique and compared bit for bit: the activation codes and block exponents.  The rank-r intermediate T is a real-valued
sum that the GPU forms in fp32 (exact integer partial sums per block of 32, scaled and added in fp32) and the oracle in
fp64, so its MXINT8 image may differ by one code where T sits next to a rounding boundary (and a block's exponent by
one where its maximum sits next to 127 * 2^e): the codes are required to agree almost everywhere and never to differ
by more than one step, and the output is compared (a) with the oracle's own forward at a tolerance that allows those
flips and (b) tightly with the oracle's sums evaluated on the GPU's own image of T, which pins the block-scaled GEMM
with its digit planes and its fused branch stage."""
import numpy as np
import pytest

from oracle import lq_oracle_mxint as I
from tests.helpers import assert_y_close, gpu_forward, rel_fro

pytestmark = pytest.mark.gpu


def _layer(rng, K, N, r, branch, bias=True):
    layer = {"main": "mxint4a8", "branch": branch if r else "none", "rank": r, "K": K, "N": N,
             "bias": (rng.standard_normal(N) * 0.05).astype(np.float16) if bias else None}
    layer["Wq"], layer["ew"] = I.q_columns(rng.standard_normal((K, N)) * 0.02, 4)
    if r:
        bits = I.FACTOR_BITS[branch]
        layer["L1q"], layer["e1"] = I.q_columns(rng.standard_normal((K, r)) * 0.05, bits)
        layer["L2q"], layer["e2"] = I.q_columns(rng.standard_normal((r, N)) * 0.05, bits)
    return layer


def _y_from_gpu_t(layer, ref, tq_gpu, et_gpu):
    """The oracle's output with the GPU's image of T in place of its own."""
    Y = ref["Y"].copy()
    r = layer["rank"]
    for tq, et, sign in ((ref["tq"], ref["et"], -1.0), (tq_gpu, et_gpu, 1.0)):
        t64 = tq.astype(np.float64)
        for c in range(-(-r // 32)):
            j0, j1 = c * 32, min(r, (c + 1) * 32)
            Y += sign * (np.exp2(et[:, c].astype(np.float64))[:, None] * np.exp2(layer["e2"][c, :].astype(np.float64))[None, :] *
                         (t64[:, j0:j1] @ layer["L2q"][j0:j1, :].astype(np.float64)))
    return Y


def _check(layer, X):
    ref = I.forward(X, layer)
    Y32, ex = gpu_forward(layer, X, out_f32=True)
    assert np.isfinite(Y32).all()
    assert np.array_equal(ex["qx"].astype(np.int16), ref["xa"]), "activation codes differ"
    assert np.array_equal(ex["sx"], ref["ex"]), "activation block exponents differ"
    r = layer["rank"]
    if r:
        tq_gpu = ex["tq"].astype(np.int16)
        et_gpu = ex["sT"].astype(np.int16)
        t_gpu = I.deq_mxint(tq_gpu, et_gpu)
        t_ref = I.deq_mxint(ref["tq"], ref["et"])
        same = (t_gpu == t_ref)
        assert same.mean() >= 0.995, f"only {same.mean():.4f} of the intermediate's codes agree"
        step = np.repeat(np.exp2(np.maximum(et_gpu, ref["et"]).astype(np.float64)), 32, axis=1)[:, :r]
        assert (np.abs(t_gpu - t_ref) <= step).all()              # never more than one code step of the coarser exponent
        Yt = _y_from_gpu_t(layer, ref, tq_gpu, et_gpu)
        assert rel_fro(Y32, Yt) <= 2e-5
        assert_y_close(Y32, Yt, True, tol=1e-4)
        assert rel_fro(Y32, ref["Y"]) <= 5e-3
    else:
        assert rel_fro(Y32, ref["Y"]) <= 2e-5
        assert_y_close(Y32, ref["Y"], True, tol=1e-4)
    Y16, _ = gpu_forward(layer, X, out_f32=False, export=False)
    assert rel_fro(Y16, ref["Y"]) <= (5e-3 if r else 1e-3)


@pytest.mark.parametrize("branch,r", [("none", 0), ("mxint8", 64), ("mxint4", 64), ("mxint8", 32), ("mxint8", 40),
                                      ("mxint4", 128), ("mxint4", 96), ("mxint4", 24)])
def test_mxint8_forward_table_3_integer_rows(branch, r):
    """MXINT4 weights x MXINT8 activations with MXINT8 factors of rank 64 or MXINT4 factors of rank 128 (Table 3's two
    integer rows) and neighbours, on a PixArt-shaped layer slice, several row tiles and a ragged tail."""
    rng = np.random.default_rng(20 + r)
    M, K, N = 300, 1152, 384
    X = (rng.standard_normal((M, K))).astype(np.float16)
    X[:, rng.choice(K, 8, replace=False)] *= 20
    _check(_layer(rng, K, N, r, branch), X)


def test_mxint8_ragged_shapes_and_edge_values():
    """K and N that are not multiples of the tiles, one row, zero rows / zero blocks, values at the fp16 extremes,
    block maxima exactly on and just above 127 * 2^e."""
    rng = np.random.default_rng(5)
    K, N, r = 200, 136, 24
    layer = _layer(rng, K, N, r, "mxint8")
    X = (rng.standard_normal((37, K)) * 3).astype(np.float16)
    X[3, :] = 0
    X[5, 32:64] = 0
    X[7, 0] = 65504; X[7, 1] = -65504
    X[9, :32] = 0; X[9, 0] = 127.0; X[9, 1] = 0.5; X[9, 2] = 1.5; X[9, 3] = -2.5         # ties at exponent 0
    X[10, :32] = 0; X[10, 0] = 127.5; X[10, 1] = 1.0; X[10, 2] = 3.0                       # just above: exponent 1, ties
    X[11, :] = 6e-8                                                                        # fp16 subnormals
    _check(layer, X)
    _check(layer, X[:1])


def test_mxint8_full_size_layer_sampled_rows():
    """The qkv shape of the PixArt block at M = 8192 in the launch configuration the benchmark times; sampled rows
    against the oracle."""
    import torch
    from paper_2604_18117_b200 import binding as B
    from tests.helpers import import_oracle_mxint_layer
    rng = np.random.default_rng(77)
    M, K, N, r = 8192, 1152, 3456, 64
    layer = _layer(rng, K, N, r, "mxint8")
    X = rng.standard_normal((M, K)).astype(np.float16)
    X[:, rng.choice(K, 8, replace=False)] *= 20
    h, cfg = import_oracle_mxint_layer(layer)
    B.lq_set_option("store_qb", 0)
    B.lq_layer_to_device(h, 0)
    act = B.lq_act_create(h, M, 0)
    try:
        Xd = torch.from_numpy(X).cuda()
        Yd = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
        st = torch.cuda.current_stream().cuda_stream
        B.lq_quantize_act(h, Xd.data_ptr(), M, act, st)
        B.lq_linear_forward(h, act, Yd.data_ptr(), B.OUT_F16, st)
        torch.cuda.synchronize()
        assert B.lq_get_device_status(0)[0] == 0
        rows = np.sort(rng.choice(M, 96, replace=False))
        rows[0], rows[-1] = 0, M - 1
        ref = I.forward(X[rows], layer)
        Y = Yd.cpu().numpy()[rows].astype(np.float64)
        assert np.isfinite(Y).all()
        assert rel_fro(Y, ref["Y"]) <= 5e-3
    finally:
        B.lq_act_free(act)
        B.lq_layer_free(h)


@pytest.mark.parametrize("branch,r", [("mxint8", 64), ("mxint4", 128)])
def test_mxint8_host_entry_point_pipelines_row_chunks(branch, r):
    """lq_linear_forward_host with 8-bit activation codes: the row-chunk views of the activation record (two code planes
    per row, scale bytes per plane, the intermediate's one or two containers) must give the same bits as one call over
    all rows, and the exported codes of all chunks must match the oracle."""
    import torch
    from paper_2604_18117_b200 import binding as B
    from tests.helpers import import_oracle_mxint_layer
    rng = np.random.default_rng(8)
    M, K, N = 1300, 1152, 392                              # five chunks, the last one ragged; N not a multiple of 128
    X = rng.standard_normal((M, K)).astype(np.float16)
    layer = _layer(rng, K, N, r, branch)
    ref = I.forward(X, layer)
    h, cfg = import_oracle_mxint_layer(layer)
    B.lq_layer_to_device(h, 0)
    act = B.lq_act_create(h, M, 0)
    try:
        st = torch.cuda.current_stream().cuda_stream
        Xp = torch.from_numpy(X).pin_memory()
        Yp = torch.full((M, N), float("nan"), dtype=torch.float16).pin_memory()
        B.lq_linear_forward_host(h, act, Xp.data_ptr(), M, Yp.data_ptr(), B.OUT_F16, st)
        assert B.lq_get_device_status(0)[0] == 0
        Yh = Yp.numpy().copy()
        ex = B.lq_act_export(act, M, cfg, st)
        assert np.array_equal(ex["qx"].astype(np.int16), ref["xa"]) and np.array_equal(ex["sx"], ref["ex"])
        Xd = torch.from_numpy(X).cuda()
        Yd = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
        B.lq_quantize_act(h, Xd.data_ptr(), M, act, st)
        B.lq_linear_forward(h, act, Yd.data_ptr(), B.OUT_F16, st)
        torch.cuda.synchronize()
        ex2 = B.lq_act_export(act, M, cfg, st)
        assert np.array_equal(ex["tq"], ex2["tq"]) and np.array_equal(ex["sT"], ex2["sT"])
        assert np.array_equal(Yh, Yd.cpu().numpy())
        assert rel_fro(Yh, ref["Y"]) <= 5e-3
    finally:
        B.lq_act_free(act)
        B.lq_layer_free(h)


@pytest.mark.parametrize("M,K,N,r,branch", [(1, 32, 8, 0, "none"), (129, 96, 136, 8, "mxint8"), (257, 8192, 128, 128, "mxint4"),
                                            (5, 160, 264, 33, "mxint8"), (1000, 40, 2000, 24, "mxint4"), (333, 5600, 24, 48, "mxint8")])
def test_mxint8_edge_shapes(M, K, N, r, branch):
    """One row, K below a block pair, the largest K and rank, ranks that end inside a block, N not a multiple of 128,
    values from tiny to large."""
    rng = np.random.default_rng(M + K)
    X = (rng.standard_normal((M, K)) * rng.choice([0.01, 1.0, 30.0])).astype(np.float16)
    _check(_layer(rng, K, N, r, branch, bias=(N % 16 == 0)), X)
