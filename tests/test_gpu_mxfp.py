"""GPU parity of the MXFP path (MXFP4e2 residual weights, MXFP8e4 activations for both branches, MXFP8/6/4 factors;
Section 4.3, Tables 3-4, Appendix A.3) against oracle/lq_oracle_mxfp.py, through the C ABI.

What is unique and compared bit for bit: the activation codes and block exponents.  The rank-r intermediate T is a
real-valued sum that the GPU forms in fp32 (tensor-core partial sums per block of 32, scaled and added in fp32) and
the oracle in fp64, so its MXFP8e4 image may differ where T sits next to a rounding boundary: the codes are required
to agree almost everywhere and never to differ by more than one e4m3 step, and the output is compared (a) with the
oracle's own forward at a tolerance that allows those flips and (b) tightly with the oracle's sums evaluated on the
GPU's own image of T, which pins the block-scaled GEMM and its fused branch stage."""
import numpy as np
import pytest

from oracle import lq_oracle_mxfp as F
from paper_2604_18117_b200 import binding as B
from tests.helpers import assert_y_close, gpu_forward, rel_fro

pytestmark = pytest.mark.gpu


def _layer(rng, K, N, r, branch, bias=True):
    layer = {"main": "mxfp4", "branch": branch if r else "none", "rank": r, "K": K, "N": N,
             "bias": (rng.standard_normal(N) * 0.05).astype(np.float16) if bias else None}
    layer["Wv"], layer["ew"] = F.q_columns(rng.standard_normal((K, N)) * 0.02, "e2m1")
    if r:
        fmt = F.BRANCH_FORMAT[branch]
        layer["L1v"], layer["e1"] = F.q_columns(rng.standard_normal((K, r)) * 0.05, fmt)
        layer["L2v"], layer["e2"] = F.q_columns(rng.standard_normal((r, N)) * 0.05, fmt)
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
                         (t64[:, j0:j1] @ layer["L2v"][j0:j1, :].astype(np.float64)))
    return Y


def _check(layer, X):
    ref = F.forward(X, layer)
    Y32, ex = gpu_forward(layer, X, out_f32=True)
    assert np.isfinite(Y32).all()
    assert np.array_equal(B.e4m3_decode(ex["qx"]), ref["xa"]), "activation elements differ"
    assert np.array_equal(ex["sx"], ref["ex"]), "activation block exponents differ"
    r = layer["rank"]
    if r:
        tq_gpu = B.e4m3_decode(ex["tq"])
        et_gpu = ex["sT"].astype(np.int16)
        t_gpu = F.deq_mxfp(tq_gpu, et_gpu)
        t_ref = F.deq_mxfp(ref["tq"], ref["et"])
        same = (t_gpu == t_ref)
        assert same.mean() >= 0.995, f"only {same.mean():.4f} of the intermediate's codes agree"
        # never more than one e4m3 step (2^-3 of the value's binade; blocks may also differ by one exponent)
        assert (np.abs(t_gpu - t_ref) <= 0.1251 * np.maximum(np.abs(t_ref), np.abs(t_gpu)) + 1e-30).all()
        Yt = _y_from_gpu_t(layer, ref, tq_gpu, et_gpu)
        assert rel_fro(Y32, Yt) <= 2e-5
        assert_y_close(Y32, Yt, True, tol=1e-4)
        assert rel_fro(Y32, ref["Y"]) <= 5e-3
    else:
        assert rel_fro(Y32, ref["Y"]) <= 2e-5
        assert_y_close(Y32, ref["Y"], True, tol=1e-4)
    Y16, _ = gpu_forward(layer, X, out_f32=False, export=False)
    assert rel_fro(Y16, ref["Y"]) <= (5e-3 if r else 1e-3)


@pytest.mark.parametrize("branch,r", [("none", 0), ("mxfp8", 64), ("mxfp6", 86), ("mxfp4", 128), ("mxfp8", 32)])
def test_mxfp_forward_tables_3_and_4_configurations(branch, r):
    """Rank / format pairs of Table 3 (64 x MXFP8e4, 86 x MXFP6e2, 128 x MXFP4e2 at equal memory) on a PixArt-shaped
    layer slice, several row tiles and a ragged tail."""
    rng = np.random.default_rng(10 + r)
    M, K, N = 300, 1152, 384
    X = (rng.standard_normal((M, K))).astype(np.float16)
    X[:, rng.choice(K, 8, replace=False)] *= 20
    _check(_layer(rng, K, N, r, branch), X)


@pytest.mark.parametrize("M,K,N,r,branch", [(1, 32, 8, 0, "none"), (129, 96, 136, 8, "mxfp8"), (257, 8192, 128, 128, "mxfp4"),
                                            (5, 160, 264, 33, "mxfp6"), (1000, 40, 2000, 24, "mxfp8"), (333, 5600, 24, 48, "mxfp8")])
def test_mxfp_edge_shapes(M, K, N, r, branch):
    """One row, K below a block pair, the largest K, ranks that end inside a block, N not a multiple of 128."""
    rng = np.random.default_rng(M + K)
    X = (rng.standard_normal((M, K)) * rng.choice([0.01, 1.0, 30.0])).astype(np.float16)
    _check(_layer(rng, K, N, r, branch, bias=(N % 16 == 0)), X)


def test_mxfp_degenerate_inputs():
    """Zero rows, zero blocks, fp16 subnormals, the largest fp16 values: exponents and elements stay exact."""
    rng = np.random.default_rng(3)
    M, K, N, r = 130, 256, 136, 40
    X = rng.standard_normal((M, K)).astype(np.float16)
    X[0] = 0
    X[1, :64] = 0
    X[2] = np.float16(6.0e-8)
    X[3] = np.float16(65504)
    X[4, ::2] = np.float16(-65504)
    X[5] = (rng.integers(-8, 9, K) * 2.0 ** -20).astype(np.float16)
    _check(_layer(rng, K, N, r, "mxfp8"), X)


@pytest.mark.parametrize("branch,r", [("mxfp6", 64), ("mxfp6", 128), ("none", 0)])
def test_mxfp6_activations_table_4_rows(branch, r):
    """The rank study's unified 6-bit rows (Table 4): MXFP6e2 activations - X for both branches and the rank-r
    intermediate - with MXFP6e2 factors; the activation elements must lie on the e2m3 grid and match the oracle bit for
    bit, the rest as for 8-bit activations."""
    rng = np.random.default_rng(40 + r)
    M, K, N = 300, 1152, 384
    X = (rng.standard_normal((M, K))).astype(np.float16)
    X[:, rng.choice(K, 8, replace=False)] *= 20
    X[5, :64] = 0
    X[6, :32] = [7.5, 7.75, 8.0, 0.0625, 0.1875, -0.3125] + [0.0] * 26       # the clamp, a binade change, subnormal ties
    layer = _layer(rng, K, N, r, branch)
    layer["act"] = "e2m3"
    _check(layer, X)


def test_mxfp_host_entry_point_pipelines_row_chunks():
    """lq_linear_forward_host with an MXFP layer: the row-chunk views of the activation record (element bytes, scale bytes
    in chunks of 128 rows, the intermediate and its scale bytes) must give the same bits as one call over all rows."""
    import torch
    from tests.helpers import import_oracle_mxfp_layer
    rng = np.random.default_rng(9)
    M, K, N, r = 1300, 1152, 392, 64                       # five chunks, the last one ragged; N not a multiple of 128
    X = rng.standard_normal((M, K)).astype(np.float16)
    layer = _layer(rng, K, N, r, "mxfp8")
    ref = F.forward(X, layer)
    h, cfg = import_oracle_mxfp_layer(layer)
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
        assert np.array_equal(B.e4m3_decode(ex["qx"]), ref["xa"]) and np.array_equal(ex["sx"], ref["ex"])
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
