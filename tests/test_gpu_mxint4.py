"""GPU parity of the MXINT4 main branch (Appendix A.3: blocks of 32 values, power-of-two E8M0 scales; the
residual-branch format of Table 2): codes and block exponents bit for bit against the oracle, Y within a relative
Frobenius error of 1e-3 (fp16 output) / 2e-5 (fp32 output: the tensor core sums the block-scaled products in fp32)."""
import numpy as np
import pytest

from oracle import lq_oracle as O
from paper_2604_18117_b200 import inputs as I
from tests.helpers import assert_codes_equal, assert_y_close, gpu_forward, rel_fro

pytestmark = pytest.mark.gpu

TOL_F16 = 1e-3
TOL_F32 = 2e-5


def _mx_layer(rng, K, N, r, branch, wscale=0.02, bias=True):
    layer = {"main": "mxint4", "branch": branch if r > 0 else "none", "rank": r, "K": K, "N": N,
             "bias": (rng.standard_normal(N) * 0.05).astype(np.float16) if bias else None}
    W = rng.standard_normal((K, N)) * wscale
    W[:: max(1, K // 7), :] *= 10                                       # outlier input channels: exponents vary per block
    layer["Wq"], layer["ew"] = O.q_weight_main_mx(W)
    if r > 0 and branch == "w16a16":
        layer["L1h"], _ = O.q_factor(rng.standard_normal((K, r)) * 0.05, None)
        layer["L2h"], _ = O.q_factor(rng.standard_normal((r, N)) * 0.05, None)
    elif r > 0:
        bw, _ = O.BRANCH_BITS[branch]
        layer["L1q"], layer["sL1"] = O.q_factor(rng.standard_normal((K, r)) * 0.05, bw)
        layer["L2q"], layer["sL2"] = O.q_factor(rng.standard_normal((r, N)) * 0.05, bw)
    return layer


def _check(layer, X):
    ref = O.forward(X, layer)
    Y32, ex = gpu_forward(layer, X, out_f32=True)
    assert np.isfinite(Y32).all()
    assert_codes_equal(ex, ref, layer["branch"])
    e32 = rel_fro(Y32, ref["Y"])
    assert e32 <= TOL_F32, f"fp32 output error {e32}"
    etol = 1e-3 if layer["branch"] == "w16a16" else 5 * TOL_F32   # the tensor core sums up to K exact products in its own order
    assert_y_close(Y32, ref["Y"], True, tol=etol)
    Y16, _ = gpu_forward(layer, X, out_f32=False, export=False)
    e16 = rel_fro(Y16, ref["Y"])
    assert e16 <= TOL_F16, f"fp16 output error {e16}"
    assert_y_close(Y16, ref["Y"], False, tol=etol)
    return e32, e16


def test_mx_integer_exact_product_with_varied_exponents():
    """Integer codes times per-block powers of two on both sides: every product is exact, so Y must equal the oracle's
    fp64 sum to fp32 rounding - and a wrong scale byte, block id or row/column mapping changes Y by a factor of two or more."""
    rng = np.random.default_rng(0)
    M, K, N = 256, 512, 384
    ea = rng.integers(-3, 4, size=(M, K // 32)); eb = rng.integers(-5, 2, size=(K // 32, N))
    Xi = rng.integers(-7, 8, size=(M, K)); Xi[:, ::32] = 7
    Wi = rng.integers(-7, 8, size=(K, N)); Wi[::32, :] = 7
    X = (Xi * np.exp2(np.repeat(ea, 32, axis=1))).astype(np.float16)
    W = Wi * np.exp2(np.repeat(eb, 32, axis=0))
    layer = {"main": "mxint4", "branch": "none", "rank": 0, "K": K, "N": N, "bias": None}
    layer["Wq"], layer["ew"] = O.q_weight_main_mx(W)
    assert np.array_equal(layer["Wq"], Wi) and np.array_equal(layer["ew"], eb)
    ref = O.forward(X, layer)
    assert np.array_equal(ref["qx"], Xi) and np.array_equal(ref["ex"], ea)
    Y, ex = gpu_forward(layer, X, out_f32=True)
    assert_codes_equal(ex, ref, "none")
    assert rel_fro(Y, ref["Y"]) <= 1e-6
    assert np.abs(Y - ref["Y"]).max() <= 1e-5 * np.abs(ref["Y"]).max()


@pytest.mark.parametrize("branch", ["none", "w8a8", "w6a6", "w4a8", "w16a16"])
def test_mx_small_shapes_all_branches(branch):
    rng = np.random.default_rng(1)
    M, K, N, r = 200, 328, 200, 0 if branch == "none" else 32          # ragged M, N; K = 10.25 blocks
    X = rng.standard_normal((M, K)).astype(np.float16)
    X[:, 7] *= 20
    X[3, :] = 0; X[4, :64] = 0; X[5, :] = np.float16(2.0 ** -24)
    _check(_mx_layer(rng, K, N, r, branch), X)


def test_mx_wide_and_narrow_tiles_long_k():
    rng = np.random.default_rng(2)
    M, K, N, r = 300, 4608, 392, 64
    X = rng.standard_normal((M, K)).astype(np.float16)
    X[:, rng.integers(0, K, 8)] *= 20
    _check(_mx_layer(rng, K, N, r, "w8a8"), X)


def test_mx_sana_shape_sampled_rows():
    """K = 5600, N = 2240 at M = 8192 with the seeded benchmark activations; 160 sampled rows against the oracle."""
    rng = np.random.default_rng(3)
    wl = I.workload(3)
    spec = I.SANA_LAYERS[3]
    X, _, _ = I.layer_inputs(wl, spec, M=8192)
    layer = _mx_layer(rng, spec.K, spec.N, 32, "w4a8")
    rows = np.unique(np.concatenate([[0, 127, 128, 8191], rng.choice(8192, 156, replace=False)]))
    ref = O.forward(X[rows], layer)
    Y, ex = gpu_forward(layer, X, out_f32=False)
    assert np.array_equal(ex["qx"][rows], ref["qx"])
    assert np.array_equal(ex["sx"][rows], ref["ex"])
    assert np.array_equal(ex["tq"][rows], ref["tq"])
    assert np.isfinite(Y.astype(np.float32)).all()
    assert rel_fro(Y[rows], ref["Y"]) <= TOL_F16


@pytest.mark.parametrize("spec", I.PIXART_LAYERS, ids=lambda s: s.name)
def test_mx_config1_pixart_block_linears(spec):
    """The benchmark's launch configuration (M = 8192, r = 32, W8A8 branch) with the MXINT4 main branch: the seeded
    config-1 activations, 160 sampled rows against the oracle.  qkv and fc1 share the work by tiles, attn-out and fc2
    (nine 128-column units per row block, few tiles per CTA) by units."""
    rng = np.random.default_rng(4)
    wl = I.workload(1)
    X, _, _ = I.layer_inputs(wl, spec, M=8192)
    layer = _mx_layer(rng, spec.K, spec.N, 32, "w8a8")
    rows = np.unique(np.concatenate([[0, 1, 127, 128, 8063, 8064, 8190, 8191], rng.choice(8192, 152, replace=False)]))
    ref = O.forward(X[rows], layer)
    Y, ex = gpu_forward(layer, X, out_f32=False)
    assert np.array_equal(ex["qx"][rows], ref["qx"])
    assert np.array_equal(ex["sx"][rows], ref["ex"])
    assert np.array_equal(ex["tq"][rows], ref["tq"])
    assert np.isfinite(Y.astype(np.float32)).all()
    assert (np.abs(Y.astype(np.float32)).sum(axis=1) > 0).all()
    assert rel_fro(Y[rows], ref["Y"]) <= TOL_F16


@pytest.mark.parametrize("r,branch", [(128, "w8a8"), (16, "w6a6"), (0, "none"), (64, "w16a16")])
def test_mx_odd_unit_count_ragged_rows_and_ranks(r, branch):
    """N = 1152 (nine units: one 128-wide tile per row block), ragged M, ranks up to the maximum (four branch MMAs)."""
    rng = np.random.default_rng(5)
    M, K, N = 1000, 1152, 1152
    X = rng.standard_normal((M, K)).astype(np.float16)
    X[:, rng.integers(0, K, 8)] *= 20
    _check(_mx_layer(rng, K, N, r, branch), X)


def test_mx_host_entry_point_pipelines_row_chunks():
    """lq_linear_forward_host with an MXINT4 layer: the row-chunk views of the activation record (codes, scale bytes in
    chunks of 128 rows, branch codes) must give the same bits as one call over all rows."""
    import torch
    from paper_2604_18117_b200 import binding as B
    from tests.helpers import import_oracle_layer
    rng = np.random.default_rng(6)
    M, K, N, r = 1300, 1152, 392, 32                       # five chunks, the last one ragged; N not a multiple of 128
    X = rng.standard_normal((M, K)).astype(np.float16)
    layer = _mx_layer(rng, K, N, r, "w8a8")
    ref = O.forward(X, layer)
    h, cfg = import_oracle_layer(layer)
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
        assert_codes_equal(ex, ref, "w8a8", with_qb=False)
        Xd = torch.from_numpy(X).cuda()
        Yd = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
        B.lq_quantize_act(h, Xd.data_ptr(), M, act, st)
        B.lq_linear_forward(h, act, Yd.data_ptr(), B.OUT_F16, st)
        torch.cuda.synchronize()
        assert np.array_equal(Yh, Yd.cpu().numpy())
        assert rel_fro(Yh, ref["Y"]) <= TOL_F16
    finally:
        B.lq_act_free(act)
        B.lq_layer_free(h)


@pytest.mark.parametrize("ctas", [0, 7])
@pytest.mark.parametrize("M,K,N,r,branch", [(1, 32, 8, 0, "none"), (129, 96, 136, 8, "w6a6"), (257, 8192, 128, 128, "w8a8"),
                                            (5, 160, 264, 32, "w16a16"), (1000, 40, 2000, 24, "w8a8"), (333, 5600, 24, 48, "w16a16")])
def test_mx_edge_shapes(ctas, M, K, N, r, branch):
    """One row, one block of K, the maximum K and rank, N below one tile, K and N that end inside a tile - with one CTA per
    SM and with seven CTAs (long runs of tiles per CTA)."""
    from paper_2604_18117_b200 import binding as B
    rng = np.random.default_rng(11)
    X = rng.standard_normal((M, K)).astype(np.float16)
    X[:, rng.integers(0, K, 2)] *= 20
    layer = _mx_layer(rng, K, N, r, branch)
    ref = O.forward(X, layer)
    B.lq_set_option("gemm_ctas", ctas)
    try:
        Y32, ex = gpu_forward(layer, X, out_f32=True)
        Y16, _ = gpu_forward(layer, X, out_f32=False, export=False)
    finally:
        B.lq_set_option("gemm_ctas", 0)
    assert_codes_equal(ex, ref, layer["branch"])
    assert np.isfinite(Y32).all()
    # fp16 reference branch: T is rounded to fp16 from an fp32 sum here and from an fp64 sum in the oracle
    assert rel_fro(Y32, ref["Y"]) <= (3e-4 if branch == "w16a16" else TOL_F32)
    assert rel_fro(Y16, ref["Y"]) <= TOL_F16
