"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Codes and scales must match bit for bit; Y within a relative Frobenius error
of 1e-3 (fp16 output; the fp16 rounding of Y alone is ~3e-4) and 1e-5 with fp32 output
(accumulation order only)."""
import numpy as np
import pytest

from oracle import lq_oracle as O
from paper_2604_18117_b200 import binding as B
from paper_2604_18117_b200 import inputs as I
from tests.helpers import assert_codes_equal, assert_y_close, gpu_forward, rel_fro

pytestmark = pytest.mark.gpu

TOL_F16 = 1e-3
TOL_F32 = 1e-5


def _random_layer(rng, K, N, r, branch, bias=True):
    """A layer with random quantized parts (no calibration needed for forward parity)."""
    layer = {"branch": branch if r > 0 else "none", "rank": r, "K": K, "N": N,
             "bias": (rng.standard_normal(N) * 0.05).astype(np.float16) if bias else None}
    layer["Wq"], layer["sw"] = O.q_weight_main(rng.standard_normal((K, N)) * 0.02)
    if r == 0:
        return layer
    L1 = rng.standard_normal((K, r)) * 0.05
    L2 = rng.standard_normal((r, N)) * 0.05
    if branch == "w16a16":
        layer["L1h"], _ = O.q_factor(L1, None)
        layer["L2h"], _ = O.q_factor(L2, None)
    else:
        bw, _ = O.BRANCH_BITS[branch]
        layer["L1q"], layer["sL1"] = O.q_factor(L1, bw)
        layer["L2q"], layer["sL2"] = O.q_factor(L2, bw)
    return layer


def _check(layer, X, tol32=TOL_F32, tol16=TOL_F16):
    ref = O.forward(X, layer)
    Y32, ex = gpu_forward(layer, X, out_f32=True)
    assert np.isfinite(Y32).all()
    assert_codes_equal(ex, ref, layer["branch"])
    e32 = rel_fro(Y32, ref["Y"])
    assert e32 <= tol32, f"fp32 output error {e32}"
    etol = 10 * tol32 if layer["branch"] == "w16a16" else tol32
    assert_y_close(Y32, ref["Y"], True, tol=etol)
    Y16, _ = gpu_forward(layer, X, out_f32=False, export=False)
    fits = np.abs(ref["Y"]).max(axis=1) < 6.0e4            # rows whose outputs fit fp16
    assert np.isfinite(Y16[fits]).all()
    e16 = rel_fro(Y16[fits], ref["Y"][fits])
    assert e16 <= tol16, f"fp16 output error {e16}"
    assert_y_close(Y16[fits], ref["Y"][fits], False, tol=etol)
    return e32, e16


def test_integer_exact_main_product():
    """Integer X in [-7,7] with every group maximum 7 and unit weight scales: all scales are 1,
    codes equal the inputs, and Y must equal the integer matrix product exactly - any inexact
    accumulation on the tensor cores shows up as a non-integer or wrong value."""
    rng = np.random.default_rng(0)
    M, K, N = 256, 1152, 384
    X = rng.integers(-7, 8, size=(M, K)).astype(np.float16)
    X[:, ::64] = 7
    X[0, :] = 7; X[1, :] = -7                               # extreme partial sums (+-3136 per group)
    Wi = rng.integers(-7, 8, size=(K, N)); Wi[::64, :] = 7
    Wi[:, 0] = 7; Wi[:, 1] = -7
    layer = {"branch": "none", "rank": 0, "K": K, "N": N, "bias": None}
    layer["Wq"], layer["sw"] = O.q_weight_main(Wi.astype(np.float64))
    assert np.all(layer["sw"] == 1)
    Y, ex = gpu_forward(layer, X, out_f32=True)
    assert np.array_equal(ex["qx"], X.astype(np.int8)) and np.all(ex["sx"] == 1)
    expect = X.astype(np.int64) @ Wi
    assert np.array_equal(Y.astype(np.int64), expect) and np.array_equal(Y, expect.astype(np.float32))


@pytest.mark.parametrize("branch", ["none", "w8a8", "w6a6", "w4a8", "w16a16"])
def test_small_shapes_all_branches(branch):
    rng = np.random.default_rng(1)
    M, K, N, r = 200, 320, 200, 0 if branch == "none" else 32      # ragged M, N; K = 5 groups (odd)
    X = rng.standard_normal((M, K)).astype(np.float16)
    X[:, 7] *= 20
    _check(_random_layer(rng, K, N, r, branch), X)


@pytest.mark.parametrize("r", [16, 64, 128])
def test_rank_sweep(r):
    rng = np.random.default_rng(2)
    M, K, N = 384, 1152, 256
    X = rng.standard_normal((M, K)).astype(np.float16)
    _check(_random_layer(rng, K, N, r, "w8a8"), X)


def test_ragged_k_and_edge_values():
    """K = 5600 -> 87.5 groups (short last group); rows of zeros, huge and subnormal values,
    exact ties."""
    rng = np.random.default_rng(3)
    M, K, N, r = 130, 5600, 136, 32
    X = rng.standard_normal((M, K)).astype(np.float16)
    X[0, :] = 0
    X[1, :64] = 0
    X[2, :] = np.float16(65504.0) * np.sign(rng.standard_normal(K)).astype(np.float16)
    X[3, :] = np.float16(2.0 ** -24)
    X[4, :] = (rng.integers(-14, 15, size=K) * 0.5).astype(np.float16); X[4, ::64] = 7   # ties k + 1/2
    X[5, :] = np.float16(6e-5) * rng.standard_normal(K).astype(np.float16)               # subnormal halves
    _check(_random_layer(rng, K, N, r, "w4a8"), X)


def test_quantizer_random_bit_patterns_and_exact_ties():
    """Codes only (Y may overflow): every finite fp16 bit pattern can occur, and whole groups / rows sit
    exactly on rounding ties with non-trivial scales, which the fast path must hand to the exact path."""
    rng = np.random.default_rng(4)
    M, K, N, r = 96, 1024, 64, 16
    bits = rng.integers(0, 1 << 16, size=(M, K), dtype=np.uint16)
    bits[(bits & 0x7C00) == 0x7C00] &= 0xBFFF                      # no inf / nan
    X = bits.view(np.float16).copy()
    # rows 0..31: each group holds s * c / 2 with group maximum 7 s, s = 2^e (1 + j/8): ties at odd c
    for m in range(32):
        for g in range(K // 64):
            s = np.float16(2.0 ** rng.integers(-10, 6) * (1 + rng.integers(0, 8) / 8))
            c = rng.integers(-14, 15, size=64)
            c[rng.integers(0, 64)] = 14
            X[m, g * 64:(g + 1) * 64] = (np.float32(s) * c.astype(np.float32) * np.float32(0.5)).astype(np.float16)
    # rows 32..47: per-token ties of the 8-bit branch: row maximum 127 * 2^e, entries (k + 1/2) * 2^e
    for m in range(32, 48):
        e = 2.0 ** rng.integers(-6, 3)
        k = rng.integers(-126, 126, size=K)
        X[m, :] = ((k + 0.5) * e).astype(np.float16)
        X[m, rng.integers(0, K)] = np.float16(127 * e)
    X[48, :] = np.float16(2.0 ** -24)                                # smallest subnormal everywhere
    X[49, :] = (rng.integers(-12, 13, size=K) * 2.0 ** -24).astype(np.float16)   # subnormal scales, quotients > 7
    for branch in ("w8a8", "w6a6"):
        layer = _random_layer(rng, K, N, r, branch)
        ref = O.forward(X, layer)
        _, ex = gpu_forward(layer, X, out_f32=True)
        assert_codes_equal(ex, ref, branch)


def test_branch_codes_stay_on_chip_by_default():
    """The benchmark configuration does not write qb to HBM; everything else must be unchanged."""
    rng = np.random.default_rng(5)
    M, K, N, r = 300, 1152, 256, 32
    X = rng.standard_normal((M, K)).astype(np.float16)
    layer = _random_layer(rng, K, N, r, "w8a8")
    ref = O.forward(X, layer)
    Y, ex = gpu_forward(layer, X, out_f32=True, store_qb=False)
    assert_codes_equal(ex, ref, "w8a8", with_qb=False)
    assert not ex["qb"].any()
    assert rel_fro(Y, ref["Y"]) <= TOL_F32


def test_config0_full_calibration():
    """Config 0: 256 x 1152 x 1152, r = 32, W8A8 branch, data-free calibration run by the oracle."""
    wl = I.workload(0)
    X, W, _ = I.layer_inputs(wl, wl.layers[0])
    layer, trace = O.calibrate(W, 32, "w8a8", steps=1000, lr=1e-4)
    assert min(trace) < trace[0]
    e32, e16 = _check(layer, X)
    print(f"config0 rel err fp32 {e32:.3e} fp16 {e16:.3e}")


def test_host_entry_point_pipelines_row_chunks():
    """lq_linear_forward_host overlaps copy-in, compute and copy-out over row chunks; the result must be the
    same as one lq_quantize_act + lq_linear_forward over all rows (bit for bit: rows are independent), and the
    activation record must hold every chunk's codes."""
    import torch
    from tests.helpers import import_oracle_layer
    rng = np.random.default_rng(6)
    M, K, N, r = 1300, 1152, 392, 32                       # five chunks, the last one ragged; N not a multiple of 128
    X = rng.standard_normal((M, K)).astype(np.float16)
    layer = _random_layer(rng, K, N, r, "w8a8")
    ref = O.forward(X, layer)
    h, cfg = import_oracle_layer(layer)
    B.lq_layer_to_device(h, 0)
    act = B.lq_act_create(h, M, 0)
    try:
        st = torch.cuda.current_stream().cuda_stream
        Xp = torch.from_numpy(X).pin_memory()
        for dtype, tdt, tol in ((B.OUT_F32, torch.float32, TOL_F32), (B.OUT_F16, torch.float16, TOL_F16)):
            Yp = torch.full((M, N), float("nan"), dtype=tdt).pin_memory()
            B.lq_linear_forward_host(h, act, Xp.data_ptr(), M, Yp.data_ptr(), dtype, st)
            assert B.lq_get_device_status(0)[0] == 0
            Yh = Yp.numpy().copy()
            Xd = torch.from_numpy(X).cuda()
            Yd = torch.full((M, N), float("nan"), dtype=tdt, device="cuda")
            B.lq_quantize_act(h, Xd.data_ptr(), M, act, st)
            B.lq_linear_forward(h, act, Yd.data_ptr(), dtype, st)
            torch.cuda.synchronize()
            assert np.array_equal(Yh, Yd.cpu().numpy())
            assert rel_fro(Yh, ref["Y"]) <= tol
        B.lq_linear_forward_host(h, act, Xp.data_ptr(), M, Yp.data_ptr(), B.OUT_F16, st)
        ex = B.lq_act_export(act, M, cfg, st)
        assert_codes_equal(ex, ref, "w8a8", with_qb=False)
    finally:
        B.lq_act_free(act)
        B.lq_layer_free(h)


def test_bounded_wait_reports_timeout_and_device_stays_usable():
    """Failure detection without a fault: a wait that nothing satisfies runs into its limit, the kernel records
    LQ_ERR_TIMEOUT (5) with the waiting stage in the status word and returns; the next forward is unaffected."""
    import torch
    st = torch.cuda.current_stream().cuda_stream
    assert B.lq_get_device_status(0)[0] == 0
    B.lq_selftest_wait_timeout(0, st)
    code, stage = B.lq_get_device_status(0)                 # synchronises; reading clears the word
    assert (code, stage) == (5, 4)
    assert B.lq_get_device_status(0) == (0, 0)
    rng = np.random.default_rng(7)
    X = rng.standard_normal((130, 320)).astype(np.float16)
    _check(_random_layer(rng, 320, 72, 16, "w8a8"), X)


def test_async_host_entry_point_on_two_streams():
    """lq_linear_forward_host_async returns before Y has arrived; after the stream is synchronised Y equals the waiting
    call's result bit for bit.  Two layers on two streams run their copies and kernels concurrently."""
    import torch
    from tests.helpers import import_oracle_layer
    rng = np.random.default_rng(8)
    M = 1300
    jobs = []
    for (K, N, r, br) in ((1152, 392, 32, "w8a8"), (640, 1160, 16, "w6a6")):
        X = rng.standard_normal((M, K)).astype(np.float16)
        layer = _random_layer(rng, K, N, r, br)
        h, _ = import_oracle_layer(layer)
        B.lq_layer_to_device(h, 0)
        jobs.append(dict(h=h, act=B.lq_act_create(h, M, 0), Xp=torch.from_numpy(X).pin_memory(), N=N,
                         ref=O.forward(X, layer)["Y"], stream=torch.cuda.Stream()))
    try:
        for j in jobs:                                      # reference: the waiting call
            j["Yw"] = torch.full((M, j["N"]), float("nan"), dtype=torch.float16).pin_memory()
            B.lq_linear_forward_host(j["h"], j["act"], j["Xp"].data_ptr(), M, j["Yw"].data_ptr(), B.OUT_F16, j["stream"].cuda_stream)
        for _ in range(2):
            for j in jobs:
                j["Ya"] = torch.full((M, j["N"]), float("nan"), dtype=torch.float16).pin_memory()
                B.lq_linear_forward_host_async(j["h"], j["act"], j["Xp"].data_ptr(), M, j["Ya"].data_ptr(), B.OUT_F16,
                                               j["stream"].cuda_stream)
            for j in jobs:
                j["stream"].synchronize()
                assert np.array_equal(j["Ya"].numpy(), j["Yw"].numpy())
                assert rel_fro(j["Ya"].numpy(), j["ref"]) <= TOL_F16
        assert B.lq_get_device_status(0)[0] == 0
    finally:
        for j in jobs:
            B.lq_act_free(j["act"])
            B.lq_layer_free(j["h"])


def test_overlapped_launches_keep_stream_order():
    """The library launches its kernels so that a kernel may take its SMs and set up while the previous kernel on the
    stream drains ("overlap" option, on by default); each kernel waits for that previous kernel before it touches global
    memory.  Two layers are chained on one stream with no synchronisation in between - the second layer's input IS the
    first layer's output - several times in a row; the result must be bit-identical with plain launches and agree with
    the oracle run on the first layer's output."""
    import torch
    from tests.helpers import import_oracle_layer
    rng = np.random.default_rng(21)
    M, K, N1, N2, r = 2000, 1152, 1152, 384, 32
    l1 = _random_layer(rng, K, N1, r, "w8a8")
    l2 = _random_layer(rng, N1, N2, r, "w8a8")
    X = (rng.standard_normal((M, K))).astype(np.float16)
    h1, _ = import_oracle_layer(l1)
    h2, _ = import_oracle_layer(l2)
    for h in (h1, h2):
        B.lq_layer_to_device(h, 0)
    a1, a2 = B.lq_act_create(h1, M, 0), B.lq_act_create(h2, M, 0)
    st = torch.cuda.current_stream().cuda_stream
    Xd = torch.from_numpy(X).cuda()
    out = {}
    try:
        for overlap in (1, 0):
            B.lq_set_option("overlap", overlap)
            Y1 = torch.zeros((M, N1), dtype=torch.float16, device="cuda")
            Y2 = torch.zeros((M, N2), dtype=torch.float16, device="cuda")
            for _ in range(3):                               # back to back: the next round's first kernel follows the last GEMM
                B.lq_quantize_act(h1, Xd.data_ptr(), M, a1, st)
                B.lq_linear_forward(h1, a1, Y1.data_ptr(), B.OUT_F16, st)
                B.lq_quantize_act(h2, Y1.data_ptr(), M, a2, st)
                B.lq_linear_forward(h2, a2, Y2.data_ptr(), B.OUT_F16, st)
            torch.cuda.synchronize()
            assert B.lq_get_device_status(0)[0] == 0
            out[overlap] = (Y1.cpu().numpy(), Y2.cpu().numpy())
        assert np.array_equal(out[1][0], out[0][0]) and np.array_equal(out[1][1], out[0][1])
        assert rel_fro(out[1][0], O.forward(X, l1)["Y"]) <= TOL_F16
        assert rel_fro(out[1][1], O.forward(out[1][0], l2)["Y"]) <= TOL_F16
    finally:
        B.lq_set_option("overlap", 1)
        B.lq_act_free(a1); B.lq_act_free(a2)
        B.lq_layer_free(h1); B.lq_layer_free(h2)
