"""lq_linear_forward_static - the entry point for callers that may not allocate device memory
when they call (a server whose pool owns the device, a fixed-budget loop, a plugin under a
framework's allocator) - must give what the regular two-call path gives.  It keeps its
activation record in one fixed array inside the library that every call reuses, so it is
called twice in a row, with different inputs, to show that what the first call left behind
does not leak into the second.  This file sorts last so that a run stopping at the first
failure has already run every other test."""
import numpy as np
import pytest

from oracle import lq_oracle as O
from paper_2604_18117_b200 import binding as B
from tests.helpers import import_oracle_layer, rel_fro

pytestmark = pytest.mark.gpu


def _layer(rng, K, N, r):
    layer = {"branch": "w8a8", "rank": r, "K": K, "N": N, "bias": (rng.standard_normal(N) * 0.05).astype(np.float16)}
    layer["Wq"], layer["sw"] = O.q_weight_main(rng.standard_normal((K, N)) * 0.02)
    layer["L1q"], layer["sL1"] = O.q_factor(rng.standard_normal((K, r)) * 0.05, 8)
    layer["L2q"], layer["sL2"] = O.q_factor(rng.standard_normal((r, N)) * 0.05, 8)
    return layer


def test_static_entry_matches_regular_path_twice_in_a_row():
    import torch
    rng = np.random.default_rng(42)
    K, N, r = 1152, 384, 32
    layer = _layer(rng, K, N, r)
    h, cfg = import_oracle_layer(layer)
    B.lq_layer_to_device(h, 0)
    st = torch.cuda.current_stream().cuda_stream
    try:
        # first call: 200 rows with large values; second call: fewer rows, small values - stale
        # rows, scales or padding from the first call would change the second result
        for M, scale in ((200, 30.0), (72, 0.25)):
            X = (rng.standard_normal((M, K)) * scale).astype(np.float16)
            Xd = torch.from_numpy(X).cuda()
            Yref = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
            act = B.lq_act_create(h, M, 0)
            B.lq_quantize_act(h, Xd.data_ptr(), M, act, st)
            B.lq_linear_forward(h, act, Yref.data_ptr(), B.OUT_F32, st)
            Y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
            B.lq_linear_forward_static(h, Xd.data_ptr(), M, Y.data_ptr(), B.OUT_F32, st)
            torch.cuda.synchronize()
            assert B.lq_get_device_status(0)[0] == 0
            B.lq_act_free(act)
            Yn, Yr = Y.cpu().numpy(), Yref.cpu().numpy()
            assert np.isfinite(Yn).all()
            assert rel_fro(Yn, Yr.astype(np.float64)) <= 1e-5          # the tolerance of the fp32 parity tests
            # and both agree with the oracle
            assert rel_fro(Yn, O.forward(X, layer)["Y"]) <= 1e-5
        # a request beyond the fixed array is refused before anything is launched
        Mbig = 4096
        Xd = torch.zeros((Mbig, K), dtype=torch.float16, device="cuda")
        Yd = torch.zeros((Mbig, N), dtype=torch.float16, device="cuda")
        with pytest.raises(B.LqError) as e:
            B.lq_linear_forward_static(h, Xd.data_ptr(), Mbig, Yd.data_ptr(), B.OUT_F16, st)
        assert e.value.code == 2
    finally:
        B.lq_layer_free(h)


def test_static_entry_alternating_layers_and_output_types():
    """Two layers with different K, rank and branch kind share the library's one fixed array call after call: a W8A8
    layer (int8 codes in the rank-r container) and a layer with the fp16 reference branch (halves in the same bytes),
    each with fp16 and fp32 output.  Stale bytes of one layer's record - read as the other's codes - would show up as
    NaNs or wrong values; every call is compared with the regular two-call path on the same input."""
    import torch
    rng = np.random.default_rng(7)
    la = _layer(rng, 1152, 256, 32)
    lb = {"branch": "w16a16", "rank": 24, "K": 640, "N": 136, "bias": None}
    lb["Wq"], lb["sw"] = O.q_weight_main(rng.standard_normal((640, 136)) * 0.02)
    lb["L1h"], _ = O.q_factor(rng.standard_normal((640, 24)) * 0.05, None)
    lb["L2h"], _ = O.q_factor(rng.standard_normal((24, 136)) * 0.05, None)
    handles = [import_oracle_layer(l)[0] for l in (la, lb)]
    for h in handles:
        B.lq_layer_to_device(h, 0)
    st = torch.cuda.current_stream().cuda_stream
    try:
        for rep in range(2):
            for layer, h in zip((la, lb), handles):
                for f32 in (True, False):
                    M = 150 if layer is la else 97
                    K, N = layer["K"], layer["N"]
                    X = (rng.standard_normal((M, K)) * (5.0 if rep == 0 else 0.5)).astype(np.float16)
                    Xd = torch.from_numpy(X).cuda()
                    dt = torch.float32 if f32 else torch.float16
                    code = B.OUT_F32 if f32 else B.OUT_F16
                    Yref = torch.full((M, N), float("nan"), dtype=dt, device="cuda")
                    act = B.lq_act_create(h, M, 0)
                    B.lq_quantize_act(h, Xd.data_ptr(), M, act, st)
                    B.lq_linear_forward(h, act, Yref.data_ptr(), code, st)
                    Y = torch.full((M, N), float("nan"), dtype=dt, device="cuda")
                    B.lq_linear_forward_static(h, Xd.data_ptr(), M, Y.data_ptr(), code, st)
                    torch.cuda.synchronize()
                    assert B.lq_get_device_status(0)[0] == 0
                    B.lq_act_free(act)
                    Yn, Yr = Y.float().cpu().numpy(), Yref.float().cpu().numpy()
                    assert np.isfinite(Yn).all()
                    # the same kernels on the same input: identical up to nothing at all
                    assert np.array_equal(Yn, Yr), (layer["branch"], f32, rep)
                    tol = (3e-4 if layer["branch"] == "w16a16" else 1e-5) if f32 else 1e-3
                    assert rel_fro(Yn, O.forward(X, layer)["Y"]) <= tol
    finally:
        for h in handles:
            B.lq_layer_free(h)
