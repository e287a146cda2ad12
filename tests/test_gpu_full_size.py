"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times
(lq_quantize_act + lq_linear_forward, fp16 output, branch codes kept on chip).

Rows (tokens) are independent in every step of the path, so the CPU oracle is evaluated on a
seeded sample of rows - including the first and last rows of the first and last row tiles -
and the GPU result, computed on ALL rows, is compared on those rows: codes and scales bit for
bit, Y within a relative Frobenius error of 1e-3 (fp16 output; 1e-5 with fp32 output, 3e-4 with the fp16 reference
branch) AND within an element-wise bound (tests/helpers.py: elementwise_excess).  Inputs are the seeded
synthetic tensors of the five configurations (outlier channels, GELU-shaped fc2 inputs); the
layers come from the oracle's SVD initialisation of the seeded weight (steps = 0: forward
parity does not depend on how far calibration ran) and are imported into the library."""
import numpy as np
import pytest

from oracle import lq_oracle as O
from paper_2604_18117_b200 import binding as B
from paper_2604_18117_b200 import inputs as I
from tests.helpers import assert_y_close, import_oracle_layer, rel_fro

pytestmark = pytest.mark.gpu

TOL_F16 = 1e-3
TOL_F32 = 1e-5
TOL_F32_W16 = 3e-4   # the fp16 reference branch rounds T = X L1 to fp16: fp32 vs fp64 accumulation flips a few roundings
SAMPLE = 160


def _sample_rows(M, seed):
    rng = np.random.default_rng(seed)
    fixed = np.array([0, 1, 127, 128, M - 129, M - 128, M - 2, M - 1])
    extra = rng.choice(M, size=SAMPLE - len(fixed), replace=False)
    return np.unique(np.concatenate([fixed, extra]))


def _run_case(config, spec, M, rank, branch, seed=0, out_f32=False):
    import torch
    wl = I.workload(config, branch=branch, rank=rank, M=M)
    X, W, bias = I.layer_inputs(wl, spec, seed=seed, with_bias=True)
    layer, _ = O.calibrate(W, rank, branch, steps=0)
    layer["bias"] = bias
    rows = _sample_rows(M, seed + 17)
    ref = O.forward(X[rows], layer)

    h, cfg = import_oracle_layer(layer)
    B.lq_layer_to_device(h, 0)
    act = B.lq_act_create(h, M, 0)
    try:
        Xd = torch.from_numpy(X).cuda()
        Yd = torch.full((M, spec.N), float("nan"), dtype=torch.float32 if out_f32 else torch.float16, device="cuda")
        st = torch.cuda.current_stream().cuda_stream
        B.lq_quantize_act(h, Xd.data_ptr(), M, act, st)
        B.lq_linear_forward(h, act, Yd.data_ptr(), B.OUT_F32 if out_f32 else B.OUT_F16, st)
        torch.cuda.synchronize()
        code, stage = B.lq_get_device_status(0)
        assert code == 0, f"device status {code} at stage {stage}"
        ex = B.lq_act_export(act, M, cfg, st)
        Y = Yd.cpu().numpy()
    finally:
        B.lq_act_free(act)
        B.lq_layer_free(h)
    assert np.array_equal(ex["qx"][rows], ref["qx"]), "qx differs"
    assert np.array_equal(ex["sx"][rows].view(np.uint16), ref["sx"].view(np.uint16)), "sx differs"
    if branch in ("w8a8", "w6a6", "w4a8"):
        assert np.array_equal(ex["sXb"][rows].view(np.uint32), ref["sXb"].view(np.uint32)), "sXb differs"
        assert np.array_equal(ex["tq"][rows], ref["tq"]), "tq differs"
        assert np.array_equal(ex["sT"][rows].view(np.uint32), ref["sT"].view(np.uint32)), "sT differs"
    assert np.isfinite(Y.astype(np.float32)).all(), "unwritten or non-finite outputs"
    err = rel_fro(Y[rows], ref["Y"])
    tol32 = TOL_F32_W16 if branch == "w16a16" else TOL_F32
    assert err <= (tol32 if out_f32 else TOL_F16), f"output error {err}"
    assert_y_close(Y[rows], ref["Y"], out_f32, tol=10 * tol32 if branch == "w16a16" else tol32)
    # every row tile was written: nothing left at the NaN fill, and no row is all zero by accident
    assert (np.abs(Y.astype(np.float32)).sum(axis=1) > 0).all()
    return err


@pytest.mark.parametrize("spec", I.PIXART_LAYERS, ids=lambda s: s.name)
def test_config1_pixart_block_linears(spec):
    _run_case(1, spec, 8192, 32, "w8a8")


@pytest.mark.parametrize("spec", I.PIXART_LAYERS, ids=lambda s: s.name)
def test_config1_pixart_block_linears_fp32_output(spec):
    """The same launches with fp32 output: the tight tolerance (accumulation order only) at the full size."""
    _run_case(1, spec, 8192, 32, "w8a8", out_f32=True)


@pytest.mark.parametrize("branch", ["w16a16", "w6a6", "w4a8", "none"])
def test_config2_branch_precision_sweep(branch):
    """qkv and fc2 shapes of config 1 with every other branch precision (W8A8 is covered above)."""
    rank = 0 if branch == "none" else 32
    _run_case(2, I.PIXART_LAYERS[0], 8192, rank, branch)
    _run_case(2, I.PIXART_LAYERS[3], 8192, rank, branch)
    _run_case(2, I.PIXART_LAYERS[1], 8192, rank, branch, out_f32=True)


@pytest.mark.parametrize("spec", I.SANA_LAYERS, ids=lambda s: s.name)
def test_config3_sana_block_linears(spec):
    """Hidden 2240 / 5600: N is not a multiple of 128 and K = 5600 ends in a half group."""
    _run_case(3, spec, 8192, 32, "w4a8")
    if spec.name in ("out", "mlp_down"):
        _run_case(3, spec, 8192, 32, "w4a8", out_f32=True)


@pytest.mark.parametrize("rank", [16, 32, 64, 128])
@pytest.mark.parametrize("spec", I.PIXART_LAYERS, ids=lambda s: s.name)
def test_config4_stack_rows_and_rank_sweep(spec, rank):
    """M = 32768 rows (batch 8 x 4096 tokens; the 16384-token x batch 2 case has the same row count), every layer
    shape at every rank of the sweep; the rank-32 cases also with fp32 output."""
    _run_case(4, spec, 32768, rank, "w8a8", out_f32=(rank == 32))
