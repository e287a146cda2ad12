"""Per-role timeline of the GEMM kernels (lq_gemm_kernel, lq_gemm_mx_kernel), from clock stamps inside the kernel.

    python -m paper_2604_18117_b200.timeline [--main sint4|mxint4|mxfp4] [--layer qkv|attn_out|fc1|fc2] [--rows 8192]
                                             [--trace N]

Builds liblq_timeline.so (the library's sources with -DLQ_TIMELINE), runs one config-1 layer through it and prints,
for CTA 0 and each stamped warp (TMA producer, MMA issuer, first and last drain warp), the median number of SM
clocks between consecutive stamps, keyed by the pair of events - i.e. how long each step of the role's loop takes
in steady state (the first tile is left out).  --trace N also prints N raw stamps per role.  The regular library
carries none of this code; stamps cost one 8-byte store each, so absolute times are those of the stamped build.

Events: P_SLOT_FREE (producer saw a free operand stage), P_ISSUED (its copies are issued); M_ACC_FREE (issuer saw a
free accumulator), M_STAGE_FULL (operands landed), M_ISSUED (the stage's MMAs and commit are issued), TILE (tile
boundary); D_OPEN (drain starts waiting), D_ACC_FULL (accumulator handed over), D_WAITED / D_LOADED (slice in
registers, accumulator handed back), D_HALF, D_DONE (arithmetic of the stage done), D_EPI_BEGIN / D_EPI_END (stores).
"""
from __future__ import annotations

import argparse
import ctypes as C
import statistics
from collections import defaultdict

import numpy as np

EV = {1: "P_SLOT_FREE", 2: "P_ISSUED", 3: "M_STAGE_FULL", 4: "M_ACC_FREE", 5: "M_ISSUED", 6: "D_OPEN", 7: "D_ACC_FULL",
      8: "D_LOADED", 9: "D_DONE", 10: "D_EPI_BEGIN", 11: "D_EPI_END", 12: "TILE", 13: "D_HALF", 14: "D_LD_ISSUED",
      15: "D_WAITED"}
ROLES = ("producer", "mma_issuer", "drain_first", "drain_last")
LISTS, CAP = 4, 8192
MASK40 = (1 << 40) - 1


def decode(words):
    out = []
    for row in words:
        lst = []
        for w in row:
            if int(w) == 0:
                break
            lst.append((int(w) >> 48, (int(w) >> 40) & 0xFF, int(w) & MASK40))
        out.append(lst)
    return out


def step_medians(lst, skip):
    """Median clocks between consecutive stamps, keyed by (previous event, event); the first `skip` stamps are left out."""
    d = defaultdict(list)
    for (e0, _, c0), (e1, _, c1) in zip(lst[skip:], lst[skip + 1:]):
        d[(e0, e1)].append(c1 - c0)
    return {k: (statistics.median(v), len(v)) for k, v in d.items()}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--main", default="sint4", choices=["sint4", "mxint4", "mxfp4"])
    ap.add_argument("--layer", default="qkv")
    ap.add_argument("--rows", type=int, default=8192)
    ap.add_argument("--trace", type=int, default=0, help="also print this many raw stamps per role from the second tile on")
    args = ap.parse_args()
    import torch
    from paper_2604_18117_b200 import binding as B, build as BUILD, inputs as I
    B.LIB_PATH = BUILD.build(timeline=True)
    wl = I.workload(1, M=args.rows)
    spec = {s.name: s for s in wl.layers}[args.layer]
    X, W, bias = I.layer_inputs(wl, spec, with_bias=True)
    if args.main == "mxfp4":
        cfg = B.lq_config_default(spec.K, spec.N, 64, "mxfp8")
    else:
        cfg = B.lq_config_default(spec.K, spec.N, wl.rank, wl.branch)
        if args.main == "mxint4":
            cfg.group = 32
    cfg.steps = 0
    h, _ = B.lq_calibrate(cfg, W, bias)
    B.lq_layer_to_device(h, 0)
    act = B.lq_act_create(h, args.rows, 0)
    Xd = torch.from_numpy(X).cuda()
    Yd = torch.empty((args.rows, spec.N), dtype=torch.float16, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    buf = np.zeros((LISTS, CAP), dtype=np.uint64)
    fn = getattr(B.lib(), "lq_debug_timeline" if args.main == "sint4" else "lq_debug_timeline_mx")
    fn.argtypes = [C.c_void_p]
    fn.restype = C.c_int
    for _ in range(3):                                   # the last launch's stamps are the ones read back
        B.lq_quantize_act(h, Xd.data_ptr(), args.rows, act, st)
        torch.cuda.synchronize()
        assert fn(buf.ctypes.data) == 0
        B.lq_linear_forward(h, act, Yd.data_ptr(), B.OUT_F16, st)
    torch.cuda.synchronize()
    assert fn(buf.ctypes.data) == 0
    assert B.lq_get_device_status(0)[0] == 0
    stamps = decode(buf)
    t0 = min(s[0][2] for s in stamps if s)
    t1 = max(s[-1][2] for s in stamps if s)
    print(f"{args.main} layer {spec.name}: K = {spec.K}, N = {spec.N}, rows = {args.rows}; CTA 0 active for {t1 - t0} clocks")
    for role, lst in zip(ROLES, stamps):
        if not lst:
            continue
        # leave the first tile out: skip up to and including the first tile-boundary / epilogue-end stamp
        skip = next((i + 1 for i, (e, _, _) in enumerate(lst) if e in (11, 12)), len(lst) // 8)
        if role == "producer":
            skip = min(len(lst) // 4, 24)
        print(f"  {role}: {len(lst)} stamps, {lst[-1][2] - lst[0][2]} clocks from first to last")
        for (e0, e1), (m, n) in sorted(step_medians(lst, skip).items(), key=lambda kv: -kv[1][0] * kv[1][1]):
            print(f"      {EV.get(e0, e0):>13s} -> {EV.get(e1, e1):<13s} median {m:8.0f} clocks  x {n:4d}  = {m * n:9.0f}")
    if args.trace:
        for role, lst in zip(ROLES, stamps):
            print(f"  trace {role} (clocks since CTA start):")
            skip = min(len(lst) // 3, 40)
            for e, tag, c in lst[skip:skip + args.trace]:
                print(f"      {c - t0:10d}  {EV.get(e, e):13s} {tag}")
    B.lq_act_free(act)
    B.lq_layer_free(h)


if __name__ == "__main__":
    main()
