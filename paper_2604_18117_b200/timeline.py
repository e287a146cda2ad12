"""Per-role timeline of the SINT4 GEMM kernel (lq_gemm_kernel), from clock stamps inside the kernel.

    python -m paper_2604_18117_b200.timeline [--layer qkv|attn_out|fc1|fc2] [--rows 8192]

Builds liblq_timeline.so (the library's sources with -DLQ_TIMELINE), runs one config-1 layer through it and prints,
for CTA 0, where the cycles of a tile go in each role: the MMA warp (waiting for operands, waiting for a free
accumulator, issuing), the first and the last drain warp (waiting for a full accumulator, loading it from tensor
memory, scaling and accumulating, epilogue).  Cycles are SM clocks (clock64); the regular library carries none of
this code.
"""
from __future__ import annotations

import argparse
import ctypes as C
import statistics
import sys

import numpy as np

EV = {1: "P_SLOT_FREE", 2: "P_ISSUED", 3: "M_STAGE_FULL", 4: "M_ACC_FREE", 5: "M_ISSUED", 6: "D_OPEN", 7: "D_ACC_FULL",
      8: "D_LOADED", 9: "D_DONE", 10: "D_EPI_BEGIN", 11: "D_EPI_END", 12: "TILE", 13: "D_HALF", 14: "D_LD_ISSUED",
      15: "D_WAITED"}
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


def med(v):
    return statistics.median(v) if v else float("nan")


def analyse(stamps, G, has_branch):
    """Returns a dict of median cycle counts per group (steady state: the first tile is left out)."""
    res = {}
    groups_per_tile = G + (1 if has_branch else 0)
    for name, lst in (("drain_first", stamps[2]), ("drain_last", stamps[3])):
        ev = [(e, t, c) for e, t, c in lst]
        wait, load, arith, period, epi = [], [], [], [], []
        opened = {}
        last_done = None
        seen = 0
        for e, tag, c in ev:
            if e == 6:
                opened[tag] = c
            elif e == 7:
                full_at = c
                w = c - opened.get(tag, c)
            elif e == 8:
                loaded_at = c
            elif e == 9:
                seen += 1
                if seen > groups_per_tile:          # past the first tile
                    wait.append(w)
                    load.append(loaded_at - full_at)
                    arith.append(c - loaded_at)
                    if last_done is not None and tag != 0:
                        period.append(c - last_done)
                last_done = c
            elif e == 10:
                epi_begin = c
            elif e == 11:
                epi.append(c - epi_begin)
        res[name] = {"wait_for_accumulator": med(wait), "first_chunk_to_last_load_landed": med(load),
                     "last_load_to_arithmetic_done": med(arith), "group_period": med(period), "epilogue": med(epi),
                     "groups": len(wait)}
    ev = stamps[1]
    wait_full, wait_acc, issue, period = [], [], [], []
    prev = None
    last_issue = None
    for e, tag, c in ev:
        if e == 3:
            if prev is not None:
                wait_full.append(c - prev)
        elif e == 4:
            wait_acc.append(c - prev if prev is not None else 0)
        elif e == 5:
            issue.append(c - prev if prev is not None else 0)
            if last_issue is not None:
                period.append(c - last_issue)
            last_issue = c
        prev = c
    skip = groups_per_tile
    res["mma_warp"] = {"wait_for_operand_stage": med(wait_full[skip // 2:]), "wait_for_free_accumulator": med(wait_acc[skip:]),
                       "issue_two_mmas_and_commit": med(issue[skip:]), "group_period": med(period[skip:]), "groups": len(issue)}
    ev = stamps[0]
    w, iss = [], []
    prev = None
    for e, tag, c in ev:
        if e == 1 and prev is not None:
            w.append(c - prev)
        if e == 2 and prev is not None:
            iss.append(c - prev)
        prev = c
    res["producer"] = {"wait_for_free_stage": med(w[4:]), "issue_copies": med(iss[4:]), "stages": len(iss)}
    return res


def main():
    ap = argparse.ArgumentParser()
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
    cfg = B.lq_config_default(spec.K, spec.N, wl.rank, wl.branch)
    cfg.steps = 0
    h, _ = B.lq_calibrate(cfg, W, bias)
    B.lq_layer_to_device(h, 0)
    act = B.lq_act_create(h, args.rows, 0)
    Xd = torch.from_numpy(X).cuda()
    Yd = torch.empty((args.rows, spec.N), dtype=torch.float16, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    buf = np.zeros((LISTS, CAP), dtype=np.uint64)
    fn = B.lib().lq_debug_timeline
    fn.argtypes = [C.c_void_p]
    fn.restype = C.c_int
    for _ in range(3):                                   # the last launch's stamps are the ones read back
        B.lq_quantize_act(h, Xd.data_ptr(), args.rows, act, st)
        torch.cuda.synchronize()
        assert fn(buf.ctypes.data) == 0
        B.lq_linear_forward(h, act, Yd.data_ptr(), B.OUT_F16, st)
    torch.cuda.synchronize()
    assert fn(buf.ctypes.data) == 0
    stamps = decode(buf)
    G = -(-spec.K // 64)
    res = analyse(stamps, G, wl.rank > 0)
    t0 = min(s[0][2] for s in stamps if s)
    t1 = max(s[-1][2] for s in stamps if s)
    print(f"layer {spec.name}: K = {spec.K}, N = {spec.N}, rows = {args.rows}, groups per tile = {G} + branch; "
          f"CTA 0 active for {t1 - t0} cycles")
    for role, d in res.items():
        print(f"  {role}:")
        for k, v in d.items():
            print(f"      {k:36s} {v}")
    if args.trace:
        names = ["producer", "mma_warp", "drain_first", "drain_last"]
        start = {0: 2 * (G // 2 + 1) + 8, 1: 3 * (G + 1) + 10, 2: 4 * (G + 1) + 8, 3: 4 * (G + 1) + 8}
        for li, lst in enumerate(stamps):
            print(f"  trace {names[li]} (cycles since CTA start):")
            for e, tag, c in lst[start[li]:start[li] + args.trace]:
                print(f"      {c - t0:9d}  {EV.get(e, e):14s} {tag}")
    B.lq_act_free(act)
    B.lq_layer_free(h)


if __name__ == "__main__":
    sys.exit(main())
