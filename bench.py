#!/usr/bin/env python
"""Benchmark of the LoRaQ fused quantized-linear hot path on B200.

One "step" = one pass of the whole hot path (activation quantizer + down-projection, then the
W4A4 tensor-core GEMM with fused per-group scales / up-projection / bias) over every linear of
one PixArt-class transformer block (qkv, attn-out, fc1, fc2; hidden 1152, MLP 4608) at
M = 4096 tokens x batch 2 = 8192 rows, rank 32, W8A8 branch - seeded synthetic tensors that
stand in for the paper's PixArt-Sigma activations and weights.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  `value` is TOPS (2MKN + 2Mr(K+N) algorithmic ops per layer) with inputs
resident in HBM; `e2e` is the same metric through lq_linear_forward_host_async (pinned host X in,
host Y out, one stream per layer, all synchronised at the end of the step: copies inside the timed region); `roofline` describes the GEMM kernel against the
8-bit-operand tensor peak (2 x the measured bf16 cuBLAS peak); `cpu_baseline` is the CPU oracle
timed on a 256-row sample of the same layers.  With N > 1 (torchrun) every rank runs the same
rows-sharded workload independently (rows are independent: no collective on the data path).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "fused_w4a4_loraq_linear_throughput"
UNIT = "TOPS"
SAMPLE_ROWS = 256


def layer_ops(M, K, N, r):
    return 2.0 * M * K * N + 2.0 * M * r * (K + N)


def gemm_ops(M, K, N, r):
    return 2.0 * M * K * N + 2.0 * M * r * N


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def gemm_traffic_bytes(main="sint4"):
    """DRAM bytes of one step's GEMM launches as measured by ncu (profiles/gemm*_dram_traffic.json),
    or None when the GEMM source differs from the one that was profiled (or none was taken)."""
    import hashlib
    stem = "lq_gemm_mx" if main == "mxint4" else "lq_gemm"
    rec = os.path.join(ROOT, "profiles", "gemm_mx_dram_traffic.json" if main == "mxint4" else "gemm_dram_traffic.json")
    src = os.path.join(ROOT, "paper_2604_18117_b200", "csrc", stem + ".cu")
    try:
        d = json.load(open(rec))
        if hashlib.sha256(open(src, "rb").read()).hexdigest() != d[stem + "_cu_sha256"]:
            return None
        return int(d["dram_bytes_per_step"])
    except (OSError, KeyError, ValueError):
        return None


class ClockSampler:
    """Samples nvidia-smi clocks / throttle reasons while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows, self.proc, self.index = [], None, index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([t.strip() for t in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx = float(r[1])
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


def blas_threads() -> int:
    """Threads numpy's BLAS (the oracle's matmul) runs on; the rest of the oracle is single-threaded."""
    try:
        from threadpoolctl import threadpool_info
        n = [d.get("num_threads", 1) for d in threadpool_info() if d.get("user_api") == "blas"]
        return int(max(n)) if n else 1
    except Exception:
        return os.cpu_count() or 1


def build_workload(args):
    from paper_2604_18117_b200 import inputs as I
    wl = I.workload(args.config, branch=args.branch, rank=args.rank)
    return I, wl


def run_reference(args):
    """Reference arm: the CPU oracle as it stands, on a bounded row sample of the same layers."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import lq_oracle as O
    I, wl = build_workload(args)
    layers = []
    for spec in wl.layers:
        X, W, _ = I.layer_inputs(wl, spec, M=SAMPLE_ROWS)
        layer, _ = O.calibrate(W, wl.rank, wl.branch, steps=args.calib_steps, main=args.main)
        layers.append((spec, X, layer))
    ops_sample = sum(layer_ops(SAMPLE_ROWS, s.K, s.N, wl.rank) for s, _, _ in layers)
    for _ in range(args.warmup):
        for _, X, layer in layers:
            O.forward(X, layer)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        for _, X, layer in layers:
            O.forward(X, layer)
    dt = time.perf_counter() - t0
    value = ops_sample * args.steps / dt / 1e12
    cores = blas_threads()
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "impl": "reference", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(wl, args) | {"rows_per_step": SAMPLE_ROWS},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"{SAMPLE_ROWS} seeded rows of each of the {len(layers)} layers per step"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


MAIN_NAMES = {"sint4": "SINT4 group 64 (fp16 scales)", "mxint4": "MXINT4 block 32 (power-of-two scales)"}


def workload_config(wl, args):
    return {"workload": f"config{wl.config}: PixArt-class block linears (qkv 1152->3456, attn-out 1152->1152, "
                        f"fc1 1152->4608, fc2 4608->1152), M={wl.M} rows (4096 tokens x batch 2), rank {wl.rank}, "
                        f"main W4A4 {MAIN_NAMES[args.main]}, branch {wl.branch}" if wl.config in (1, 2) else f"config{wl.config}",
            "main": args.main, "rows": wl.M, "rank": wl.rank, "branch": wl.branch, "layers": [s.name for s in wl.layers],
            "calibration_steps": args.calib_steps,
            "l2": ("L2 flushed (256 MiB write) before every timed step; layers inside a step run back to back"
                   if args.l2 == "flush" else
                   "no explicit flush: one step reads 132 MB of X and writes 170 MB of Y plus 66 MB of codes, the L2 holds 126 MB"),
            "parallelism": f"rows sharded x{args.gpus}, no collective"}


def cpu_baseline(wl, I, args):
    """The oracle on this machine's host cores: 256 sampled rows per layer, all layers, repeated
    until about 10 s have passed."""
    from oracle import lq_oracle as O
    layers = []
    for spec in wl.layers:
        X, W, _ = I.layer_inputs(wl, spec, M=SAMPLE_ROWS)
        layer, _ = O.calibrate(W, wl.rank, wl.branch, steps=0, main=args.main)
        layers.append((spec, X, layer))
    ops = sum(layer_ops(SAMPLE_ROWS, s.K, s.N, wl.rank) for s, _, _ in layers)
    for _, X, layer in layers:
        O.forward(X, layer)
    n, t0 = 0, time.perf_counter()
    while True:
        for _, X, layer in layers:
            O.forward(X, layer)
        n += 1
        dt = time.perf_counter() - t0
        if dt > 10.0 or n >= 200:
            break
    return {"value": ops * n / dt / 1e12, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "sample": f"{SAMPLE_ROWS} seeded rows of each of the {len(layers)} layers, {n} passes in {dt:.1f} s "
                      f"(numpy/BLAS threads as configured on the box)"}


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2604_18117_b200 import binding as B
    from paper_2604_18117_b200 import build as BUILD

    from paper_2604_18117_b200 import dist_util as D
    world, rank, local = D.env_ranks()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device(f"cuda:{local}")
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    BUILD.build()
    I, wl = build_workload(args)
    M, r = wl.M, wl.rank
    st = torch.cuda.current_stream().cuda_stream

    layers = []
    for spec in wl.layers:
        Xh, W, bias = I.layer_inputs(wl, spec, seed=D.shard_seed(0, rank), with_bias=True)
        cfg = B.lq_config_default(spec.K, spec.N, r, wl.branch)
        cfg.steps = args.calib_steps
        if args.main == "mxint4":
            cfg.group = 32
        h, _ = B.lq_calibrate(cfg, W, bias)
        B.lq_layer_to_device(h, local)
        act = B.lq_act_create(h, M, local)
        Xd = torch.from_numpy(Xh).to(dev)
        Yd = torch.empty((M, spec.N), dtype=torch.float16, device=dev)
        Xp = torch.from_numpy(Xh).pin_memory()
        Yp = torch.empty((M, spec.N), dtype=torch.float16).pin_memory()
        layers.append(dict(spec=spec, h=h, act=act, Xd=Xd, Yd=Yd, Xp=Xp, Yp=Yp))
    ops_step = sum(layer_ops(M, L["spec"].K, L["spec"].N, r) for L in layers)
    gops_step = sum(gemm_ops(M, L["spec"].K, L["spec"].N, r) for L in layers)
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)

    def step(timed=None):
        if args.l2 == "flush":
            flush.zero_()
        if timed is not None:
            timed["s"].record()
        for i, L in enumerate(layers):
            if timed is not None:
                timed["q0"][i].record()
            B.lq_quantize_act(L["h"], L["Xd"].data_ptr(), M, L["act"], st)
            if timed is not None:
                timed["g0"][i].record()
            B.lq_linear_forward(L["h"], L["act"], L["Yd"].data_ptr(), B.OUT_F16, st)
            if timed is not None:
                timed["g1"][i].record()
        if timed is not None:
            timed["e"].record()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    ev = lambda: torch.cuda.Event(enable_timing=True)
    timers = [dict(s=ev(), e=ev(), q0=[ev() for _ in layers], g0=[ev() for _ in layers], g1=[ev() for _ in layers])
              for _ in range(args.steps)]
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        t_wait = time.perf_counter()          # nvidia-smi needs a moment before its first line: keep the GPU busy meanwhile
        while not sampler.rows and time.perf_counter() - t_wait < 3.0:
            step()
            torch.cuda.synchronize()
    barrier()
    n_before = len(sampler.rows)
    t_timed = time.perf_counter()
    for t in timers:
        step(t)
    barrier()
    timed_wall = time.perf_counter() - t_timed
    clocks = None
    if rank == 0:
        # The timed region of a short run is over before nvidia-smi (one line per 100 ms) reports: repeat the same
        # steps, untimed, until at least 1.5 s of this load have been sampled.
        extended = False
        while time.perf_counter() - t_timed < 1.5:
            extended = True
            step()
            torch.cuda.synchronize()
        sampler.rows = sampler.rows[n_before:]
        clocks = sampler.stop()
        clocks["window"] = (f"timed region of {timed_wall * 1e3:.0f} ms" +
                            (" plus untimed repeats of the same steps up to 1.5 s" if extended else ""))
    barrier()
    step_ms = [t["s"].elapsed_time(t["e"]) for t in timers]
    gemm_ms = [sum(a.elapsed_time(b) for a, b in zip(t["g0"], t["g1"])) for t in timers]
    quant_ms = [sum(a.elapsed_time(b) for a, b in zip(t["q0"], t["g0"])) for t in timers]
    per_layer = []
    for i, L in enumerate(layers):
        q = float(np.mean([t["q0"][i].elapsed_time(t["g0"][i]) for t in timers]))
        g = float(np.mean([t["g0"][i].elapsed_time(t["g1"][i]) for t in timers]))
        sp = L["spec"]
        per_layer.append({"layer": sp.name, "K": sp.K, "N": sp.N, "quantize_us": q * 1e3, "gemm_us": g * 1e3,
                          "gemm_tops": gemm_ops(M, sp.K, sp.N, r) / (g * 1e-3) / 1e12,
                          "pair_tops": layer_ops(M, sp.K, sp.N, r) / ((q + g) * 1e-3) / 1e12})
    total_ms = float(sum(step_ms))
    code, stage = B.lq_get_device_status(local)
    if code != 0:
        raise SystemExit(f"device status {code} (stage {stage}) after the timed region")
    total_ms_max = D.max_over_ranks(total_ms, world, dev)

    # end to end: pinned host X -> device -> K1 -> K2 -> pinned host Y, every step
    # one stream per layer: a layer's output travels to the host while the next layer's input travels to the device
    e2e_streams = [torch.cuda.Stream(device=dev) for _ in layers]

    def e2e_step():
        for L, es in zip(layers, e2e_streams):
            B.lq_linear_forward_host_async(L["h"], L["act"], L["Xp"].data_ptr(), M, L["Yp"].data_ptr(), B.OUT_F16, es.cuda_stream)
        for es in e2e_streams:
            es.synchronize()

    for _ in range(2):
        e2e_step()
    barrier()
    e2e_steps = max(3, min(args.steps, 10))
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    e2e_s = D.max_over_ranks(e2e_s, world, dev)

    if rank == 0:
        peaks = measured_peaks()
        peak_tops = 2.0 * peaks["bf16_tflops"]
        gemm_avg_ms = float(np.mean(gemm_ms))
        achieved = gops_step / (gemm_avg_ms * 1e-3) / 1e12
        # algorithmic bytes per row of the quantizer: X read once (2K); packed 4-bit codes (K/2), 8-bit branch
        # codes (K), fp16 group scales (2G), the per-token scale (4), r intermediate codes and their scale (4)
        # (MXINT4: one scale byte per block of 32 instead)
        sc_bytes = (lambda K: -(-K // 32)) if args.main == "mxint4" else (lambda K: 2 * (-(-K // 64)))
        k1_bytes = sum(M * (2 * L["spec"].K + L["spec"].K // 2 + L["spec"].K + sc_bytes(L["spec"].K) + 4 + r + 4)
                       for L in layers)
        quant_avg_ms = float(np.mean(quant_ms))
        line = {
            "metric": METRIC, "value": D.job_throughput(ops_step, args.steps, total_ms_max, world) / 1e12, "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": total_ms_max / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "e4m3 (exact int4 codes) / int8 operands, fp32 accumulate", "data": "synthetic",
            "config": workload_config(wl, args),
            "tokens_per_s": D.job_throughput(M, args.steps, total_ms_max, world),
            "e2e": {"value": D.job_throughput(ops_step, e2e_steps, e2e_s * 1e3, world) / 1e12, "unit": UNIT,
                    "h2d_bytes_per_step": int(sum(M * L["spec"].K * 2 for L in layers)),
                    "d2h_bytes_per_step": int(sum(M * L["spec"].N * 2 for L in layers)),
                    "ms_per_step": e2e_s / e2e_steps * 1e3},
            "gpu_launches": args.steps * len(layers) * (3 if wl.branch == "w16a16" else 2),
            "roofline": {"kernel": ("lq_gemm_mx_kernel" if args.main == "mxint4" else "lq_gemm_kernel") +
                                   " (4 launches per step, one per layer)", "bound": "tensor",
                         "achieved": achieved, "peak": peak_tops, "unit": "TOP/s", "frac": achieved / peak_tops,
                         "traffic": gemm_traffic_bytes(args.main), "traffic_note": "DRAM read + write bytes of the four GEMM "
                         "launches of one step from one ncu capture; null when the kernel source changed since",
                         "peak_source": f"2 x bf16_tflops ({peaks['bf16_tflops']}) of {peaks['source']}: 8-bit operands, "
                                        f"nominal ratio 2 to bf16",
                         "avg_launch_ms_sum": gemm_avg_ms},
            "roofline_quantizer": {"kernel": "lq_quant_kernel + down-projection", "bound": "hbm",
                                   "achieved": k1_bytes / (quant_avg_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                                   "unit": "GB/s", "frac": k1_bytes / (quant_avg_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                   "avg_ms_sum": quant_avg_ms},
            "layers": per_layer,
            "clocks": clocks,
        }
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = cpu_baseline(wl, I, args)
        print(json.dumps(line))
    for L in layers:
        B.lq_act_free(L["act"])
        B.lq_layer_free(L["h"])
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=1)
    ap.add_argument("--rank", type=int, default=32)
    ap.add_argument("--branch", default=None)
    ap.add_argument("--main", default="sint4", choices=["sint4", "mxint4"],
                    help="main-branch 4-bit format: sint4 = blocks of 64 with fp16 scales (the headline configuration), "
                         "mxint4 = blocks of 32 with power-of-two scales applied by the tensor core")
    ap.add_argument("--calib-steps", type=int, default=2, dest="calib_steps")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--l2", default="flush", choices=["flush", "working-set"],
                    help="flush: write 256 MiB before every step; working-set: rely on one step touching more than the L2 holds")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
