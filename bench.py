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
host Y out, one stream per layer, all synchronised at the end of the step: copies inside the timed region);
`roofline` describes the GEMM kernel against the 8-bit-operand tensor peak (2 x the measured bf16 cuBLAS burst peak),
with the fractions against the nominal and the sustained peak and against the composite bound
max(t_tensor, t_drain, t_HBM) per layer beside it; `mxint4` (default run only) is the same step with the MXINT4 main
branch; `cpu_baseline` is the CPU oracle timed on a 256-row sample of the same layers.  `--config 4` runs the whole
PixArt-class stack (28 blocks x 4 linears back to back, M = 32768, no L2 flush) and reports tokens/s.  With N > 1
(torchrun) every rank runs the same rows-sharded workload independently (rows are independent: no collective on the
data path).
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


NOMINAL_8BIT_TOPS = 4500.0      # dense 8-bit-operand class figure of the part (context, not the denominator of `frac`)
SMS, FP32_LANES, SM_MAX_HZ = 148, 128, 1.965e9
STACK_BLOCKS = 28
MXFP_RANK, MXFP_BRANCH = 64, "mxfp8"   # Table 3's MXFP8e4 row: rank 64 at the memory of an fp16 rank-32 branch
MXINT_RANK, MXINT_BRANCH = 64, "mxint8"   # Table 3's MXINT8 row
STUDY = {"mxfp4": (MXFP_RANK, MXFP_BRANCH), "mxint4a8": (MXINT_RANK, MXINT_BRANCH)}   # formats with a branch of their own


def layer_bounds(M, K, N, r, main, peaks):
    """Lower bounds (seconds) of one layer's two kernels from the algorithmic figures:
    K2 tensor: ops / (2 x bf16 burst); K2 drain (SINT4 only): 2 fp32 operations per output and group (G groups + the
    branch) on 128 lanes per SM at the maximum SM clock; K2 HBM: packed 4-bit codes, scales, branch codes in, fp16 Y
    out, weights once; K1 HBM: X in, codes and scales out."""
    mx = main in ("mxint4", "mxfp4", "mxint4a8")
    G = -(-K // (32 if mx else 64))
    sc = G if mx else 2 * G
    t_tensor = gemm_ops(M, K, N, r) / (2.0 * peaks["bf16_tflops"] * 1e12)
    t_drain = 0.0 if mx else 2.0 * M * N * (-(-K // 64) + (1 if r else 0)) / (SMS * FP32_LANES * SM_MAX_HZ)
    k2_bytes = M * (K // 2 + sc + r + 4) + 2 * M * N + (K * N // 2 + sc * N + r * N + 4 * N)
    # quantizer output: packed 4-bit codes + 8-bit branch codes (MXFP: ONE 8-bit code stream for both branches)
    k1_bytes = M * (2 * K + (K if main in ("mxfp4", "mxint4a8") else K // 2 + K) + sc + 4 + r + 4)
    t_hbm2 = k2_bytes / (peaks["hbm_gbs"] * 1e9)
    t_hbm1 = k1_bytes / (peaks["hbm_gbs"] * 1e9)
    return {"t_tensor_us": t_tensor * 1e6, "t_drain_us": t_drain * 1e6, "t_hbm_gemm_us": t_hbm2 * 1e6,
            "t_hbm_quant_us": t_hbm1 * 1e6, "gemm_bound_us": max(t_tensor, t_drain, t_hbm2) * 1e6, "k1_bytes": k1_bytes}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


TRAFFIC_RECORDS = {"mxint4a8": ("gemm_mxint4a8_dram_traffic.json", "lq_gemm_mx_kernel"), "sint4": ("gemm_dram_traffic.json", "lq_gemm_kernel"), "mxint4": ("gemm_mx_dram_traffic.json", "lq_gemm_mx_kernel"),
                   "mxfp4": ("gemm_mxfp_dram_traffic.json", "lq_gemm_mx_kernel")}


def gemm_traffic_bytes(main="sint4"):
    """DRAM bytes of one step's GEMM launches as measured by ncu (profiles/gemm*_dram_traffic.json, written by
    paper_2604_18117_b200.ncu_summary), or None when the kernel's sources differ from the ones that were profiled
    (or no capture was taken)."""
    from paper_2604_18117_b200.ncu_summary import sources_sha256
    name, kernel = TRAFFIC_RECORDS[main]
    try:
        d = json.load(open(os.path.join(ROOT, "profiles", name)))
        if d["kernel"] != kernel or d["sources_sha256"] != sources_sha256(kernel):
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


def oracle_layer(W, wl, args, steps):
    """(calibrated oracle layer, its forward, the rank it used) for the format --main names."""
    if args.main == "mxfp4":
        from oracle import lq_oracle_mxfp as OF
        layer, _ = OF.calibrate(W, MXFP_RANK, MXFP_BRANCH, steps=steps)
        return layer, OF.forward, MXFP_RANK
    if args.main == "mxint4a8":
        from oracle import lq_oracle_mxint as OI
        layer, _ = OI.calibrate(W, MXINT_RANK, MXINT_BRANCH, steps=steps)
        return layer, OI.forward, MXINT_RANK
    from oracle import lq_oracle as O
    layer, _ = O.calibrate(W, wl.rank, wl.branch, steps=steps, main=args.main)
    return layer, O.forward, wl.rank


def run_reference(args):
    """Reference arm: the CPU oracle as it stands, on a bounded row sample of the same layers."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    I, wl = build_workload(args)
    layers = []
    for spec in wl.layers:
        X, W, _ = I.layer_inputs(wl, spec, M=SAMPLE_ROWS)
        layer, fwd, r = oracle_layer(W, wl, args, args.calib_steps)
        layers.append((spec, X, layer))
    ops_sample = sum(layer_ops(SAMPLE_ROWS, s.K, s.N, r) for s, _, _ in layers)
    for _ in range(args.warmup):
        for _, X, layer in layers:
            fwd(X, layer)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        for _, X, layer in layers:
            fwd(X, layer)
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


MAIN_NAMES = {"sint4": "SINT4 group 64 (fp16 scales)", "mxint4": "MXINT4 block 32 (power-of-two scales)",
              "mxfp4": "MXFP4e2 weights x MXFP8e4 activations, block 32 (power-of-two scales)",
              "mxint4a8": "MXINT4 weights x MXINT8 activations, block 32 (power-of-two scales; 8-bit codes as two 4-bit digit planes)"}


def workload_config(wl, args):
    if args.main in STUDY:        # the mixed-precision study's formats have their own branch: rank and format of Table 3's rows
        import dataclasses
        wl = dataclasses.replace(wl, rank=STUDY[args.main][0], branch=STUDY[args.main][1])
    if wl.config in (1, 2):
        desc = (f"config{wl.config}: PixArt-class block linears (qkv 1152->3456, attn-out 1152->1152, fc1 1152->4608, "
                f"fc2 4608->1152), M={wl.M} rows (4096 tokens x batch 2), rank {wl.rank}, main W4A4 {MAIN_NAMES[args.main]}, "
                f"branch {wl.branch}")
    elif wl.config == 4:
        desc = (f"config4: full PixArt-class stack, {STACK_BLOCKS} blocks x (qkv, attn-out, fc1, fc2) run back to back, "
                f"M={wl.M} rows (batch 8 x 4096 tokens; the 2048px case, 16384 tokens x batch 2, has the same row count and "
                f"the same launches), rank {wl.rank}, main W4A4 {MAIN_NAMES[args.main]}, branch {wl.branch}; one calibrated "
                f"layer and one X / Y buffer per distinct shape, reused by all blocks; no L2 flush inside the stack")
    elif wl.config == 3:
        desc = (f"config3: SANA-class block linears (qkv 2240->6720, out 2240->2240, up 2240->5600, down 5600->2240), "
                f"M={wl.M} rows, rank {wl.rank}, main W4A4 {MAIN_NAMES[args.main]}, branch {wl.branch}")
    else:
        desc = f"config{wl.config}"
    return {"workload": desc,
            "main": args.main, "rows": wl.M, "rank": wl.rank, "branch": wl.branch, "layers": [s.name for s in wl.layers],
            "calibration_steps": args.calib_steps,
            "l2": ("no flush: one pass of the stack touches 112 x (X + codes + Y) = far more than the 126 MB L2; per-launch "
                   "times are those of the first block of each pass" if wl.config == 4 else
                   "L2 flushed (256 MiB write) before every timed step; layers inside a step run back to back"
                   if args.l2 == "flush" else
                   "no explicit flush: one step reads 132 MB of X and writes 170 MB of Y plus 66 MB of codes, the L2 holds 126 MB"),
            "timing": ("`value` and `ms_per_step`: K steps with one CUDA-event pair around each step and nothing between the "
                       "launches (launches overlap their set-up with the previous kernel's tail, as for a user); per-layer and "
                       "per-kernel times (`layers`, `roofline`): the same K steps repeated with events around every launch, "
                       "which serialises the launches - their step time is `ms_per_step_instrumented`"),
            "parallelism": f"rows sharded x{args.gpus}, no collective"}


def cpu_baseline(wl, I, args):
    """The oracle on this machine's host cores: 256 sampled rows per layer, all layers, repeated
    until about 10 s have passed."""
    layers = []
    for spec in wl.layers:
        X, W, _ = I.layer_inputs(wl, spec, M=SAMPLE_ROWS)
        layer, fwd, r = oracle_layer(W, wl, args, 0)
        layers.append((spec, X, layer))
    ops = sum(layer_ops(SAMPLE_ROWS, s.K, s.N, r) for s, _, _ in layers)
    for _, X, layer in layers:
        fwd(X, layer)
    n, t0 = 0, time.perf_counter()
    while True:
        for _, X, layer in layers:
            fwd(X, layer)
        n += 1
        dt = time.perf_counter() - t0
        if dt > 10.0 or n >= 200:
            break
    return {"value": ops * n / dt / 1e12, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "sample": f"{SAMPLE_ROWS} seeded rows of each of the {len(layers)} layers, {n} passes in {dt:.1f} s; the oracle is "
                      f"numpy: its matrix products run on `cores` BLAS threads, everything else (quantizers, scaling) on one"}


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
    # one process per node builds (a stale library would otherwise be rebuilt by every rank at once into the same files)
    if local == 0:
        BUILD.build()
    if world > 1:
        dist.barrier()
    I, wl = build_workload(args)
    M, r = wl.M, wl.rank
    st = torch.cuda.current_stream().cuda_stream
    stack = wl.config == 4
    repeats = STACK_BLOCKS if stack else 1           # the stack runs its four distinct layers 28 times back to back
    peaks = measured_peaks()
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def setup(main):
        layers = []
        for spec in wl.layers:
            Xh, W, bias = I.layer_inputs(wl, spec, seed=D.shard_seed(0, rank), with_bias=True)
            if main in STUDY:
                cfg = B.lq_config_default(spec.K, spec.N, *STUDY[main])
            else:
                cfg = B.lq_config_default(spec.K, spec.N, r, wl.branch)
            cfg.steps = args.calib_steps
            if main == "mxint4":
                cfg.group = 32
            h, _ = B.lq_calibrate(cfg, W, bias)
            B.lq_layer_to_device(h, local)
            act = B.lq_act_create(h, M, local)
            Xd = torch.from_numpy(Xh).to(dev)
            Yd = torch.empty((M, spec.N), dtype=torch.float16, device=dev)
            layers.append(dict(spec=spec, h=h, act=act, Xd=Xd, Yd=Yd, Xh=Xh))
        return layers

    def teardown(layers):
        for L in layers:
            B.lq_act_free(L["act"])
            B.lq_layer_free(L["h"])

    def measure(main, layers, steps, sample_clocks):
        """Device-resident timing: `steps` steps with one event pair around each step (this is `value`: nothing sits between
        the launches, so the library's overlapped launches work as they do for a user), then the same `steps` steps again
        with events around every launch (per-layer and per-kernel times; their own step time is reported beside)."""
        r = STUDY[main][0] if main in STUDY else wl.rank
        def step(timed=None):
            if args.l2 == "flush" and not stack:
                flush.zero_()
            if timed is not None:
                timed["s"].record()
            for rep in range(repeats):
                for i, L in enumerate(layers):
                    ev = timed is not None and rep == 0 and "q0" in timed
                    if ev:
                        timed["q0"][i].record()
                    B.lq_quantize_act(L["h"], L["Xd"].data_ptr(), M, L["act"], st)
                    if ev:
                        timed["g0"][i].record()
                    B.lq_linear_forward(L["h"], L["act"], L["Yd"].data_ptr(), B.OUT_F16, st)
                    if ev:
                        timed["g1"][i].record()
            if timed is not None:
                timed["e"].record()

        for _ in range(max(args.warmup, 3)):
            step()
        ev = lambda: torch.cuda.Event(enable_timing=True)
        timers = [dict(s=ev(), e=ev(), q0=[ev() for _ in layers], g0=[ev() for _ in layers], g1=[ev() for _ in layers])
                  for _ in range(steps)]
        sampler = ClockSampler(local)
        if rank == 0 and sample_clocks:
            sampler.start()
            t_wait = time.perf_counter()          # nvidia-smi needs a moment before its first line: keep the GPU busy meanwhile
            while not sampler.rows and time.perf_counter() - t_wait < 3.0:
                step()
                torch.cuda.synchronize()
        barrier()
        n_before = len(sampler.rows)
        t_timed = time.perf_counter()
        plain = [dict(s=ev(), e=ev()) for _ in range(steps)]
        for t in plain:
            step(t)
        barrier()
        timed_wall = time.perf_counter() - t_timed
        for t in timers:                          # the instrumented pass
            step(t)
        barrier()
        clocks = None
        if rank == 0 and sample_clocks:
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
        code, stage = B.lq_get_device_status(local)
        if code != 0:
            raise SystemExit(f"device status {code} (stage {stage}) after the timed region")
        step_ms = [t["s"].elapsed_time(t["e"]) for t in plain]
        step_ms_instrumented = float(np.mean([t["s"].elapsed_time(t["e"]) for t in timers]))
        per_layer = []
        for i, L in enumerate(layers):
            q = float(np.mean([t["q0"][i].elapsed_time(t["g0"][i]) for t in timers]))
            g = float(np.mean([t["g0"][i].elapsed_time(t["g1"][i]) for t in timers]))
            sp = L["spec"]
            bd = layer_bounds(M, sp.K, sp.N, r, main, peaks)
            per_layer.append({"layer": sp.name, "K": sp.K, "N": sp.N, "quantize_us": q * 1e3, "gemm_us": g * 1e3,
                              "gemm_tops": gemm_ops(M, sp.K, sp.N, r) / (g * 1e-3) / 1e12,
                              "pair_tops": layer_ops(M, sp.K, sp.N, r) / ((q + g) * 1e-3) / 1e12,
                              "bounds_us": {k: round(v, 2) for k, v in bd.items() if k.endswith("_us")},
                              "k1_bytes": bd["k1_bytes"]})
        total_ms_max = D.max_over_ranks(float(sum(step_ms)), world, dev)
        return {"total_ms": total_ms_max, "steps": steps, "layers": per_layer, "clocks": clocks,
                "ms_per_step_instrumented": step_ms_instrumented}

    def summarise(main, res):
        """value / roofline records of one measured format."""
        r = STUDY[main][0] if main in STUDY else wl.rank
        ops_step = repeats * sum(layer_ops(M, L["K"], L["N"], r) for L in res["layers"])
        gops_block = sum(gemm_ops(M, L["K"], L["N"], r) for L in res["layers"])
        gemm_ms = sum(L["gemm_us"] for L in res["layers"]) * 1e-3
        quant_ms = sum(L["quantize_us"] for L in res["layers"]) * 1e-3
        achieved = gops_block / (gemm_ms * 1e-3) / 1e12
        burst, sust = 2.0 * peaks["bf16_tflops"], 2.0 * (peaks["bf16_tflops_sustained"] or peaks["bf16_tflops"])
        bound_gemm_ms = sum(L["bounds_us"]["gemm_bound_us"] for L in res["layers"]) * 1e-3
        bound_quant_ms = sum(L["bounds_us"]["t_hbm_quant_us"] for L in res["layers"]) * 1e-3
        k1_bytes = sum(L["k1_bytes"] for L in res["layers"])
        kname = "lq_gemm_mx_kernel" if main in ("mxint4", "mxfp4", "mxint4a8") else "lq_gemm_kernel"
        roof = {"kernel": kname + " (one launch per layer)", "bound": "tensor",
                "achieved": achieved, "peak": burst, "unit": "TOP/s", "frac": achieved / burst,
                "traffic": gemm_traffic_bytes(main),
                "traffic_note": "DRAM read + write bytes of the four GEMM launches of one block from one ncu capture; null when "
                                "the kernel source changed since",
                "peak_source": f"2 x bf16_tflops ({peaks['bf16_tflops']}) of {peaks['source']}: 8-bit operands, nominal "
                               f"ratio 2 to bf16",
                "frac_of_nominal_4500": achieved / NOMINAL_8BIT_TOPS,
                "frac_of_2x_bf16_sustained": achieved / sust,
                "composite_bound": {"what": "sum over layers of max(t_tensor at 2 x bf16 burst, t_drain: 2 fp32 ops per output "
                                            "and group on 148 x 128 lanes at 1965 MHz (SINT4 only), t_HBM of the GEMM)",
                                    "bound_ms": bound_gemm_ms, "measured_ms": gemm_ms, "frac": bound_gemm_ms / gemm_ms},
                "pair_sum_of_bounds": {"what": "quantizer HBM bound + GEMM composite bound (the two kernels run one after "
                                               "the other)", "bound_ms": bound_gemm_ms + bound_quant_ms,
                                       "measured_ms": gemm_ms + quant_ms,
                                       "frac": (bound_gemm_ms + bound_quant_ms) / (gemm_ms + quant_ms)},
                "avg_launch_ms_sum": gemm_ms}
        roofq = {"kernel": "lq_quant_kernel (activation quantizer + down-projection, one launch per layer)", "bound": "hbm",
                 "achieved": k1_bytes / (quant_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                 "frac": k1_bytes / (quant_ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "avg_ms_sum": quant_ms}
        return {"value": D.job_throughput(ops_step, res["steps"], res["total_ms"], world) / 1e12,
                "ms_per_step": res["total_ms"] / res["steps"],
                "ms_per_step_instrumented": res["ms_per_step_instrumented"],
                "tokens_per_s": D.job_throughput(M, res["steps"], res["total_ms"], world),
                "roofline": roof, "roofline_quantizer": roofq}

    layers = setup(args.main)
    res = measure(args.main, layers, args.steps, True)
    summ = summarise(args.main, res)

    # end to end: pinned host X -> device -> K1 -> K2 -> pinned host Y, every step
    # one stream per layer: a layer's output travels to the host while the next layer's input travels to the device
    for L in layers:
        L["Xp"] = torch.from_numpy(L["Xh"]).pin_memory()
        L["Yp"] = torch.empty((M, L["spec"].N), dtype=torch.float16).pin_memory()
    e2e_streams = [torch.cuda.Stream(device=dev) for _ in layers]

    def e2e_step():
        for rep in range(repeats):
            for L, es in zip(layers, e2e_streams):
                B.lq_linear_forward_host_async(L["h"], L["act"], L["Xp"].data_ptr(), M, L["Yp"].data_ptr(), B.OUT_F16, es.cuda_stream)
        for es in e2e_streams:
            es.synchronize()

    for _ in range(1 if stack else 2):
        e2e_step()
    barrier()
    e2e_steps = 2 if stack else max(3, min(args.steps, 10))
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    e2e_s = D.max_over_ranks(e2e_s, world, dev)
    ops_step = repeats * sum(layer_ops(M, L["spec"].K, L["spec"].N, STUDY[args.main][0] if args.main in STUDY else r) for L in layers)
    specs = [L["spec"] for L in layers]
    teardown(layers)

    mx = None
    if args.main == "sint4" and wl.config == 1 and not args.no_mxint4:
        # the same step with the MXINT4 main branch (Table 2's format), whose block scales the tensor core applies itself
        mx_layers = setup("mxint4")
        mx_res = measure("mxint4", mx_layers, args.steps, True)
        mx_s = summarise("mxint4", mx_res)
        mx = {"what": "the same step with the MXINT4 main branch (blocks of 32, power-of-two scales, tcgen05 block-scaled MMA)",
              "value": mx_s["value"], "unit": UNIT, "ms_per_step": mx_s["ms_per_step"], "ms_per_step_instrumented": mx_s["ms_per_step_instrumented"], "tokens_per_s": mx_s["tokens_per_s"],
              "roofline": mx_s["roofline"], "roofline_quantizer": mx_s["roofline_quantizer"], "layers": mx_res["layers"],
              "clocks": mx_res["clocks"]}
        teardown(mx_layers)
    fp = None
    if args.main == "sint4" and wl.config == 1 and not args.no_mxint4:
        # and with the MXFP formats of the mixed-precision study (Tables 3-4): MXFP4e2 weights, MXFP8e4 activations for
        # both branches, MXFP8e4 factors of rank 64; every scale is applied by the tensor core
        fp_layers = setup("mxfp4")
        fp_res = measure("mxfp4", fp_layers, args.steps, True)
        fp_s = summarise("mxfp4", fp_res)
        fp = {"what": f"the same layer shapes with MXFP4e2 residual weights, MXFP8e4 activations and a rank-{MXFP_RANK} {MXFP_BRANCH} branch",
              "value": fp_s["value"], "unit": UNIT, "ms_per_step": fp_s["ms_per_step"], "ms_per_step_instrumented": fp_s["ms_per_step_instrumented"], "tokens_per_s": fp_s["tokens_per_s"],
              "roofline": fp_s["roofline"], "roofline_quantizer": fp_s["roofline_quantizer"], "layers": fp_res["layers"],
              "clocks": fp_res["clocks"]}
        teardown(fp_layers)
    i8 = None
    if args.main == "sint4" and wl.config == 1 and not args.no_mxint4:
        # and the study's integer row: MXINT4 weights, MXINT8 activations for both branches (two digit planes per 8-bit
        # code, so the kernel issues twice the MMAs the op count credits), MXINT8 factors of rank 64
        i8_layers = setup("mxint4a8")
        i8_res = measure("mxint4a8", i8_layers, args.steps, True)
        i8_s = summarise("mxint4a8", i8_res)
        i8 = {"what": f"the same layer shapes with MXINT4 residual weights, MXINT8 activations and a rank-{MXINT_RANK} {MXINT_BRANCH} branch",
              "value": i8_s["value"], "unit": UNIT, "ms_per_step": i8_s["ms_per_step"], "ms_per_step_instrumented": i8_s["ms_per_step_instrumented"], "tokens_per_s": i8_s["tokens_per_s"],
              "roofline": i8_s["roofline"], "roofline_quantizer": i8_s["roofline_quantizer"], "layers": i8_res["layers"],
              "clocks": i8_res["clocks"]}
        teardown(i8_layers)

    if rank == 0:
        nl = len(specs)
        line = {
            "metric": METRIC, "value": summ["value"], "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": summ["ms_per_step"], "ms_per_step_instrumented": summ["ms_per_step_instrumented"],
            "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "e4m3 (exact int4 codes) / int8 operands, fp32 accumulate", "data": "synthetic",
            "config": workload_config(wl, args),
            "tokens_per_s": summ["tokens_per_s"],
            "e2e": {"value": D.job_throughput(ops_step, e2e_steps, e2e_s * 1e3, world) / 1e12, "unit": UNIT,
                    "h2d_bytes_per_step": int(repeats * sum(M * sp.K * 2 for sp in specs)),
                    "d2h_bytes_per_step": int(repeats * sum(M * sp.N * 2 for sp in specs)),
                    "ms_per_step": e2e_s / e2e_steps * 1e3},
            "gpu_launches": args.steps * repeats * nl * 2 * (1 + (mx is not None) + (fp is not None) + (i8 is not None)),
            "roofline": summ["roofline"],
            "roofline_quantizer": summ["roofline_quantizer"],
            "layers": res["layers"],
            "clocks": res["clocks"],
        }
        if mx is not None:
            line["mxint4"] = mx
        if fp is not None:
            line["mxfp4"] = fp
        if i8 is not None:
            line["mxint4a8"] = i8
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = cpu_baseline(wl, I, args)
        print(json.dumps(line))
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
    ap.add_argument("--main", default="sint4", choices=["sint4", "mxint4", "mxfp4", "mxint4a8"],
                    help="main-branch 4-bit format: sint4 = blocks of 64 with fp16 scales (the headline configuration), "
                         "mxint4 = blocks of 32 with power-of-two scales applied by the tensor core")
    ap.add_argument("--calib-steps", type=int, default=2, dest="calib_steps")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-mxint4", action="store_true", dest="no_mxint4",
                    help="leave out the MXINT4 sub-record that the default (config 1, sint4) run adds")
    ap.add_argument("--l2", default="flush", choices=["flush", "working-set"],
                    help="flush: write 256 MiB before every step; working-set: rely on one step touching more than the L2 holds")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
