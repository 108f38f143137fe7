#!/usr/bin/env python
"""Benchmark of the CWAC hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4|cfg1|cfg2|cfg3|rn50|cfg5] [--impl ours|reference]

A *step* is one pass of the whole hot path over one batch of synthetic input:
  phase A  for every layer of the workload: CWAC statistics + closed-form solve on the layer's calibration
           pair and the fold (qwt_cwac_calibrate_batch, or qwt_cwac_calibrate + qwt_cwac_fold per layer);
  phase B  for every layer: the CWAC-fused quantized linear forward (qwt_qlinear_cwac_forward).
`value` is the GEMM throughput of phase B (2*M*N*K operations per layer / phase-B device time, TOPS);
the calibration half of the metric (8 bytes per row and channel / phase-A device time, GB/s) is in
`calibration`.  `ms_per_step` covers both phases.  All inputs are resident in HBM before the timed
region; `e2e` repeats phase B through the host-buffer entry point with the copies inside the timing and
`e2e_calibration` does the same for the fit (qwt_cwac_calibrate_host).

The headline workload is the tensor-bound one (config 4, the LLaMA-7B shaped layers); on one GPU the same line
carries, in `per_config`, the same two figures with their roofline fractions for every other workload
(configs 1, 2, 3, the ResNet-50 shaped pointwise convolutions, and the calibration sweep of config 5),
each measured on its own full shapes with fewer steps.  Prints ONE JSON line on rank 0.

With --gpus N > 1 and no torchrun environment the script starts the N ranks itself (one process per GPU,
rendezvous on 127.0.0.1); every rank runs its own copy of the workload (row shards, no collective).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "CWAC-fused W8A8 GEMM TOPS & % INT8 peak; calibration GB/s & % HBM peak"
UNIT = "TOPS"

# Fallback peaks of this B200 pool when MEASURED_PEAKS.json is absent.
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
INT8_OVER_BF16 = 2.0      # nominal dense ratio (4.5 POPS int8 : 2.25 PFLOPS bf16)

# DRAM bytes moved per algorithmic byte, per kernel and workload, from ncu captures: a small tracked table whose rows
# name the summary under profiles/ they were read from and the hash of the kernel source at capture time.
TRAFFIC_TABLE = os.path.join(ROOT, "paper_2505_20932_b200", "ncu_traffic.json")
CSRC = os.path.join(ROOT, "paper_2505_20932_b200", "csrc")


def source_hash(files):
    h = hashlib.sha256()
    for f in files:
        with open(os.path.join(CSRC, f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def traffic_ratio(key):
    """(ratio, provenance) for `key`, or (None, why) when there is no capture or the kernel source has changed since."""
    try:
        with open(TRAFFIC_TABLE) as f:
            row = json.load(f)[key]
    except (OSError, KeyError, ValueError):
        return None, "no ncu capture recorded for this kernel and workload"
    if row.get("source_sha") != source_hash(row["source_files"]):
        return None, f"kernel source changed since the capture in {row['profile']}"
    return float(row["dram_bytes_per_algorithmic_byte"]), row["profile"]


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": FALLBACK_BF16_TFLOPS,
            "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# --------------------------------------------------------------------------------------------- clocks

class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake_slowdown",
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop_evt.wait(self.period)

    def stop(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2)
        return {"sm_mhz": (statistics.median(self.samples) if self.samples else None),
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# --------------------------------------------------------------------------------------------- workload on the device

class Layer:
    """Device-resident state of one quantized linear layer (inputs, parameters, outputs, scratch)."""
    pass


def _quant_rows(B, torch, X, qmax):
    r, c = X.shape
    q = torch.empty((r, c), dtype=torch.int8, device=X.device)
    s = torch.empty(r, dtype=torch.float32, device=X.device)
    B.qwt_quantize_rows_i8(X, r, c, c, qmax, q, s)
    return q, s


def build_layer(B, torch, WL, spec, seed, device, calib_rows=None, keep_calib_inputs=False):
    L = Layer()
    L.spec = spec
    M, K, N = spec.M, spec.K, spec.N
    R = spec.calib_rows if calib_rows is None else calib_rows
    L.R = R
    L.wfmt = B.QWT_W_INT8 if spec.w_bits == 8 else B.QWT_W_INT4_PACKED
    L.out_mode = B.QWT_OUT_INT8_PER_TOKEN if spec.out == "int8" else B.QWT_OUT_BF16
    X = WL.device_activations(spec.act, M, K, seed, spec.name + "|infer", device)
    L.Xq, L.xs = _quant_rows(B, torch, X, 127)
    del X
    W = WL.device_weights(N, K, seed, spec.name, device=device)
    qmax = 127 if spec.w_bits == 8 else 7
    Wq, L.ws = _quant_rows(B, torch, W, qmax)
    if spec.w_bits == 4:
        L.W = torch.empty((N, K // 2), dtype=torch.uint8, device=device)
        B.qwt_pack_int4(Wq, N, K, L.W)
    else:
        L.W = Wq
    g = torch.Generator(device=device)
    g.manual_seed(seed * 7919 + 13)
    L.bias = torch.randn(N, generator=g, device=device) * 0.01
    # calibration pair (Section 3.3): Y_full and Y_quant of the same calibration tokens
    Xc = WL.device_activations(spec.act, R, K, seed, spec.name + "|calib", device)
    Xcq, xcs = _quant_rows(B, torch, Xc, 127)
    L.q_out = torch.empty((R, N), dtype=torch.float32, device=device)
    wsb = B.qwt_qlinear_workspace_bytes(R, N, K, L.wfmt, B.QWT_OUT_FP32)
    ws = torch.empty(max(wsb, 256), dtype=torch.uint8, device=device)
    B.qwt_qlinear_cwac_forward(Xcq, xcs, L.W, L.wfmt, L.ws, L.bias, R, N, K, B.QWT_OUT_FP32, L.q_out, None, ws, wsb)
    B.qwt_qlinear_check_status(ws)
    if spec.planted:
        a_star, b_star = WL.host_planted_cwac(N, seed, spec.name)
        a_s, b_s = torch.from_numpy(a_star).to(device), torch.from_numpy(b_star).to(device)
        L.fp_out = L.q_out * a_s[None, :] + b_s[None, :]
        sd = L.q_out[: min(R, 4096)].std(dim=0)
        L.fp_out += torch.randn((R, N), generator=g, device=device) * (0.01 * sd)[None, :]
    else:
        L.fp_out = torch.addmm(L.bias, Xc, W.t())
    # the quantized calibration inputs of the first layers are kept for the in-layer calibration figure
    L.Xcq, L.xcs = (Xcq, xcs) if keep_calib_inputs else (None, None)
    del Xc, Xcq, xcs, W
    L.a = torch.empty(N, dtype=torch.float32, device=device)
    L.b = torch.empty(N, dtype=torch.float32, device=device)
    L.fs = torch.empty(N, dtype=torch.float32, device=device)
    L.fb = torch.empty(N, dtype=torch.float32, device=device)
    L.cws_bytes = B.qwt_cwac_workspace_bytes(R, N)
    L.cws = torch.empty(max(L.cws_bytes, 256), dtype=torch.uint8, device=device)
    ydt = torch.int8 if spec.out == "int8" else torch.bfloat16
    L.Y = torch.empty((M, N), dtype=ydt, device=device)
    L.ys = torch.empty(M, dtype=torch.float32, device=device) if spec.out == "int8" else None
    L.fws_bytes = B.qwt_qlinear_workspace_bytes(M, N, K, L.wfmt, L.out_mode)
    L.fws = torch.empty(max(L.fws_bytes, 256), dtype=torch.uint8, device=device)
    L.calib_bytes = 8 * R * N
    out_b = 1 if spec.out == "int8" else 2
    wb = K if spec.w_bits == 8 else K // 2
    L.fwd_bytes = M * K + N * wb + M * N * out_b + 4 * M + 8 * N + (4 * M if spec.out == "int8" else 0)
    return L


class CalibBatch:
    """All layers' calibration problems (with their folds) for the batched entry point, and its workspace."""

    def __init__(self, B, layers, device):
        import torch
        self.probs = B.calib_problems((L.fp_out, L.q_out, L.R, L.spec.N, L.spec.N, L.a, L.b, L.ws, L.bias, L.fs, L.fb)
                                      for L in layers)
        self.wsb = B.qwt_cwac_calibrate_batch_workspace_bytes(self.probs)
        self.ws = torch.empty(max(self.wsb, 256), dtype=torch.uint8, device=device)
        self.groups = (len(layers) + 47) // 48        # launches of the statistics kernel per call


def phase_a(B, layers, stream, side=None, batch=None):
    """Calibrate + fold every layer: one batched call (statistics of all layers in one launch, reduce + solve + fold
    in a second), or layer by layer.  Layer by layer the independent layers alternate over two streams when `side` is
    given: the small solve / fold kernels of one layer then run under the next layer's statistics pass."""
    if batch is not None:
        B.qwt_cwac_calibrate_batch(batch.probs, None, batch.ws, batch.wsb, stream)
        return
    if side is not None:
        side.wait_stream(stream)
    for i, L in enumerate(layers):
        s = L.spec
        st = stream if (side is None or i % 2 == 0) else side
        B.qwt_cwac_calibrate(L.fp_out, L.q_out, L.R, s.N, s.N, L.a, L.b, None, L.cws, L.cws_bytes, st)
        B.qwt_cwac_fold(L.ws, L.bias, L.a, L.b, s.N, L.fs, L.fb, st)
    if side is not None:
        stream.wait_stream(side)


def phase_b(B, layers, stream, sides=()):
    """Fused forward of every layer; like phase A the independent layers may be dealt over several streams, so
    that one call's launch latency and tail run under its neighbours."""
    lanes = [stream] + list(sides)
    for sd in sides:
        sd.wait_stream(stream)
    for i, L in enumerate(layers):
        s = L.spec
        B.qwt_qlinear_cwac_forward(L.Xq, L.xs, L.W, L.wfmt, L.fs, L.fb, s.M, s.N, s.K, L.out_mode, L.Y, L.ys,
                                   L.fws, L.fws_bytes, lanes[i % len(lanes)])
    for sd in sides:
        stream.wait_stream(sd)


def workload_layers(WL, name):
    if name == "cfg1":
        return WL.config_layers(1), "config 1: single W8A8 layer 788x384->1536, CWAC fit on 32 images"
    if name == "cfg2":
        return WL.config_layers(2), "config 2: DeiT-S W8A8 stack, 12 blocks x (qkv, proj, fc1, fc2), batch 64x197 tokens, CWAC fit per layer on 512 images"
    if name == "cfg3":
        return WL.config_layers(3), "config 3: ViT-B W4A8 stack, 12 blocks, batch 128x197 tokens, BF16 out, CWAC fit on 1024 images"
    if name == "cfg4":
        return WL.config_layers(4), "config 4: LLaMA-7B shaped W8A8 layers at M=2048 and 8192, CWAC planted and refit from 128x2048 tokens"
    if name == "rn50":
        return WL.resnet50_pointwise_layers(), "ResNet-50 shaped pointwise convolutions (first and last 1x1 convolution of a bottleneck in each of the four stages, NHWC: M = 32 x H x W pixels), W8A8, CWAC fit on 32 images"
    raise ValueError(name)


# --------------------------------------------------------------------------------------------- CPU oracle timing

def oracle_block_time(layers_host, calib_rows_cap):
    """Times the oracle (as it stands) on host copies of a few layers.  Returns (fwd_ops, fwd_s, cal_bytes, cal_s)."""
    from oracle import qwt_oracle as O
    fwd_ops = cal_bytes = 0
    fwd_s = cal_s = 0.0
    for h in layers_host:
        t0 = time.perf_counter()
        a, b, _ = O.cwac_fit(h["fp_out"], h["q_out"])
        fs, fb = O.cwac_fold(h["ws"], h["bias"], a, b)
        t1 = time.perf_counter()
        acc = O.int_matmul(h["Xq"], h["Wq"])
        z = O.forward_folded(acc, h["xs"], fs, fb)
        if h["out"] == "int8":
            O.requant_per_token(z)
        else:
            O.to_bf16_bits(z)
        t2 = time.perf_counter()
        cal_s += t1 - t0
        fwd_s += t2 - t1
        cal_bytes += 8 * h["fp_out"].shape[0] * h["fp_out"].shape[1]
        fwd_ops += 2 * h["Xq"].shape[0] * h["Wq"].shape[0] * h["Xq"].shape[1]
    return fwd_ops, fwd_s, cal_bytes, cal_s


def host_copy_of_layer(L, rows_cap, calib_cap, O=None):
    from oracle import qwt_oracle as Or
    s = L.spec
    m = min(s.M, rows_cap)
    r = min(L.R, calib_cap)
    W = L.W.cpu().numpy()
    if s.w_bits == 4:
        W = Or.unpack_int4(W)
    return {"Xq": L.Xq[:m].cpu().numpy(), "xs": L.xs[:m].cpu().numpy(), "Wq": W, "ws": L.ws.cpu().numpy(),
            "bias": L.bias.cpu().numpy(), "fp_out": L.fp_out[:r].cpu().numpy(), "q_out": L.q_out[:r].cpu().numpy(),
            "out": s.out}


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


# --------------------------------------------------------------------------------------------- reference arm

def run_reference(args):
    """Times the CPU oracle on the host cores: each step = a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from oracle import qwt_oracle as O
    from paper_2505_20932_b200 import workload as WL
    specs, desc = workload_layers(WL, args.workload)
    specs = specs[:4]
    rows_cap, calib_cap = 1024, 8192
    hosts = []
    for sp in specs:
        m, r = min(sp.M, rows_cap), min(sp.calib_rows, calib_cap)
        d = WL.host_layer_inputs(sp, seed=args.seed, rows=m, calib_rows=r)
        qmax = 127 if sp.w_bits == 8 else 7
        Xq, xs = O.quantize_rows_sym(d["X"], 127)
        Wq, ws = O.quantize_rows_sym(d["W"], qmax)
        Xcq, xcs = O.quantize_rows_sym(d["Xc"], 127)
        q_out = O.dequant(O.int_matmul(Xcq, Wq), xcs, ws, d["bias"]).astype(np.float32)
        if sp.planted:
            fp_out = (q_out * d["a_star"] + d["b_star"]).astype(np.float32)
        else:
            fp_out = O.linear_fp(d["Xc"], d["W"], d["bias"]).astype(np.float32)
        hosts.append({"Xq": Xq, "xs": xs, "Wq": Wq, "ws": ws, "bias": d["bias"], "fp_out": fp_out, "q_out": q_out,
                      "out": sp.out})
    for _ in range(args.warmup):
        oracle_block_time(hosts, calib_cap)
    t_f = t_c = 0.0
    t0 = time.perf_counter()
    for _ in range(args.steps):
        ops, fs_, cb, cs_ = oracle_block_time(hosts, calib_cap)
        t_f += fs_
        t_c += cs_
    total = time.perf_counter() - t0
    value = ops * args.steps / t_f / 1e12
    sample = (f"first {len(specs)} layers of the workload, first {rows_cap} tokens (forward) and first {calib_cap} "
              f"calibration rows (fit) of each, per step")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": total / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": desc, "l2": "n/a (CPU)"},
        "calibration": {"value": cb * args.steps / t_c / 1e9, "unit": "GB/s"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# --------------------------------------------------------------------------------------------- our arm

class Ctx:
    """What every measurement needs: the binding, torch, the workload module, the process group and the peaks."""
    pass


def make_ctx():
    import torch
    import torch.distributed as dist

    from paper_2505_20932_b200 import binding as B     # raises if libqwt2.so is missing: no fallback
    from paper_2505_20932_b200 import workload as WL
    c = Ctx()
    c.torch, c.dist, c.B, c.WL = torch, dist, B, WL
    c.world = int(os.environ.get("WORLD_SIZE", "1"))
    c.rank = int(os.environ.get("RANK", "0"))
    c.local = int(os.environ.get("LOCAL_RANK", "0"))
    if c.world > 1:
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{c.local}"))
    torch.cuda.set_device(c.local)
    c.device = f"cuda:{c.local}"
    torch.backends.cuda.matmul.allow_tf32 = False
    c.peaks = load_peaks()
    c.int8_peak = c.peaks["bf16_tflops"] * INT8_OVER_BF16
    c.int8_peak_sus = c.peaks["bf16_tflops_sustained"] * INT8_OVER_BF16
    c.stream = torch.cuda.current_stream()
    return c


def barrier(c):
    c.torch.cuda.synchronize()
    if c.world > 1:
        c.dist.barrier()
    c.torch.cuda.synchronize()


def max_over_ranks(c, values):
    t = c.torch.tensor(values, dtype=c.torch.float64, device=c.device)
    if c.world > 1:
        c.dist.all_reduce(t, op=c.dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def measure_layers(c, args, specs, steps, warmup, calib_cap, keep_calib_inputs=0, sampler=None):
    """Builds the layers of one workload on the device and times `steps` steps (phase A, phase B) of it.
    Returns (result dict, layers).  Times are the maximum over ranks of the CUDA-event durations."""
    torch, B, WL = c.torch, c.B, c.WL
    layers = [build_layer(B, torch, WL, sp, args.seed + 1000 * c.rank + i, c.device,
                          calib_rows=(min(sp.calib_rows, calib_cap) if calib_cap else None),
                          keep_calib_inputs=(c.rank == 0 and i < keep_calib_inputs))
              for i, sp in enumerate(specs)]
    torch.cuda.synchronize()
    stream = c.stream
    batch = None if args.calibration == "per-layer" else CalibBatch(B, layers, c.device)
    for _ in range(warmup):
        phase_a(B, layers, stream, batch=batch)
        phase_b(B, layers, stream)
    for L in layers:
        if L.fws_bytes:
            B.qwt_qlinear_check_status(L.fws)
    barrier(c)

    # The library calls of each phase are recorded once into a CUDA graph (stream capture) and replayed per
    # step, so that the timed region holds the device work and not the host's per-call launch overhead.
    graphs = None
    launches_per_step = None
    if not args.no_graph:
        cap = torch.cuda.Stream()
        cap.wait_stream(stream)
        graphs = []
        B.qwt_launch_count_reset()
        sides = [torch.cuda.Stream() for _ in range(3)]
        with torch.cuda.stream(cap):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=cap):
                phase_a(B, layers, cap, sides[0], batch=batch)
            graphs.append(g)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=cap):
                phase_b(B, layers, cap, sides[: args.forward_streams - 1])
            graphs.append(g)
        launches_per_step = B.qwt_launch_count()      # launches recorded = launches per replayed step
        stream.wait_stream(cap)
        for g in graphs:                               # one untimed replay
            g.replay()
        barrier(c)

    if sampler is not None:
        sampler.start()                                 # clocks are sampled during the timed region only
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    B.qwt_launch_count_reset()
    for k in range(steps):
        ev[k][0].record(stream)
        if graphs is None:
            phase_a(B, layers, stream, batch=batch)
        else:
            graphs[0].replay()
        ev[k][1].record(stream)
        if graphs is None:
            phase_b(B, layers, stream)
        else:
            graphs[1].replay()
        ev[k][2].record(stream)
    barrier(c)
    clocks = sampler.stop() if sampler is not None else None
    launches = B.qwt_launch_count() if graphs is None else launches_per_step * steps
    t_a = sum(e[0].elapsed_time(e[1]) for e in ev) * 1e-3
    t_b = sum(e[1].elapsed_time(e[2]) for e in ev) * 1e-3
    t_all = ev[0][0].elapsed_time(ev[-1][2]) * 1e-3
    for L in layers:
        B.qwt_qlinear_check_status(L.fws)
    t_a, t_b, t_all = max_over_ranks(c, [t_a, t_b, t_all])
    r = {"t_a": t_a, "t_b": t_b, "t_all": t_all, "steps": steps, "launches": int(launches), "clocks": clocks,
         "fwd_ops": sum(L.spec.ops for L in layers), "cal_bytes": sum(L.calib_bytes for L in layers),
         "fwd_bytes": sum(L.fwd_bytes for L in layers), "n_layers": len(layers),
         "cal_launches_per_step": (len(layers) if batch is None else batch.groups), "batched": batch is not None}
    del graphs, batch
    return r, layers


def forward_roofline(c, r, key):
    """Phase B against min(tensor roof, HBM roof) of the workload's own operations and algorithmic bytes."""
    p = c.peaks
    tops = r["fwd_ops"] * r["steps"] / r["t_b"] / 1e12                    # per GPU
    t_min_compute = r["fwd_ops"] / (c.int8_peak * 1e12)
    t_min_hbm = r["fwd_bytes"] / (p["hbm_gbs"] * 1e9)
    ratio, prov = traffic_ratio(key)
    n_launch = r["n_layers"] * r["steps"]
    roof = {"kernel": "qlinear_cwac_kernel", "launches": n_launch, "avg_launch_ms": r["t_b"] / n_launch * 1e3,
            "algorithmic_bytes_per_launch": r["fwd_bytes"] / r["n_layers"],
            "algorithmic_ops_per_launch": r["fwd_ops"] / r["n_layers"],
            "traffic": None if ratio is None else ratio * r["fwd_bytes"] / r["n_layers"], "traffic_source": prov,
            "min_time_ms_tensor": t_min_compute * 1e3, "min_time_ms_hbm": t_min_hbm * 1e3,
            "frac_of_roofline": max(t_min_compute, t_min_hbm) / (r["t_b"] / r["steps"])}
    if t_min_compute >= t_min_hbm:
        roof.update({"bound": "tensor", "achieved": tops, "peak": c.int8_peak, "unit": "TOP/s", "frac": tops / c.int8_peak,
                     "peak_source": f"2 x bf16 burst, of {p['source']}", "frac_of_sustained": tops / c.int8_peak_sus})
    else:
        ach = r["fwd_bytes"] * r["steps"] / r["t_b"] / 1e9
        roof.update({"bound": "hbm", "achieved": ach, "peak": p["hbm_gbs"], "unit": "GB/s", "frac": ach / p["hbm_gbs"],
                     "peak_source": f"of {p['source']}", "tensor_frac": tops / c.int8_peak})
    return tops, roof


def calibration_roofline(c, r, key):
    p = c.peaks
    n_launch = r["cal_launches_per_step"] * r["steps"]
    per_launch = r["cal_bytes"] * r["steps"] / n_launch
    ach = r["cal_bytes"] * r["steps"] / r["t_a"] / 1e9                     # per GPU
    ratio, prov = traffic_ratio(key)
    return ach, {"kernel": "cwac_stats_batch_kernel" if r["batched"] else "cwac_stats_kernel", "bound": "hbm",
                 "achieved": ach, "peak": p["hbm_gbs"], "unit": "GB/s", "frac": ach / p["hbm_gbs"],
                 "peak_source": f"copy (read + write), of {p['source']}",
                 "traffic": None if ratio is None else ratio * per_launch, "traffic_source": prov,
                 "algorithmic_bytes_per_launch": per_launch, "launches": n_launch,
                 "avg_launch_ms": r["t_a"] / n_launch * 1e3,
                 "note": ("duration = phase A (one statistics launch for all layers + one reduce/solve/fold launch) / launches"
                          if r["batched"] else "duration = phase A (stats + reduce/solve + fold kernels of every layer) / launches")}


def read_only_hbm_gbs(c):
    """A read-only stream over 4 GiB (the library's sum reduction), best of 5: a second denominator for the statistics
    pass, which only reads, beside the read + write copy figure of the measured peaks."""
    torch = c.torch
    try:
        x = torch.empty(1 << 30, dtype=torch.float32, device=c.device).fill_(1.0)
        for _ in range(2):
            x.sum()
        best = None
        for _ in range(5):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            x.sum()
            e1.record()
            torch.cuda.synchronize()
            t = e0.elapsed_time(e1) * 1e-3
            best = t if best is None else min(best, t)
        return x.numel() * 4 / best / 1e9
    except Exception:
        return None


def e2e_forward(c, layers, steps):
    """Phase B through the host-buffer entry point: pinned host X / x_scale in, host Y / y_scale out, per layer."""
    torch, B = c.torch, c.B
    host = []
    for L in layers:
        s = L.spec
        hx = torch.empty((s.M, s.K), dtype=torch.int8).pin_memory()
        hx.copy_(L.Xq)
        hxs = L.xs.cpu().pin_memory()
        hy = torch.empty(L.Y.shape, dtype=L.Y.dtype).pin_memory()
        hys = torch.empty(s.M, dtype=torch.float32).pin_memory() if L.ys is not None else None
        sb = B.qwt_qlinear_host_staging_bytes(s.M, s.N, s.K, L.wfmt, L.out_mode)
        host.append((hx, hxs, hy, hys, sb))
    sb_max = max(h[4] for h in host)
    staging = torch.empty(sb_max, dtype=torch.uint8, device=c.device)

    def one_pass():
        for L, (hx, hxs, hy, hys, sb) in zip(layers, host):
            s = L.spec
            B.qwt_qlinear_cwac_forward_host(hx.data_ptr(), hxs.data_ptr(), L.W, L.wfmt, L.fs, L.fb, s.M, s.N, s.K,
                                            L.out_mode, hy.data_ptr(), None if hys is None else hys.data_ptr(),
                                            staging, sb_max, c.stream)
    one_pass()
    barrier(c)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n = max(1, min(steps, 5))
    e0.record(c.stream)
    for _ in range(n):
        one_pass()
    e1.record(c.stream)
    barrier(c)
    (t,) = max_over_ranks(c, [e0.elapsed_time(e1) * 1e-3])
    h2d = sum(h[0].numel() + h[1].numel() * 4 for h in host)
    d2h = sum(h[2].numel() * h[2].element_size() + (h[3].numel() * 4 if h[3] is not None else 0) for h in host)
    ops = sum(L.spec.ops for L in layers)
    return {"value": c.world * ops * n / t / 1e12, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "steps": n,
            "what": "phase B through qwt_qlinear_cwac_forward_host: pinned host X/x_scale in, host Y/y_scale out, per layer"}


def e2e_calibration(c, layers, max_bytes=3 << 30):
    """The fit through the host-matrix entry point (qwt_cwac_calibrate_host): pinned host fp_out / q_out streamed to
    the device in chunks while earlier chunks are reduced, a and b back on the host.  A bounded subset: the first
    layers whose pairs fit `max_bytes` of pinned memory."""
    torch, B = c.torch, c.B
    chosen, total = [], 0
    for L in layers:
        if total + L.calib_bytes > max_bytes and chosen:
            break
        chosen.append(L)
        total += L.calib_bytes
        if total > max_bytes:
            break
    host = []
    for L in chosen:
        N = L.spec.N
        hf = torch.empty((L.R, N), dtype=torch.float32).pin_memory()
        hq = torch.empty((L.R, N), dtype=torch.float32).pin_memory()
        hf.copy_(L.fp_out)
        hq.copy_(L.q_out)
        ha, hb = torch.empty(N).pin_memory(), torch.empty(N).pin_memory()
        sb = B.qwt_cwac_host_staging_bytes(L.R, N)
        host.append((hf, hq, ha, hb, sb))
    staging = torch.empty(max(h[4] for h in host), dtype=torch.uint8, device=c.device)

    def one_pass():
        for L, (hf, hq, ha, hb, sb) in zip(chosen, host):
            B.qwt_cwac_calibrate_host(hf.data_ptr(), hq.data_ptr(), L.R, L.spec.N, L.spec.N, ha.data_ptr(), hb.data_ptr(),
                                      None, staging, sb, c.stream)
    one_pass()
    barrier(c)
    worst = max(float((h[2] - L.a.cpu()).abs().max()) for L, h in zip(chosen, host))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n = 2
    e0.record(c.stream)
    for _ in range(n):
        one_pass()
    e1.record(c.stream)
    barrier(c)
    (t,) = max_over_ranks(c, [e0.elapsed_time(e1) * 1e-3])
    return {"value": c.world * total * n / t / 1e9, "unit": "GB/s", "h2d_bytes_per_step": total,
            "d2h_bytes_per_step": sum(8 * L.spec.N for L in chosen), "steps": n, "layers": len(chosen),
            "max_abs_diff_of_a_vs_phase_A": worst,
            "what": "qwt_cwac_calibrate_host: pinned host fp_out/q_out in (chunked, overlapped with the reduction), a/b out"}


def in_layer_calibration(c, layers, n=4):
    """Calibration inside the layer (the statistics accumulated in the layer's own epilogue, the quantized output never
    stored) on the first layers: an extra figure outside the timed region, checked against phase A's fit."""
    torch, B = c.torch, c.B
    us, moved, worst, used = 0.0, 0, 0.0, 0
    for L in layers[:n]:
        if L.Xcq is None:
            continue
        s = L.spec
        wsb = B.qwt_qlinear_cwac_calibrate_workspace_bytes(L.R, s.N, s.K, L.wfmt)
        ws = torch.empty(wsb, dtype=torch.uint8, device=c.device)
        a2, b2 = torch.empty_like(L.a), torch.empty_like(L.b)

        def call():
            B.qwt_qlinear_cwac_calibrate(L.Xcq, L.xcs, L.W, L.wfmt, L.ws, L.bias, L.fp_out, s.N, L.R, s.N, s.K,
                                         None, a2, b2, None, ws, wsb, c.stream)
        call()
        q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        q0.record(c.stream)
        for _ in range(3):
            call()
        q1.record(c.stream)
        torch.cuda.synchronize()
        B.qwt_qlinear_check_status(ws)
        us += q0.elapsed_time(q1) * 1e3 / 3
        moved += 4 * L.R * s.N + L.R * s.K + s.N * (s.K if s.w_bits == 8 else s.K // 2)
        worst = max(worst, float(((a2 - L.a).abs() / L.a.abs().clamp_min(1e-6)).max()))
        used += 1
        del ws
        L.Xcq = L.xcs = None
    if not used:
        return None
    gbs = moved / us / 1e3
    return {"value": gbs, "unit": "GB/s", "us": us, "layers": used, "frac_hbm_peak": gbs / c.peaks["hbm_gbs"],
            "bytes": "4 R N (fp_out) + R K (codes) + weights", "max_rel_diff_of_a_vs_phase_A": worst}


def library_int8_matmul_tops(c):
    """An on-box INT8 reference point: the library's plain int8 x int8 -> int32 matmul (no epilogue) at 8192^3, timed
    outside the timed region.  Context for the "% INT8 peak" figures, not part of the path."""
    torch = c.torch
    try:
        a8 = torch.randint(-127, 128, (8192, 8192), dtype=torch.int8, device=c.device)
        b8 = torch.randint(-127, 128, (8192, 8192), dtype=torch.int8, device=c.device).t()
        for _ in range(3):
            torch._int_mm(a8, b8)
        best = None
        for _ in range(5):
            q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            q0.record()
            torch._int_mm(a8, b8)
            q1.record()
            torch.cuda.synchronize()
            t = q0.elapsed_time(q1) * 1e-3
            best = t if best is None else min(best, t)
        return 2 * 8192 ** 3 / best / 1e12
    except Exception:
        return None


def calibration_sweep(c, steps, warmup, seed):
    """Config 5: 2048 images x 197 tokens, widths 768 / 2304 / 3072, quantization noise at 8 and 4 bits.  A step =
    qwt_cwac_calibrate on each of the six pairs (8 bytes per row and channel).  The pairs are drawn on the device one
    at a time (they are 2.5-9.9 GB each)."""
    torch, B, WL = c.torch, c.B, c.WL
    R = WL.CALIB_SWEEP_ROWS
    rows, total_bytes, total_s = [], 0, 0.0
    B.qwt_launch_count_reset()
    for C_ in WL.CALIB_SWEEP_WIDTHS:
        for bits in WL.CALIB_SWEEP_BITS:
            fp, q, _ = WL.device_calib_pair(R, C_, bits, seed=seed, device=c.device)
            a = torch.empty(C_, dtype=torch.float32, device=c.device)
            b = torch.empty(C_, dtype=torch.float32, device=c.device)
            wsb = B.qwt_cwac_workspace_bytes(R, C_)
            ws = torch.empty(max(wsb, 256), dtype=torch.uint8, device=c.device)
            for _ in range(warmup):
                B.qwt_cwac_calibrate(fp, q, R, C_, C_, a, b, None, ws, wsb, c.stream)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(c.stream)
            for _ in range(steps):
                B.qwt_cwac_calibrate(fp, q, R, C_, C_, a, b, None, ws, wsb, c.stream)
            e1.record(c.stream)
            torch.cuda.synchronize()
            t = e0.elapsed_time(e1) * 1e-3 / steps
            byt = 8 * R * C_
            rows.append({"channels": C_, "bits": bits, "ms": t * 1e3, "gbs": byt / t / 1e9,
                         "frac_hbm_peak": byt / t / 1e9 / c.peaks["hbm_gbs"], "a_mean": float(a.mean().item())})
            total_bytes += byt
            total_s += t
            del fp, q, a, b, ws
    return rows, total_bytes, total_s, int(B.qwt_launch_count())


RESNET50_3X3 = [   # (H = W, C = C_out) of the 3 x 3 convolution inside a bottleneck of stages 2, 3, 4; batch 32
    (28, 128), (14, 256), (7, 512),
]


def conv_entry(c, steps, batch=32):
    """CNN-shaped k x k layers: the ResNet-50 3 x 3 bottleneck convolutions (stride 1, pad 1) of the stages whose channel
    count the implicit-GEMM path takes (C % 128 == 0), per-token (per-pixel) INT8 output, timed through
    qwt_qconv2d_cwac_forward and, for comparison, through qwt_im2col_i8 + qwt_qlinear_cwac_forward."""
    torch, B = c.torch, c.B
    g = torch.Generator(device=c.device)
    g.manual_seed(12345)
    layers = []
    for hw, ch in RESNET50_3X3:
        X = torch.randn((batch, hw, hw, ch), generator=g, device=c.device)
        Xq = (X / (X.abs().max() / 127.0)).round().clamp_(-127, 127).to(torch.int8)    # per-tensor codes (inputs only)
        Wq = torch.randint(-127, 128, (ch, 3, 3, ch), generator=g, device=c.device, dtype=torch.int8)
        fs = torch.rand(ch, generator=g, device=c.device) * 2e-4 + 1e-4
        fb = torch.randn(ch, generator=g, device=c.device) * 0.01
        M, K = batch * hw * hw, 9 * ch
        Y = torch.empty((M, ch), dtype=torch.int8, device=c.device)
        ys = torch.empty(M, dtype=torch.float32, device=c.device)
        wsb = B.qwt_qconv2d_workspace_bytes(batch, hw, hw, ch, ch, 3, 3, 1, 1, B.QWT_OUT_INT8_PER_TOKEN)
        ws = torch.empty(max(wsb, 256), dtype=torch.uint8, device=c.device)
        P = torch.empty((M, K), dtype=torch.int8, device=c.device)
        xs = torch.full((M,), 0.02, dtype=torch.float32, device=c.device)
        wsb2 = B.qwt_qlinear_workspace_bytes(M, ch, K, B.QWT_W_INT8, B.QWT_OUT_INT8_PER_TOKEN)
        ws2 = torch.empty(max(wsb2, 256), dtype=torch.uint8, device=c.device)
        layers.append(dict(hw=hw, ch=ch, M=M, K=K, Xq=Xq, Wq=Wq, fs=fs, fb=fb, Y=Y, ys=ys, ws=ws, wsb=wsb, P=P, xs=xs,
                           ws2=ws2, wsb2=wsb2))

    def implicit(st):
        for L in layers:
            B.qwt_qconv2d_cwac_forward(L["Xq"], 0.02, L["Wq"], L["fs"], L["fb"], batch, L["hw"], L["hw"], L["ch"], L["ch"],
                                       3, 3, 1, 1, B.QWT_OUT_INT8_PER_TOKEN, L["Y"], L["ys"], L["ws"], L["wsb"], st)

    def patches(st):
        for L in layers:
            B.qwt_im2col_i8(L["Xq"], batch, L["hw"], L["hw"], L["ch"], 3, 3, 1, 1, L["P"], st)
            B.qwt_qlinear_cwac_forward(L["P"], L["xs"], L["Wq"], B.QWT_W_INT8, L["fs"], L["fb"], L["M"], L["ch"], L["K"],
                                       B.QWT_OUT_INT8_PER_TOKEN, L["Y"], L["ys"], L["ws2"], L["wsb2"], st)

    def timed(fn):
        for _ in range(3):
            fn(c.stream)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(c.stream)
        for _ in range(steps):
            fn(c.stream)
        e1.record(c.stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e-3 / steps

    B.qwt_launch_count_reset()
    t_imp = timed(implicit)
    launches = B.qwt_launch_count()
    t_pat = timed(patches)
    for L in layers:
        B.qwt_qlinear_check_status(L["ws"])
    ops = sum(2 * L["M"] * L["ch"] * L["K"] for L in layers)
    byt = sum(L["Xq"].numel() + L["Wq"].numel() + L["M"] * L["ch"] + 4 * L["M"] + 8 * L["ch"] for L in layers)
    t_min = max(ops / (c.int8_peak * 1e12), byt / (c.peaks["hbm_gbs"] * 1e9))
    return {"workload": "ResNet-50 shaped 3 x 3 convolutions (stride 1, pad 1; 28 x 28 x 128, 14 x 14 x 256, 7 x 7 x 512; batch 32), "
                        "W8A8, per-tensor activation scale, per-pixel INT8 output; direct calls",
            "layers": len(layers), "steps": steps,
            "forward": {"tops": ops / t_imp / 1e12, "ms_per_step": t_imp * 1e3, "bound": "tensor",
                        "frac_int8_peak_burst": ops / t_imp / 1e12 / c.int8_peak, "frac_of_roofline": t_min / t_imp,
                        "min_time_ms": t_min * 1e3, "path": "implicit GEMM (qwt_qconv2d_cwac_forward)",
                        "through_patch_matrix_tops": ops / t_pat / 1e12,
                        "through_patch_matrix_ms": t_pat * 1e3},
            "calibration": None, "gpu_launches": int(launches)}


PER_CONFIG = [   # (workload, calibration-row cap or 0, why the cap)
    ("cfg1", 0, None),
    ("cfg2", 0, None),
    ("cfg3", 100864, "512 of the config's 1024 calibration images: the 48 pairs at full length are 134 GB"),
    ("rn50", 0, None),
]


def per_config_entries(c, args):
    """The two halves of the metric for every other workload, each on its own full shapes (fewer steps)."""
    torch = c.torch
    out = []
    steps = max(3, min(args.steps, 5))
    for name, cap, why in PER_CONFIG:
        if name == args.workload:
            continue
        specs, desc = workload_layers(c.WL, name)
        r, layers = measure_layers(c, args, specs, steps, 3, cap)
        tops, roof_f = forward_roofline(c, r, f"qlinear_cwac_kernel@{name}")
        gbs, roof_c = calibration_roofline(c, r, "cwac_stats_kernel")
        out.append({"workload": desc, "layers": r["n_layers"], "steps": steps, "calib_rows_cap": cap or None,
                    "calib_rows_cap_reason": why,
                    "forward": {"tops": tops, "ms_per_step": r["t_b"] / steps * 1e3, "bound": roof_f["bound"],
                                "frac_int8_peak_burst": tops / c.int8_peak, "frac_of_roofline": roof_f["frac_of_roofline"],
                                "min_time_ms": max(roof_f["min_time_ms_tensor"], roof_f["min_time_ms_hbm"])},
                    "calibration": {"gbs": gbs, "ms_per_step": r["t_a"] / steps * 1e3, "frac_hbm_peak": roof_c["frac"],
                                    "bytes_per_step": r["cal_bytes"]},
                    "gpu_launches": r["launches"]})
        del layers, r
        torch.cuda.empty_cache()
    out.append(conv_entry(c, steps))
    torch.cuda.empty_cache()
    if args.workload != "cfg5":
        rows, total_bytes, total_s, launches = calibration_sweep(c, steps, 3, args.seed)
        gbs = total_bytes / total_s / 1e9
        out.append({"workload": "config 5: CWAC calibration sweep, 403456 rows x {768, 2304, 3072} channels, 8- and 4-bit noise",
                    "steps": steps, "forward": None,
                    "calibration": {"gbs": gbs, "ms_per_step": total_s * 1e3, "frac_hbm_peak": gbs / c.peaks["hbm_gbs"],
                                    "bytes_per_step": total_bytes, "pairs": rows},
                    "gpu_launches": launches})
        torch.cuda.empty_cache()
    return out


def run_ours(args):
    c = make_ctx()
    torch, B, WL = c.torch, c.B, c.WL
    specs, desc = workload_layers(WL, args.workload)
    specs = specs[args.first_layer:]
    if args.layers:
        specs = specs[: args.layers]
    # every rank owns a full copy of the workload with its own seed (row shards of a larger batch): weak scaling
    if args.out:
        import dataclasses
        specs = [dataclasses.replace(sp, out=args.out) for sp in specs]
    calib_cap = args.calib_rows if args.calib_rows >= 0 else DEFAULT_CALIB_CAP.get(args.workload, 0)

    r, layers = measure_layers(c, args, specs, args.steps, args.warmup, calib_cap, keep_calib_inputs=4,
                               sampler=ClockSampler(c.local))
    clocks = r["clocks"]
    world = c.world
    tops_gpu, roof_fwd = forward_roofline(c, r, f"qlinear_cwac_kernel@{args.workload}")
    cal_gpu, roof_cal = calibration_roofline(c, r, "cwac_stats_kernel")
    tops, cal_gbs = world * tops_gpu, world * cal_gpu
    dominant = roof_cal if r["t_a"] >= r["t_b"] else roof_fwd

    e2e = None if args.no_e2e else e2e_forward(c, layers, args.steps)
    e2e_cal = None if args.no_e2e else e2e_calibration(c, layers)
    in_layer = in_layer_calibration(c, layers) if c.rank == 0 else None
    lib_int8 = library_int8_matmul_tops(c) if (c.rank == 0 and not args.no_library_int8) else None
    read_gbs = read_only_hbm_gbs(c) if c.rank == 0 else None

    cpu = None
    if c.rank == 0 and world == 1 and not args.no_cpu:
        rows_cap, calib_cpu = args.cpu_rows, args.cpu_calib_rows
        hl = [host_copy_of_layer(L, rows_cap, calib_cpu) for L in layers[:4]]
        ops, fs_, cb, cs_ = oracle_block_time(hl, calib_cpu)
        cpu = {"value": ops / fs_ / 1e12, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
               "sample": (f"first {len(hl)} layers, first {rows_cap} tokens (forward: integer product, dequant+CWAC, "
                          f"requant) and first {calib_cpu} calibration rows (fit) of each; {fs_ + cs_:.1f} s of CPU work; "
                          "BLAS matmul threaded, elementwise numpy single-threaded"),
               "calibration_gbs": cb / cs_ / 1e9, "host_cpus": os.cpu_count()}
        del hl
    fwd_bytes, cal_bytes, n_layers = r["fwd_bytes"], r["cal_bytes"], r["n_layers"]
    del layers
    torch.cuda.empty_cache()

    per_config = None
    if world == 1 and not args.no_per_config and not args.layers and not args.first_layer:
        per_config = per_config_entries(c, args)

    if c.rank == 0:
        line = {
            "metric": METRIC, "value": tops, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": r["t_all"] / args.steps * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "int8", "data": "synthetic",
            "config": {"workload": desc, "layers": n_layers, "first_layer": args.first_layer,
                       "calib_rows_cap": calib_cap or None, "out_override": args.out or None,
                       "l2": "inputs larger than L2: every step streams "
                             f"{cal_bytes / 1e9:.1f} GB of calibration pairs and cycles {n_layers} distinct layer buffer sets "
                             f"({fwd_bytes / 1e6:.0f} MB)", "parallelism": f"row shards x{world}, no collective",
                       "launch": "direct calls" if args.no_graph else "CUDA graph replay of the recorded library calls"},
            "calibration": {"value": cal_gbs, "unit": "GB/s", "ms_per_step": r["t_a"] / args.steps * 1e3,
                            "frac_hbm_peak": cal_gpu / c.peaks["hbm_gbs"],
                            "hbm_read_only_gbs": read_gbs,
                            "frac_hbm_read_only": None if not read_gbs else cal_gpu / read_gbs,
                            "denominators": "frac_hbm_peak: measured read + write copy; frac_hbm_read_only: a read-only "
                                            "sum reduction over 4 GiB timed in this run (the statistics pass only reads)"},
            "forward": {"ms_per_step": r["t_b"] / args.steps * 1e3, "frac_int8_peak_burst": tops_gpu / c.int8_peak,
                        "frac_int8_peak_sustained": tops_gpu / c.int8_peak_sus,
                        "frac_int8_datasheet_4500": tops_gpu / 4500.0,
                        "library_int8_matmul_8192_tops": lib_int8,
                        "min_time_ms": max(roof_fwd["min_time_ms_tensor"], roof_fwd["min_time_ms_hbm"]),
                        "frac_of_roofline": roof_fwd["frac_of_roofline"]},
            "roofline": dominant, "rooflines": [roof_cal, roof_fwd],
            "cpu_baseline": cpu, "e2e": e2e, "e2e_calibration": e2e_cal, "calibration_in_layer": in_layer,
            "per_config": per_config, "gpu_launches": r["launches"], "clocks": clocks,
        }
        print(json.dumps(line))
    if world > 1:
        c.dist.barrier()
        c.dist.destroy_process_group()
    return 0


def run_calibration_sweep(args):
    """`--workload cfg5`: the calibration sweep as a line of its own, GB/s, single GPU."""
    c = make_ctx()
    sampler = ClockSampler(c.local)
    sampler.start()
    rows, total_bytes, total_s, launches = calibration_sweep(c, args.steps, args.warmup, args.seed)
    clocks = sampler.stop()
    gbs = total_bytes / total_s / 1e9
    ratio, prov = traffic_ratio("cwac_stats_kernel")
    line = {"metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": total_s * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": "config 5: CWAC calibration sweep, 403456 rows x {768, 2304, 3072} channels, 8- and 4-bit noise",
                       "l2": "inputs larger than L2 (2.5-9.9 GB per pair)"},
            "roofline": {"kernel": "cwac_stats_kernel", "bound": "hbm", "achieved": gbs, "peak": c.peaks["hbm_gbs"],
                         "unit": "GB/s", "frac": gbs / c.peaks["hbm_gbs"], "peak_source": f"of {c.peaks['source']}",
                         "traffic": None if ratio is None else ratio * total_bytes / len(rows), "traffic_source": prov},
            "pairs": rows, "cpu_baseline": None, "e2e": None, "gpu_launches": launches, "clocks": clocks}
    print(json.dumps(line))
    return 0


# Calibration rows per layer when --calib-rows is not given: config 4's 14 pairs at the full 262144 rows are 178 GB.
DEFAULT_CALIB_CAP = {"cfg4": 65536}


def spawn_ranks(args):
    """`--gpus N` without a torchrun environment: start the N ranks here (one process per GPU, rendezvous on
    127.0.0.1).  NCCL's own communicator log is left on and goes to one file per rank beside the temporary files."""
    import tempfile
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    env = dict(os.environ)
    if "NCCL_DEBUG" not in env:
        logdir = tempfile.mkdtemp(prefix="qwt_nccl_")
        env.update(NCCL_DEBUG="INFO", NCCL_DEBUG_SUBSYS="INIT", NCCL_DEBUG_FILE=os.path.join(logdir, "nccl_rank_%p.log"))
        sys.stderr.write(f"NCCL communicator log: {logdir}\n")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd, env=env)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4", choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg5", "rn50"])
    ap.add_argument("--layers", type=int, default=0, help="only the first L layers of the workload (0 = all)")
    ap.add_argument("--first-layer", type=int, default=0, help="skip this many layers of the workload")
    ap.add_argument("--calib-rows", type=int, default=-1,
                    help="cap the calibration rows per layer (0 = the config's own; default: the config's own except "
                         "65536 for cfg4, whose pairs at full length do not fit one GPU)")
    ap.add_argument("--out", default="", choices=["", "int8", "bf16"], help="override the output stage")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="skip the per_config entries (the other workloads)")
    ap.add_argument("--calibration", default="batch", choices=["batch", "per-layer"],
                    help="phase A through the batched entry point (one statistics launch for all layers) or one "
                         "calibrate + fold call per layer")
    ap.add_argument("--forward-streams", type=int, default=2, choices=[1, 2, 3, 4],
                    help="streams the forward calls of phase B alternate over inside the graph")
    ap.add_argument("--no-library-int8", action="store_true", help="skip timing the library int8 matmul reference point")
    ap.add_argument("--no-graph", action="store_true", help="issue every library call from the host in the timed region")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--cpu-rows", type=int, default=4096)
    ap.add_argument("--cpu-calib-rows", type=int, default=32768)
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        return run_reference(args)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return spawn_ranks(args)
    if args.workload == "cfg5":
        return run_calibration_sweep(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
