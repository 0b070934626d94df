#!/usr/bin/env python
"""Benchmark of the encoder-layer operator library on B200.

One step = one forward pass of the BERT-large-shaped post-LN encoder layer
(batch 32 x seq 512, hidden 1024, 16 heads, FFN 4096) through
``pd_encoder_layer_fwd``: it runs every operator of the library (bf16 GEMMs with
fused bias / GELU / residual epilogues, attention, softmax, LayerNorm) on one
batch of seeded synthetic input.  The headline value is bf16 TFLOP/s counted
over the six dense contractions (446.68 GFLOP per step).  The standalone
operators at their configured and paper shapes are timed separately and
reported under "ops" (GB/s for the row operators, TFLOP/s for the GEMM).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl pd|reference]

With N > 1 (launched by torch.distributed.run) every rank runs an independent
replica on its own batch shard: the path has no exchange step, so there is no
data-path collective; NCCL is used for the timing barrier and the max over ranks.
``--impl reference`` times the CPU oracle (rank 0 only) on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2511_03586_b200 import inputs  # noqa: E402  (seeded generators only)

NOMINAL_HBM_GBS = 8000.0
NOMINAL_BF16_TFLOPS = 2250.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel at the FFN-up / configured
# GEMM shape, from the ncu capture summarised in profiles/gemm_bf16_tcgen05_pair_16384x4096x1024.md.  Set to None
# whenever that kernel changes until the counters are taken again.
DOMINANT_KERNEL_DRAM_TRAFFIC_BYTES = 42.002176e6 + 80.332544e6
METRIC = "achieved HBM GB/s (row ops) and bf16 TFLOP/s (GEMM, layer) as % of roofline"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    except Exception:
        return dict(FALLBACK_PEAKS, source="fallback")


# ----------------------------------------------------------------------------
# clocks during the timed region (NVML, read-only)
# ----------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
               0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}

    def __init__(self, index: int, period_s: float = 0.02):
        self.index, self.period = index, period_s
        self.sm, self.power_w, self.reasons, self.max_mhz = [], [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nv = None

    def _sample(self):
        try:
            self.sm.append(int(self._nv.nvmlDeviceGetClockInfo(self._h, self._nv.NVML_CLOCK_SM)))
            self.power_w.append(self._nv.nvmlDeviceGetPowerUsage(self._h) / 1000.0)
            mask = int(self._nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
            for bit, name in self.REASONS.items():
                if mask & bit and name != "gpu_idle":
                    self.reasons.add(name)
        except Exception:
            pass

    def _run(self):
        while not self._stop.is_set():
            self._sample()
            self._stop.wait(self.period)

    def __enter__(self):
        if self._nv:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        if self._thread:
            self._sample()
            self._stop.set()
            self._thread.join()

    def summary(self):
        return {"sm_mhz": statistics.median(self.sm) if self.sm else None, "sm_max_mhz": self.max_mhz,
                "power_w": statistics.median(self.power_w) if self.power_w else None,
                "reasons": sorted(self.reasons), "samples": len(self.sm)}


# ----------------------------------------------------------------------------
# CPU oracle legs
# ----------------------------------------------------------------------------
def oracle_layer_seconds(n_seq: int, seed: int = 0, seq: int = 512):
    """Runs the CPU oracle's encoder layer on `n_seq` sequences of the workload (cut to `seq` tokens when the
    time budget asks for a smaller sample); returns (seconds, flops of the sample)."""
    import oracle
    shape = inputs.EncoderLayerShape(batch=n_seq, seq=seq)
    p = inputs.encoder_layer_inputs(shape, seed=seed)
    w = {m: inputs.bf16_bits_to_f32(p[m + "_bits"]) for m in ("w_qkv", "w_o", "w_ffn1", "w_ffn2")}
    x = inputs.bf16_bits_to_f32(p["x_bits"])
    oracle.softmax(np.zeros((1, 4)))  # load / build the library outside the timed part
    t0 = time.perf_counter()
    oracle.encoder_layer(x, w["w_qkv"], p["b_qkv"], w["w_o"], p["b_o"], w["w_ffn1"], p["b_ffn1"], w["w_ffn2"],
                         p["b_ffn2"], p["ln1_gamma"], p["ln1_beta"], p["ln2_gamma"], p["ln2_beta"],
                         batch=n_seq, seq=shape.seq, heads=shape.heads, ln_eps=shape.ln_eps)
    return time.perf_counter() - t0, shape.gemm_flops()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    # One sequence of 512 tokens takes about 5 s on one core.  The whole run is held to about 150 s by
    # cutting the sampled sequence shorter when many steps are asked for.
    seq = 512
    while seq > 32 and (args.warmup + args.steps) * 5.0 * seq / 512 > 150.0:
        seq //= 2
    times = []
    flops = 0.0
    for i in range(args.warmup + args.steps):
        dt, flops = oracle_layer_seconds(1, seed=i, seq=seq)
        if i >= args.warmup:
            times.append(dt)
    sec = sum(times) / max(len(times), 1)
    value = flops / sec / 1e12
    sample = f"one sequence (batch 1 x seq {seq}" + ("" if seq == 512 else " of 512") + ") per step, full layer"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "bert-large post-LN encoder layer fwd, batch 32 x seq 512, hidden 1024, 16 heads, ffn 4096",
                   "sample": sample},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": 1, "kind": "oracle", "sample": sample,
                         "host_cores": os.cpu_count()},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)
    return 0


# ----------------------------------------------------------------------------
# GPU arm
# ----------------------------------------------------------------------------
def time_launches(torch, fn, n_iter, n_warm=3):
    """Average device milliseconds of fn(i) over n_iter launches (CUDA events on the launching stream).

    The launches are captured once into a CUDA graph and the graph is replayed for the timed run, so that
    launches far shorter than the host's launch cost (a 1 MiB softmax) are limited by the device, not by
    Python; if capture is not possible the launches are issued directly."""
    for i in range(n_warm):
        fn(i)
    torch.cuda.synchronize()
    graph = None
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                for i in range(n_iter):
                    fn(n_warm + i)
        torch.cuda.current_stream().wait_stream(side)
        graph = g
    except Exception:
        graph = None
        torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if graph is not None:
        graph.replay()
        torch.cuda.synchronize()
        e0.record()
        graph.replay()
        e1.record()
    else:
        e0.record()
        for i in range(n_iter):
            fn(n_warm + i)
        e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / n_iter


def ops_suite(torch, api, peaks, only: str = ""):
    """Standalone operators at the configured and the paper's shapes.  Buffers rotate
    through a pool larger than L2 so that every launch reads from HBM.  `only`
    restricts the suite to the operators whose name contains it."""
    out = {}
    L2_POOL = 400 << 20

    def wanted(name):
        return only in name

    def pool_size(bytes_per_set):
        return max(2, min(256, -(-L2_POOL // bytes_per_set)))

    def rowop_entry(name, ms, bytes_moved, note=None):
        gbs = bytes_moved / ms / 1e6
        e = {"ms": ms, "GB/s": gbs, "frac_measured": gbs / peaks["hbm_gbs"], "frac_nominal": gbs / NOMINAL_HBM_GBS}
        if note:
            e["note"] = note
        out[name] = e

    for rows, cols, note in ((256, 512, "configured shape: 1 MiB, launch-latency-bound"), (24576, 512, "paper shape"),
                             (262144, 512, "attention rows of the layer")):
        if not wanted(f"softmax_{rows}x{cols}"):
            continue
        x = torch.from_numpy(inputs.softmax_inputs(min(rows, 24576), cols)["x"]).cuda()
        if rows > x.shape[0]:
            x = x.repeat(-(-rows // x.shape[0]), 1)[:rows].contiguous()
        n = pool_size(rows * cols * 8)
        xs = [x.clone() for _ in range(n)]
        ys = [torch.empty_like(x) for _ in range(n)]
        iters = max(20, min(2000, int(3e9 / (rows * cols * 8))))
        ms = time_launches(torch, lambda i: api.pd_softmax(xs[i % n], ys[i % n]), iters)
        rowop_entry(f"softmax_{rows}x{cols}", ms, rows * cols * 8, note)
        del xs, ys

    for rows, cols, note in ((4096, 1024, "configured shape"), (16384, 1024, "paper shape"), (4096, 4096, "paper shape"),
                             (2048, 24576, "long rows: one 256-thread CTA per row, 24 float4 per thread")):
        if not wanted(f"layernorm_{rows}x{cols}"):
            continue
        p = inputs.layernorm_inputs(rows, cols)
        x = torch.from_numpy(p["x"]).cuda()
        g, b = torch.from_numpy(p["gamma"]).cuda(), torch.from_numpy(p["beta"]).cuda()
        n = pool_size(rows * cols * 8)
        xs = [x.clone() for _ in range(n)]
        ys = [torch.empty_like(x) for _ in range(n)]
        iters = max(20, min(2000, int(3e9 / (rows * cols * 8))))
        ms = time_launches(torch, lambda i: api.pd_layernorm(xs[i % n], g, b, 1e-5, ys[i % n]), iters)
        rowop_entry(f"layernorm_{rows}x{cols}", ms, rows * cols * 8 + cols * 8, note)
        if rows * cols * 8 <= (32 << 20):
            # what a plain device copy of the same bytes reaches in the same harness: the ceiling at this size,
            # where a launch lasts a few microseconds and its ramp-up and tail no longer vanish
            ms = time_launches(torch, lambda i: ys[i % n].copy_(xs[i % n]), iters)
            rowop_entry(f"context_copy_{rows}x{cols}", ms, rows * cols * 8,
                        "torch copy_ of the same bytes, for context: not part of the library")
        del xs, ys

    rows, cols = 3072, 4096
    if wanted(f"rmsnorm_{rows}x{cols}"):
        p = inputs.rmsnorm_inputs(rows, cols)
        x = torch.from_numpy(p["x"]).cuda()
        g = torch.from_numpy(p["gamma"]).cuda()
        n = pool_size(rows * cols * 8)
        xs = [x.clone() for _ in range(n)]
        ys = [torch.empty_like(x) for _ in range(n)]
        ms = time_launches(torch, lambda i: api.pd_rmsnorm(xs[i % n], g, 1e-5, ys[i % n]), 40)
        rowop_entry(f"rmsnorm_{rows}x{cols}", ms, rows * cols * 8 + cols * 4, "paper shape")
        del xs, ys

    rows, cols = 4096, 4096
    if wanted(f"reducemean_{rows}x{cols}"):
        x = torch.from_numpy(inputs.rmsnorm_inputs(rows, cols)["x"]).cuda()
        n = pool_size(rows * cols * 4)
        xs = [x.clone() for _ in range(n)]
        ys = [torch.empty(rows, dtype=torch.float32, device="cuda") for _ in range(n)]
        ms = time_launches(torch, lambda i: api.pd_reducemean(xs[i % n], ys[i % n]), 60)
        rowop_entry(f"reducemean_{rows}x{cols}", ms, rows * cols * 4 + rows * 4, "paper shape")
        del xs, ys

    rows, cols = 16384, 4096
    if wanted(f"bias_gelu_residual_{rows}x{cols}"):
        p = inputs.bias_gelu_residual_inputs(rows, cols)
        xs = [torch.from_numpy(p["x"]).cuda() for _ in range(2)]
        rs = [torch.from_numpy(p["r"]).cuda() for _ in range(2)]
        os_ = [torch.empty_like(xs[0]) for _ in range(2)]
        bias = torch.from_numpy(p["bias"]).cuda()
        ms = time_launches(torch, lambda i: api.pd_bias_gelu_residual(xs[i % 2], bias, rs[i % 2], os_[i % 2]), 20)
        rowop_entry(f"bias_gelu_residual_{rows}x{cols}", ms, rows * cols * 12 + cols * 4, "configured shape")
        del xs, rs, os_, p

    def bf16_rand(*shape, scale=1.0):
        return (torch.randn(*shape, device="cuda") * scale).to(torch.bfloat16)

    def gemm_entry(name, ms, flops, note):
        tf = flops / ms / 1e9
        # a few milliseconds of launches at boost clocks: the burst peak is the one that applies
        out[name] = {"ms": ms, "TFLOP/s": tf, "frac_measured_burst": tf / peaks["bf16_tflops"],
                     "frac_measured_sustained": tf / peaks["bf16_tflops_sustained"],
                     "frac_nominal": tf / NOMINAL_BF16_TFLOPS, "note": note}

    # small problems of the paper's operator table: less than one wave of tiles, bound by latency, not by the tensor pipe
    M, N, K = 768, 1024, 1024
    if wanted(f"gemm_{M}x{N}x{K}"):
        a, b = bf16_rand(M, K), bf16_rand(K, N, scale=K ** -0.5)
        c = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
        ms = time_launches(torch, lambda i: api.pd_gemm_bf16(a, b, c), 200)
        gemm_entry(f"gemm_{M}x{N}x{K}_cbf16", ms, 2.0 * M * N * K, "paper shape (matmul); operands L2-resident")
    B_, M, K, N = 192, 256, 128, 256
    if wanted(f"bmm_{B_}x{M}x{K}x{N}"):
        a, b = bf16_rand(B_, M, K), bf16_rand(B_, K, N, scale=K ** -0.5)
        c = torch.empty(B_, M, N, dtype=torch.bfloat16, device="cuda")
        ms = time_launches(torch, lambda i: api.pd_gemm_bf16(a, b, c), 200)
        gemm_entry(f"bmm_{B_}x{M}x{K}x{N}_cbf16", ms, 2.0 * B_ * M * N * K, "paper shape (bmm); operands L2-resident")
    M, N, K = 256, 448, 4096
    if wanted(f"swiglu_{M}x{N}x{K}"):
        x, wg, wu = bf16_rand(M, K), bf16_rand(K, N, scale=K ** -0.5), bf16_rand(K, N, scale=K ** -0.5)
        y = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
        ms = time_launches(torch, lambda i: api.pd_swiglu_gemm(x, wg, wu, y), 200)
        gemm_entry(f"swiglu_{M}x{N}x{K}", ms, 4.0 * M * N * K, "paper shape (swiglu: gate and up products + SiLU * up)")
    M, N, K = 16384, 1024, 1024
    if wanted(f"gemm_layernorm_{M}x{N}x{K}"):
        as_ = [bf16_rand(M, K) for _ in range(3)]
        rs = [bf16_rand(M, N) for _ in range(3)]
        ys = [torch.empty(M, N, dtype=torch.bfloat16, device="cuda") for _ in range(3)]
        b = bf16_rand(K, N, scale=K ** -0.5)
        bias, gam, bet = torch.randn(N, device="cuda"), torch.rand(N, device="cuda") + 0.5, torch.randn(N, device="cuda")
        ms = time_launches(torch, lambda i: api.pd_gemm_bias_residual_layernorm(as_[i % 3], b, bias, rs[i % 3], gam, bet,
                                                                                 1e-5, y=ys[i % 3]), 50)
        gemm_entry(f"gemm_layernorm_{M}x{N}x{K}", ms, 2.0 * M * N * K, "the layer's output projection + residual + LayerNorm")
        del as_, rs, ys
    M, N, K = 16384, 4096, 1024
    if wanted(f"gemm_bias_gelu_{M}x{N}x{K}"):
        as_ = [bf16_rand(M, K) for _ in range(3)]
        cs = [torch.empty(M, N, dtype=torch.bfloat16, device="cuda") for _ in range(3)]
        b, bias = bf16_rand(K, N, scale=K ** -0.5), torch.randn(N, device="cuda")
        ms = time_launches(torch, lambda i: api.pd_gemm_bias_act(as_[i % 3], b, bias, None, act=api.ACT_GELU, c=cs[i % 3]), 30)
        gemm_entry(f"gemm_bias_gelu_{M}x{N}x{K}", ms, 2.0 * M * N * K, "the layer's FFN-up projection + bias + GELU")
        del as_, cs

    M, K, N = 16384, 1024, 4096
    if not wanted(f"gemm_{M}x{N}x{K}"):
        return out
    g = inputs.gemm_inputs(M, N, K)
    a = torch.from_numpy(g["a_bits"][0].view(np.int16)).cuda().view(torch.bfloat16)
    b = torch.from_numpy(g["b_bits"][0].view(np.int16)).cuda().view(torch.bfloat16)
    as_, bs = [a.clone() for _ in range(3)], [b.clone() for _ in range(3)]
    for cd, nm in ((torch.bfloat16, "bf16"), (torch.float32, "f32")):
        cs = [torch.empty(M, N, dtype=cd, device="cuda") for _ in range(3)]
        ms = time_launches(torch, lambda i: api.pd_gemm_bf16(as_[i % 3], bs[i % 3], cs[i % 3]), 30)
        tf = 2.0 * M * N * K / ms / 1e9
        out[f"gemm_{M}x{N}x{K}_c{nm}"] = {"ms": ms, "TFLOP/s": tf, "frac_measured_burst": tf / peaks["bf16_tflops"],
                                          "frac_measured_sustained": tf / peaks["bf16_tflops_sustained"],
                                          "frac_nominal": tf / NOMINAL_BF16_TFLOPS, "note": "configured shape"}
        del cs
    # the vendor library on the same shape, same timing method: context only, never on the product path
    cs = [torch.empty(M, N, dtype=torch.bfloat16, device="cuda") for _ in range(3)]
    ms = time_launches(torch, lambda i: torch.matmul(as_[i % 3], bs[i % 3], out=cs[i % 3]), 30)
    out[f"context_cublas_{M}x{N}x{K}_cbf16"] = {"ms": ms, "TFLOP/s": 2.0 * M * N * K / ms / 1e9,
                                               "note": "torch.matmul (cuBLAS), for context: not part of the library"}
    return out


def run_pd(args):
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    from paper_2511_03586_b200 import api  # fails loudly when libpd.so is missing

    peaks = load_peaks()
    if args.ops_only:
        if rank == 0:
            print(json.dumps({"ops": ops_suite(torch, api, peaks, args.ops_filter), "peaks": peaks}), flush=True)
        return 0
    shape = inputs.EncoderLayerShape(batch=args.batch)
    p = inputs.encoder_layer_inputs(shape, seed=rank)

    def bf16_dev(bits):
        return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)

    params = api.EncoderLayerParams(
        **{m: bf16_dev(p[m + "_bits"]) for m in ("w_qkv", "w_o", "w_ffn1", "w_ffn2")},
        **{v: torch.from_numpy(p[v]).cuda() for v in ("b_qkv", "b_o", "b_ffn1", "b_ffn2", "ln1_gamma", "ln1_beta",
                                                       "ln2_gamma", "ln2_beta")})
    x_host = torch.from_numpy(p["x_bits"].view(np.int16)).view(torch.bfloat16).pin_memory()
    y_host = torch.empty_like(x_host).pin_memory()
    x = x_host.cuda()
    y = torch.empty_like(x)
    ws = torch.empty(api.pd_encoder_layer_workspace_bytes(shape.batch, shape.seq, shape.hidden, shape.heads, shape.ffn),
                     dtype=torch.uint8, device="cuda")
    kw = dict(batch=shape.batch, seq=shape.seq, heads=shape.heads, ln_eps=shape.ln_eps, workspace=ws)
    api.pd_clear_device_status()

    def step():
        api.pd_encoder_layer_fwd(params, x, y=y, **kw)

    def barrier():
        if world > 1:
            dist.barrier()

    # ---- device-resident throughput ------------------------------------------
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local_rank) as clocks:
        torch.cuda.synchronize()
        e0.record()
        for _ in range(args.steps):
            step()
        e1.record()
        torch.cuda.synchronize()
    barrier()
    ms = e0.elapsed_time(e1) / args.steps

    # ---- end to end: pinned host input -> device -> layer -> pinned host output ------------------
    # Every step copies its own input in and its own output out inside the timed region.  The copies run on
    # their own streams with double-buffered device and host tensors, so that step i+1's upload and step
    # i-1's download overlap step i's kernels (the library call takes the stream it is given).
    h2d, d2h, comp = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.current_stream()
    xs = [x, torch.empty_like(x)]
    ys = [y, torch.empty_like(y)]
    y_hosts = [y_host, torch.empty_like(y_host).pin_memory()]
    up_done = [torch.cuda.Event() for _ in range(2)]
    comp_done = [torch.cuda.Event() for _ in range(2)]
    down_done = [torch.cuda.Event() for _ in range(2)]

    def e2e_step(i):
        k = i & 1
        with torch.cuda.stream(h2d):
            h2d.wait_event(comp_done[k])       # the layer two steps back has finished reading xs[k]
            xs[k].copy_(x_host, non_blocking=True)
            up_done[k].record(h2d)
        comp.wait_event(up_done[k])
        comp.wait_event(down_done[k])           # ys[k] has been downloaded
        api.pd_encoder_layer_fwd(params, xs[k], y=ys[k], **kw)
        comp_done[k].record(comp)
        with torch.cuda.stream(d2h):
            d2h.wait_event(comp_done[k])
            y_hosts[k].copy_(ys[k], non_blocking=True)
            down_done[k].record(d2h)

    e2e_steps = max(4, min(args.steps, 100))
    for i in range(4):
        e2e_step(i)
    torch.cuda.synchronize()
    barrier()
    e0.record()
    for i in range(e2e_steps):
        e2e_step(i)
    comp.wait_stream(d2h)
    e1.record()
    torch.cuda.synchronize()
    barrier()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps

    from paper_2511_03586_b200 import replicas
    ms, e2e_ms = replicas.max_over_ranks([ms, e2e_ms], device="cuda")
    timeout_code = api.pd_get_device_status()
    flops = shape.gemm_flops()
    stage_names = api.pd_encoder_layer_stage_names()

    # ---- per-stage device times (CUDA events recorded by the library around each launch) and the standalone
    # operators: rank 0, before the long run below heats the board, so that they are burst measurements
    stages, ops = None, None
    if rank == 0:
        runs = []
        for _ in range(7):
            _, st = api.pd_encoder_layer_fwd_profiled(params, x, y=y, **kw)
            runs.append(st)
        stages = {n: statistics.median(r[n] for r in runs[2:]) for n in stage_names}
        if world == 1 and not args.no_ops:
            ops = ops_suite(torch, api, peaks, args.ops_filter)
            timeout_code = timeout_code or api.pd_get_device_status()

    # ---- sustained: at least `--sustained-seconds` of back-to-back steps, long enough for the board to settle at
    # its power cap; clocks and power sampled throughout, so that runs of different lengths can be compared through
    # ms x MHz (the step's cost in SM cycles)
    sustained = None
    if args.sustained_seconds > 0:
        n_sus = max(args.steps, int(args.sustained_seconds * 1e3 / ms) + 1)
        barrier()
        with ClockSampler(local_rank, period_s=0.05) as sus_clocks:
            torch.cuda.synchronize()
            e0.record()
            for _ in range(n_sus):
                step()
            e1.record()
            torch.cuda.synchronize()
        barrier()
        sus_ms = e0.elapsed_time(e1) / n_sus
        sustained = {"steps": n_sus, "ms_per_step": sus_ms, "clocks": sus_clocks.summary()}

    if sustained is not None:
        sustained["ms_per_step"] = replicas.max_over_ranks([sustained["ms_per_step"]], device="cuda")[0]
        timeout_code = timeout_code or api.pd_get_device_status()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    value = world * flops / ms / 1e9

    # dominant kernel: the tcgen05 GEMM; its largest launch is the FFN-up projection (= the configured GEMM shape)
    T, H, F = shape.tokens, shape.hidden, shape.ffn
    dom_flops = 2.0 * T * H * F
    dom_tf = dom_flops / stages["ffn_up_gemm"] / 1e9
    # The stage time comes from single steps, each enqueued and waited for on its own (the profiled call
    # synchronises): the board is at its boost clock, so the peak that applies is the burst one.
    roofline = {"bound": "tensor", "kernel": "gemm_bf16_tcgen05_pair_kernel<B[K,N], bf16 out> (ffn_up_gemm launch)",
                "achieved": dom_tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": dom_tf / peaks["bf16_tflops"],
                "peak_source": f"{peaks['source']} burst cuBLAS bf16 (the launch is timed inside single synchronised "
                               f"steps, at boost clocks)",
                "launch_ms": stages["ffn_up_gemm"],
                "frac_of_sustained_peak": dom_tf / peaks["bf16_tflops_sustained"],
                "frac_of_nominal": dom_tf / NOMINAL_BF16_TFLOPS,
                "traffic": DOMINANT_KERNEL_DRAM_TRAFFIC_BYTES, "algorithmic_bytes": 2.0 * (T * H + H * F + T * F)}

    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"bert-large post-LN encoder layer fwd, batch {shape.batch} x seq {shape.seq} per GPU, "
                               f"hidden {shape.hidden}, {shape.heads} heads, ffn {shape.ffn} (configs[4])",
                   "headline": "value = bf16 TFLOP/s of the whole layer step (six dense contractions); the row "
                               "operators' GB/s and the standalone GEMM are under 'ops'",
                   "flops_per_step_per_gpu": flops,
                   "l2": "no flush between steps: one step reads and writes about 0.37 GiB (X 32, qkv 96, ctx 32, "
                         "h1 32, mid 128, Y 32, weights 24 MiB), three times the 126 MB L2",
                   "parallelism": "replicas only" if world > 1 else "single GPU", "sigma_reading": "N(a, b): b is the std"},
        "timed_as": ("burst" if ms * args.steps < 1000.0 else "sustained") +
                    f": {ms * args.steps:.0f} ms of back-to-back steps; see 'sustained' for the long run",
        "frac_of_measured_burst_peak": value / world / peaks["bf16_tflops"],
        "frac_of_measured_sustained_peak": value / world / peaks["bf16_tflops_sustained"],
        "frac_of_nominal_peak": value / world / NOMINAL_BF16_TFLOPS,
        "clocks": clocks.summary(),
        "e2e": {"value": world * flops / e2e_ms / 1e9, "unit": "TFLOP/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": x_host.numel() * 2, "d2h_bytes_per_step": y_host.numel() * 2},
        "gpu_launches": api.pd_encoder_layer_kernel_count(shape.batch, shape.seq, shape.hidden, shape.heads,
                                                          shape.ffn) * args.steps,
        "device_timeout_code": timeout_code,
        "stages_ms": stages,
        "stages_note": "per launch, from single synchronised steps (boost clocks)",
        "roofline": roofline,
        "peaks": peaks,
    }
    if sustained is not None:
        c = sustained["clocks"]
        sustained["value"] = world * flops / sustained["ms_per_step"] / 1e9
        sustained["unit"] = "TFLOP/s"
        sustained["frac_of_measured_sustained_peak"] = sustained["value"] / world / peaks["bf16_tflops_sustained"]
        sustained["ms_x_mhz"] = sustained["ms_per_step"] * c["sm_mhz"] if c["sm_mhz"] else None
        line["sustained"] = sustained
        line["ms_x_mhz"] = ms * line["clocks"]["sm_mhz"] if line["clocks"]["sm_mhz"] else None
    if ops is not None:
        line["ops"] = ops
    line["device_timeout_code"] = timeout_code
    if world == 1 and not args.no_cpu_baseline:
        n_seq = 2
        sec, fl = oracle_layer_seconds(n_seq)
        line["cpu_baseline"] = {"value": fl / sec / 1e12, "unit": "TFLOP/s", "cores": 1, "kind": "oracle",
                                "sample": f"{n_seq} of the {shape.batch} sequences (batch {n_seq} x seq 512), full layer, "
                                          f"{sec:.1f} s", "host_cores": os.cpu_count()}
    if timeout_code:
        # a bounded wait ran out inside a tensor-core kernel: that kernel returned early, the numbers above do not
        # describe completed work
        line["invalid"] = f"device status {timeout_code}: a kernel gave up on a wait; timings are not of completed work"
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()
    return 1 if timeout_code else 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=("pd", "reference"), default="pd")
    ap.add_argument("--batch", type=int, default=32, help="sequences per GPU")
    ap.add_argument("--no-ops", action="store_true", help="skip the standalone-operator suite")
    ap.add_argument("--ops-only", action="store_true", help="run only the standalone-operator suite")
    ap.add_argument("--ops-filter", default="", help="substring selecting operators of the suite")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip timing the CPU oracle")
    ap.add_argument("--sustained-seconds", type=float, default=2.0,
                    help="length of the additional long run of back-to-back steps (0: skip it)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_pd(args)


if __name__ == "__main__":
    sys.exit(main())
