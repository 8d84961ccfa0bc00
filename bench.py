#!/usr/bin/env python
"""Benchmark of the ASER W4A8 + low-rank linear forward pass on B200.

One "step" is one pass of the whole hot path over one batch of synthetic tokens:
aser_quant_act (smooth, int8-quantize, T = X~ L_A^T) followed by aser_linear_w4a8_lr
(int4 x int8 GEMM, dequantisation, + T L_B^T, fp16 store).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line (rank 0).  With N > 1 (launched by torch.distributed.run) every rank
runs an independent replica of the same workload: the path shards over tokens with no
exchange step, so no collective is on the data path; `value` is the sum over ranks.
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

import aser_synth as synth  # noqa: E402

L2_BYTES = 126 * 1024 * 1024

WORKLOADS = {
    # name: (config id, M, N, K, r, gated_input, outlier_gain, sigma_w, bound)
    "c2_decode_m8": (2, 8, 4096, 4096, 64, False, 30.0, 0.02, "hbm"),
    "c2_decode_m1": (2, 1, 4096, 4096, 64, False, 30.0, 0.02, "hbm"),
    "c3_prefill_gate_up": (3, 2048, 14336, 4096, 64, False, 30.0, 0.02, "tensor"),
    "c3_prefill_down": (3, 2048, 4096, 14336, 64, True, 30.0, 0.02, "tensor"),
    "c3_small": (3, 2048, 4096, 4096, 64, False, 30.0, 0.02, "tensor"),
    "c5_decode_m16_8192": (5, 16, 8192, 8192, 64, False, 50.0, 0.015, "hbm"),
    "c5_decode_m16_28672": (5, 16, 28672, 8192, 64, False, 50.0, 0.015, "hbm"),
    "c5_prefill_m4096_8192": (5, 4096, 8192, 8192, 64, False, 50.0, 0.015, "tensor"),
}

# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel under ncu, taken
# with the kernel as it stands in this tree; the summaries with the commands are under profiles/
# (<kernel>_<workload>.txt).  Workloads without a capture of the current kernel report null.
NCU_DRAM_BYTES_PER_LAUNCH = {
    "c2_decode_m8": 8.71e6,           # linear_decode: mean of two launches, 8.45 and 8.98 MB read, 0 written back
    "c3_prefill_gate_up": 52.36e6,    # linear_tc: 37.9 MB read + 14.5 MB written (output partly still in L2)
}


def dominant_kernel(M, N, K):
    """Name of the kernel the library runs for the integer product at this shape (few tokens and
    at most 64 MB of packed weights: the streaming kernel; otherwise the tensor-core kernel)."""
    return "linear_decode_kernel" if M <= 16 and N * K // 2 <= (64 << 20) else "linear_tc_kernel"
DEFAULT_WORKLOAD = "c2_decode_m8"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def algorithmic_bytes_linear(M, N, K, r):
    """Bytes the int GEMM + epilogue kernel must move once: packed weights, scales, int8
    activations, fp16 output, and with compensation L_B and T."""
    b = N * K // 2 + 4 * N + M * K + 4 * M + 2 * M * N
    if r:
        b += 2 * N * r + 2 * M * r
    return b


def algorithmic_bytes_act(M, K, r):
    b = 2 * M * K + M * K + 4 * M + 4 * K
    if r:
        b += 2 * r * K + 2 * M * r
    return b


def make_inputs(name, index=0):
    cfg, M, N, K, r, gated, gain, sigma, _ = WORKLOADS[name]
    lay = synth.make_layer(M, N, K, seed=synth.seed_for(cfg, 100 * index + (M % 97)),
                           outlier_gain=gain, sigma_w=sigma, n_cal=8, gated_input=gated)
    s = synth.standin_smoothing_vector(K, lay.outlier_idx, 24.0)
    L_A, L_B = synth.standin_factors(N, K, r, seed=lay.meta["seed"], scale_a=0.01, scale_b=0.01)
    return lay, s, L_A, L_B


# ---------------------------------------------------------------------------
# clocks sampled while the GPU is busy
# ---------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap",
               0x8: "hw_slowdown", 0x10: "sync_boost", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
               0x100: "display_clock_setting"}

    def __init__(self, index):
        self.samples, self.reasons, self.stop = [], set(), False
        self.max_mhz = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None
        self.t = threading.Thread(target=self.run, daemon=True)

    def run(self):
        while not self.stop and self.nv is not None:
            try:
                mhz = self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)
                util = self.nv.nvmlDeviceGetUtilizationRates(self.h).gpu
                get = getattr(self.nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                    self.nv.nvmlDeviceGetCurrentClocksThrottleReasons
                mask = get(self.h)
                self.samples.append((mhz, util))
                for bit, nm in self.REASONS.items():
                    if mask & bit and nm != "gpu_idle":
                        self.reasons.add(nm)
            except Exception:
                pass
            time.sleep(0.005)

    def __enter__(self):
        self.t.start()
        return self

    def __exit__(self, *a):
        self.stop = True
        self.t.join(timeout=2)

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        mhz = [m for m, _ in self.samples]
        return {"sm_mhz": statistics.median(mhz), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(mhz)}


# ---------------------------------------------------------------------------
# CPU oracle leg (the only part of this file that touches oracle/)
# ---------------------------------------------------------------------------
def time_oracle(name, reps=3):
    from oracle import forward as F
    cfg, M, N, K, r, *_ = WORKLOADS[name]
    lay, s, L_A, L_B = make_inputs(name)
    cores = len(os.sched_getaffinity(0))
    F.set_threads(cores)
    q, w_scale = F.quant_w4(lay.W, s)
    Wq = F.pack_w4(q)
    # bounded sample: at most 64 token rows through the integer product
    rows = None if M <= 64 else np.arange(64)
    m_eff = M if rows is None else 64
    best = float("inf")
    for _ in range(reps):
        t0 = time.perf_counter()
        F.forward(lay.X if rows is None else lay.X[:64], s, Wq, w_scale, L_A, L_B)
        best = min(best, time.perf_counter() - t0)
    F.set_threads(1)
    tops = 2.0 * m_eff * N * K / best / 1e12
    sample = (f"full call (M={M})" if rows is None else f"first 64 of {M} token rows") + \
        f", best of {reps}, all stages of the oracle forward"
    return dict(value=tops, unit="TOPS", cores=cores, kind="oracle", sample=sample,
                seconds=best, m_rows=m_eff)


def run_reference(args, rank, world):
    if rank != 0:
        return
    name = args.workload
    cfg, M, N, K, r, *_ = WORKLOADS[name]
    from oracle import forward as F
    lay, s, L_A, L_B = make_inputs(name)
    cores = len(os.sched_getaffinity(0))
    F.set_threads(cores)
    q, w_scale = F.quant_w4(lay.W, s)
    Wq = F.pack_w4(q)
    m_eff = min(M, 64)
    X = lay.X[:m_eff]
    for _ in range(max(1, min(args.warmup, 2))):
        F.forward(X, s, Wq, w_scale, L_A, L_B)
    steps = max(1, min(args.steps, 20))
    t0 = time.perf_counter()
    for _ in range(steps):
        F.forward(X, s, Wq, w_scale, L_A, L_B)
    dt = (time.perf_counter() - t0) / steps
    tops = 2.0 * m_eff * N * K / dt / 1e12
    sample = f"{m_eff} of {M} token rows per step, {steps} steps"
    line = dict(impl="reference", metric="aser_w4a8_lowrank_linear_tops", value=tops, unit="TOPS",
                n_gpus=args.gpus, steps=steps, warmup=args.warmup, ms_per_step=dt * 1e3,
                higher_is_better=True, scaling="weak", vs_baseline=None, dtype="int8",
                data="synthetic", config=dict(workload=name, M=M, N=N, K=K, r=r),
                cpu_baseline=dict(value=tops, unit="TOPS", cores=cores, kind="oracle", sample=sample),
                e2e=dict(value=tops, unit="TOPS", h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                gpu_launches=0)
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------
# multi-rank aggregation (replicas: no collective on the data path)
# ---------------------------------------------------------------------------
def max_over_ranks_ms(ms: float, world: int, device=None) -> float:
    """Slowest rank's device time: the job is as fast as its slowest replica."""
    if world == 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tops(ops_per_rank_step: float, ms_per_step: float, world: int) -> float:
    """Aggregate throughput of `world` independent replicas that each finish a step in ms_per_step."""
    return world * ops_per_rank_step / (ms_per_step * 1e-3) / 1e12


# ---------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------
class Bench:
    def __init__(self, name, device):
        import torch
        import paper_2411_07762_b200 as aser
        self.torch, self.aser, self.name = torch, aser, name
        cfg, M, N, K, r, gated, gain, sigma, bound = WORKLOADS[name]
        self.M, self.N, self.K, self.r, self.bound = M, N, K, r, bound
        per_set = N * K // 2 + 2 * r * (N + K) + 3 * M * K
        # rotate over enough distinct operand sets that no step finds its operands in L2
        self.n_sets = 1 if per_set > 2 * L2_BYTES else int(np.ceil(2.2 * L2_BYTES / per_set))
        lay, s, L_A, L_B = make_inputs(name)
        dev = device
        t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
        self.s = t(s)
        self.layers, self.X = [], []
        base = aser.AserLinear(t(lay.W), self.s, t(L_A), t(L_B), M)
        self.layers.append(base)
        self.X.append(t(lay.X))
        g = torch.Generator(device="cpu").manual_seed(1234)
        for i in range(1, self.n_sets):
            # further operand sets: same shapes and value ranges; packed weights are the base
            # set's bytes rolled by a set-dependent offset (contents do not affect timing)
            L = object.__new__(aser.AserLinear)
            L.__dict__.update(base.__dict__)
            L.Wk = torch.roll(base.Wk, shifts=8192 * i)
            L.w_scale = base.w_scale.clone()
            L.L_A = torch.roll(base.L_A, shifts=i, dims=0).contiguous()
            L.L_B = torch.roll(base.L_B, shifts=i, dims=0).contiguous()
            L.Xq = torch.empty_like(base.Xq)
            L.a_scale = torch.empty_like(base.a_scale)
            L.T = torch.empty_like(base.T)
            L.Y = torch.empty_like(base.Y)
            self.layers.append(L)
            self.X.append(torch.roll(self.X[0], shifts=i, dims=1).contiguous())
        self.host_X = self.X[0].cpu().pin_memory()
        self.host_Y = torch.empty((M, N), dtype=torch.float16).pin_memory()
        torch.cuda.synchronize()

    def step(self, i, lowrank=True):
        # the library's whole forward pass: quantization and linear kernel, overlapped
        self.layers[i % self.n_sets](self.X[i % self.n_sets], lowrank)

    def linear_only(self, i, lowrank=True):
        self.layers[i % self.n_sets].linear(self.M, lowrank)

    def quant_only(self, i):
        self.layers[i % self.n_sets].quant(self.X[i % self.n_sets])

    def time_graph(self, fn, steps, chunk=None):
        """Device time (ms) of exactly `steps` calls of fn(i), replayed from CUDA graphs."""
        torch = self.torch
        chunk = min(steps, chunk or max(self.n_sets * 4, 64))
        graphs = []
        sizes = [chunk] * (steps // chunk) + ([steps % chunk] if steps % chunk else [])
        made = {}
        side = torch.cuda.Stream()
        for sz in set(sizes):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(g, stream=side):
                    for i in range(sz):
                        fn(i)
            made[sz] = g
        torch.cuda.synchronize()
        graphs = [made[sz] for sz in sizes]
        st = torch.cuda.current_stream()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st)
        for g in graphs:
            g.replay()
        e1.record(st)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)


def run_ours(args, rank, world, local_rank):
    import torch
    import torch.distributed as dist
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    peaks = load_peaks()
    name = args.workload
    b = Bench(name, dev)
    M, N, K, r = b.M, b.N, b.K, b.r
    ops = 2.0 * M * N * K

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms):
        return max_over_ranks_ms(ms, world, dev)

    W = max(args.warmup, 3)
    for i in range(W):
        b.step(i)
    torch.cuda.synchronize()
    for i in range(b.n_sets):       # every operand set touched once before capture
        b.step(i)
        b.step(i, lowrank=False)
    for L in b.layers:
        b.aser.check_status(L.ws)

    with ClockSampler(local_rank) as clk:
        barrier()
        ms_total = b.time_graph(b.step, args.steps)
        barrier()
        ms_total = max_over_ranks(ms_total)
        # dominant kernel alone (same launch configuration), for the roofline
        ms_lin = b.time_graph(b.linear_only, args.steps) / args.steps
        ms_lin_plain = b.time_graph(lambda i: b.linear_only(i, False), args.steps) / args.steps
        ms_act = b.time_graph(b.quant_only, args.steps) / args.steps
        ms_plain_step = b.time_graph(lambda i: b.step(i, False), args.steps) / args.steps
        # end to end from host buffers through the C ABI
        L0 = b.layers[0]
        for _ in range(3):
            L0.forward_host(b.host_X, b.host_Y)
        torch.cuda.synchronize()
        n_e2e = min(args.steps, 2000)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        for i in range(n_e2e):
            b.layers[i % b.n_sets].forward_host(b.host_X, b.host_Y)
        e1.record()
        torch.cuda.synchronize()
        ms_e2e = max_over_ranks(e0.elapsed_time(e1)) / n_e2e
        clocks = clk.summary()
    for L in b.layers:
        b.aser.check_status(L.ws)

    ms_step = ms_total / args.steps
    tops = whole_job_tops(ops, ms_step, world)
    traffic = NCU_DRAM_BYTES_PER_LAUNCH.get(name)
    bytes_lin = algorithmic_bytes_linear(M, N, K, r)
    if b.bound == "hbm":
        achieved = bytes_lin / (ms_lin * 1e-3) / 1e9
        roof = dict(bound="hbm", achieved=achieved, peak=peaks["hbm_gbs"], unit="GB/s",
                    frac=achieved / peaks["hbm_gbs"], traffic=traffic,
                    peak_source=peaks["source"] + " copy bandwidth")
    else:
        peak = 2.0 * peaks["bf16_tflops"]   # int8 : bf16 dense nominal ratio is 2
        achieved = ops / (ms_lin * 1e-3) / 1e12
        roof = dict(bound="tensor", achieved=achieved, peak=peak, unit="TOP/s",
                    frac=achieved / peak, traffic=traffic,
                    peak_source=peaks["source"] + " bf16 burst x2 (int8:bf16 nominal)",
                    library_int8_gemm_8192_tops=library_int8_gemm_tops(torch, dev))
    roof.update(kernel=dominant_kernel(M, N, K), us_per_launch=ms_lin * 1e3,
                algorithmic_bytes=bytes_lin, ops=ops)

    line = dict(
        metric="aser_w4a8_lowrank_linear_tops", value=tops, unit="TOPS", n_gpus=world,
        steps=args.steps, warmup=W, ms_per_step=ms_step, higher_is_better=True, scaling="weak",
        vs_baseline=None, dtype="int8", data="synthetic",
        config=dict(workload=name, M=M, N=N, K=K, r=r,
                    l2="rotating %d distinct operand sets (%.0f MB) between steps" % (
                        b.n_sets, b.n_sets * (N * K // 2 + 2 * r * (N + K) + 3 * M * K) / 1e6)
                    if b.n_sets > 1 else "operands of one step exceed 2x L2",
                    timing="CUDA-graph replay, CUDA events", replicas=world),
        us_per_call=dict(step=ms_step * 1e3, quant_act=ms_act * 1e3, linear_lr=ms_lin * 1e3,
                         linear_plain=ms_lin_plain * 1e3, step_plain=ms_plain_step * 1e3),
        lowrank_overhead=dict(linear=ms_lin / ms_lin_plain - 1.0, step=ms_step / ms_plain_step - 1.0),
        roofline=roof,
        e2e=dict(value=world * ops / (ms_e2e * 1e-3) / 1e12, unit="TOPS",
                 h2d_bytes_per_step=M * K * 2, d2h_bytes_per_step=M * N * 2,
                 us_per_step=ms_e2e * 1e3, steps=n_e2e),
        gpu_launches=2 * args.steps,
        clocks=clocks,
    )
    if rank == 0 and world == 1 and not args.no_cpu:
        line["cpu_baseline"] = time_oracle(name)
    if rank == 0 and world == 1 and args.extra:
        line["extra_points"] = extra_points(args, dev, peaks, skip=name)
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def extra_points(args, dev, peaks, skip):
    """Other workloads of the sweep, each timed like the headline (kernel pair and GEMM alone)."""
    import torch
    out = []
    for name in ("c2_decode_m1", "c3_prefill_gate_up", "c3_prefill_down", "c5_decode_m16_28672"):
        if name == skip:
            continue
        b = Bench(name, dev)
        M, N, K, r = b.M, b.N, b.K, b.r
        steps = 200 if b.bound == "hbm" else 20
        for i in range(max(3, b.n_sets)):
            b.step(i)
            b.step(i, False)
        torch.cuda.synchronize()
        ms_step = b.time_graph(b.step, steps) / steps
        ms_lin = b.time_graph(b.linear_only, steps) / steps
        ms_plain = b.time_graph(lambda i: b.linear_only(i, False), steps) / steps
        ms_act = b.time_graph(b.quant_only, steps) / steps
        ops = 2.0 * M * N * K
        pt = dict(workload=name, M=M, N=N, K=K, r=r, us_step=ms_step * 1e3, us_linear_lr=ms_lin * 1e3,
                  us_linear_plain=ms_plain * 1e3, us_quant_act=ms_act * 1e3,
                  tops_step=ops / (ms_step * 1e-3) / 1e12, tops_linear=ops / (ms_lin * 1e-3) / 1e12,
                  lowrank_overhead_linear=ms_lin / ms_plain - 1.0)
        if b.bound == "hbm":
            gbs = algorithmic_bytes_linear(M, N, K, r) / (ms_lin * 1e-3) / 1e9
            pt.update(bound="hbm", gbs_linear=gbs, frac=gbs / peaks["hbm_gbs"])
        else:
            pt.update(bound="tensor", frac=pt["tops_linear"] / (2.0 * peaks["bf16_tflops"]))
        pt["quant_act_gbs"] = algorithmic_bytes_act(M, K, r) / (ms_act * 1e-3) / 1e9
        out.append(pt)
        del b
        torch.cuda.empty_cache()
    return out


# ---------------------------------------------------------------------------
# sweeps over the other benchmark configurations (not the headline line)
# ---------------------------------------------------------------------------
class SweepLayer:
    """One weight matrix packed once, stand-in factors of the largest rank, and rolled copies of
    the packed weights; `point(M, r)` gives operand sets (views and fresh intermediates) for one
    (tokens, rank) point, as many as it takes to exceed twice the L2 size between reuses."""

    def __init__(self, dev, cfg, index, N, K, r_max, M_max, gain, sigma, gated=False):
        import torch
        import paper_2411_07762_b200 as aser
        self.torch, self.aser, self.dev = torch, aser, dev
        self.N, self.K, self.r_max = N, K, r_max
        lay = synth.make_layer(M_max, N, K, seed=synth.seed_for(cfg, index), outlier_gain=gain,
                               sigma_w=sigma, n_cal=8, gated_input=gated)
        t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
        self.s = t(synth.standin_smoothing_vector(K, lay.outlier_idx, 24.0))
        L_A, L_B = synth.standin_factors(N, K, max(r_max, 16), seed=lay.meta["seed"],
                                         scale_a=0.01, scale_b=0.01)
        self.L_A, self.L_B = t(L_A), t(L_B)
        Wq, self.w_scale = aser.pack_w4(t(lay.W), self.s)
        self.Wk = [aser.repack_w4(Wq)]
        del Wq
        self.X = t(lay.X)
        torch.cuda.empty_cache()

    def point(self, M, r):
        torch, aser = self.torch, self.aser
        N, K = self.N, self.K
        per_set = N * K // 2 + 2 * r * (N + K) + 3 * M * K + 2 * M * N
        n_sets = 1 if per_set > 2 * L2_BYTES else int(np.ceil(2.2 * L2_BYTES / per_set))
        while len(self.Wk) < n_sets:
            self.Wk.append(torch.roll(self.Wk[0], shifts=8192 * len(self.Wk)))
        sets = []
        for i in range(n_sets):
            L = object.__new__(aser.AserLinear)
            L.N, L.K, L.r, L.s, L.max_tokens = N, K, r, self.s, M
            L.L_A = torch.roll(self.L_A[:r], shifts=i, dims=0).contiguous() if r else None
            L.L_B = torch.roll(self.L_B[:, :r], shifts=i, dims=0).contiguous() if r else None
            L.Wk, L.w_scale = self.Wk[i], self.w_scale
            L.Xq = torch.empty((M, K), dtype=torch.int8, device=self.dev)
            L.a_scale = torch.empty((M,), dtype=torch.float32, device=self.dev)
            L.T = torch.empty((M, max(r, 1)), dtype=torch.bfloat16, device=self.dev)
            L.Y = torch.empty((M, N), dtype=torch.float16, device=self.dev)
            L.ws = aser.new_workspace(M, N, K, r, self.dev)
            X = self.X[:M] if i == 0 else torch.roll(self.X[:M], shifts=i, dims=1).contiguous()
            sets.append((L, X))
        return sets


def time_calls(torch, fn, steps):
    """Device time (us per call) of `steps` calls of fn(i) replayed from one CUDA graph."""
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            for i in range(steps):
                fn(i)
    torch.cuda.synchronize()
    best = float("inf")
    for _ in range(3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        g.replay()
        e1.record()
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1))
    return best * 1e3 / steps


def time_point(torch, aser, sets, M, N, K, r, peaks):
    n = len(sets)
    steps = 240 if M <= 128 else (48 if M <= 1024 else 16)
    steps = max(steps, 2 * n)
    for L, X in sets:                      # warm-up, every operand set touched
        for _ in range(3):
            L(X)
    torch.cuda.synchronize()
    us_step = time_calls(torch, lambda i: sets[i % n][0](sets[i % n][1]), steps)
    us_lin = time_calls(torch, lambda i: sets[i % n][0].linear(M, True), steps)
    us_act = time_calls(torch, lambda i: sets[i % n][0].quant(sets[i % n][1]), steps)
    for L, _ in sets:
        aser.check_status(L.ws)
    ops = 2.0 * M * N * K
    gbs = algorithmic_bytes_linear(M, N, K, r) / (us_lin * 1e-6) / 1e9
    tops = ops / (us_lin * 1e-6) / 1e12
    return dict(M=M, N=N, K=K, r=r, us_step=us_step, us_linear=us_lin, us_quant_act=us_act,
                tops_linear=tops, tops_step=ops / (us_step * 1e-6) / 1e12, gbs_linear=gbs,
                frac_hbm=gbs / peaks["hbm_gbs"], frac_tensor=tops / (2.0 * peaks["bf16_tflops"]),
                quant_act_gbs=algorithmic_bytes_act(M, K, r) / (us_act * 1e-6) / 1e9,
                operand_sets=n)


def library_int8_gemm_tops(torch, dev, n=8192, reps=10):
    """Yardstick only: the vendor library's plain int8 x int8 -> int32 GEMM at n^3 (best of `reps`),
    printed beside the int8 peak that the fractions use (2 x the measured bf16 figure)."""
    try:
        a = torch.randint(-127, 128, (n, n), dtype=torch.int8, device=dev)
        b = torch.randint(-127, 128, (n, n), dtype=torch.int8, device=dev)
        for _ in range(3):
            torch._int_mm(a, b)
        torch.cuda.synchronize()
        best = float("inf")
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            torch._int_mm(a, b)
            e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        return 2.0 * n ** 3 / (best * 1e-3) / 1e12
    except Exception as exc:    # the yardstick is optional; the product path never depends on it
        return "unavailable: %s" % type(exc).__name__


def run_sweep(args, local_rank):
    """`--sweep c4`: the seven linears of a decoder block at 4096 tokens, rank 128, each alone and
    all back to back.  `--sweep c5`: the 70B-class grid (two shapes x five token counts x five
    ranks) with the low-rank overhead against the rank-0 point.  One JSON line."""
    import torch
    import paper_2411_07762_b200 as aser
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    peaks = load_peaks()
    points = []
    lib_int8 = library_int8_gemm_tops(torch, dev)
    with ClockSampler(local_rank) as clk:
        if args.sweep == "c4":
            M, r = 4096, 128
            block = []
            for i, (nm, K, N) in enumerate(synth.DECODER_BLOCK_LINEARS):
                sl = SweepLayer(dev, 4, i, N, K, r, M, 30.0, 0.02)
                sets = sl.point(M, r)
                plain = sl.point(M, 0)
                pt = time_point(torch, aser, sets, M, N, K, r, peaks)
                p0 = time_point(torch, aser, plain, M, N, K, 0, peaks)
                pt.update(layer=nm, us_linear_plain=p0["us_linear"], us_step_plain=p0["us_step"],
                          lowrank_overhead_linear=pt["us_linear"] / p0["us_linear"] - 1.0,
                          lowrank_overhead_step=pt["us_step"] / p0["us_step"] - 1.0)
                points.append(pt)
                block.append(sets[0])
                del plain
            def whole_block(i):
                for L, X in block:
                    L(X)
            us_block = time_calls(torch, whole_block, 8)
            ops_block = sum(2.0 * M * p["N"] * p["K"] for p in points)
            summary = dict(us_block=us_block, sum_of_layers_us=sum(p["us_step"] for p in points),
                           tops_block=ops_block / (us_block * 1e-6) / 1e12,
                           frac_tensor_block=ops_block / (us_block * 1e-6) / 1e12 / (2.0 * peaks["bf16_tflops"]))
        else:
            summary = {}
            for N in (8192, 28672):
                sl = SweepLayer(dev, 5, N // 1024, N, 8192, 256, 4096, 50.0, 0.015)
                for M in (1, 16, 128, 1024, 4096):
                    base = None
                    for r in (0, 32, 64, 128, 256):
                        sets = sl.point(M, r)
                        pt = time_point(torch, aser, sets, M, N, 8192, r, peaks)
                        if r == 0:
                            base = pt
                        pt.update(lowrank_overhead_linear=pt["us_linear"] / base["us_linear"] - 1.0,
                                  lowrank_overhead_step=pt["us_step"] / base["us_step"] - 1.0)
                        points.append(pt)
                        del sets
                        torch.cuda.empty_cache()
                del sl
                torch.cuda.empty_cache()
        clocks = clk.summary()
    line = dict(sweep=args.sweep, unit_time="us per call, CUDA-graph replay, best of 3",
                peaks=dict(hbm_gbs=peaks["hbm_gbs"], int8_tops=2.0 * peaks["bf16_tflops"],
                           source=peaks["source"], library_int8_gemm_8192_tops=lib_int8),
                points=points, clocks=clocks, **summary)
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle timing")
    ap.add_argument("--no-extra", dest="extra", action="store_false",
                    help="skip the additional sweep points")
    ap.add_argument("--sweep", choices=["c4", "c5"], default=None,
                    help="time the decoder-block linears (c4) or the 70B-class grid (c5) instead")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if args.sweep:
        if rank == 0:
            run_sweep(args, local_rank)
        return
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
