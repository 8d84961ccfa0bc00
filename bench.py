#!/usr/bin/env python
"""Benchmark of the ASER W4A8 + low-rank linear forward pass on B200.

One "step" is one pass of the whole hot path over one batch of synthetic tokens: for every
linear layer of the workload, the activation kernel (smooth, int8-quantize, T = X~ L_A^T)
followed by the linear kernel (int4 x int8 GEMM, dequantisation, + T L_B^T, fp16 store),
through the library's public entry points.  The default workload is the largest configuration:
all seven linears of a Llama-3-8B-shaped decoder block at 4096 tokens, rank 128.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line (rank 0).  With N > 1 (launched by torch.distributed.run) every rank runs
an independent replica of the same workload: the path shards over tokens with no exchange
step, so no collective is on the data path; `value` is the sum over ranks.

Timing.  Every quantity is the MEDIAN over at least ten repeats of a CUDA-graph replay bracketed
by CUDA events on the replaying stream.  A repeat of the headline region is exactly `--steps`
steps; a region shorter than 20 ms is replayed back to back inside the same pair of events until
it is longer, so the figures do not depend on `--steps`.  The spread of the repeats is reported.
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
MIN_REGION_MS = 20.0
REPEATS = 10
DATASHEET_INT8_TOPS = 4500.0      # dense int8, vendor figure for this part
DATASHEET_HBM_GBS = 8000.0        # "about 8 TB/s", vendor figure

# A workload is a list of linear layers (name, K, N, input group); layers of one input group read
# the same activation tensor (q/k/v of an attention block, gate/up of an MLP).
WORKLOADS = {
    "c4_decoder_block": dict(cfg=4, M=4096, r=128, gain=30.0, sigma=0.02, bound="tensor",
                             layers=[("q", 4096, 4096, 0), ("k", 4096, 1024, 0), ("v", 4096, 1024, 0),
                                     ("o", 4096, 4096, 1), ("gate", 4096, 14336, 2),
                                     ("up", 4096, 14336, 2), ("down", 14336, 4096, 3)],
                             gated_groups=(3,)),
    "c2_decode_m8": dict(cfg=2, M=8, r=64, gain=30.0, sigma=0.02, bound="hbm",
                         layers=[("proj", 4096, 4096, 0)]),
    "c2_decode_m1": dict(cfg=2, M=1, r=64, gain=30.0, sigma=0.02, bound="hbm",
                         layers=[("proj", 4096, 4096, 0)]),
    "c3_prefill_gate_up": dict(cfg=3, M=2048, r=64, gain=30.0, sigma=0.02, bound="tensor",
                               layers=[("gate_up", 4096, 14336, 0)]),
    "c3_prefill_down": dict(cfg=3, M=2048, r=64, gain=30.0, sigma=0.02, bound="tensor",
                            layers=[("down", 14336, 4096, 0)], gated_groups=(0,)),
    "c5_decode_m16_8192": dict(cfg=5, M=16, r=64, gain=50.0, sigma=0.015, bound="hbm",
                               layers=[("proj", 8192, 8192, 0)]),
    "c5_decode_m16_28672": dict(cfg=5, M=16, r=64, gain=50.0, sigma=0.015, bound="hbm",
                                layers=[("proj", 8192, 28672, 0)]),
    "c5_prefill_m4096_8192": dict(cfg=5, M=4096, r=64, gain=50.0, sigma=0.015, bound="tensor",
                                  layers=[("proj", 8192, 8192, 0)]),
    "c5_prefill_m4096_28672": dict(cfg=5, M=4096, r=64, gain=50.0, sigma=0.015, bound="tensor",
                                   layers=[("proj", 8192, 28672, 0)]),
}
E2E_STREAMS = 4          # streams the end-to-end measurement spreads the layers over
DEFAULT_WORKLOAD = "c4_decoder_block"
EXTRA_POINTS = ("c2_decode_m8", "c2_decode_m1", "c3_prefill_gate_up", "c3_prefill_down",
                "c5_decode_m16_8192", "c5_decode_m16_28672", "c5_prefill_m4096_8192",
                "c5_prefill_m4096_28672")

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel under ncu, taken with
# the kernel as it stands in this tree; the summary with the command is
# profiles/launches_c4_decoder_block_step.txt.  The workload's figure is the average over its
# linear_tc launches; "<workload>/<layers>" is the launch of that layer or fused group.  Workloads
# without a capture of the current kernel report null.
NCU_DRAM_BYTES_PER_LAUNCH = {
    "c4_decoder_block": 1056.9e6 / 5,
    "c4_decoder_block/q+k+v": 36.8e6, "c4_decoder_block/o": 27.6e6, "c4_decoder_block/gate": 166.7e6,
    "c4_decoder_block/up": 189.1e6, "c4_decoder_block/down": 636.9e6,
}


def dominant_kernel(M, N, K):
    """Name of the kernel the library runs for the integer product at this shape (few tokens and
    at most 64 MB of packed weights: the streaming kernel; otherwise the tensor-core kernel)."""
    return "linear_decode_kernel" if M <= 16 and N * K // 2 <= (64 << 20) else "linear_tc_kernel"


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


def workload_ops(w):
    return sum(2.0 * w["M"] * N * K for _, K, N, _ in w["layers"])


def workload_config(name):
    """The `config` object of the JSON line: the workload only, the same for both arms."""
    w = WORKLOADS[name]
    per_step = step_bytes(w)
    return dict(workload=name, tokens=w["M"], rank=w["r"],
                layers=[dict(name=nm, K=K, N=N) for nm, K, N, _ in w["layers"]],
                l2=("operands of one step (%.0f MB) exceed L2" % (per_step / 1e6)) if per_step > 2 * L2_BYTES
                else "distinct operand sets rotated between steps, more than 2x L2 in all")


def step_bytes(w):
    """Device bytes one step touches (weights, factors, activations in and out)."""
    M, r = w["M"], w["r"]
    b = 0
    groups = set()
    for _, K, N, g in w["layers"]:
        b += N * K // 2 + 2 * r * (N + K) + M * K + 2 * M * N
        if g not in groups:
            groups.add(g)
            b += 2 * M * K
    return b


def make_layer_inputs(w, li, index=0):
    """Seeded synthetic tensors of layer `li` of the workload (see aser_synth)."""
    _, K, N, g = w["layers"][li]
    gated = g in w.get("gated_groups", ())
    lay = synth.make_layer(w["M"], N, K, seed=synth.seed_for(w["cfg"], 100 * index + 10 * li + (w["M"] % 7)),
                           outlier_gain=w["gain"], sigma_w=w["sigma"], n_cal=8, gated_input=gated)
    s = synth.standin_smoothing_vector(K, lay.outlier_idx, 24.0)
    L_A, L_B = synth.standin_factors(N, K, w["r"], seed=lay.meta["seed"], scale_a=0.01, scale_b=0.01)
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
        busy = [m for m, u in self.samples if u > 0] or [m for m, _ in self.samples]
        return {"sm_mhz": statistics.median(busy), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(busy)}


# ---------------------------------------------------------------------------
# CPU oracle legs (the only part of this file that touches oracle/)
# ---------------------------------------------------------------------------
def oracle_pass(F, packed, rows):
    """One oracle forward over the first `rows` token rows of every layer of the workload."""
    for X, s, Wq, w_scale, L_A, L_B in packed:
        F.forward(X[:rows], s, Wq, w_scale, L_A, L_B)


def oracle_setup(name):
    from oracle import forward as F
    w = WORKLOADS[name]
    packed = []
    for li in range(len(w["layers"])):
        lay, s, L_A, L_B = make_layer_inputs(w, li)
        q, w_scale = F.quant_w4(lay.W, s)
        packed.append((lay.X, s, F.pack_w4(q), w_scale, L_A, L_B))
    return F, w, packed


def time_oracle(name):
    """The oracle as it stands on the host cores: all cores on up to 1024 token rows of every
    layer (about ten seconds of CPU work on sixteen cores for the decoder block), and a single
    thread on up to 64 rows (a bounded sample; the int product is the plain triple loop)."""
    F, w, packed = oracle_setup(name)
    cores = len(os.sched_getaffinity(0))
    unit_ops = sum(2.0 * N * K for _, K, N, _ in w["layers"])     # per token row
    out = {}
    for label, threads, rows, reps in (("all_cores", cores, min(w["M"], 1024), 1), ("single_thread", 1, min(w["M"], 64), 1)):
        F.set_threads(threads)
        best = float("inf")
        for _ in range(reps):
            t0 = time.perf_counter()
            oracle_pass(F, packed, rows)
            best = min(best, time.perf_counter() - t0)
        out[label] = dict(tops=unit_ops * rows / best / 1e12, seconds=best, rows=rows, threads=threads)
    F.set_threads(1)
    a = out["all_cores"]
    return dict(value=a["tops"], unit="TOPS", cores=cores, kind="oracle",
                sample="first %d of %d token rows of every layer, one run, all stages of the oracle forward"
                       % (a["rows"], w["M"]),
                seconds=a["seconds"],
                single_thread=dict(value=out["single_thread"]["tops"], unit="TOPS",
                                   sample="first %d token rows, one run" % out["single_thread"]["rows"],
                                   seconds=out["single_thread"]["seconds"]))


def run_reference(args, rank, world):
    """`--impl reference`: the CPU oracle, as it stands, on the same workload; each step is a
    bounded sample (64 token rows of every layer) on all host cores."""
    if rank != 0:
        return
    name = args.workload
    F, w, packed = oracle_setup(name)
    cores = len(os.sched_getaffinity(0))
    F.set_threads(cores)
    rows = min(w["M"], 64)
    unit_ops = sum(2.0 * N * K for _, K, N, _ in w["layers"])
    t0 = time.perf_counter()
    oracle_pass(F, packed, rows)
    once = time.perf_counter() - t0
    budget = 90.0                                   # seconds for warm-up plus timed steps
    steps = max(1, min(args.steps, int(budget * 0.8 / once)))
    warm = max(0, min(args.warmup, int(budget * 0.2 / once)))
    for _ in range(warm):
        oracle_pass(F, packed, rows)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_pass(F, packed, rows)
    dt = (time.perf_counter() - t0) / steps
    F.set_threads(1)
    tops = unit_ops * rows / dt / 1e12
    sample = "first %d of %d token rows of every layer per step, %d steps" % (rows, w["M"], steps)
    line = dict(impl="reference", metric="aser_w4a8_lowrank_linear_tops", value=tops, unit="TOPS",
                n_gpus=args.gpus, steps=steps, warmup=warm, ms_per_step=dt * 1e3,
                higher_is_better=True, scaling="weak", vs_baseline=None, dtype="int8",
                data="synthetic", config=workload_config(name),
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


def summarize(samples_ms):
    """Median and spread of repeated timings (ms)."""
    med = statistics.median(samples_ms)
    return dict(median=med, min=min(samples_ms), max=max(samples_ms), repeats=len(samples_ms),
                spread=(max(samples_ms) - min(samples_ms)) / med if med > 0 else 0.0)


# ---------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------
class Model:
    """Device-resident operands of a workload: one AserLinear per layer and one activation
    tensor per input group, in as many distinct operand sets as it takes for a step never to
    find its operands in L2 (one set where a single step already exceeds twice the L2 size).
    Layers of one input group run through aser_forward_shared_cat (one activation pass and one
    linear launch over the group's concatenated output channels; aser_forward_shared, one linear
    launch per layer, where the group cannot be stored fused), a layer alone in its group through
    aser_forward."""

    def __init__(self, name, device):
        import torch
        import paper_2411_07762_b200 as aser
        self.torch, self.aser, self.name = torch, aser, name
        w = WORKLOADS[name]
        self.w = w
        self.M, self.r = w["M"], w["r"]
        per_set = step_bytes(w)
        self.n_sets = 1 if per_set > 2 * L2_BYTES else int(np.ceil(2.2 * L2_BYTES / per_set))
        t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(device)
        self.group_ids = [g for _, _, _, g in w["layers"]]
        self.members = {}                       # input group -> layer indices
        self.fused = {}                         # input group -> stored as one fused projection
        for li, g in enumerate(self.group_ids):
            self.members.setdefault(g, []).append(li)
        base_layers, base_x, group_s = [], {}, {}
        for li, (nm, K, N, g) in enumerate(w["layers"]):
            lay, s, L_A, L_B = make_layer_inputs(w, li)
            if g not in base_x:
                base_x[g] = t(lay.X)
                group_s[g] = t(s)               # the layers of a group share the smoothing vector
            base_layers.append(aser.AserLinear(t(lay.W), group_s[g], t(L_A) if self.r else None,
                                               t(L_B) if self.r else None, self.M))
            del lay
        self.sets = [self._make_set(base_layers, base_x)]
        for i in range(1, self.n_sets):
            # further operand sets: same shapes and value ranges; packed weights are the base
            # set's bytes rolled by a set-dependent offset (contents do not affect timing)
            layers = []
            for b in base_layers:
                L = object.__new__(aser.AserLinear)
                L.__dict__.update(b.__dict__)
                L.Wk = torch.roll(b.Wk, shifts=8192 * i)
                L.w_scale = b.w_scale.clone()
                if self.r:
                    L.L_A = torch.roll(b.L_A, shifts=i, dims=0).contiguous()
                    L.L_B = torch.roll(b.L_B, shifts=i, dims=0).contiguous()
                L.Xq, L.a_scale = torch.empty_like(b.Xq), torch.empty_like(b.a_scale)
                L.T, L.Y = torch.empty_like(b.T), torch.empty_like(b.Y)
                layers.append(L)
            xs = {g: torch.roll(x, shifts=i, dims=1).contiguous() for g, x in base_x.items()}
            self.sets.append(self._make_set(layers, xs))
        torch.cuda.synchronize()

    def _make_set(self, layers, xs):
        """(layers, inputs, shared-input groups with and without the low-rank term)."""
        aser = self.aser
        shared, shared_plain = {}, {}
        for g, idx in self.members.items():
            if len(idx) > 1:
                # One linear launch over the concatenated output channels pays where a layer alone
                # has too few 128 x 128 tiles to fill the SMs evenly (key/value: 256 tiles on 148
                # SMs); with thousands of tiles per layer (gate/up) it measured 6 % slower than
                # one launch per layer, so those groups keep their layers apart.
                tiles = [(self.w["layers"][i][2] // 128) * ((self.M + 127) // 128) for i in idx]
                fused = (len(idx) <= 4 and all(self.w["layers"][i][2] % 128 == 0 for i in idx)
                         and min(tiles) < 4 * 148)
                Group = aser.AserSharedInputCat if fused else aser.AserSharedInput
                self.fused[g] = fused
                shared[g] = Group([layers[i] for i in idx], self.M)
                if self.r:
                    plain = []
                    for i in idx:
                        P = object.__new__(aser.AserLinear)
                        P.__dict__.update(layers[i].__dict__)
                        P.r, P.L_A, P.L_B = 0, None, None
                        plain.append(P)
                    shared_plain[g] = Group(plain, self.M)
                else:
                    shared_plain[g] = shared[g]
        return dict(layers=layers, xs=xs, shared=shared, shared_plain=shared_plain)

    # one whole pass through the public entry points
    def step(self, i, lowrank=True):
        S = self.sets[i % self.n_sets]
        for g, idx in self.members.items():
            if len(idx) > 1:
                (S["shared"] if lowrank else S["shared_plain"])[g](S["xs"][g])
            else:
                S["layers"][idx[0]](S["xs"][g], lowrank)

    def linear_only(self, i, li=None, lowrank=True):
        """The linear launches of a step (a fused group is one launch), or layer `li` on its own."""
        S = self.sets[i % self.n_sets]
        if li is not None:
            S["layers"][li].linear(self.M, lowrank)
            return
        for g, idx in self.members.items():
            if self.fused.get(g):
                (S["shared"] if lowrank else S["shared_plain"])[g].linear(self.M)
            else:
                for j in idx:
                    S["layers"][j].linear(self.M, lowrank)

    def group_linear(self, i, g, lowrank=True):
        S = self.sets[i % self.n_sets]
        if self.fused.get(g):
            (S["shared"] if lowrank else S["shared_plain"])[g].linear(self.M)
        else:
            for j in self.members[g]:
                S["layers"][j].linear(self.M, lowrank)

    def linear_launches(self):
        return sum(1 if self.fused.get(g) else len(idx) for g, idx in self.members.items())

    def quant_only(self, i, g_only=None):
        """The activation passes of a step (one per input group), or of one group."""
        S = self.sets[i % self.n_sets]
        for g, idx in self.members.items():
            if g_only is not None and g != g_only:
                continue
            if len(idx) > 1:
                S["shared"][g].quant(S["xs"][g])
            else:
                S["layers"][idx[0]].quant(S["xs"][g])

    def group_step(self, i, g, lowrank=True):
        S = self.sets[i % self.n_sets]
        idx = self.members[g]
        if len(idx) > 1:
            (S["shared"] if lowrank else S["shared_plain"])[g](S["xs"][g])
        else:
            S["layers"][idx[0]](S["xs"][g], lowrank)

    def launches_per_step(self):
        """Kernels of this library launched by one step: per input group the activation pass
        (as many kernels as the library says it runs at that shape) and one linear kernel per layer
        (one per group where the group is stored fused)."""
        n = 0
        for g, idx in self.members.items():
            K = self.w["layers"][idx[0]][1]
            n += self.aser.forward_act_launches(self.M, K, self.r * len(idx)) + (1 if self.fused.get(g) else len(idx))
        return n

    def check(self):
        for S in self.sets:
            for L in S["layers"]:
                self.aser.check_status(L.ws)
            for G in list(S["shared"].values()) + list(S["shared_plain"].values()):
                self.aser.check_status(G.ws)

    # ---- timing ----
    def capture(self, fn, calls):
        """CUDA graphs that together make exactly `calls` calls fn(0) .. fn(calls - 1)."""
        torch = self.torch
        chunk = max(1, min(calls, max(self.n_sets * 2, 4096 // max(1, 3 * len(self.group_ids)))))
        sizes = [chunk] * (calls // chunk) + ([calls % chunk] if calls % chunk else [])
        side = torch.cuda.Stream()
        graphs, start = [], 0
        for sz in sizes:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(g, stream=side):
                    for i in range(start, start + sz):
                        fn(i)
            graphs.append(g)
            start += sz
        torch.cuda.synchronize()
        return graphs

    def time_region(self, fn, calls, repeats=REPEATS, barrier=None, label=""):
        """Median device time of `calls` calls of fn, as ms per call, with the spread.  One
        repeat replays the captured region (back to back, as often as it takes to last
        MIN_REGION_MS) between two CUDA events on the replaying stream."""
        torch = self.torch
        if os.environ.get("ASER_BENCH_TRACE"):
            print("region %s %s calls=%d" % (self.name, label, calls), file=sys.stderr, flush=True)
        if self.n_sets > 1:      # a region cycles through every operand set: no set returns early
            calls = -(-calls // self.n_sets) * self.n_sets
        graphs = self.capture(fn, calls)
        st = torch.cuda.current_stream()

        def once(n_replays):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(st)
            for _ in range(n_replays):
                for g in graphs:
                    g.replay()
            e1.record(st)
            torch.cuda.synchronize()
            return e0.elapsed_time(e1)

        first = once(1)                                        # also a warm-up of the graphs
        replays = max(1, int(np.ceil(MIN_REGION_MS / max(first, 1e-3))))
        samples = []
        for _ in range(repeats):
            if barrier is not None:
                barrier()
            samples.append(once(replays) / (replays * calls))
        out = summarize(samples)
        out["calls_per_region"] = calls * replays
        return out


def library_int8_gemm_tops(torch, dev, n=8192, reps=10):
    """Yardstick only: the vendor library's plain int8 x int8 -> int32 GEMM at n^3 (best of `reps`),
    a measured s8 x s8 figure printed beside the peaks that the fractions use."""
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


def roofline_of(w, name, us_linear, peaks, lib_int8, li=None, launches=None, layer_idx=None):
    """Roofline object of the integer-product kernel for the whole workload (li None: all its
    launches together) or one layer.  HBM-bound few-token shapes: algorithmic bytes over the
    measured copy bandwidth.  Tensor-bound shapes: 2 M N K over the int8 peak, taken as twice the
    measured bf16 figure (the nominal int8 : bf16 ratio); the kernel is timed inside a replay loop
    of at least 20 ms, so the sustained figure is the denominator, and the burst figure, the
    vendor library's measured int8 GEMM and the data-sheet value are printed beside it."""
    layers = w["layers"] if li is None else [w["layers"][li]]
    if layer_idx is not None:
        layers = [w["layers"][i] for i in layer_idx]
    n_launch = launches if launches is not None else len(layers)
    M, r = w["M"], w["r"]
    ops = sum(2.0 * M * N * K for _, K, N, _ in layers)
    nbytes = sum(algorithmic_bytes_linear(M, N, K, r) for _, K, N, _ in layers)
    secs = us_linear * 1e-6
    _, K0, N0, _ = layers[0]
    key = name if (li is None and layer_idx is None) else "%s/%s" % (name, "+".join(l[0] for l in layers))
    roof = dict(kernel=dominant_kernel(M, N0, K0), launches=n_launch, us_per_launch=us_linear / n_launch,
                algorithmic_bytes=nbytes, ops=ops, algorithmic_bytes_per_launch=nbytes / n_launch,
                traffic=NCU_DRAM_BYTES_PER_LAUNCH.get(key))
    if w["bound"] == "hbm":
        achieved = nbytes / secs / 1e9
        roof.update(bound="hbm", achieved=achieved, peak=peaks["hbm_gbs"], unit="GB/s",
                    frac=achieved / peaks["hbm_gbs"], peak_source=peaks["source"] + " copy bandwidth",
                    frac_of_datasheet_8tbs=achieved / DATASHEET_HBM_GBS)
    else:
        achieved = ops / secs / 1e12
        peak = 2.0 * peaks["bf16_tflops_sustained"]
        roof.update(bound="tensor", achieved=achieved, peak=peak, unit="TOP/s", frac=achieved / peak,
                    peak_source=peaks["source"] + " bf16 sustained x2 (nominal int8:bf16 ratio)",
                    frac_of_burst_x2=achieved / (2.0 * peaks["bf16_tflops"]),
                    frac_of_datasheet_4500=achieved / DATASHEET_INT8_TOPS,
                    library_int8_gemm_8192_tops=lib_int8,
                    frac_of_library_int8=(achieved / lib_int8) if isinstance(lib_int8, float) else None)
    return roof


def measure(m, steps, peaks, lib_int8, barrier=None, max_over_ranks=lambda x: x, per_layer=True):
    """All timed quantities of one workload (ms / us per step or call)."""
    w = m.w
    t_step = m.time_region(m.step, steps, barrier=barrier, label="step")
    ms_step = max_over_ranks(t_step["median"])
    calls = max(1, min(steps, 64))
    t_step_plain = m.time_region(lambda i: m.step(i, False), calls, label="step_plain") if m.r else t_step
    t_lin = m.time_region(m.linear_only, calls, label="linear")
    t_lin_plain = m.time_region(lambda i: m.linear_only(i, None, False), calls, label="linear_plain") if m.r else t_lin
    t_act = m.time_region(m.quant_only, calls, label="quant")
    out = dict(ms_step=ms_step, step=t_step,
               us=dict(step=ms_step * 1e3, step_plain=t_step_plain["median"] * 1e3,
                       quant_act=t_act["median"] * 1e3, linear_lr=t_lin["median"] * 1e3,
                       linear_plain=t_lin_plain["median"] * 1e3),
               spread=dict(step=t_step["spread"], linear_lr=t_lin["spread"], quant_act=t_act["spread"]),
               overhead=dict(linear=t_lin["median"] / t_lin_plain["median"] - 1.0,
                             step=t_step["median"] / t_step_plain["median"] - 1.0),
               roofline=roofline_of(w, m.name, t_lin["median"] * 1e3, peaks, lib_int8, launches=m.linear_launches()))
    act_bytes = sum(algorithmic_bytes_act(w["M"], w["layers"][idx[0]][1], w["r"] * len(idx))
                    for idx in m.members.values())
    out["quant_act_gbs"] = act_bytes / (t_act["median"] * 1e-3) / 1e9
    if per_layer and len(w["layers"]) > 1:
        rows = []
        for li, (nm, K, N, _) in enumerate(w["layers"]):
            tl = m.time_region(lambda i: m.linear_only(i, li), calls, label=nm + " linear")
            tp = m.time_region(lambda i: m.linear_only(i, li, False), calls, label=nm + " linear_plain") if m.r else tl
            ops = 2.0 * w["M"] * N * K
            roof = roofline_of(w, m.name, tl["median"] * 1e3, peaks, lib_int8, li)
            rows.append(dict(layer=nm, K=K, N=N, us_linear_lr=tl["median"] * 1e3,
                             us_linear_plain=tp["median"] * 1e3,
                             tops_linear=ops / (tl["median"] * 1e-3) / 1e12, frac=roof["frac"],
                             traffic=roof["traffic"], algorithmic_bytes=roof["algorithmic_bytes"],
                             lowrank_overhead_linear=tl["median"] / tp["median"] - 1.0))
        out["layers"] = rows
        groups = []
        for g, idx in m.members.items():
            K = w["layers"][idx[0]][1]
            names = "+".join(w["layers"][i][0] for i in idx)
            ta = m.time_region(lambda i: m.quant_only(i, g), calls, label=names + " quant")
            ts = m.time_region(lambda i: m.group_step(i, g), calls, label=names + " step")
            tsp = m.time_region(lambda i: m.group_step(i, g, False), calls, label=names + " step_plain") if m.r else ts
            act_b = algorithmic_bytes_act(w["M"], K, w["r"] * len(idx))
            tgl = m.time_region(lambda i: m.group_linear(i, g), calls, label=names + " linear")
            tglp = m.time_region(lambda i: m.group_linear(i, g, False), calls, label=names + " linear_plain") if m.r else tgl
            groof = roofline_of(w, m.name, tgl["median"] * 1e3, peaks, lib_int8, layer_idx=idx,
                                launches=1 if m.fused.get(g) else len(idx))
            groups.append(dict(layers=names, K=K, stacked_rank=w["r"] * len(idx),
                               fused_linear=bool(m.fused.get(g)), linear_launches=groof["launches"],
                               us_linear_lr=tgl["median"] * 1e3, us_linear_plain=tglp["median"] * 1e3,
                               linear_frac=groof["frac"], linear_traffic=groof["traffic"],
                               linear_algorithmic_bytes=groof["algorithmic_bytes"],
                               us_quant_act=ta["median"] * 1e3, us_step=ts["median"] * 1e3,
                               us_step_plain=tsp["median"] * 1e3,
                               lowrank_overhead_step=ts["median"] / tsp["median"] - 1.0,
                               quant_act_gbs=act_b / (ta["median"] * 1e-3) / 1e9,
                               quant_act_frac_hbm=act_b / (ta["median"] * 1e-3) / 1e9 / peaks["hbm_gbs"]))
        out["input_groups"] = groups
    return out


def warm_l2_point(m):
    """The same step with ONE operand set replayed back to back (weights stay in L2): reported
    for few-token shapes, labelled as L2-warm, never used for a roofline fraction."""
    keep, m.n_sets = m.n_sets, 1
    try:
        t = m.time_region(m.step, 64)
    finally:
        m.n_sets = keep
    return t["median"] * 1e3


def run_ours(args, rank, world, local_rank):
    import torch
    import torch.distributed as dist
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    peaks = load_peaks()
    name = args.workload
    w = WORKLOADS[name]
    m = Model(name, dev)
    ops = workload_ops(w)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    W = max(args.warmup, 3)
    for i in range(max(W, m.n_sets)):       # warm-up; every operand set touched once before capture
        m.step(i)
        if m.r:
            m.step(i, lowrank=False)
    torch.cuda.synchronize()
    m.check()
    lib_int8 = library_int8_gemm_tops(torch, dev) if rank == 0 else None

    with ClockSampler(local_rank) as clk:
        barrier()
        res = measure(m, args.steps, peaks, lib_int8, barrier=barrier if world > 1 else None,
                      max_over_ranks=lambda ms: max_over_ranks_ms(ms, world, dev))
        barrier()
        # end to end from pinned host buffers through the C ABI (aser_forward_host per layer):
        # every step copies each layer's input to the device and its output back.  The layers go
        # out on a few streams in turn (every layer has its own device buffers), so that one layer's
        # copy back overlaps the next layer's copy in and kernels: the link carries both directions.
        layers, xs = m.sets[0]["layers"], m.sets[0]["xs"]
        host_x = {g: x.cpu().pin_memory() for g, x in xs.items()}
        host_y = [torch.empty((m.M, L.N), dtype=torch.float16).pin_memory() for L in layers]
        side = [torch.cuda.Stream(device=dev) for _ in range(E2E_STREAMS)]

        def e2e_step():
            for i, (L, g, y) in enumerate(zip(layers, m.group_ids, host_y)):
                with torch.cuda.stream(side[i % E2E_STREAMS]):
                    L.forward_host(host_x[g], y)

        def e2e_region(n):
            """n steps on the side streams, bracketed by events on the current stream."""
            cur = torch.cuda.current_stream()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(cur)
            for st in side:
                st.wait_event(e0)
            for _ in range(n):
                e2e_step()
            for st in side:
                done = torch.cuda.Event()
                done.record(st)
                cur.wait_event(done)
            e1.record(cur)
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / n
        e2e_region(3)
        samples = []
        n_inner = max(1, int(np.ceil(MIN_REGION_MS / max(res["ms_step"] * 4, 0.05))))
        for _ in range(REPEATS):
            barrier()
            samples.append(e2e_region(n_inner))
        ms_e2e = max_over_ranks_ms(statistics.median(samples), world, dev)
        clocks = clk.summary()
    m.check()

    ms_step = res["ms_step"]
    line = dict(
        metric="aser_w4a8_lowrank_linear_tops", value=whole_job_tops(ops, ms_step, world), unit="TOPS",
        n_gpus=world, steps=args.steps, warmup=W, ms_per_step=ms_step, higher_is_better=True,
        scaling="weak", vs_baseline=None, dtype="int8", data="synthetic", config=workload_config(name),
        timing=dict(method="CUDA-graph replay between CUDA events; median of %d repeats, each exactly "
                           "--steps steps and at least %.0f ms" % (REPEATS, MIN_REGION_MS),
                    step_ms=res["step"], spread=res["spread"], replicas=world,
                    operand_sets=m.n_sets),
        us_per_call=res["us"], lowrank_overhead=res["overhead"], roofline=res["roofline"],
        quant_act_gbs=res["quant_act_gbs"],
        peaks=dict(hbm_gbs=peaks["hbm_gbs"], hbm_datasheet_gbs=DATASHEET_HBM_GBS,
                   int8_tops_sustained_x2=2.0 * peaks["bf16_tflops_sustained"],
                   int8_tops_burst_x2=2.0 * peaks["bf16_tflops"], int8_datasheet_tops=DATASHEET_INT8_TOPS,
                   library_int8_gemm_8192_tops=lib_int8, source=peaks["source"]),
        e2e=dict(value=world * ops / (ms_e2e * 1e-3) / 1e12, unit="TOPS",
                 h2d_bytes_per_step=sum(m.M * K * 2 for _, K, _, _ in w["layers"]),
                 d2h_bytes_per_step=sum(m.M * N * 2 for _, _, N, _ in w["layers"]),
                 us_per_step=ms_e2e * 1e3, steps=REPEATS * n_inner, streams=E2E_STREAMS),
        gpu_launches=m.launches_per_step() * args.steps,
        clocks=clocks,
    )
    if "layers" in res:
        line["layers"] = res["layers"]
        line["input_groups"] = res["input_groups"]
    if w["bound"] == "hbm":
        line["l2_warm_us_step"] = warm_l2_point(m)
    del m
    torch.cuda.empty_cache()
    if rank == 0 and world == 1 and args.extra:
        line["extra_points"] = extra_points(dev, peaks, lib_int8, skip=name)
        line["variants"] = variant_points(dev)
    if rank == 0 and world == 1 and not args.no_cpu:
        line["cpu_baseline"] = time_oracle(name)
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def extra_points(dev, peaks, lib_int8, skip):
    """The other configurations, each measured like the headline: own roofline object, low-rank
    overhead of the kernel and of the step, and for few-token shapes the L2-warm step time."""
    import torch
    out = []
    for name in EXTRA_POINTS:
        if name == skip:
            continue
        w = WORKLOADS[name]
        m = Model(name, dev)
        for i in range(max(3, m.n_sets)):
            m.step(i)
            m.step(i, False)
        torch.cuda.synchronize()
        steps = 64 if w["bound"] == "hbm" else 8
        res = measure(m, steps, peaks, lib_int8, per_layer=False)
        m.check()
        _, K, N, _ = w["layers"][0]
        pt = dict(workload=name, M=w["M"], N=N, K=K, r=w["r"], us_per_call=res["us"],
                  tops_step=workload_ops(w) / (res["ms_step"] * 1e-3) / 1e12,
                  lowrank_overhead=res["overhead"], roofline=res["roofline"],
                  quant_act_gbs=res["quant_act_gbs"], spread=res["spread"], operand_sets=m.n_sets)
        if w["bound"] == "hbm":
            pt["l2_warm_us_step"] = warm_l2_point(m)
        out.append(pt)
        del m
        torch.cuda.empty_cache()
    return out


def time_callable(torch, fn, calls=8, repeats=REPEATS):
    """Median ms per call of fn() replayed from a CUDA graph (regions of at least MIN_REGION_MS)."""
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            for _ in range(calls):
                fn()
    torch.cuda.synchronize()

    def once(n):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)
    n = max(1, int(np.ceil(MIN_REGION_MS / max(once(1), 1e-3))))
    return statistics.median(once(n) / (n * calls) for _ in range(repeats))


def variant_points(dev):
    """The paper's own variant beside the default, on one 4096 x 4096 layer at 2048 tokens, rank 64,
    512 calibration tokens, factors built on the device (aser_construct):
      default  smoothing s = sqrt(max|X_c| / max|W_c|) on the seeded outlier channels, all columns
               quantized, T in bf16;
      split    the paper's m_i = mean|X_i| / min over the f = 32 outlier channels of
               mean|X| * mean|W| (Sec. 4.2 Eq. 11), those columns kept out of the int4 matrix and
               carried by the factors (Eq. 12), T as bf16 pairs (rank 128 in the linear kernel).
    Reports the time of a step and the reconstruction error ||Y - X W^T||_F / ||X W^T||_F against
    the fp32 product of the fp16 operands, with plain W4A8 (no factors) as the yardstick."""
    import torch
    import paper_2411_07762_b200 as aser
    N = K = 4096
    M, r, f = 2048, 64, 32
    lay = synth.make_layer(M, N, K, seed=synth.seed_for(2, 4242), outlier_gain=30.0, sigma_w=0.02, n_cal=512)
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    W, X, Xc = t(lay.W), t(lay.X), t(lay.X_cal)
    exact = X.float() @ W.float().t()
    den = float(exact.norm())
    out = {}
    # default
    idx = torch.from_numpy(lay.outlier_idx).to(dev)
    s = torch.ones(K, dtype=torch.float32, device=dev)
    s[idx] = torch.sqrt(Xc[:, idx].float().abs().amax(0) / W[:, idx].float().abs().amax(0))
    c = aser.construct(W, s, Xc, r)
    layer = aser.AserLinear(W, s, c["L_A"].contiguous(), c["L_B"], M)
    assert torch.equal(layer.Wq, c["Wq"])
    Y = layer(X).float()
    out["default"] = dict(rel_error=float((Y - exact).norm()) / den, us_step=time_callable(torch, lambda: layer(X)) * 1e3)
    Yp = layer(X, lowrank=False).float()
    out["plain_w4a8"] = dict(rel_error=float((Yp - exact).norm()) / den,
                             us_step=time_callable(torch, lambda: layer(X, lowrank=False)) * 1e3)
    # the paper's smoothing rule and outlier split
    xbar, wbar = Xc.float().abs().mean(0), W.float().abs().mean(0)
    idx_f = torch.topk(xbar * wbar, f).indices.sort().values
    m = torch.ones(K, dtype=torch.float32, device=dev)
    m[idx_f] = xbar[idx_f] / xbar[idx_f].min()
    c2 = aser.construct(W, m, Xc, r, split_idx=idx_f.to(torch.int32))
    Wk = aser.repack_w4(c2["Wq"])
    LA2, LB2 = c2["L_A"].contiguous(), aser.pair_up_projection(c2["L_B"])
    ws = aser.new_workspace(M, N, K, 2 * r)
    bufs = (torch.empty((M, K), dtype=torch.int8, device=dev), torch.empty((M,), dtype=torch.float32, device=dev),
            torch.empty((M, 2 * r), dtype=torch.bfloat16, device=dev))
    Y2 = torch.empty((M, N), dtype=torch.float16, device=dev)

    def split_step():
        Xq, sc, T = aser.quant_act_ws(X, m, LA2, ws=ws, out=bufs, t_pair=True)
        aser.linear_w4a8_lr(Xq, sc, Wk, c2["w_scale"], T, LB2, N, ws, Y=Y2)
    split_step()
    aser.check_status(ws)
    out["paper_split"] = dict(rel_error=float((Y2.float() - exact).norm()) / den,
                              us_step=time_callable(torch, split_step) * 1e3, f=f)
    out["shape"] = dict(M=M, N=N, K=K, r=r, n_cal=512)
    return out


# ---------------------------------------------------------------------------
# the 70B-class grid (not the headline line)
# ---------------------------------------------------------------------------
def run_sweep(args, local_rank):
    """`--sweep c5`: two shapes x five token counts x five ranks with the low-rank overhead
    against the rank-0 point.  One JSON line."""
    import torch
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    peaks = load_peaks()
    lib_int8 = library_int8_gemm_tops(torch, dev)
    points = []
    with ClockSampler(local_rank) as clk:
        for N in (8192, 28672):
            for M in (1, 16, 128, 1024, 4096):
                base = None
                for r in (0, 32, 64, 128, 256):
                    nm = "sweep_c5_%d_%d_%d" % (N, M, r)
                    WORKLOADS[nm] = dict(cfg=5, M=M, r=r, gain=50.0, sigma=0.015,
                                         bound="hbm" if M <= 16 else "tensor",
                                         layers=[("proj", 8192, N, 0)])
                    m = Model(nm, dev)
                    for i in range(max(3, m.n_sets)):
                        m.step(i)
                    torch.cuda.synchronize()
                    calls = 64 if M <= 128 else 8
                    t_step = m.time_region(m.step, calls, repeats=5)
                    t_lin = m.time_region(m.linear_only, calls, repeats=5)
                    t_act = m.time_region(m.quant_only, calls, repeats=5)
                    m.check()
                    ops = 2.0 * M * N * 8192
                    us_lin, us_step = t_lin["median"] * 1e3, t_step["median"] * 1e3
                    pt = dict(M=M, N=N, K=8192, r=r, us_step=us_step, us_linear=us_lin,
                              us_quant_act=t_act["median"] * 1e3,
                              tops_linear=ops / (us_lin * 1e-6) / 1e12,
                              gbs_linear=algorithmic_bytes_linear(M, N, 8192, r) / (us_lin * 1e-6) / 1e9,
                              operand_sets=m.n_sets)
                    pt["frac_hbm"] = pt["gbs_linear"] / peaks["hbm_gbs"]
                    pt["frac_tensor"] = pt["tops_linear"] / (2.0 * peaks["bf16_tflops_sustained"])
                    if r == 0:
                        base = pt
                    pt.update(lowrank_overhead_linear=us_lin / base["us_linear"] - 1.0,
                              lowrank_overhead_step=us_step / base["us_step"] - 1.0)
                    points.append(pt)
                    del m
                    del WORKLOADS[nm]
                    torch.cuda.empty_cache()
        clocks = clk.summary()
    line = dict(sweep=args.sweep, unit_time="us per call, CUDA-graph replay, median of 5 repeats of >= 20 ms",
                peaks=dict(hbm_gbs=peaks["hbm_gbs"], int8_tops_sustained_x2=2.0 * peaks["bf16_tflops_sustained"],
                           int8_tops_burst_x2=2.0 * peaks["bf16_tflops"], source=peaks["source"],
                           library_int8_gemm_8192_tops=lib_int8),
                points=points, clocks=clocks)
    print(json.dumps(line), flush=True)


def run_profile(args, local_rank):
    """Plain launches for a profiler (no graphs, no timing): `--profile step` runs whole steps,
    `--profile <layer>` only that layer's activation pass and linear kernel."""
    import torch
    torch.cuda.set_device(local_rank)
    m = Model(args.workload, torch.device("cuda", local_rank))
    names = [nm for nm, _, _, _ in m.w["layers"]]
    if args.profile != "step" and args.profile not in names:
        raise SystemExit("--profile takes 'step' or one of %s" % names)
    per = m.launches_per_step()
    for i in range(args.warmup + args.steps):
        if args.profile == "step":
            m.step(i)
        else:
            li = names.index(args.profile)
            S = m.sets[i % m.n_sets]
            S["layers"][li](S["xs"][m.group_ids[li]])
            per = m.aser.forward_act_launches(m.M, m.w["layers"][li][1], m.r) + 1
    torch.cuda.synchronize()
    m.check()
    print(json.dumps(dict(profile=args.profile, workload=args.workload, launches_per_iteration=per,
                          warmup=args.warmup, steps=args.steps)), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle timing")
    ap.add_argument("--no-extra", dest="extra", action="store_false",
                    help="skip the other configurations' points")
    ap.add_argument("--profile", default=None, metavar="WHAT",
                    help="for a profiler: run W warm-up steps and K steps eagerly and exit, printing nothing "
                         "but the launch count ('step' = whole steps, or a layer name = that layer's "
                         "activation pass and linear kernel only)")
    ap.add_argument("--sweep", choices=["c5"], default=None,
                    help="time the 70B-class grid (two shapes x five token counts x five ranks) instead")
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
    if args.profile:
        if rank == 0:
            run_profile(args, local_rank)
        return
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
