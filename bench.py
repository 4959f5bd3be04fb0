#!/usr/bin/env python
"""Benchmark of the DGQ hot path on one B200 (or N independent replicas, one per rank).

One step = one pass of the whole path over one batch of synthetic, seeded tensors shaped like
the 64x64-latent level of the Stable Diffusion v1.4 UNet at batch 2 (classifier-free guidance):

  * transformer-block linears, W8A8, per-token dynamic activation scales over 8 calibrated
    channel groups: activation quantizer + proj_in, q/k/v (one quantizer call feeds three
    projections, stacked into a single 320 -> 960 GEMM), out (320 -> 320), GEGLU FF 320 -> 2560 and
    1280 -> 320, 8192 tokens;
  * cross-attention with prompt-specific log2 score quantization, B = 2, 8 heads,
    4096 queries x 40, 77 keys, 8-bit scores;
  * the level's ResBlock 3x3 convolution, 320 -> 320 on 2 x 64 x 64, W4A6, 16 channel groups,
    as an implicit GEMM (activation quantizer + conv).

Calibration and weight preparation are offline and untimed.  Buffers rotate over enough
distinct sets that the footprint exceeds L2, so the timed kernels read HBM.

`value` is the algorithmic int8 throughput of the whole step (2 M N K_real of every GEMM and
conv, divided by the full step time including quantizers and attention).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2501_04304_b200 import synth  # noqa: E402

SEED = 1
TOKENS, BATCH = 4096, 2
M = TOKENS * BATCH
LINEARS = [  # name, N, K, input id
    # q, k and v read the same quantized activation: their weights are stacked into one 320 -> 960 GEMM
    ("proj_in", 320, 320, "a"), ("qkv", 960, 320, "b"),
    ("out", 320, 320, "c"), ("ff1", 2560, 320, "d"), ("ff2", 320, 1280, "e"),
]
INPUT_C = {"a": 320, "b": 320, "c": 320, "d": 320, "e": 1280}
ATT = dict(B=2, H=8, nq=4096, nk=77, d=40, bits=8)
CONV = dict(n=2, h=64, w=64, c=320, N=320)
WORKLOAD = ("sdv14_64x64_level_batch2: W8A8 transformer linears (proj_in, q/k/v stacked 320->960, out 320->320, FF 320->2560, "
            "1280->320; 8192 tokens; dynamic per-token scales, 8 channel groups) + log2 cross-attention "
            "(B2 H8 nq4096 d40 nk77, 8-bit) + W4A6 3x3 conv 320->320 on 2x64x64 (16 groups)")


def gemm_ops():
    ops = sum(2.0 * M * N * K for _, N, K, _ in LINEARS)
    ops += 2.0 * CONV["n"] * CONV["h"] * CONV["w"] * CONV["N"] * 9 * CONV["c"]
    return ops


def attn_bytes():
    a = ATT
    return 2.0 * a["B"] * a["nq"] * a["H"] * a["d"] * 2 + 2.0 * a["B"] * a["nk"] * a["H"] * a["d"] * 2


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm=float(d["hbm_gbs"]), bf16=float(d["bf16_tflops"]),
                    bf16_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


# Plain-ALU bound of the per-group epilogue: every accumulator element of every channel group takes one
# int32 -> fp32 conversion, which the SM issues at 16 per clock and sub-partition (64 per SM).
CVT_PER_CLK_SM = 64


def alu_peak_gelems(n_sm=148, sm_mhz=1965.0):
    """Conversions per second of the whole GPU, in 1e9 elements / s."""
    return CVT_PER_CLK_SM * n_sm * sm_mhz * 1e6 / 1e9


def gemm_launch_rooflines(peaks, int8_peak_tops, n_sm, sm_mhz):
    """Per GEMM launch of the step: (ops, bytes, group elements) and its own roofline time in us: the slowest of
    tensor, HBM and epilogue-conversion time."""
    out = []
    alu = alu_peak_gelems(n_sm, sm_mhz)
    for name, N, K, key in LINEARS:
        ops, byts, el = 2.0 * M * N * K, M * K + N * K + 2.0 * M * N, float(M) * N * 8
        out.append((name, ops, byts, el))
    c = CONV
    Mc = c["n"] * c["h"] * c["w"]
    out.append(("conv", 2.0 * Mc * c["N"] * 9 * c["c"], Mc * c["c"] + c["N"] * 9 * c["c"] / 2 + 2.0 * Mc * c["N"],
                float(Mc) * c["N"] * 16))
    res = []
    for name, ops, byts, el in out:
        t = {"tensor": ops / int8_peak_tops / 1e6, "hbm": byts / peaks["hbm"] / 1e3, "alu": el / alu / 1e3}
        bound = max(t, key=t.get)
        res.append({"launch": name, "bound": bound, "roofline_us": t[bound], "t_us": t})
    return res


class ClockSampler(threading.Thread):
    """Samples SM clocks and throttle reasons with ONE long-running `nvidia-smi -lms` child, started before
    the warm-up so that no process is spawned while a timed region runs; `mark()` opens the window whose
    samples are reported."""

    QUERY = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.rows, self.t_mark, self.proc = index, [], None, None

    def run(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "50"], stdout=subprocess.PIPE, text=True)
            for line in self.proc.stdout:
                f = [x.strip() for x in line.strip().split(",")]
                if len(f) >= 6:
                    self.rows.append((time.monotonic(), f))
        except Exception:
            pass

    def mark(self):
        self.t_mark = time.monotonic()

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()      # the exact child this object started
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
        self.join(timeout=5)
        rows = [f for t, f in self.rows if self.t_mark is None or t >= self.t_mark] or [f for _, f in self.rows[-1:]]
        mhz, reasons, max_mhz = [], set(), None
        for f in rows:
            try:
                mhz.append(float(f[0]))
                max_mhz = float(f[1])
            except ValueError:
                continue
            for n, v in zip(self.NAMES, f[2:]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(mhz)) if mhz else None, "sm_max_mhz": max_mhz, "reasons": sorted(reasons),
                "samples": len(mhz)}


# ------------------------------------------------------------------------------------------ CUDA arm
class Workload:
    """Calibrated layers, prepared weights and rotating buffer sets on one GPU."""

    def __init__(self, torch, b, n_sets):
        self.torch, self.b, self.n_sets = torch, b, n_sets
        dev = "cuda"
        self.groups, self.weights, self.biases = {}, {}, {}
        # one grouping per distinct layer input; calibrated on 4 further draws
        for key, C in INPUT_C.items():
            Xcal = torch.from_numpy(synth.activations(SEED, 100 + ord(key), 4, TOKENS, C)).to(dev)
            self.groups[key] = b.calibrate_groups(Xcal, TOKENS, 8, 8, b.DIM_CHANNEL)
            del Xcal
        for i, (name, N, K, key) in enumerate(LINEARS):
            W = torch.from_numpy(synth.weights(SEED, 200 + i, N, K)).to(dev)
            self.weights[name] = b.weight_prepare(self.groups[key], W, 8)
            self.biases[name] = torch.from_numpy(synth.bias(SEED, 300 + i, N)).to(dev)
        c = CONV
        Xcal = torch.from_numpy(synth.activations(SEED, 150, 4, c["h"] * c["w"], c["c"], token_outliers=False)).to(dev)
        self.conv_groups = b.calibrate_groups(Xcal, c["h"] * c["w"], 6, 16, b.DIM_CHANNEL)
        del Xcal
        self.conv_desc = (c["n"], c["h"], c["w"], c["c"])
        Wc = torch.from_numpy(synth.conv_weights(SEED, 250, c["N"], c["c"])).to(dev)
        self.conv_weight = b.weight_prepare(self.conv_groups, Wc, 4, conv=self.conv_desc)
        self.conv_bias = torch.from_numpy(synth.bias(SEED, 350, c["N"])).to(dev)
        self.conv_ws = torch.empty(b.linear_workspace_bytes(self.conv_groups, self.conv_weight, M), dtype=torch.uint8,
                                   device=dev)   # the 4-bit conv weights are expanded into it by every call
        # host inputs (pinned) and device buffer sets
        self.host = {}
        for key, C in INPUT_C.items():
            self.host[key] = torch.from_numpy(synth.activations(SEED, 10 + ord(key), BATCH, TOKENS, C)).pin_memory()
        self.host["conv"] = torch.from_numpy(
            synth.activations(SEED, 60, c["n"], c["h"] * c["w"], c["c"], token_outliers=False)).pin_memory()
        a = ATT
        Q, K, V = synth.attention_inputs(SEED, a["B"], a["H"], a["nq"], a["nk"], a["d"])
        self.host["Q"], self.host["K"], self.host["V"] = [torch.from_numpy(x).pin_memory() for x in (Q, K, V)]
        ws_bytes = b.cross_attn_workspace_bytes(a["B"], a["H"], a["nq"], a["nk"], a["d"])
        self.sets = []
        for _ in range(n_sets):
            s = {"in": {k: v.to(dev) for k, v in self.host.items()}}
            s["codes"], s["ds"], s["dz"] = {}, {}, {}
            for key in INPUT_C:
                g = self.groups[key]
                s["codes"][key] = torch.empty((M, g.K_pad), dtype=torch.uint8, device=dev)
                s["ds"][key] = torch.empty((M, g.G), dtype=torch.float32, device=dev)
                s["dz"][key] = torch.empty((M, g.G), dtype=torch.int32, device=dev)
            s["conv_codes"] = torch.empty((M, self.conv_groups.K_pad), dtype=torch.uint8, device=dev)
            s["out"] = {name: torch.empty((M, N), dtype=torch.float16, device=dev) for name, N, _, _ in LINEARS}
            s["conv_out"] = torch.empty((M, c["N"]), dtype=torch.float16, device=dev)
            s["attn_out"] = torch.empty((a["B"], a["nq"], a["H"], a["d"]), dtype=torch.float16, device=dev)
            s["attn_ws"] = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
            self.sets.append(s)
        self.host_out = {k: torch.empty((M, 320), dtype=torch.float16).pin_memory() for k in ("ff2", "conv")}
        self.host_out["attn"] = torch.empty((a["B"], a["nq"], a["H"], a["d"]), dtype=torch.float16).pin_memory()

    def set_bytes(self):
        tot = 0
        s = self.sets[0]
        for v in list(s["in"].values()) + list(s["codes"].values()) + list(s["out"].values()) + \
                [s["conv_codes"], s["conv_out"], s["attn_out"]]:
            tot += v.numel() * v.element_size()
        return tot

    KINDS = ("quantize", "gemm", "attention")
    KIND_STEPS = 6

    def launch_kind(self, kind, i):
        """Enqueues the kernels of one kind of one step on buffer set i (order of a step: every
        activation quantizer, then every GEMM and the conv, then the cross-attention)."""
        b = self.b
        s = self.sets[i % self.n_sets]
        if kind == "quantize":
            for key in INPUT_C:
                b.quantize_act_into(self.groups[key], s["in"][key], s["codes"][key], s["ds"][key], s["dz"][key],
                                    mode=b.MODE_DYNAMIC_TOKEN)
            b.quantize_act_into(self.conv_groups, s["in"]["conv"], s["conv_codes"], None, None,
                                layout=b.CODES_S8_CENTRED)
        elif kind == "gemm":
            for name, N, K, key in LINEARS:
                b.linear(self.groups[key], self.weights[name], s["codes"][key], mode=b.MODE_DYNAMIC_TOKEN,
                         dyn_scale=s["ds"][key], dyn_zp=s["dz"][key], bias=self.biases[name], out=s["out"][name])
            b.linear(self.conv_groups, self.conv_weight, s["conv_codes"], layout=b.CODES_S8_CENTRED,
                     bias=self.conv_bias, out=s["conv_out"], conv=self.conv_desc, workspace=self.conv_ws)
        else:
            b.cross_attn_logq(s["in"]["Q"], s["in"]["K"], s["in"]["V"], ATT["bits"], out=s["attn_out"],
                              workspace=s["attn_ws"])

    def step(self, i):
        for kind in self.KINDS:
            self.launch_kind(kind, i)

    def capture(self):
        """Per buffer set: one CUDA graph of the whole step (what `value` is timed on).  Per kind: one
        graph that holds that kind's launches of KIND_STEPS consecutive steps (rotating over the buffer
        sets), which the per-kernel split is timed on: the boundary between two graph replays is then
        paid once per KIND_STEPS steps and not once per step."""
        torch = self.torch
        self.step_graphs, self.stream = [], torch.cuda.Stream()
        with torch.cuda.stream(self.stream):
            n0 = self.b.launch_count()
            for i in range(self.n_sets):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=self.stream):
                    self.step(i)
                self.step_graphs.append(g)
            self.launches_per_step = (self.b.launch_count() - n0) // self.n_sets
            self.kind_graphs = {}
            for kind in self.KINDS:
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=self.stream):
                    for i in range(self.KIND_STEPS):
                        self.launch_kind(kind, i)
                self.kind_graphs[kind] = g
        torch.cuda.synchronize()

    def replay_whole_step(self, i):
        self.step_graphs[i % self.n_sets].replay()

    def replay_kinds(self, marks=None):
        """KIND_STEPS steps' worth of work, kind by kind."""
        for kind in self.KINDS:
            if marks is not None:
                e = self.torch.cuda.Event(enable_timing=True)
                e.record()
                marks.append((kind, e))
            self.kind_graphs[kind].replay()

    def run_e2e(self, steps):
        """`steps` steps through host buffers, pipelined over three streams as a serving loop would be: the
        inputs of step i + 1 travel host -> device while step i computes and the results of step i - 1
        travel back.  Every step still copies all of its inputs from pinned host memory and reads all of
        its results back; a buffer set is reused only after the step that last used it has been read back.
        Returns (start event, end event): start is recorded before the first copy, end after the last read."""
        torch = self.torch
        if not hasattr(self, "e2e_streams"):
            self.e2e_streams = [torch.cuda.Stream() for _ in range(3)]
        s_in, s_run, s_out = self.e2e_streams
        cur = torch.cuda.current_stream()
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record(cur)
        for st in (s_in, s_run, s_out):
            st.wait_event(start)
        read_back = [None] * self.n_sets        # per buffer set: event "results of its last step are on the host"
        for i in range(steps):
            k = i % self.n_sets
            s = self.sets[k]
            with torch.cuda.stream(s_in):
                if read_back[k] is not None:
                    s_in.wait_event(read_back[k])
                for name, h in self.host.items():
                    s["in"][name].copy_(h, non_blocking=True)
                ev_in = torch.cuda.Event()
                ev_in.record(s_in)
            with torch.cuda.stream(s_run):
                s_run.wait_event(ev_in)
                self.step_graphs[k].replay()
                ev_run = torch.cuda.Event()
                ev_run.record(s_run)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_run)
                self.host_out["ff2"].copy_(s["out"]["ff2"], non_blocking=True)
                self.host_out["conv"].copy_(s["conv_out"], non_blocking=True)
                self.host_out["attn"].copy_(s["attn_out"], non_blocking=True)
                read_back[k] = torch.cuda.Event()
                read_back[k].record(s_out)
        for st in (s_in, s_run, s_out):
            cur.wait_stream(st)
        end.record(cur)
        return start, end

    def h2d_bytes(self):
        return int(sum(h.numel() * h.element_size() for h in self.host.values()))

    def d2h_bytes(self):
        return int(sum(h.numel() * h.element_size() for h in self.host_out.values()))


def max_over_ranks(values, world, device):
    """Replicas only: every rank times the same work on its own GPU; the job's time is the slowest rank's."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_rate(ops_per_replica, ms_per_step, world):
    """Whole-job TOPS: `world` replicas each do `ops_per_replica` per step in `ms_per_step` (max over ranks)."""
    return world * ops_per_replica / (ms_per_step * 1e-3) / 1e12


# DRAM bytes (read + written) of the six GEMM launches of one step, from one ncu capture of this
# benchmark (profiles/gq_gemm_kernel_bench_step_dram.md).  Valid only for the kernel sources it was
# taken with: any change to them turns the figure back into null.
GEMM_DRAM_BYTES_PER_STEP = 42_431_744
GEMM_SOURCES = ("paper_2501_04304_b200/csrc/linear.cuh", "paper_2501_04304_b200/csrc/common.cuh")
GEMM_SOURCES_SHA1 = "cb05aa9bf599a217ec061b934c553c7f4274a0cb"


def gemm_traffic():
    import hashlib
    h = hashlib.sha1()
    try:
        for f in GEMM_SOURCES:
            with open(os.path.join(ROOT, f), "rb") as fh:
                h.update(fh.read())
    except OSError:
        return None
    return GEMM_DRAM_BYTES_PER_STEP if h.hexdigest() == GEMM_SOURCES_SHA1 else None


def run_cuda(args):
    import torch
    import torch.distributed as dist
    from paper_2501_04304_b200 import binding as b

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    b.lib()  # fails loudly if the extension is missing

    n_sets = 3
    wl = Workload(torch, b, n_sets)
    l2_bytes = torch.cuda.get_device_properties(local).L2_cache_size
    assert wl.set_bytes() * n_sets > 2 * l2_bytes

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    sampler.start()
    for i in range(3):
        wl.step(i)
    barrier()
    wl.capture()
    for i in range(max(args.warmup, 3)):
        wl.replay_whole_step(i)
    for _ in range(2):
        wl.replay_kinds()
    barrier()
    # A step lasts a fraction of a millisecond: the K timed steps are preceded by about a second of untimed
    # replays of the same graphs, so that the clock record below has tens of samples taken under this load.
    sampler.mark()
    t_load = time.monotonic()
    i_load = 0
    while time.monotonic() - t_load < 1.0:
        for _ in range(200):
            wl.replay_whole_step(i_load)
            i_load += 1
        torch.cuda.synchronize()
    # timed region: K whole steps, one graph replay each
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for i in range(args.steps):
        wl.replay_whole_step(i)
    e1.record()
    barrier()
    launches = wl.launches_per_step * args.steps
    ms_total = e0.elapsed_time(e1)
    # at least K steps again, one graph per kind with an event in between, for the per-kernel split
    marks = []
    k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    kind_replays = max(1, -(-args.steps // wl.KIND_STEPS))
    kind_steps = kind_replays * wl.KIND_STEPS
    k0.record()
    for _ in range(kind_replays):
        wl.replay_kinds(marks)
    k1.record()
    barrier()
    # end to end: host buffers in, results out, every step
    wl.run_e2e(3)
    barrier()
    e2, e3 = wl.run_e2e(args.steps)
    barrier()
    ms_e2e = e2.elapsed_time(e3)
    clocks = sampler.stop()
    status = b.device_status()
    if status != 0:
        raise RuntimeError(f"a kernel recorded status {status} ({b.status_string(status)})")

    # duration of a kind = from its mark to the next mark (or to the end of the timed region)
    kind_ms = {}
    for j, (kind, ev) in enumerate(marks):
        nxt = marks[j + 1][1] if j + 1 < len(marks) else k1
        kind_ms.setdefault(kind, []).append(ev.elapsed_time(nxt))
    ms_total, ms_e2e = max_over_ranks([ms_total, ms_e2e], world, "cuda")
    ms_step = ms_total / args.steps
    ops = gemm_ops()
    value = whole_job_rate(ops, ms_step, world)
    e2e_value = whole_job_rate(ops, ms_e2e / args.steps, world)
    peaks = measured_peaks()
    int8_peak = 2.0 * peaks["bf16_sustained"]          # int8 : bf16 dense nominal ratio 4.5 : 2.25
    gemm_ms = sum(kind_ms["gemm"]) / kind_steps        # all GEMM launches of one step
    gemm_tops = ops / (gemm_ms * 1e-3) / 1e12
    attn_ms = sum(kind_ms["attention"]) / kind_steps
    quant_ms = sum(kind_ms["quantize"]) / kind_steps
    quant_bytes = 3.0 * (M * sum(INPUT_C.values()) + M * CONV["c"])
    props = torch.cuda.get_device_properties(local)
    sm_mhz = clocks.get("sm_max_mhz") or 1965.0
    int8_burst = 2.0 * peaks["bf16"]
    launches_rf = gemm_launch_rooflines(peaks, int8_peak, props.multi_processor_count, sm_mhz)
    # the resource that binds most of the step's GEMM time, and the step's GEMM roofline = sum of the launches' own
    sums = {k: sum(l["t_us"][k] for l in launches_rf) for k in ("tensor", "hbm", "alu")}
    bound = max(sums, key=sums.get)
    own_us = sum(l["roofline_us"] for l in launches_rf)
    gemm_elems = sum(float(M) * N * 8 for _, N, _, _ in LINEARS) + float(M) * CONV["N"] * 16
    gemm_bytes = sum(M * K + N * K + 2.0 * M * N for _, N, K, _ in LINEARS) + M * CONV["c"] + CONV["N"] * 9 * CONV["c"] / 2 \
        + 2.0 * M * CONV["N"]
    if bound == "tensor":
        ach, peak, unit = gemm_tops, int8_peak, "TOP/s"
    elif bound == "hbm":
        ach, peak, unit = gemm_bytes / (gemm_ms * 1e-3) / 1e9, peaks["hbm"], "GB/s"
    else:
        ach, peak, unit = gemm_elems / (gemm_ms * 1e-3) / 1e9, alu_peak_gelems(props.multi_processor_count, sm_mhz), "Gelem/s"
    out = {
        "metric": "group-quant GEMM TOPS & %INT8 peak; log-quant cross-attn GB/s & %HBM",
        "value": value, "unit": "TOPS", "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int8", "data": "synthetic",
        "config": {"workload": WORKLOAD, "l2": f"{n_sets} rotating buffer sets, {wl.set_bytes() * n_sets >> 20} MiB "
                   f"> L2 {l2_bytes >> 20} MiB", "parallelism": "replicas only" if world > 1 else "single gpu"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "TOPS", "h2d_bytes_per_step": wl.h2d_bytes(),
                "d2h_bytes_per_step": wl.d2h_bytes(), "ms_per_step": ms_e2e / args.steps},
        "gpu_launches": int(launches),
        "roofline": {"bound": bound, "achieved": ach, "peak": peak, "unit": unit,
                     "frac": ach / peak, "traffic": gemm_traffic(),
                     "frac_int8_peak": gemm_tops / int8_peak, "frac_int8_peak_burst": gemm_tops / int8_burst,
                     "frac_own_rooflines": own_us / (gemm_ms * 1e3),
                     "own_rooflines": "sum over the 6 launches of the slowest of each launch's tensor, HBM and "
                                      "epilogue-conversion time, divided by the measured time",
                     "launches": [{k: (round(v, 3) if isinstance(v, float) else v) for k, v in l.items() if k != "t_us"}
                                  for l in launches_rf],
                     "alu_peak": f"{CVT_PER_CLK_SM} int32->fp32 conversions per clock and SM x "
                                 f"{props.multi_processor_count} SMs x {sm_mhz:.0f} MHz",
                     "traffic_unit": "DRAM bytes per step over the 6 launches (ncu); outputs are still in L2 when a launch ends",
                     "kernel": "gq_gemm_kernel (6 launches per step, timed on one CUDA graph of the GEMM launches of 6 consecutive steps)",
                     "peak_source": f"int8 = 2 x bf16 sustained, HBM = copy bandwidth, {peaks['source']}"},
        "kernels": {
            "gemm": {"ms_per_step": gemm_ms, "tops": gemm_tops, "frac_int8_peak": gemm_tops / int8_peak},
            "attention": {"ms_per_step": attn_ms, "gbs": attn_bytes() / (attn_ms * 1e-3) / 1e9,
                          "frac_hbm": attn_bytes() / (attn_ms * 1e-3) / 1e9 / peaks["hbm"]},
            "quantize": {"ms_per_step": quant_ms, "gbs": quant_bytes / (quant_ms * 1e-3) / 1e9,
                         "frac_hbm": quant_bytes / (quant_ms * 1e-3) / 1e9 / peaks["hbm"]},
        },
    }
    if rank == 0:
        if world == 1 and not args.no_shapes:
            # every layer shape of the five benchmark configurations, one kernel at a time
            out["shapes"] = [time_case(torch, b, peaks, name, 5) for name in SHAPE_CASES]
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_baseline()
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------ oracle arm
def oracle_step_sample(rows=2048, attn_rows=2048, hs=32):
    """Times the oracle, as it stands, on a bounded sample of one step; returns (seconds scaled to a
    full step, description)."""
    from oracle import calibration as oc, linear as ol, attention as oa
    t_full = 0.0
    for key, C in INPUT_C.items():
        Xcal = synth.activations(SEED, 100 + ord(key), 1, TOKENS, C)
        gr = oc.calibrate(Xcal[:1024], 1024, 8, 8, dim_select=oc.DIM_CHANNEL)
        X = synth.activations(SEED, 10 + ord(key), 1, rows, C)
        t0 = time.perf_counter()
        codes, s, z = ol.quantize_dynamic_token(X, gr.col_group, gr.G, 8)
        t_q = time.perf_counter() - t0
        t_l = 0.0
        for i, (name, N, K, k2) in enumerate(LINEARS):
            if k2 != key:
                continue
            wq, sw = ol.weight_rtn(synth.weights(SEED, 200 + i, N, K), 8)
            bias = synth.bias(SEED, 300 + i, N)
            t0 = time.perf_counter()
            ol.group_linear(codes, s, z, gr.col_group, wq, sw, bias)
            t_l += time.perf_counter() - t0
        t_full += (t_q + t_l) * (M / rows)
    a = ATT
    Q, K, V = synth.attention_inputs(SEED, 1, a["H"], attn_rows, a["nk"], a["d"])
    t0 = time.perf_counter()
    oa.cross_attn_logq(Q, K, V, a["bits"])
    t_full += (time.perf_counter() - t0) * (a["B"] * a["nq"] / attn_rows)
    c = CONV

    Xcal = synth.activations(SEED, 150, 1, hs * c["w"], c["c"], token_outliers=False)
    gr = oc.calibrate(Xcal, hs * c["w"], 6, 16, dim_select=oc.DIM_CHANNEL)
    X = synth.activations(SEED, 60, 1, hs * c["w"], c["c"], token_outliers=False)
    wq, sw = ol.weight_rtn(synth.conv_weights(SEED, 250, c["N"], c["c"]), 4)
    t0 = time.perf_counter()
    codes, s, z = ol.quantize_static(X, gr, 0)
    ol.group_conv3x3(codes.reshape(1, hs, c["w"], c["c"]), gr.scale[0][0], gr.zp[0][0], gr.col_group, wq, sw,
                     synth.bias(SEED, 350, c["N"]))
    t_full += (time.perf_counter() - t0) * (c["n"] * c["h"] / hs)
    desc = (f"{rows} of {M} token rows of every linear (+ their quantizer), {attn_rows} of {a['B'] * a['nq']} "
            f"query rows of the attention (all heads), {hs} of {c['n'] * c['h']} image rows of the conv; "
            "time scaled to the full step by rows")
    return t_full, desc


def cpu_baseline():
    t, desc = oracle_step_sample()
    return {"value": gemm_ops() / t / 1e12, "unit": "TOPS", "cores": 1, "kind": "oracle", "sample": desc,
            "est_seconds_per_step": t}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    for _ in range(max(0, min(args.warmup, 1))):
        oracle_step_sample(rows=32, attn_rows=64)
    ts, desc = [], ""
    wall0 = time.perf_counter()
    for _ in range(max(1, min(args.steps, 3))):
        t, desc = oracle_step_sample()
        ts.append(t)
    wall = time.perf_counter() - wall0
    t = float(np.mean(ts))
    v = gemm_ops() / t / 1e12
    print(json.dumps({
        "impl": "reference", "metric": "group-quant GEMM TOPS & %INT8 peak; log-quant cross-attn GB/s & %HBM",
        "value": v, "unit": "TOPS", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": len(ts),
        "warmup": max(0, min(args.warmup, 1)), "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int64/f64", "data": "synthetic", "config": {"workload": WORKLOAD},
        # each step ran a bounded sample of the workload; ms_per_step is that time scaled to a whole step
        "extrapolated": True, "measured_wall_seconds": wall, "steps_requested": args.steps,
        "cpu_baseline": {"value": v, "unit": "TOPS", "cores": 1, "kind": "oracle", "sample": desc},
        "e2e": {"value": v, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------------------------------ single-kernel cases
MICRO_CASES = {
    # name: (kind, params)
    "quant_8192x320": ("quant", dict(M=8192, P=4096, C=320, G=8, dynamic=1)),
    "quant_8192x1280": ("quant", dict(M=8192, P=4096, C=1280, G=8, dynamic=1)),
    "quant_32768x320": ("quant", dict(M=32768, P=4096, C=320, G=8, dynamic=1)),
    "quant_32768x1280": ("quant", dict(M=32768, P=4096, C=1280, G=8, dynamic=1)),
    "quant_static_32768x320": ("quant", dict(M=32768, P=4096, C=320, G=16, dynamic=0)),
    "gemm_8192x320x320_w8": ("gemm", dict(M=8192, P=4096, N=320, C=320, G=8, wbits=8)),
    "gemm_8192x2560x320_w8": ("gemm", dict(M=8192, P=4096, N=2560, C=320, G=8, wbits=8)),
    "gemm_8192x320x1280_w8": ("gemm", dict(M=8192, P=4096, N=320, C=1280, G=8, wbits=8)),
    "gemm_32768x320x1280_w4": ("gemm", dict(M=32768, P=4096, N=320, C=1280, G=8, wbits=4)),
    "gemm_8192x640x640_w4": ("gemm", dict(M=8192, P=1024, N=640, C=640, G=8, wbits=4)),
    "gemm_8192x5120x640_w4": ("gemm", dict(M=8192, P=1024, N=5120, C=640, G=8, wbits=4)),
    "gemm_8192x640x2560_w4": ("gemm", dict(M=8192, P=1024, N=640, C=2560, G=8, wbits=4)),
    "gemm_2048x1280x5120_w4": ("gemm", dict(M=2048, P=256, N=1280, C=5120, G=8, wbits=4)),
    "conv_2x64x64x320": ("conv", dict(n=2, h=64, w=64, C=320, N=320, G=16)),
    "conv_8x64x64x320": ("conv", dict(n=8, h=64, w=64, C=320, N=320, G=16)),
    "conv_8x32x32x640": ("conv", dict(n=8, h=32, w=32, C=640, N=640, G=16)),
    "conv_8x16x16x1280": ("conv", dict(n=8, h=16, w=16, C=1280, N=1280, G=16)),
    "attn_2x4096x40": ("attn", dict(B=2, H=8, nq=4096, nk=77, d=40)),
    "attn_8x4096x40": ("attn", dict(B=8, H=8, nq=4096, nk=77, d=40)),
    "attn_qv_2x4096x40": ("attn", dict(B=2, H=8, nq=4096, nk=77, d=40, v_bits=8)),
    "attn_8x1024x80": ("attn", dict(B=8, H=8, nq=1024, nk=77, d=80)),
    "attn_8x256x160": ("attn", dict(B=8, H=8, nq=256, nk=77, d=160)),
    "attn_sdxl_1x10x1024x64": ("attn", dict(B=1, H=10, nq=1024, nk=77, d=64)),
    "gemm_sdxl_1024x5120x640_w8": ("gemm", dict(M=1024, P=1024, N=5120, C=640, G=8, wbits=8)),
    # the remaining layer shapes of the benchmark configurations
    "cfg1_gemm_256x320x320_w8": ("gemm", dict(M=256, P=256, N=320, C=320, G=4, wbits=8, explicit=1)),
    "gemm_32768x320x320_w4": ("gemm", dict(M=32768, P=4096, N=320, C=320, G=8, wbits=4)),
    "gemm_32768x2560x320_w4": ("gemm", dict(M=32768, P=4096, N=2560, C=320, G=8, wbits=4)),
    "gemm_616x320x768_w4": ("gemm", dict(M=616, P=77, N=320, C=768, G=8, wbits=4)),
    "gemm_616x640x768_w4": ("gemm", dict(M=616, P=77, N=640, C=768, G=8, wbits=4)),
    "gemm_616x1280x768_w4": ("gemm", dict(M=616, P=77, N=1280, C=768, G=8, wbits=4)),
    "gemm_2048x1280x1280_w4": ("gemm", dict(M=2048, P=256, N=1280, C=1280, G=8, wbits=4)),
    "gemm_2048x10240x1280_w4": ("gemm", dict(M=2048, P=256, N=10240, C=1280, G=8, wbits=4)),
    "gemm_512x1280x1280_w4": ("gemm", dict(M=512, P=64, N=1280, C=1280, G=8, wbits=4)),
    "gemm_512x10240x1280_w4": ("gemm", dict(M=512, P=64, N=10240, C=1280, G=8, wbits=4)),
    "gemm_512x1280x5120_w4": ("gemm", dict(M=512, P=64, N=1280, C=5120, G=8, wbits=4)),
    "conv_8x8x8x1280": ("conv", dict(n=8, h=8, w=8, C=1280, N=1280, G=16)),
    "attn_8x64x160": ("attn", dict(B=8, H=8, nq=64, nk=77, d=160)),
    "selfattn_2x4096x40": ("selfattn", dict(B=2, H=8, n=4096, d=40)),
    "selfattn_8x1024x80": ("selfattn", dict(B=8, H=8, n=1024, d=80)),
    "selfattn_8x256x160": ("selfattn", dict(B=8, H=8, n=256, d=160)),
}


# The layer shapes of the five benchmark configurations, timed one kernel at a time by the default run
# ("shapes" in its JSON line): config 1; config 2 (W8A8, 8192 tokens); config 3 and 5 (cross-attention at the
# four resolutions, batch 2 and 8); config 4 (W4A8 transformer linears of the four levels at batch 8); config 5
# (W4A6 3x3 convs at batch 8).
SHAPE_CASES = [
    "cfg1_gemm_256x320x320_w8",
    "gemm_8192x320x320_w8", "gemm_8192x2560x320_w8", "gemm_8192x320x1280_w8",
    "attn_2x4096x40",
    "gemm_32768x320x320_w4", "gemm_32768x2560x320_w4", "gemm_32768x320x1280_w4", "gemm_616x320x768_w4",
    "gemm_8192x640x640_w4", "gemm_8192x5120x640_w4", "gemm_8192x640x2560_w4", "gemm_616x640x768_w4",
    "gemm_2048x1280x1280_w4", "gemm_2048x10240x1280_w4", "gemm_2048x1280x5120_w4", "gemm_616x1280x768_w4",
    "gemm_512x1280x1280_w4", "gemm_512x10240x1280_w4", "gemm_512x1280x5120_w4",
    "conv_8x64x64x320", "conv_8x32x32x640", "conv_8x16x16x1280", "conv_8x8x8x1280",
    "attn_8x4096x40", "attn_8x1024x80", "attn_8x256x160", "attn_8x64x160",
    "quant_8192x320", "quant_32768x1280",
]


def time_case(torch, b, peaks, name, steps):
    """Times one single-kernel case: a CUDA graph of back-to-back launches that rotate over buffer sets
    larger than L2, replayed and timed with CUDA events (median of `steps` replays after 3 warm-up replays).
    Returns the record with the case's own roofline: the slowest of its algorithmic bytes at the measured copy
    bandwidth, its operations at the measured burst tensor peak and, for the GEMMs, its per-group epilogue
    conversions at the SMs' conversion rate."""
    kind, p = MICRO_CASES[name]
    fns, algo_bytes, algo_ops, algo_elems = [], 0.0, 0.0, 0.0
    if kind in ("quant", "gemm", "conv"):
        conv = None
        if kind == "conv":
            P, M, C, bits, tok = p["h"] * p["w"], p["n"] * p["h"] * p["w"], p["C"], 6, False
            conv = (p["n"], p["h"], p["w"], C)
        else:
            P, M, C, bits, tok = p["P"], p["M"], p["C"], 8, True
        Xcal = torch.from_numpy(synth.activations(SEED, 100, 2, P, C, token_outliers=tok)).cuda()
        g = b.calibrate_groups(Xcal, P, bits, p["G"], b.DIM_CHANNEL,
                               b.OUTLIER_EXPLICIT if p.get("explicit") else b.OUTLIER_KMEANS)
        Xh = synth.activations(SEED, 1, -(-M // P), P, C, token_outliers=tok)[:M]
        per_set = M * C * 2 + M * g.K_pad + (M * p.get("N", 0) * 2)
        n_sets = max(2, int(3 * 126e6 // per_set) + 1)
        dyn = kind == "gemm" or (kind == "quant" and p["dynamic"])
        mode = b.MODE_DYNAMIC_TOKEN if dyn else b.MODE_STATIC
        layout = b.CODES_S8_CENTRED if kind == "conv" else b.CODES_U8
        sets = []
        for _ in range(n_sets):
            X = torch.from_numpy(Xh).cuda()
            Xq = torch.empty((M, g.K_pad), dtype=torch.uint8, device="cuda")
            ds = torch.empty((M, g.G), dtype=torch.float32, device="cuda") if dyn else None
            dz = torch.empty((M, g.G), dtype=torch.int32, device="cuda") if dyn else None
            b.quantize_act_into(g, X, Xq, ds, dz, mode=mode, layout=layout)
            Y = torch.empty((M, p["N"]), dtype=torch.float16, device="cuda") if kind != "quant" else None
            sets.append((X, Xq, ds, dz, Y))
        if kind == "quant":
            fns = [lambda s=s: b.quantize_act_into(g, s[0], s[1], s[2], s[3], mode=mode, layout=layout) for s in sets]
            algo_bytes = 3.0 * M * C + (8.0 * M * g.G if dyn else 0)
        else:
            if kind == "conv":
                W = torch.from_numpy(synth.conv_weights(SEED, 2, p["N"], C)).cuda()
                w = b.weight_prepare(g, W, 4, conv=conv)
                kreal, wb = 9 * C, 4
            else:
                W = torch.from_numpy(synth.weights(SEED, 2, p["N"], C)).cuda()
                w = b.weight_prepare(g, W, p["wbits"])
                kreal, wb = C, p["wbits"]
            bias = torch.from_numpy(synth.bias(SEED, 3, p["N"])).cuda()
            ws_need = b.linear_workspace_bytes(g, w, M)      # 4-bit weights are expanded into it by every call
            ws = torch.empty(ws_need, dtype=torch.uint8, device="cuda") if ws_need else None
            fns = [lambda s=s: b.linear(g, w, s[1], mode=mode, layout=layout, dyn_scale=s[2], dyn_zp=s[3],
                                        bias=bias, out=s[4], conv=conv, workspace=ws) for s in sets]
            algo_ops = 2.0 * M * p["N"] * kreal
            algo_bytes = M * C + p["N"] * kreal * wb / 8 + 2.0 * M * p["N"]
            algo_elems = float(M) * p["N"] * g.G
        extra = {"K_pad": g.K_pad, "G": g.G}
    elif kind == "selfattn":
        rng = np.random.default_rng(SEED)
        shape = (p["B"], p["n"], p["H"], p["d"])
        n_sets = max(2, int(3 * 126e6 // (4 * 2 * np.prod(shape))) + 1)
        sets = [tuple(torch.from_numpy(rng.normal(0, 1, shape).astype(np.float16)).cuda() for _ in range(3))
                + (torch.empty(shape, dtype=torch.float16, device="cuda"),) for _ in range(n_sets)]
        fns = [lambda s=s: b.self_attn_logq(s[0], s[1], s[2], 8, out=s[3]) for s in sets]
        algo_bytes = 4.0 * 2 * np.prod(shape)
        algo_ops = 4.0 * p["B"] * p["H"] * p["n"] * p["n"] * p["d"]      # Q K^T and P V, once each
        extra = {}
    else:
        a = p
        Q, K, V = synth.attention_inputs(SEED, a["B"], a["H"], a["nq"], a["nk"], a["d"])
        per_set = 2 * Q.size * 2
        n_sets = max(2, int(3 * 126e6 // per_set) + 1)
        ws_bytes = b.cross_attn_workspace_bytes(a["B"], a["H"], a["nq"], a["nk"], a["d"])
        sets = [(torch.from_numpy(Q).cuda(), torch.from_numpy(K).cuda(), torch.from_numpy(V).cuda(),
                 torch.empty(Q.shape, dtype=torch.float16, device="cuda"),
                 torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")) for _ in range(n_sets)]
        fns = [lambda s=s: b.cross_attn_logq(s[0], s[1], s[2], 8, out=s[3], workspace=s[4],
                                             v_bits=p.get("v_bits", 0)) for s in sets]
        algo_bytes = 2.0 * Q.size * 2 + 2.0 * K.size * 2
        extra = {}
    reps = max(1, 24 // len(fns))
    for f in fns:
        f()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            for _ in range(reps):
                for f in fns:
                    f()
    n_launch = reps * len(fns)
    torch.cuda.synchronize()
    times = []
    for _ in range(3 + steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        graph.replay()
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1) * 1e3 / n_launch)
    us = float(np.median(times[3:]))
    rec = {"case": name, "us": us, "gbs": algo_bytes / us / 1e3, "frac_hbm": algo_bytes / us / 1e3 / peaks["hbm"],
           "sets": len(fns), **extra}
    t_hbm_us, t_tc_us = algo_bytes / peaks["hbm"] / 1e3, 0.0
    t_alu_us = algo_elems / alu_peak_gelems(torch.cuda.get_device_properties(0).multi_processor_count) / 1e3
    if algo_ops:
        rec["tops"] = algo_ops / us / 1e6
        if kind == "selfattn":      # fp16 operands: the measured bf16 peak is the denominator
            rec["frac_f16_peak"] = rec["tops"] / peaks["bf16"]
            t_tc_us = algo_ops / peaks["bf16"] / 1e6
        else:
            rec["frac_int8_peak"] = rec["tops"] / (2 * peaks["bf16"])
            t_tc_us = algo_ops / (2 * peaks["bf16"]) / 1e6
    t = {"tensor": t_tc_us, "hbm": t_hbm_us, "alu": t_alu_us}
    rec["bound"] = max(t, key=t.get)
    rec["roofline_us"] = t[rec["bound"]]
    rec["frac_roofline"] = rec["roofline_us"] / us
    assert b.device_status() == 0
    del sets, fns, graph
    return {k: (round(v, 4) if isinstance(v, float) else v) for k, v in rec.items()}


def run_micro(args):
    """Times single kernels (see time_case) and prints one JSON line per case."""
    import torch
    from paper_2501_04304_b200 import binding as b
    torch.cuda.set_device(0)
    peaks = measured_peaks()
    for name in [n for n in MICRO_CASES if args.micro == "all" or n.startswith(args.micro)]:
        print(json.dumps(time_case(torch, b, peaks, name, args.steps)), flush=True)


def rank_launch_command(n, argv):
    """The command that runs this script as n ranks of one node (replicas only), one GPU each."""
    import socket
    with socket.socket() as so:
        so.bind(("127.0.0.1", 0))
        port = so.getsockname()[1]
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *argv]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-shapes", action="store_true", help="skip the per-shape single-kernel timings")
    ap.add_argument("--micro", default=None, help="time single kernels: 'all' or a case-name prefix")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not args.micro:
        # started without a launcher: start one rank per GPU of this node and let them print the line
        sys.exit(subprocess.call(rank_launch_command(args.gpus, sys.argv[1:])))
    if args.micro:
        run_micro(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
