#!/usr/bin/env python
"""Benchmark of the DiG token-mixer hot path on B200.

A step is one pass of the whole hot path over one batch of synthetic, seeded input: for every
scan direction of the workload (one DiG block each) the gate transform, GLA forward, GLA backward
and, where the workload has one, the SREM depthwise conv.  Every block owns its own input and
output buffers.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C5] [--impl ours|reference]

Headline (`value`): the largest single-GPU workload (C5: 128 x 128 grid, 16 heads of 72 channels,
four scan directions + conv).  K steps are captured as CUDA-graph replays and timed with CUDA
events; the K-step region is repeated until at least a second of device time has been measured and
the median repetition is reported, with the spread and the SM clock sampled meanwhile.  The other
workloads (C1 - C4 and the chunk sweep of C4) follow as `sweep` entries: a whole step each, median
of 20 repetitions with the L2 flushed before every one ("cold") and without ("warm"), forward and
backward also on their own, each with its roofline fractions and clock record.

Prints one JSON line (rank 0).  N > 1 (torchrun) shards nothing across ranks: every rank runs the
same workload on its own GPU (weak scaling over independent batches, no collective in the path).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "gla_fwd_bwd_tokens_per_s"
UNIT = "tokens/s"
TILE = 64                      # tokens per tile of the tcgen05 kernels, whatever chunk size was asked for
FAMILY = {1: "fma", 2: "tensor", 3: "mma"}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def executed_tile(family, chunk):
    """Tokens per tile the kernels actually work on: the tcgen05 family always uses 64-token tiles
    (shorter chunks are sub-chunks of a tile whose other rows are zero), the others the chunk itself."""
    return TILE if family == 2 else chunk


def flops_per_token_head(wl, tile):
    """(algorithmic, executed) flops per (token, head) for fwd+bwd: causal-useful work without the
    backward's recomputation, and full tile x tile blocks with it."""
    dk, dv, C = wl.d_k, wl.d_v, tile
    alg = 3 * (C + 1) * (dk + dv) + 12 * dk * dv
    exe = 2 * C * (dk + dv) + 4 * dk * dv + 2 * C * (3 * dk + 2 * dv) + 10 * dk * dv
    if not wl.backward:
        alg = (C + 1) * (dk + dv) + 4 * dk * dv
        exe = 2 * C * (dk + dv) + 4 * dk * dv
    return alg, exe


def bytes_per_token_head(wl):
    """Algorithmic HBM bytes per (token, head): every operand touched once per pass; bf16 (or fp32)
    tensors, fp32 gate and gate gradient."""
    e = 2 if wl.dtype == "bf16" else 4
    dk, dv = wl.d_k, wl.d_v
    fwd = e * (2 * dk + dv) + 4 * dk + e * dv
    bwd = e * (2 * dk + 2 * dv) + 4 * dk + e * (2 * dk + dv) + 4 * dk
    return fwd, (bwd if wl.backward else 0)


def step_work(wl, family):
    """Algorithmic bytes and executed flops of one step (all blocks) of a workload."""
    fwd_b, bwd_b = bytes_per_token_head(wl)
    th = wl.B * wl.L * wl.H
    e = 2 if wl.dtype == "bf16" else 4
    nb = len(wl.directions)
    conv_b = 2 * e * wl.B * wl.L * wl.H * wl.d_v if wl.conv else 0
    alg_f, exe_f = flops_per_token_head(wl, executed_tile(family, wl.chunk))
    return {"bytes": nb * (th * (fwd_b + bwd_b) + conv_b), "flops_alg": nb * th * alg_f, "flops_exec": nb * th * exe_f}


def roofline_fracs(work, seconds, peaks):
    t_hbm = work["bytes"] / (peaks["hbm_gbs"] * 1e9)
    t_tc = work["flops_exec"] / (peaks["bf16_tflops_sustained"] * 1e12)
    return {"hbm_frac": t_hbm / seconds, "tensor_frac_exec": t_tc / seconds, "frac": max(t_hbm, t_tc) / seconds,
            "bound": "hbm" if t_hbm >= t_tc else "tensor",
            "tflops_alg": work["flops_alg"] / seconds / 1e12, "tflops_exec": work["flops_exec"] / seconds / 1e12,
            "gbs_alg": work["bytes"] / seconds / 1e9}


def kernel_alg_bytes(wl):
    """Algorithmic bytes per launch of the kernels that have a plain bandwidth model."""
    fwd_b, bwd_b = bytes_per_token_head(wl)
    th = wl.B * wl.L * wl.H
    e = 2 if wl.dtype == "bf16" else 4
    out = {}
    for name in ("sweep_fwd", "mma_chunk_out", "fma_chunk_out"):
        out[name] = fwd_b * th
    for name in ("sweep_bwd", "mma_chunk_bwd", "fma_chunk_bwd"):
        out[name] = bwd_b * th
    out["gate_logsigmoid"] = (e + 4) * th * wl.d_k
    out["srem_dwconv3x3"] = 2 * e * wl.B * wl.L * wl.H * wl.d_v
    return out


def source_hash():
    h = hashlib.sha256()
    src = os.path.join(ROOT, "paper_2405_18428_b200", "csrc")
    for f in sorted(os.listdir(src)):
        if f.endswith((".cu", ".cuh")):
            h.update(open(os.path.join(src, f), "rb").read())
    return h.hexdigest()[:16]


def recorded_traffic(kernel, workload):
    """DRAM bytes per launch of a kernel from the ncu capture recorded beside the profile summaries;
    None when no capture exists for this kernel and workload or the kernel sources changed since."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(path):
        return None
    try:
        rec = json.load(open(path))
    except ValueError:
        return None
    if rec.get("source_hash") != source_hash():
        return None
    for r in rec.get("kernels", []):
        if r["kernel"].startswith(kernel) and r["workload"] == workload:
            return r["dram_bytes_per_launch"]
    return None


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while a timed region runs (read only)."""

    def __init__(self, index):
        self.samples, self.reasons, self.stop_flag, self.thread, self.max_mhz = [], set(), False, None, None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20,
                 "hw_thermal_slowdown": 0x40, "hw_power_brake": 0x80}
        while not self.stop_flag:
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for n, bit in names.items():
                    if r & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            time.sleep(0.005)

    def start(self):
        if self.nv is not None:
            self.thread = threading.Thread(target=self._loop, daemon=True)
            self.thread.start()
        return self

    def stop(self):
        self.stop_flag = True
        if self.thread is not None:
            self.thread.join()
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


class Block:
    """Device buffers of one DiG block (one scan direction) of the workload."""

    def __init__(self, wl, direction, x, torch, dig):
        dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda().to(
            torch.bfloat16 if wl.dtype == "bf16" else torch.float32)
        self.wl, self.direction = wl, direction
        self.q, self.k, self.v, self.g, self.dO = (dev(x[n]) for n in ("q", "k", "v", "g", "dO"))
        ost = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
        self.gate = torch.empty(self.q.shape, dtype=torch.float32, device="cuda")
        self.out = torch.empty(self.v.shape, dtype=ost, device="cuda")
        self.grads = (torch.empty(self.q.shape, dtype=ost, device="cuda"), torch.empty(self.q.shape, dtype=ost, device="cuda"),
                      torch.empty(self.v.shape, dtype=ost, device="cuda"), torch.empty(self.q.shape, dtype=torch.float32, device="cuda"))
        dt = dig.DIG_BF16 if wl.dtype == "bf16" else dig.DIG_F32
        need = dig.dig_gla_workspace_bytes(wl.B, wl.H, wl.grid_h, wl.grid_w, wl.d_k, wl.d_v, wl.chunk, dt, int(wl.backward))
        self.ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda")
        self.tau = x["tau"]
        if wl.conv:
            self.cx, self.cw = dev(x["conv_x"]), dev(x["conv_w"])
            self.cy = torch.empty_like(self.cx)

    def run(self, dig, part="all"):
        """part: "all" (the step), "fwd" (gate transform + forward), "bwd" (backward alone)."""
        wl = self.wl
        if part in ("all", "fwd"):
            dig.dig_gate_logsigmoid(self.g, self.tau, self.gate)
            dig.dig_gla_fwd(self.q, self.k, self.v, self.gate, wl.grid_h, wl.grid_w, wl.chunk, self.direction,
                            out=self.out, workspace=self.ws)
        if wl.backward and part in ("all", "bwd"):
            dig.dig_gla_bwd(self.q, self.k, self.v, self.gate, self.dO, wl.grid_h, wl.grid_w, wl.chunk,
                            self.direction, grads=self.grads, workspace=self.ws)
        if wl.conv and part == "all":
            dig.dig_srem_dwconv(self.cx, self.cw, None, wl.grid_h, wl.grid_w, self.direction, y=self.cy)

    def host_io(self, torch):
        """Pinned host mirrors for the end-to-end leg."""
        ins = [self.q, self.k, self.v, self.g, self.dO] + ([self.cx] if self.wl.conv else [])
        outs = [self.out, *self.grads] + ([self.cy] if self.wl.conv else [])
        self.h_in = [torch.empty(t.shape, dtype=t.dtype).pin_memory().copy_(t) for t in ins]
        self.h_out = [torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in outs]
        self.d_in, self.d_out_t = ins, outs
        return (sum(t.numel() * t.element_size() for t in ins), sum(t.numel() * t.element_size() for t in outs))

    def run_e2e(self, dig, torch):
        """One block end to end: inputs from pinned host memory, the library calls, results back to
        pinned host memory.  The copies run on two side streams so that the two PCIe directions and
        the kernels of neighbouring blocks overlap; events order every reuse of a buffer."""
        cur = torch.cuda.current_stream()
        if not hasattr(self, "s_in"):
            self.s_in, self.s_out = Block.copy_streams(torch)
            self.ev_run = self.ev_back = None
        if self.ev_run is not None:
            self.s_in.wait_event(self.ev_run)          # last step's kernels have read the inputs
        else:
            self.s_in.wait_stream(cur)
        with torch.cuda.stream(self.s_in):
            for h, d in zip(self.h_in, self.d_in):
                d.copy_(h, non_blocking=True)
            ev_in = self.s_in.record_event()
        cur.wait_event(ev_in)
        if self.ev_back is not None:
            cur.wait_event(self.ev_back)               # last step's results have left the device
        self.run(dig)
        self.ev_run = cur.record_event()
        self.s_out.wait_event(self.ev_run)
        with torch.cuda.stream(self.s_out):
            for h, d in zip(self.h_out, self.d_out_t):
                h.copy_(d, non_blocking=True)
            self.ev_back = self.s_out.record_event()

    _streams = None

    @staticmethod
    def copy_streams(torch):
        if Block._streams is None:
            Block._streams = (torch.cuda.Stream(), torch.cuda.Stream())
        return Block._streams

    @staticmethod
    def join_copies(torch):
        """Make the current stream wait for every copy issued so far."""
        if Block._streams is not None:
            for s in Block._streams:
                torch.cuda.current_stream().wait_stream(s)


def make_blocks(wl, torch, dig):
    from paper_2405_18428_b200.inputs import make_inputs
    blocks = []
    for i, d in enumerate(wl.directions):
        x = make_inputs(wl.scaled(seed=wl.seed + i))
        blocks.append(Block(wl, d, x, torch, dig))
    return blocks


def max_over_ranks(ms, dist, device="cuda"):
    """Step time of the job = the slowest rank's (ranks run independent replicas of the workload)."""
    if dist is None:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_tokens_per_s(tokens_per_step_per_rank, steps, world, ms):
    """Whole-job throughput: every rank processes its own copy of the workload (weak scaling)."""
    return tokens_per_step_per_rank * steps * world / (ms * 1e-3)


def time_steps(blocks, dig, torch, steps, warmup, dist, e2e=False, before_timed=None, part="all"):
    """K steps of plain stream launches between two CUDA events (barrier + synchronize on both sides)."""
    for _ in range(warmup):
        for b in blocks:
            b.run_e2e(dig, torch) if e2e else b.run(dig, part)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    if before_timed is not None:
        before_timed()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(steps):
        for b in blocks:
            b.run_e2e(dig, torch) if e2e else b.run(dig, part)
    if e2e:
        Block.join_copies(torch)
    t1.record()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    return max_over_ranks(t0.elapsed_time(t1), dist)


def capture_step(blocks, dig, torch, part="all"):
    """One step (or its forward / backward part) as a CUDA graph: the kernels and their order are
    those of the plain launches, only the host-side launch cost goes away.  None if capture fails."""
    try:
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            for b in blocks:
                b.run(dig, part)          # first calls outside the capture (per-kernel attribute set-up)
            torch.cuda.synchronize()
            with torch.cuda.graph(graph, stream=side):
                for b in blocks:
                    b.run(dig, part)
        torch.cuda.synchronize()
        return graph
    except Exception:
        return None


def time_replays(graph, torch, steps, dist):
    """`steps` replays of a captured step between two CUDA events."""
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(steps):
        graph.replay()
    t1.record()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    return max_over_ranks(t0.elapsed_time(t1), dist)


def median_single(run_once, torch, reps, flush=None):
    """Median (and min, max) over `reps` single timed runs, optionally with the L2 flushed before each."""
    ts = []
    for _ in range(reps):
        if flush is not None:
            flush.zero_()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        run_once()
        t1.record()
        torch.cuda.synchronize()
        ts.append(t0.elapsed_time(t1))
    ts.sort()
    return {"median_ms": float(np.median(ts)), "min_ms": ts[0], "max_ms": ts[-1], "reps": reps}


def profile_kernels(blocks, dig, torch, steps):
    """Per-kernel device time of `steps` steps, every launch bracketed by two CUDA events."""
    for b in blocks:
        b.run(dig)
    torch.cuda.synchronize()
    dig.dig_profile_enable(True)
    for _ in range(steps):
        for b in blocks:
            b.run(dig)
    torch.cuda.synchronize()
    prof = dig.dig_profile_read()
    dig.dig_profile_enable(False)
    total = sum(t for n, t in prof.values() if n) or 1.0
    return {k: {"launches": n, "ms_per_launch": t / n, "share": t / total} for k, (n, t) in prof.items() if n}


def kernel_rooflines(shares, wl, peaks):
    """Achieved algorithmic GB/s of every kernel with a bandwidth model, against the measured copy bandwidth."""
    alg = kernel_alg_bytes(wl)
    out = {}
    for k, s in shares.items():
        if k in alg and alg[k] > 0:
            a = alg[k] / (s["ms_per_launch"] * 1e-3) / 1e9
            out[k] = {"bound": "hbm", "achieved": a, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": a / peaks["hbm_gbs"],
                      "algorithmic_bytes_per_launch": alg[k], "us_per_launch": s["ms_per_launch"] * 1e3,
                      "traffic": recorded_traffic(k, wl.name), "peak_source": peaks["source"]}
    return out


def sweep_entry(name, wl, torch, dig, peaks, local, flush, reps=20):
    dt = dig.DIG_BF16 if wl.dtype == "bf16" else dig.DIG_F32
    fam = dig.dig_gla_query_impl(wl.d_k, wl.d_v, wl.chunk, dt, int(wl.backward))
    blocks = make_blocks(wl, torch, dig)
    sampler = ClockSampler(local).start()
    res = {"L": wl.L, "B": wl.B, "H": wl.H, "d": wl.d_k, "chunk_requested": wl.chunk,
           "tile_executed": executed_tile(fam, wl.chunk), "storage": wl.dtype, "kernel_family": FAMILY.get(fam, str(fam)),
           "directions": list(wl.directions), "conv": wl.conv, "backward": wl.backward}
    graphs = {p: capture_step(blocks, dig, torch, p) for p in (("all", "fwd", "bwd") if wl.backward else ("all",))}
    run = {p: (g.replay if g is not None else (lambda p=p: [b.run(dig, p) for b in blocks])) for p, g in graphs.items()}
    for p in run:
        for _ in range(3):
            run[p]()
    torch.cuda.synchronize()
    res["step_cold"] = median_single(run["all"], torch, reps, flush)
    res["step_warm"] = median_single(run["all"], torch, reps, None)
    if wl.backward:
        res["fwd_cold"] = median_single(run["fwd"], torch, reps, flush)
        res["bwd_cold"] = median_single(run["bwd"], torch, reps, flush)
    sec = res["step_cold"]["median_ms"] * 1e-3
    res["tokens_per_s"] = wl.B * wl.L * len(wl.directions) / sec
    res["roofline"] = roofline_fracs(step_work(wl, fam), sec, peaks)
    shares = profile_kernels(blocks, dig, torch, 3)
    rl = kernel_rooflines(shares, wl, peaks)
    dom = max(shares, key=lambda k: shares[k]["share"])
    res["dominant_kernel"] = {"name": dom, "share": shares[dom]["share"], **(rl.get(dom) or {})}
    res["clocks"] = sampler.stop()
    res["launch"] = "cuda_graph" if graphs["all"] is not None else "eager"
    del blocks, graphs, run
    torch.cuda.empty_cache()
    return res


def multi_direction_entry(wl, torch, dig, flush, reps=20):
    """Sums over the four scan orders (Algorithm 3) of one workload: the library's entry points, which add
    every order's fp32 results into one set of buffers, against four single-order calls plus torch adds."""
    from paper_2405_18428_b200.inputs import make_inputs
    x = make_inputs(wl, conv=False)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda().to(torch.bfloat16)
    q, k, v, g, dO = (dev(x[n]) for n in ("q", "k", "v", "g", "dO"))
    gate = dig.dig_gate_logsigmoid(g, x["tau"])
    dirs = (0, 1, 2, 3)
    dt = dig.DIG_BF16
    ws1 = torch.empty(dig.dig_gla_workspace_bytes(wl.B, wl.H, wl.grid_h, wl.grid_w, wl.d_k, wl.d_v, wl.chunk, dt, 1), dtype=torch.uint8, device="cuda")
    wsm = torch.empty(dig.dig_gla_multi_workspace_bytes(wl.B, wl.H, wl.grid_h, wl.grid_w, wl.d_k, wl.d_v, wl.chunk, dt, 1), dtype=torch.uint8, device="cuda")
    outs = [torch.empty_like(v) for _ in dirs]
    grads = [(torch.empty_like(q), torch.empty_like(q), torch.empty_like(v), torch.empty(q.shape, dtype=torch.float32, device="cuda")) for _ in dirs]
    out_m = torch.empty_like(v)
    grads_m = (torch.empty_like(q), torch.empty_like(q), torch.empty_like(v), torch.empty(q.shape, dtype=torch.float32, device="cuda"))

    def separate():
        for i, d in enumerate(dirs):
            dig.dig_gla_fwd(q, k, v, gate, wl.grid_h, wl.grid_w, wl.chunk, d, out=outs[i], workspace=ws1)
            dig.dig_gla_bwd(q, k, v, gate, dO, wl.grid_h, wl.grid_w, wl.chunk, d, grads=grads[i], workspace=ws1)
        o = outs[0] + outs[1] + outs[2] + outs[3]
        gs = [grads[0][j] + grads[1][j] + grads[2][j] + grads[3][j] for j in range(4)]
        return o, gs

    def fused():
        dig.dig_gla_fwd_multi(q, k, v, gate, wl.grid_h, wl.grid_w, dirs, wl.chunk, out=out_m, workspace=wsm)
        dig.dig_gla_bwd_multi(q, k, v, gate, dO, wl.grid_h, wl.grid_w, dirs, wl.chunk, grads=grads_m, workspace=wsm)

    for _ in range(3):
        separate()
        fused()
    torch.cuda.synchronize()
    th = wl.B * wl.L * wl.H
    fwd_b, bwd_b = bytes_per_token_head(wl)
    d = wl.d_k
    # output bytes per (token, head) with d = d_k = d_v, bf16 results and an fp32 gate gradient:
    #   separate: 4 orders x 12d stored, then the adds read 4 x 12d and store 12d            -> 108 d
    #   entry points: fp32 sums of out, dq, dk, dv (16d): stored once, read + stored 3 times, read once
    #   more and rounded to 8d; the gate gradient (4d) stored once, read + stored 3 times      -> 164 d
    sep_out, fus_out = th * 108 * d, th * 164 * d
    return {"workload": wl.name, "directions": list(dirs),
            "four_calls_plus_adds": median_single(separate, torch, reps, flush),
            "multi_entry_points": median_single(fused, torch, reps, flush),
            "output_bytes_model": {"four_calls_plus_adds": sep_out, "multi_entry_points": fus_out,
                                   "inputs_each": 4 * th * (fwd_b + bwd_b),
                                   "note": "both read q, k, v, dO and the gates once per order; the entry points form the sums in fp32 "
                                           "and round once, at the price of fp32 read-add-store traffic on the outputs"}}


def next_rows_entry(torch, dig, peaks, flush, reps=20):
    """The operators beyond the timed step, each timed alone (median of `reps` single calls, L2 flushed before
    each): conv backward, output gate forward / backward, the full gate alpha^T beta forward + backward, and a
    forward pass cut in two pieces that hand the state over.  Algorithmic bytes are the tensors each one must
    read and write once (bf16 tensors, fp32 gates and parameter gradients neglected)."""
    from paper_2405_18428_b200.inputs import CONFIGS, make_inputs
    out = {}
    hbm = peaks["hbm_gbs"]

    def entry(run, alg_bytes, extra=None):
        for _ in range(3):
            run()
        torch.cuda.synchronize()
        t = median_single(run, torch, reps, flush)
        gbs = alg_bytes / (t["median_ms"] * 1e-3) / 1e9
        e = {**t, "algorithmic_bytes": alg_bytes, "achieved_gbs": gbs, "hbm_frac": gbs / hbm, "peak_source": peaks["source"]}
        if extra:
            e.update(extra)
        return e

    # conv backward and output gate on the shape of the largest config (16384 tokens x 1152 channels)
    wl = CONFIGS["C5"]
    D = wl.H * wl.d_v
    n = wl.B * wl.L * D
    g = torch.Generator(device="cuda").manual_seed(5)
    x = torch.randn(wl.B, wl.L, D, device="cuda", generator=g).to(torch.bfloat16)
    dy = torch.randn(wl.B, wl.L, D, device="cuda", generator=g).to(torch.bfloat16)
    w = (torch.randn(3, 3, D, device="cuda", generator=g) / 3).to(torch.bfloat16)
    out["conv_backward"] = entry(lambda: dig.dig_srem_dwconv_bwd(x, w, dy, wl.grid_h, wl.grid_w, 0),
                                 6 * n, {"shape": [wl.B, wl.grid_h, wl.grid_w, D], "bytes_model": "x, dy read, dx written: 6 B per element"})
    o = x.view(wl.B, wl.L, wl.H, wl.d_v)
    r = dy.view(wl.B, wl.L, wl.H, wl.d_v)
    dz = torch.randn(wl.B, wl.L, wl.H, wl.d_v, device="cuda", generator=g).to(torch.bfloat16)
    ln_w = torch.ones(wl.d_v, device="cuda")
    ln_b = torch.zeros(wl.d_v, device="cuda")
    out["output_gate_forward"] = entry(lambda: dig.dig_gla_outgate_fwd(o, r, ln_w, ln_b), 6 * n,
                                       {"shape": [wl.B, wl.L, wl.H, wl.d_v], "bytes_model": "o, r read, z written: 6 B per element"})
    out["output_gate_backward"] = entry(lambda: dig.dig_gla_outgate_bwd(o, r, dz, ln_w, ln_b), 10 * n,
                                        {"shape": [wl.B, wl.L, wl.H, wl.d_v], "bytes_model": "o, r, dz read, d_o, d_r written: 10 B per element"})
    del x, dy, w, o, r, dz
    torch.cuda.empty_cache()

    # the full gate (served by the warp-level tensor-core family) and the state hand-over, on the 4096-token config
    wl = CONFIGS["C3"]
    xin = make_inputs(wl, conv=False)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda().to(torch.bfloat16)
    q, k, v, gg, dO = (dev(xin[m]) for m in ("q", "k", "v", "g", "dO"))
    gate = dig.dig_gate_logsigmoid(gg, xin["tau"])
    bgate = dig.dig_gate_logsigmoid(dev(xin["g"][..., ::-1]), xin["tau"])       # d_k = d_v here: the key gate's logits, channels reversed
    th = wl.B * wl.L * wl.H
    fwd_b, bwd_b = bytes_per_token_head(wl)
    beta_bytes = th * (fwd_b + bwd_b + 4 * wl.d_v * 3)        # bgate read by both passes, dbgate written

    def beta():
        dig.dig_gla_fwd_beta(q, k, v, gate, bgate, wl.grid_h, wl.grid_w, wl.chunk, 0)
        dig.dig_gla_bwd_beta(q, k, v, gate, bgate, dO, wl.grid_h, wl.grid_w, wl.chunk, 0)

    def alpha_only():
        dig.dig_gla_fwd(q, k, v, gate, wl.grid_h, wl.grid_w, wl.chunk, 0)
        dig.dig_gla_bwd(q, k, v, gate, dO, wl.grid_h, wl.grid_w, wl.chunk, 0)

    out["full_gate_fwd_bwd"] = entry(beta, beta_bytes, {"workload": wl.name, "kernel_family": "mma", "tokens_per_s": None})
    out["full_gate_fwd_bwd"]["tokens_per_s"] = wl.B * wl.L / (out["full_gate_fwd_bwd"]["median_ms"] * 1e-3)
    out["full_gate_fwd_bwd"]["alpha_only_same_config"] = entry(alpha_only, th * (fwd_b + bwd_b), {"kernel_family": "tensor"})

    # forward pass of the first and the second half of the rows of the grid, the state of the first handed to the second
    half = wl.grid_h // 2
    Lh = half * wl.grid_w
    parts = [tuple(t[:, :Lh].contiguous() for t in (q, k, v, gate)), tuple(t[:, Lh:].contiguous() for t in (q, k, v, gate))]

    def two_pieces():
        _, s = dig.dig_gla_fwd_state(*parts[0], None, half, wl.grid_w, wl.chunk, 0, want_s_out=True)
        dig.dig_gla_fwd_state(*parts[1], s, wl.grid_h - half, wl.grid_w, wl.chunk, 0, want_s_out=False)

    out["state_handover_forward"] = entry(two_pieces, th * fwd_b, {"workload": wl.name, "pieces": 2})
    out["state_handover_forward"]["one_call"] = entry(lambda: dig.dig_gla_fwd(q, k, v, gate, wl.grid_h, wl.grid_w, wl.chunk, 0), th * fwd_b)
    return out


def cpu_baseline(wl, budget_s=16.0, threads=None):
    """The fp64 oracle, as it stands, on a bounded sample of the workload: whole (batch, head)
    pairs, every scan direction of the workload, gate + fwd + bwd (+ conv on those batches)."""
    import oracle
    from paper_2405_18428_b200.inputs import make_inputs
    cores = max(1, len(os.sched_getaffinity(0))) if threads is None else threads
    # one (b, h) pair costs about L*dk*dv*(2 + 8) fp64 multiply-adds at ~1e9/s per core, per direction
    per_pair = wl.L * wl.d_k * wl.d_v * 10 / 1.0e9 * len(wl.directions)
    pairs_budget = max(1, int(0.5 * budget_s * cores / max(per_pair, 1e-9)))
    nh = max(1, min(wl.H, pairs_budget))
    nb = max(1, min(wl.B, pairs_budget // wl.H)) if nh == wl.H else 1
    sub = wl.scaled(B=nb, H=nh)
    x = make_inputs(sub)
    t0 = time.perf_counter()
    passes = 0
    while True:
        for d in wl.directions:
            a = oracle.gate(x["g"], x["tau"])
            oracle.gla_fwd(x["q"], x["k"], x["v"], a, sub.grid_h, sub.grid_w, d, threads=cores)
            if wl.backward:
                oracle.gla_bwd(x["q"], x["k"], x["v"], a, x["dO"], sub.grid_h, sub.grid_w, d, threads=cores)
            if wl.conv:
                oracle.dwconv(x["conv_x"], x["conv_w"], None, sub.grid_h, sub.grid_w, d)
        passes += 1
        if time.perf_counter() - t0 >= 0.5 * budget_s:
            break
    dt = time.perf_counter() - t0
    # tokens of a full-width batch this much head-work corresponds to (the heads are independent recurrences)
    tokens = nb * wl.L * len(wl.directions) * passes * (nh / wl.H)
    return {"value": tokens / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{nb} of {wl.B} batches x {nh} of {wl.H} heads (tokens scaled by the head fraction), "
                      f"directions {list(wl.directions)}, gate+fwd{'+bwd' if wl.backward else ''}{'+conv' if wl.conv else ''}, "
                      f"{passes} passes, {dt:.2f} s wall on {cores} threads"}, dt, tokens


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    for _ in range(max(0, min(args.warmup, 1))):
        cpu_baseline(wl, budget_s=2.0)
    tot_t, tot_tok, last = 0.0, 0, None
    steps = max(1, min(args.steps, 5))
    for _ in range(steps):
        last, dt, tok = cpu_baseline(wl, budget_s=8.0)
        tot_t += dt
        tot_tok += tok
    value = tot_tok / tot_t
    last["value"] = value
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": 1e3 * tot_t / steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "B": wl.B, "H": wl.H, "grid": [wl.grid_h, wl.grid_w], "d_k": wl.d_k,
                   "d_v": wl.d_v, "note": "fp64 token-by-token CPU oracle on a bounded sample per step"},
        "cpu_baseline": last,
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="C5")
    ap.add_argument("--chunk", type=int, default=0)
    ap.add_argument("--grid", type=int, nargs=2, default=None, metavar=("H", "W"),
                    help="patch grid to use instead of the workload's (a reduced copy of a workload, e.g. for a profiler capture)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--family", default="auto", choices=["auto", "fma", "tensor", "mma"])
    ap.add_argument("--eager", action="store_true", help="time plain stream launches instead of CUDA-graph replays")
    ap.add_argument("--min-seconds", type=float, default=1.0, help="device time the repeated K-step region must add up to")
    ap.add_argument("--no-sweep", action="store_true", help="skip the other workloads (C1 - C4 and the chunk sweep of C4)")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle baseline")
    args = ap.parse_args()

    from paper_2405_18428_b200.inputs import CONFIGS
    wl = CONFIGS[args.workload]
    if args.chunk:
        wl = wl.scaled(chunk=args.chunk)
    if args.grid:
        wl = wl.scaled(name=f"{wl.name}@{args.grid[0]}x{args.grid[1]}", grid_h=args.grid[0], grid_w=args.grid[1])
    if args.impl == "reference":
        return run_reference(args, wl)

    import torch
    from paper_2405_18428_b200 import dig
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist = dist_mod
    dig.lib()      # fails loudly if the CUDA library is missing
    dig.dig_set_impl({"auto": dig.DIG_IMPL_AUTO, "fma": dig.DIG_IMPL_FMA, "tensor": dig.DIG_IMPL_TENSOR, "mma": dig.DIG_IMPL_MMA}[args.family])
    peaks = load_peaks()
    W = max(args.warmup, 3)
    K = args.steps
    dt_id = dig.DIG_BF16 if wl.dtype == "bf16" else dig.DIG_F32
    impl = dig.dig_gla_query_impl(wl.d_k, wl.d_v, wl.chunk, dt_id, int(wl.backward))

    blocks = make_blocks(wl, torch, dig)
    tokens_per_step = wl.B * wl.L * len(blocks)

    # ---- headline: K steps per repetition, repeated until min-seconds of device time have been measured
    ms_eager = time_steps(blocks, dig, torch, K, W, dist)
    graph = None if args.eager else capture_step(blocks, dig, torch)
    launch_mode = "cuda_graph" if graph is not None else "eager"
    if graph is not None:
        for _ in range(W):
            graph.replay()
    one = (lambda: time_replays(graph, torch, K, dist)) if graph is not None else (lambda: time_steps(blocks, dig, torch, K, 0, dist))
    first = one()
    reps = int(min(200, max(3, math.ceil(args.min_seconds * 1e3 / max(first, 1e-3)))))
    if dist is not None:           # every rank must run the same number of repetitions
        t = torch.tensor([reps], dtype=torch.int64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        reps = int(t.item())
    sampler = ClockSampler(local).start()
    rep_ms = [one() for _ in range(reps)]
    clocks = sampler.stop()
    ms = float(np.median(rep_ms))
    value = job_tokens_per_s(tokens_per_step, K, world, ms)
    step_s = ms * 1e-3 / K
    timing = {"repetitions": reps, "steps_per_repetition": K, "median_ms": ms, "min_ms": min(rep_ms), "max_ms": max(rep_ms),
              "timed_seconds_total": sum(rep_ms) * 1e-3,
              "ms_per_step_x_sm_mhz": (ms / K) * clocks["sm_mhz"] if clocks.get("sm_mhz") else None}

    # forward and backward on their own (same blocks, K steps of plain launches each)
    parts = {}
    if wl.backward:
        for p in ("fwd", "bwd"):
            parts[p + "_ms_per_step"] = time_steps(blocks, dig, torch, K, 2, dist, part=p) / K
    # per-kernel times: the same steps once more with every launch bracketed by two CUDA events
    shares = profile_kernels(blocks, dig, torch, min(K, 10))
    assert dig.dig_last_device_status() == dig.DIG_OK
    launches_per_step = sum(s["launches"] for s in shares.values()) // min(K, 10)

    # end-to-end: pinned host -> device copies of every input, the same calls, device -> host of every result
    h2d = d2h = 0
    for b in blocks:
        i, o = b.host_io(torch)
        h2d += i
        d2h += o
    e2e_steps = max(3, min(K, 10))
    ms_e2e = time_steps(blocks, dig, torch, e2e_steps, 3, dist, e2e=True)
    e2e_value = job_tokens_per_s(tokens_per_step, e2e_steps, world, ms_e2e)

    # rooflines: the whole step, and the kernels with a bandwidth model (the dominant one is the headline object)
    work = step_work(wl, impl)
    step_rl = roofline_fracs(work, step_s, peaks)
    krl = kernel_rooflines(shares, wl, peaks)
    gla_kernels = [k for k in shares if k in krl and k not in ("gate_logsigmoid", "srem_dwconv3x3")]
    dom = max(gla_kernels or list(shares), key=lambda k: shares[k]["share"])
    roofline = dict(krl.get(dom, {}), kernel=dom, share_of_step=shares[dom]["share"]) if dom in krl else None

    sweep = {}
    if not args.no_sweep and rank == 0 and world == 1:
        del blocks, graph
        torch.cuda.empty_cache()
        flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        for name, base, over in [("C1", "C1", {}), ("C2", "C2", {}), ("C3", "C3", {}), ("C4", "C4", {}),
                                 ("C4_chunk32", "C4", {"chunk": 32}), ("C4_chunk128", "C4", {"chunk": 128})]:
            if base == wl.name and not over:
                continue
            sweep[name] = sweep_entry(name, CONFIGS[base].scaled(**over), torch, dig, peaks, local, flush)
        # many short sequences (a training batch at 256 x 256 pixels): more sequences than resident CTAs, so sequences
        # are not cut into segments and the forward pass is the forward sweep alone
        sweep["many_sequences"] = sweep_entry("many_sequences", CONFIGS["C2"].scaled(name="B128_L256", B=128, grid_h=16, grid_w=16, directions=(0,), conv=False),
                                              torch, dig, peaks, local, flush)
        sweep["multi"] = multi_direction_entry(CONFIGS["C2"], torch, dig, flush)
        sweep["next_rows"] = next_rows_entry(torch, dig, peaks, flush)
        sweep["note"] = ("one whole step of each workload per timing (its scan directions and conv), captured as a CUDA graph; "
                         "cold = 256 MB written before every timing, warm = back to back; median of 20; roofline from the cold step; "
                         "the tcgen05 kernels work on 64-token tiles for every requested chunk size (tile_executed)")

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu, _, _ = cpu_baseline(wl)
        one_thread, _, _ = cpu_baseline(wl, budget_s=8.0, threads=1)
        cpu["single_thread"] = {"value": one_thread["value"], "sample": one_thread["sample"]}

    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": {2: "f16", 3: "tf32", 1: "f32"}.get(impl, "f32"), "data": "synthetic",
            "config": {"workload": wl.name, "B": wl.B, "H": wl.H, "grid": [wl.grid_h, wl.grid_w], "L": wl.L,
                       "d_k": wl.d_k, "d_v": wl.d_v, "chunk_requested": wl.chunk, "tile_executed": executed_tile(impl, wl.chunk),
                       "storage": wl.dtype, "operands": "fp16 tiles, fp32 accumulation" if impl == 2 else None,
                       "directions": list(wl.directions), "conv": wl.conv, "blocks_per_step": len(wl.directions),
                       "launch": launch_mode, "ms_per_step_eager": ms_eager / K, **parts,
                       "kernel_family": FAMILY.get(impl, str(impl)),
                       "l2": "each block has its own buffers; a step streams far more than the 126 MB L2, no flush needed",
                       "step_roofline": step_rl, "timing": timing},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": ms_e2e / e2e_steps,
                    "copies": "pinned host buffers, two side streams (both PCIe directions overlap the kernels)"},
            "gpu_launches": launches_per_step * K,
            "roofline": roofline, "kernel_rooflines": krl, "kernels": shares, "cpu_baseline": cpu, "sweep": sweep}))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
