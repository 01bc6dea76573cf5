#!/usr/bin/env python
"""Benchmark of the SBP linear-layer hot path on B200.

A step is one pass of the whole path over one batch of synthetic input: draw the keep set once
(the same set serves every SBP layer of the step), build the forward cache of every layer, run the
SBP backward (db, dW, dX) of every layer.  Default workload: the four linear layers of a ViT-B/16
block (qkv, proj, fc1, fc2; bf16, B=128, 14x14 tokens, keep ratio 0.5, random mask), with the
keep-ratio sweep {0.25, 0.5, 0.75, 1.0} reported beside the headline; `--workload vit_b16_fc1` is
the single fc1 layer at B=64.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]
    python bench.py --sweep all|vit|convnext|detection|forward|blocks|attention|sampler [--iters 24]
    python bench.py --probe

Prints one JSON line (rank 0).  ``value`` counts the backward FLOPs of the kept rows
(4 * M_keep * C_in * C_out per layer, step and GPU) over device time, with inputs resident in HBM;
``e2e`` is the same metric through ``sbp_step_host`` with pinned host tensors (copies timed).
With N > 1 every rank processes its own shard of the batch (its own sample ids); the path itself has
no exchange step, so the headline issues no collective (weak scaling); the all-reduce of dW / db that
data-parallel training adds is timed beside it.  Without torchrun, ``--gpus N`` starts the N ranks itself.
``--impl reference`` times the fp64 CPU oracle on a bounded sample of the same workload.
``--sweep`` prints per-call timing tables for every layer shape of the paper's models instead.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2210_00129_b200 import synth  # noqa: E402

METRIC = "sbp_backward_tflops_kept_rows"
UNIT = "TFLOP/s"
# dram__bytes_read + dram__bytes_write per launch of the dominant kernel (mean over the launches of one step), from
# the ncu captures summarised in profiles/ (absent = never captured, or the kernel changed since)
NCU_TRAFFIC_BYTES = {"vit_b16_block_b128": 176.0e6, "convnext_b_s1_block": 225.3e6}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL_BF16_TFLOPS = 2250.0

VIT_BLOCK = (("qkv", 768, 2304), ("proj", 768, 768), ("fc1", 768, 3072), ("fc2", 3072, 768))


def _wl(B, H, W, layers, keep_ratio=0.5, mode=0, dtype="bf16", sweep=None):
    return dict(dtype=dtype, B=B, H=H, W=W, keep_ratio=keep_ratio, mode=mode, layers=tuple(layers),
                sweep=tuple(sweep) if sweep else tuple(sorted({keep_ratio, 1.0})))


WORKLOADS = {
    # the linear layers of one ViT-B/16 block with the keep-ratio sweep
    "vit_b16_block_b128": _wl(128, 14, 14, VIT_BLOCK, sweep=(0.25, 0.5, 0.75, 1.0)),
    # single layers
    "vit_b16_fc1": _wl(64, 14, 14, [("fc1", 768, 3072)]),
    "vit_b16_fc2": _wl(64, 14, 14, [("fc2", 3072, 768)]),
    "vit_b16_fc1_b128": _wl(128, 14, 14, [("fc1", 768, 3072)]),
    "vit_b16_qkv_b128": _wl(128, 14, 14, [("qkv", 768, 2304)]),
    "vit_b16_proj_b128": _wl(128, 14, 14, [("proj", 768, 768)]),
    "convnext_b_s1_block": _wl(64, 56, 56, [("pw1", 128, 512), ("pw2", 512, 128)]),
    "convnext_b_s1_pw1": _wl(64, 56, 56, [("pw1", 128, 512)]),
    "convnext_b_s1_pw2": _wl(64, 56, 56, [("pw2", 512, 128)]),
    "convnext_b_s2_block_grid": _wl(64, 28, 28, [("pw1", 256, 1024), ("pw2", 1024, 256)], mode=1),
    "convnext_b_s3_pw1_grid": _wl(64, 14, 14, [("pw1", 512, 2048)], mode=1),
    "det_s1_block": _wl(2, 200, 334, [("pw1", 128, 512), ("pw2", 512, 128)]),
    "det_s1_pw1": _wl(2, 200, 334, [("pw1", 128, 512)]),
    "single_fp32": _wl(2, 16, 1, [("fc", 32, 64)], dtype="f32"),
    # a small block for smoke runs of the whole benchmark
    "tiny_block": _wl(4, 14, 14, [("a", 256, 384), ("b", 384, 256)], sweep=(0.5, 1.0)),
}
DEFAULT_WORKLOAD = "vit_b16_block_b128"


def config_of(name, w, n_gpus):
    """The `config` object of the JSON line: the same keys and values in both arms."""
    return {"workload": name, "B_per_gpu": w["B"], "H": w["H"], "W": w["W"],
            "layers": [f"{n}:{ci}->{co}" for n, ci, co in w["layers"]], "keep_ratio": w["keep_ratio"],
            "keep_ratio_sweep": list(w["sweep"]), "mask": "grid" if w["mode"] else "random",
            "parallelism": f"dp{n_gpus} (batch sharded by sample id)"}


def sample_offset_of(rank, B_per_gpu):
    """First global sample id of a rank's shard: rank r owns samples [r * B, (r + 1) * B)."""
    return rank * B_per_gpu


def max_over_ranks(ms, device):
    """Step time of a multi-rank run: the slowest rank's (no-op for a single process)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def bytes_of(dtype):
    return 2 if dtype == "bf16" else 4


def flops_of(w, M_keep):
    return sum(4.0 * M_keep * ci * co for _, ci, co in w["layers"])


def algorithmic_bytes(w, M, M_keep):
    """Bytes the backward calls of one step must move: kept rows of dY and X_keep and W read, dX, dW, db written."""
    es = bytes_of(w["dtype"])
    return sum(M_keep * (ci + co) * es + ci * co * es + 4.0 * ci * co + M * ci * es + 4 * co for _, ci, co in w["layers"])


class ClockSampler:
    """nvidia-smi clock / throttle-reason sampler running beside the timed region."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"], "samples": 0}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, smax, power = [], [], []
        reasons = set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [t.strip() for t in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); smax.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "reasons": sorted(reasons), "samples": len(sm)}


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def respawn_under_torchrun(n_gpus):
    """`python bench.py --gpus N` without a launcher: start the N ranks (one process per GPU) and pass their output through."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


# ----------------------------------------------------------------------------------------------
# reference arm / CPU baseline: the fp64 oracle, as it stands, on a bounded sample
# ----------------------------------------------------------------------------------------------
def oracle_sample_step(w, B_s, data_seed):
    """One whole step of the oracle on the first B_s samples of the workload; returns (seconds, flops)."""
    import oracle
    N = w["H"] * w["W"]
    M = B_s * N
    tensors = []
    for li, (_, ci, co) in enumerate(w["layers"]):
        X, Wt, dY = synth.layer_inputs(w["dtype"], M, ci, co, data_seed + li)
        tensors.append(tuple(synth.to_f64(a, w["dtype"]) for a in (X, Wt, dY)))
    t0 = time.perf_counter()
    keep, _ = oracle.sample_keep(w["mode"], B_s, w["H"], w["W"], w["keep_ratio"], 0, 0, 0)
    caches = [oracle.forward_cache(Xf, keep) for Xf, _, _ in tensors]
    for Xk, (Xf, Wf, dYf) in zip(caches, tensors):
        oracle.linear_backward(Xk, dYf, Wf, keep)
    dt = time.perf_counter() - t0
    return dt, flops_of(w, len(keep))


def pick_oracle_sample(w, target_s=12.0):
    """Samples of the batch the oracle gets: sized from a one-sample probe to ~target_s seconds."""
    import oracle
    oracle.build()
    t1, _ = oracle_sample_step(w, 1, 999)
    return int(max(1, min(w["B"], target_s / max(t1, 1e-4))))


def run_reference(args, w, name):
    import oracle
    if int(os.environ.get("RANK", "0")) != 0:
        return
    # bounded sample: the whole run (probe + warm-up + K steps) stays near a minute and a half
    B_s = pick_oracle_sample(w, target_s=min(6.0, 90.0 / (args.steps + 2)))
    for _ in range(min(args.warmup, 1)):
        oracle_sample_step(w, B_s, 1000)
    times, flops = [], 0.0
    for _ in range(args.steps):
        dt, fl = oracle_sample_step(w, B_s, 1000)
        times.append(dt); flops = fl
    total = sum(times)
    value = flops * args.steps / total / 1e12
    cores = oracle.num_threads()
    sample = f"first {B_s} of {w['B']} samples of {name} per step (whole path: sampler, caches, dW, db, dX of every layer)"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(name, w, args.gpus),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------
# CUDA arm
# ----------------------------------------------------------------------------------------------
class Job:
    """Device buffers of one workload on this rank and the step that runs the path through the C ABI."""

    def __init__(self, w, rank, n_sets=None):
        import torch
        import paper_2210_00129_b200 as sbp
        self.torch, self.sbp, self.w = torch, sbp, w
        self.lib = sbp.load_library()
        self.dtype, self.B, self.H, self.W_, self.r, self.mode = (w[k] for k in ("dtype", "B", "H", "W", "keep_ratio", "mode"))
        self.layers = w["layers"]
        self.code = sbp.SBP_BF16 if self.dtype == "bf16" else sbp.SBP_F32
        self.es = bytes_of(self.dtype)
        self.tdt = torch.bfloat16 if self.dtype == "bf16" else torch.float32
        self.M = self.B * self.H * self.W_
        self.cap = {r: self.B * sbp.sbp_keep_count(self.mode, self.H, self.W_, r) for r in set(w["sweep"]) | {self.r, 1.0}}
        self.sample_offset = sample_offset_of(rank, self.B)
        M = self.M
        # seeded host tensors: one X per distinct C_in, one dY per distinct C_out, one W per layer
        self.host = {}
        for li, (_, ci, co) in enumerate(self.layers):
            if ("X", ci) not in self.host:
                self.host[("X", ci)] = synth.gaussian_tensor((M, ci), self.dtype, 1002 + rank, 10 + len(self.host), 1.0)
            if ("dY", co) not in self.host:
                self.host[("dY", co)] = synth.gaussian_tensor((M, co), self.dtype, 1002 + rank, 10 + len(self.host), 1e-2)
            self.host[("W", li)] = synth.gaussian_tensor((ci, co), self.dtype, 1002 + rank, 500 + li, 0.02)
        # ---- buffer sets: rotate so that consecutive steps never find their inputs in the 126 MB L2 ----
        self.set_bytes = sum((M * ci + M * co + ci * co + 2 * M * ci) * self.es + ci * co * 4 for _, ci, co in self.layers)
        if n_sets is None:
            n_sets = min(max(2, int(np.ceil(3 * 126e6 / self.set_bytes)) + 1), 64)
        self.n_sets = n_sets
        self.grad_elems = sum(ci * co + co for _, ci, co in self.layers)
        self.sets = []
        for i in range(n_sets):
            s = dict(rows=torch.zeros(M, dtype=torch.int32, device="cuda"),
                     offs=torch.zeros(self.B + 1, dtype=torch.int32, device="cuda"),
                     grads=torch.zeros(self.grad_elems, dtype=torch.float32, device="cuda"), layers=[])
            off = 0
            for li, (_, ci, co) in enumerate(self.layers):
                X, dY, Wt = self.to_dev(self.host[("X", ci)]), self.to_dev(self.host[("dY", co)]), self.to_dev(self.host[("W", li)])
                if i:   # same distribution, different bits per set: roll the seeded tensors
                    X, dY = torch.roll(X, i + li, 0), torch.roll(dY, i + li, 0)
                # the cache holds a full batch so that the same sets also serve the keep = 1.0 comparison;
                # dW and db of all layers sit in one flat buffer (one all-reduce per step in data-parallel runs)
                L = dict(X=X, dY=dY, W=Wt, Xk=torch.zeros((M, ci), dtype=self.tdt, device="cuda"),
                         dW=s["grads"][off:off + ci * co].view(ci, co), db=s["grads"][off + ci * co:off + ci * co + co],
                         dX=torch.zeros((M, ci), dtype=self.tdt, device="cuda"))
                off += ci * co + co
                L["p"] = {k: L[k].data_ptr() for k in ("X", "dY", "W", "Xk", "dW", "db", "dX")}
                s["layers"].append(L)
            s["p"] = dict(rows=s["rows"].data_ptr(), offs=s["offs"].data_ptr(), cnt=s["offs"].data_ptr() + 4 * self.B)
            self.sets.append(s)
        self.ws_bytes = max(sbp.sbp_linear_backward_workspace_bytes(self.code, M, c, ci, co)
                            for c in self.cap.values() for _, ci, co in self.layers)
        self.ws = torch.empty(self.ws_bytes, dtype=torch.uint8, device="cuda")
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")
        self.stream = torch.cuda.current_stream()

    def to_dev(self, a):
        t = self.torch.from_numpy(a).cuda()
        return t.view(self.torch.bfloat16) if self.dtype == "bf16" else t

    def launches_per_step(self, r=None):
        r = self.r if r is None else r
        return 1 + sum(1 + self.sbp.sbp_linear_backward_kernel_count(self.code, self.M, self.cap[r], ci, co, True, True, True, 0)
                       for _, ci, co in self.layers)

    def step(self, i, r=None, events=None, sid=None):
        """One pass of the whole path: draw the keep set, cache the kept rows of every layer's input, run every
        layer's backward (last layer first).  `events`: one (before, after) pair per layer around its backward call."""
        r = self.r if r is None else r
        sid = self.stream.cuda_stream if sid is None else sid
        lib, code, M, capk = self.lib, self.code, self.M, self.cap[r]
        s = self.sets[i % self.n_sets]
        a = s["p"]
        rc = lib.sbp_sample_keep(self.mode, self.B, self.H, self.W_, r, 0, i, self.sample_offset, 0, a["rows"], a["offs"], sid)
        for (_, ci, co), L in zip(self.layers, s["layers"]):
            rc |= lib.sbp_forward_cache(code, L["p"]["X"], M, ci, a["rows"], a["cnt"], capk, L["p"]["Xk"], sid)
        for li in range(len(self.layers) - 1, -1, -1):
            if events is not None:
                events[li][0].record(self.stream)
            rc |= self.backward_call(i, li, r, sid)
            if events is not None:
                events[li][1].record(self.stream)
        if rc != 0:
            raise RuntimeError(f"sbp call failed with status {rc}")

    def backward_call(self, i, li, r, sid):
        """sbp_linear_backward of layer li on buffer set i (its keep set and cache must have been made at ratio r)."""
        s = self.sets[i % self.n_sets]
        _, ci, co = self.layers[li]
        q, a = s["layers"][li]["p"], s["p"]
        return self.lib.sbp_linear_backward(self.code, q["Xk"], q["dY"], q["W"], a["rows"], a["cnt"], self.M, self.cap[r], ci, co,
                                            q["dW"], q["db"], q["dX"], 0, self.ws.data_ptr(), self.ws_bytes, self.status.data_ptr(), sid)

    def timed_backward_graphs(self, r, reps):
        """Device time of every layer's backward call at keep ratio r, without the host in the loop: per layer one CUDA
        graph holding that call once per buffer set, replayed `reps` times between two events on the launch stream.
        Returns (per-layer ms per call, seconds of the timed replays)."""
        torch = self.torch
        for k in range(self.n_sets):                       # keep sets and caches of every buffer set at this ratio
            self.step(k, r)
        self.barrier()
        cap_stream = torch.cuda.Stream()
        cap_stream.wait_stream(self.stream)
        per_layer, total_s = [], 0.0
        for li in range(len(self.layers)):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=cap_stream):
                for k in range(self.n_sets):
                    if self.backward_call(k, li, r, cap_stream.cuda_stream) != 0:
                        raise RuntimeError("sbp_linear_backward failed during capture")
            g.replay()
            self.barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(self.stream)
            for _ in range(reps):
                g.replay()
            e1.record(self.stream)
            self.barrier()
            ms = max_over_ranks(e0.elapsed_time(e1), "cuda")
            per_layer.append(ms / (reps * self.n_sets))
            total_s += ms * 1e-3
        return per_layer, total_s

    def barrier(self):
        import torch.distributed as dist
        if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
            dist.barrier()
        self.torch.cuda.synchronize()

    def timed_calls(self, k_steps, r=None, inner_events=True, allreduce=False):
        """K steps of direct C-ABI calls between two events; returns (total ms over ranks, per-layer mean backward ms)."""
        torch = self.torch
        nl = len(self.layers)
        evs = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(nl)]
               if inner_events else None for _ in range(k_steps)]
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.barrier()
        e0.record(self.stream)
        for i in range(k_steps):
            self.step(i, r, evs[i])
            if allreduce:
                import torch.distributed as dist
                dist.all_reduce(self.sets[i % self.n_sets]["grads"])      # sum of dW and db of every layer over the ranks
        e1.record(self.stream)
        self.barrier()
        total_ms = max_over_ranks(e0.elapsed_time(e1), "cuda")
        if not inner_events:
            return total_ms, None
        return total_ms, [sum(e[li][0].elapsed_time(e[li][1]) for e in evs) / k_steps for li in range(nl)]

    def capture_graphs(self):
        """One captured step per buffer set (sampler, caches, backward calls through the same C-ABI calls): replaying
        them keeps the host out of the timed region.  The step counter of a captured step is fixed, so the masks
        repeat every n_sets steps; every replay still draws, gathers and multiplies from scratch."""
        torch = self.torch
        cap_stream = torch.cuda.Stream()
        cap_stream.wait_stream(self.stream)
        self.graphs = []
        for k in range(self.n_sets):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=cap_stream):
                self.step(k, sid=cap_stream.cuda_stream)
            self.graphs.append(g)
        for g in self.graphs:
            g.replay()
        self.barrier()

    def timed_graphs(self, k_steps):
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.barrier()
        e0.record(self.stream)
        for i in range(k_steps):
            self.graphs[i % self.n_sets].replay()
        e1.record(self.stream)
        self.barrier()
        return max_over_ranks(e0.elapsed_time(e1), "cuda")

    def m_keep(self):
        return int(self.sets[0]["offs"][self.B].item())


def time_e2e(job, world, steps):
    """The same metric end to end: every step copies its inputs in from pinned host tensors and all results back,
    through sbp_step_host (one call per layer).  Two streams, each with its own device arena and pinned outputs, take
    the steps alternately, so the copies of one step overlap the kernels and the copies of the step before it."""
    torch, sbp, w = job.torch, job.sbp, job.w
    M, B = job.M, job.B
    pin = lambda a: torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).pin_memory()
    host_in = {k: pin(v) for k, v in job.host.items()}
    arena_bytes = max(sbp.sbp_step_host_arena_bytes(job.code, job.mode, B, job.H, job.W_, ci, co, job.r) for _, ci, co in job.layers)
    out_dt = torch.int16 if job.dtype == "bf16" else torch.float32
    lanes = []
    for _ in range(2):
        lanes.append(dict(stream=torch.cuda.Stream(), arena=torch.empty(arena_bytes, dtype=torch.uint8, device="cuda"),
                          st=torch.zeros(len(job.layers), dtype=torch.int32).pin_memory(),
                          out=[dict(dW=torch.empty((ci, co), dtype=torch.float32).pin_memory(),
                                    db=torch.empty(co, dtype=torch.float32).pin_memory(),
                                    dX=torch.empty((M, ci), dtype=out_dt).pin_memory()) for _, ci, co in job.layers]))

    def host_step(i):
        ln = lanes[i % 2]
        for li, (_, ci, co) in enumerate(job.layers):
            o = ln["out"][li]
            sbp.sbp_step_host(job.code, job.mode, B, job.H, job.W_, ci, co, job.r, 0, i, job.sample_offset, 0,
                              host_in[("X", ci)], host_in[("dY", co)], host_in[("W", li)], o["dW"], o["db"], o["dX"], None, None,
                              ln["st"].data_ptr() + 4 * li, ln["arena"], arena_bytes, stream=ln["stream"].cuda_stream)
    for i in range(2):
        host_step(i)
    job.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(job.stream)
    for ln in lanes:
        ln["stream"].wait_stream(job.stream)
    for i in range(steps):
        host_step(i)
    for ln in lanes:
        job.stream.wait_stream(ln["stream"])
    e1.record(job.stream)
    job.barrier()
    ms = max_over_ranks(e0.elapsed_time(e1), "cuda")
    assert int((lanes[0]["st"] + lanes[1]["st"]).abs().sum().item()) == 0, "device status word set in the end-to-end steps"
    h2d = sum((M * ci + M * co + ci * co) * job.es for _, ci, co in job.layers)
    d2h = sum(ci * co * 4 + co * 4 + M * ci * job.es + 4 for _, ci, co in job.layers)
    return ms, h2d, d2h


def run_cuda(args, w, name):
    import torch
    import torch.distributed as dist
    import paper_2210_00129_b200 as sbp
    from paper_2210_00129_b200 import build as sbp_build

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.gpus != world:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE is {world}: launch one rank per GPU (or drop the launcher)")
    if rank == 0:
        sbp_build.build()
    torch.cuda.set_device(local_rank)
    if "WORLD_SIZE" in os.environ:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    sbp.load_library()
    warmup = max(args.warmup, 3)
    job = Job(w, rank)
    for i in range(warmup):
        job.step(i)
    job.barrier()
    assert int(job.status.item()) == 0, "device status word set during warm-up"
    M, M_keep = job.M, job.m_keep()
    if args.launch == "graph":
        job.capture_graphs()

    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.3)
    # The headline region replays whole captured steps.  The launch durations the roofline figure uses come from a
    # second set of replays that hold only the backward calls, layer by layer (events between the calls of a step
    # would keep a kernel from starting its launch early, and direct calls would put the host's pace into the figure).
    total_ms = job.timed_graphs(args.steps) if args.launch == "graph" else job.timed_calls(args.steps, inner_events=False)[0]
    reps = max(1, -(-args.steps // job.n_sets))                    # about K launches of every layer's backward call
    layer_ms, layer_s = job.timed_backward_graphs(w["keep_ratio"], reps)
    clocks = sampler.stop() if sampler else None
    assert int(job.status.item()) == 0, "device status word set during the timed steps"
    flops_step = flops_of(w, M_keep)
    value = flops_step * args.steps * world / (total_ms * 1e-3) / 1e12

    # ---- data-parallel runs: the same steps followed by the all-reduce (sum) of dW and db over the ranks ----
    with_allreduce = None
    if dist.is_initialized() and (world > 1 or args.allreduce):
        for i in range(3):
            job.step(i)
            dist.all_reduce(job.sets[i % job.n_sets]["grads"])
        plain_ms, _ = job.timed_calls(args.steps, inner_events=False)
        ar_ms, _ = job.timed_calls(args.steps, inner_events=False, allreduce=True)
        with_allreduce = {"ms_per_step": ar_ms / args.steps, "ms_per_step_without": plain_ms / args.steps,
                          "value": flops_step * args.steps * world / (ar_ms * 1e-3) / 1e12, "unit": UNIT,
                          "bytes_per_rank": 4 * job.grad_elems, "collective": "one NCCL all-reduce (sum) of dW and db of every layer per step",
                          "launch": "direct C-ABI calls"}

    # ---- the same kernels over the keep-ratio sweep: backward time, speed-up against keep ratio 1.0, saved activations ----
    sweep_reps = max(2, reps // 4)
    sweep = {}
    for r in sorted(set(w["sweep"]) | {1.0}):
        per_layer = layer_ms if r == w["keep_ratio"] else job.timed_backward_graphs(r, sweep_reps)[0]
        if r == w["keep_ratio"]:
            for k in range(job.n_sets):
                job.step(k, r)
            job.barrier()
        mk = job.m_keep()
        sweep[r] = dict(M_keep=mk, bwd_ms=per_layer, bwd_ms_total=sum(per_layer),
                        tflops_bwd=flops_of(w, mk) / (sum(per_layer) * 1e-3) / 1e12)
    for r, s in sweep.items():
        s["bwd_speedup_vs_keep1"] = sweep[1.0]["bwd_ms_total"] / s["bwd_ms_total"]
        s["saved_activation_frac_vs_keep1"] = (sum(s["M_keep"] * ci * job.es for _, ci, _ in job.layers) + 4 * s["M_keep"] + 4 * (job.B + 1)) / \
            sum(M * ci * job.es for _, ci, _ in job.layers)
    for i in range(3):
        job.step(i)
    job.barrier()

    e2e_steps = max(4, min(args.steps, 20))
    e2e_ms, h2d, d2h = time_e2e(job, world, e2e_steps)
    e2e_value = flops_step * e2e_steps * world / (e2e_ms * 1e-3) / 1e12

    if rank == 0:
        print(json.dumps(json_line(args, w, name, job, world, dict(
            total_ms=total_ms, calls_ms=layer_s * 1e3, layer_ms=layer_ms, clocks=clocks, value=value, M_keep=M_keep,
            with_allreduce=with_allreduce, sweep=sweep, e2e_ms=e2e_ms, e2e_steps=e2e_steps, e2e_value=e2e_value, h2d=h2d, d2h=d2h,
            warmup=warmup))))
    if dist.is_initialized():
        dist.barrier()
        dist.destroy_process_group()


def roofline_of(w, name, job, r):
    """Roofline object of the dominant kernel (tc_backward_kernel; the CUDA-core kernels for fp32 / tiny shapes):
    algorithmic work of the backward calls of one step over their measured duration, against the measured peak."""
    peaks, peak_kind = load_peaks()
    M, M_keep = job.M, r["M_keep"]
    launch_ms = sum(r["layer_ms"])
    nl = len(w["layers"])
    flops = flops_of(w, M_keep)
    by = algorithmic_bytes(w, M, M_keep)
    tc_path = w["dtype"] == "bf16" and all(min(ci, co) >= 128 for _, ci, co in w["layers"]) and M_keep >= 64
    timed_s = r["calls_ms"] * 1e-3
    clk = r["clocks"] or {}
    # a cuBLAS-style burst figure is the right denominator unless the timed region was long enough, and the clocks low
    # enough, for the part to have settled into its power-limited state
    sustained = bool(timed_s >= 1.0 and clk.get("sm_mhz") and clk.get("sm_max_mhz") and clk["sm_mhz"] < 0.9 * clk["sm_max_mhz"])
    burst_peak = float(peaks["bf16_tflops"])
    sust_peak = float(peaks.get("bf16_tflops_sustained", burst_peak))
    hbm_peak = float(peaks["hbm_gbs"])
    if not tc_path:
        peak = 148 * 128 * 2 * 1.965e9 / 1e12     # 128 fp32 FMA lanes x 148 SMs x 2 FLOP at the maximum SM clock
        out = {"kernel": "simt_dw_kernel + simt_dx_kernel", "bound": "alu", "achieved": flops / (launch_ms * 1e-3) / 1e12,
               "peak": peak, "peak_kind": "derived: 148 SMs x 128 FMA/clk x 2 x 1.965 GHz", "unit": "TFLOP/s", "traffic": None}
    elif by / (hbm_peak * 1e9) > flops / (burst_peak * 1e12):
        out = {"kernel": "tc_backward_kernel (dW and dX tiles, db on the side; timed with its reduce kernel)", "bound": "hbm",
               "achieved": by / (launch_ms * 1e-3) / 1e9, "peak": hbm_peak, "peak_kind": f"{peak_kind} copy bandwidth",
               "unit": "GB/s", "traffic": NCU_TRAFFIC_BYTES.get(name), "algorithmic_bytes_per_launch": by / nl}
    else:
        ach = flops / (launch_ms * 1e-3) / 1e12
        out = {"kernel": "tc_backward_kernel (dW and dX tiles, db on the side; timed with its reduce kernel)", "bound": "tensor",
               "achieved": ach, "peak": sust_peak if sustained else burst_peak,
               "peak_kind": f"{peak_kind} cuBLAS bf16, " + ("sustained (timed region over 1 s at reduced clocks)" if sustained
                                                          else "burst (short timed region at full clocks)"),
               "unit": "TFLOP/s", "traffic": NCU_TRAFFIC_BYTES.get(name),
               "frac_burst": ach / burst_peak, "frac_sustained": ach / sust_peak,
               "peak_nominal": NOMINAL_BF16_TFLOPS, "frac_nominal": ach / NOMINAL_BF16_TFLOPS,
               "flops_per_launch": flops / nl}
    out["frac"] = out["achieved"] / out["peak"]
    out["launches_per_step"] = nl
    out["launch_ms"] = launch_ms / nl
    out["timed_region_s"] = timed_s
    out["per_layer"] = {n: {"ms": ms, "tflops": 4.0 * M_keep * ci * co / (ms * 1e-3) / 1e12}
                        for (n, ci, co), ms in zip(w["layers"], r["layer_ms"])}
    return out


def json_line(args, w, name, job, world, r):
    import oracle
    B_s = pick_oracle_sample(w)
    cpu_s, cpu_flops = oracle_sample_step(w, B_s, 1000)
    cpu_threads = oracle.num_threads()
    B_1 = max(1, B_s // 8)                              # single-thread figure on a smaller slice
    oracle.set_num_threads(1)
    cpu1_s, cpu1_flops = oracle_sample_step(w, B_1, 1000)
    oracle.set_num_threads(cpu_threads)
    keep1 = r["sweep"][1.0]
    main = r["sweep"][w["keep_ratio"]]
    cfg = config_of(name, w, world)
    return {
        "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": r["warmup"], "ms_per_step": r["total_ms"] / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if w["dtype"] == "bf16" else "f32", "data": "synthetic",
        "config": cfg,
        "run": {"M": job.M, "M_keep": r["M_keep"],
                "l2": f"inputs larger than L2: {job.n_sets} rotating buffer sets of {job.set_bytes / 1e6:.0f} MB",
                "launch": (f"CUDA graph replay, one captured step ({1 + 2 * len(w['layers'])} C-ABI calls) per buffer set"
                           if args.launch == "graph" else "direct C-ABI calls"),
                "collective": "none in the headline (the path has no exchange step)"},
        "roofline": roofline_of(w, name, job, r),
        "cpu_baseline": {"value": cpu_flops / cpu_s / 1e12, "unit": UNIT, "cores": cpu_threads,
                         "kind": "oracle", "seconds": cpu_s,
                         "sample": f"first {B_s} of {w['B']} samples of {name}, whole path once, fp64",
                         "single_thread": {"value": cpu1_flops / cpu1_s / 1e12, "unit": UNIT, "seconds": cpu1_s,
                                           "sample": f"first {B_1} of {w['B']} samples"}},
        "e2e": {"value": r["e2e_value"], "unit": UNIT, "h2d_bytes_per_step": r["h2d"], "d2h_bytes_per_step": r["d2h"],
                "ms_per_step": r["e2e_ms"] / r["e2e_steps"], "steps": r["e2e_steps"],
                "api": "sbp_step_host, one call per layer (pinned host tensors; steps alternate between two streams so copies overlap)"},
        "gpu_launches": job.launches_per_step() * args.steps,
        "clocks": r["clocks"],
        "bwd_speedup_vs_keep1": main["bwd_speedup_vs_keep1"],
        "bwd_ms": {"keep": main["bwd_ms_total"], "keep1": keep1["bwd_ms_total"]},
        "saved_activation_frac_vs_keep1": main["saved_activation_frac_vs_keep1"],
        "keep_ratio_sweep": {str(k): {kk: (vv if not isinstance(vv, list) else [round(x, 5) for x in vv]) for kk, vv in v.items()}
                             for k, v in r["sweep"].items()},
        "with_allreduce": r["with_allreduce"],
    }


# ----------------------------------------------------------------------------------------------
# --sweep: per-call timing of every layer shape of the paper's models against the roofline of each call
# ----------------------------------------------------------------------------------------------
# For every layer of the chosen groups (ViT-B/16 MLP and attention projections at four keep ratios, ConvNeXt-B
# point-wise layers of the four stages with random and grid masks, the detection-resolution map; Sec. 5 of the paper
# gives the models) it times sbp_sample_keep, sbp_forward_cache and sbp_linear_backward (dW alone, dX alone, db alone,
# both products, all three) and prints a markdown table: microseconds, the lower bound
# t_min = max(FLOP / peak, bytes / bandwidth) of the call's algorithmic work, t_min / t, and the speed-up of the whole
# backward over keep ratio 1.0.  Each call is captured `iters` times into a CUDA graph over rotating buffer sets whose
# total size exceeds the L2 cache, the graph is replayed once untimed and once between two CUDA events.
def sweep_layers(group):
    """(name, B, H, W, C_in, C_out, keep ratio, mask mode) of every layer of a group."""
    out = []
    if group in ("vit", "all"):
        out.append(("vit_b16 fc1 B=64", 64, 14, 14, 768, 3072, 0.5, 0))
        for r in (0.25, 0.5, 0.75, 1.0):
            for nm, ci, co in (("qkv", 768, 2304), ("proj", 768, 768), ("fc1", 768, 3072), ("fc2", 3072, 768)):
                out.append((f"vit_b16 {nm} B=128 r={r}", 128, 14, 14, ci, co, r, 0))
    if group in ("convnext", "all"):
        for mode in (0, 1):
            for st, (dim, hw) in enumerate(((128, 56), (256, 28), (512, 14), (1024, 7)), 1):
                for nm, ci, co in (("pw1", dim, 4 * dim), ("pw2", 4 * dim, dim)):
                    out.append((f"convnext_b s{st} {nm} {'grid' if mode else 'random'}", 64, hw, hw, ci, co, 0.5, mode))
    if group in ("detection", "all"):
        for nm, ci, co in (("128->512", 128, 512), ("512->128", 512, 128)):
            out.append((f"detection 200x334 {nm}", 2, 200, 334, ci, co, 0.5, 0))
    return out


class GraphTimer:
    def __init__(self, iters):
        self.iters = iters
        self.stream = torch.cuda.Stream()
        self.sid = self.stream.cuda_stream

    def time_us(self, fn, n_sets):
        """fn(set index, step) enqueues one call on self.stream; returns microseconds per call."""
        with torch.cuda.stream(self.stream):
            for i in range(3):
                fn(i % n_sets, i)
            self.stream.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=self.stream):
                for i in range(self.iters):
                    fn(i % n_sets, i)
        g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        g.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / self.iters * 1e3


def measure_layer(bench, spec, pk):
    name, B, H, W_, C_in, C_out, r, mode = spec
    es = 2
    M = B * H * W_
    cap = B * sbp.sbp_keep_count(mode, H, W_, r)
    set_bytes = (2 * M * C_in + M * C_out + C_in * C_out + cap * C_in) * es + C_in * C_out * 4
    n_sets = max(3, int(400e6 // set_bytes) + 1)
    gen = torch.Generator(device="cuda").manual_seed(1234)
    sets = []
    for _ in range(n_sets):
        sets.append(dict(
            X=torch.randn(M, C_in, device="cuda", generator=gen).bfloat16(),
            dY=(torch.randn(M, C_out, device="cuda", generator=gen) * 0.01).bfloat16(),
            W=(torch.randn(C_in, C_out, device="cuda", generator=gen) * 0.02).bfloat16(),
            rows=torch.zeros(cap, dtype=torch.int32, device="cuda"),
            offs=torch.zeros(B + 1, dtype=torch.int32, device="cuda"),
            Xk=torch.zeros(cap, C_in, device="cuda", dtype=torch.bfloat16),
            dW=torch.zeros(C_in, C_out, device="cuda"), db=torch.zeros(C_out, device="cuda"),
            dX=torch.zeros(M, C_in, device="cuda", dtype=torch.bfloat16)))
    nb = sbp.sbp_linear_backward_workspace_bytes(sbp.SBP_BF16, M, cap, C_in, C_out)
    ws = torch.empty(max(nb, 16), dtype=torch.uint8, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    sid = bench.sid
    torch.cuda.synchronize()      # the buffers were filled on torch's stream; the calls below run on another

    def cnt(s):          # device-side row count (grid masks on odd maps keep 24 or 25 of 49)
        return s["offs"][B:] if mode == 1 else None

    def sample(k, i):
        s = sets[k]
        sbp.sbp_sample_keep(mode, B, H, W_, r, 0, i, 0, 0, s["rows"], s["offs"], stream=sid)

    def cache(k, i):
        s = sets[k]
        sbp.sbp_forward_cache(sbp.SBP_BF16, s["X"], M, C_in, s["rows"], cnt(s), cap, s["Xk"], stream=sid)

    def bw(k, dW, db, dX):
        s = sets[k]
        sbp.sbp_linear_backward(sbp.SBP_BF16, s["Xk"], s["dY"], s["W"], s["rows"], cnt(s), M, cap, C_in, C_out,
                                s["dW"] if dW else None, s["db"] if db else None, s["dX"] if dX else None, 0, ws, nb,
                                st, stream=sid)

    with torch.cuda.stream(bench.stream):
        for k in range(n_sets):
            sample(k, 0)
            cache(k, 0)
    bench.stream.synchronize()
    M_keep = int(sets[0]["offs"][B].item())

    t = {
        "sample": bench.time_us(sample, n_sets),
        "cache": bench.time_us(cache, n_sets),
        "db": bench.time_us(lambda k, i: bw(k, 0, 1, 0), n_sets),
        "dW": bench.time_us(lambda k, i: bw(k, 1, 0, 0), n_sets),
        "dX": bench.time_us(lambda k, i: bw(k, 0, 0, 1), n_sets),
        "dW+dX": bench.time_us(lambda k, i: bw(k, 1, 0, 1), n_sets),
        "bwd": bench.time_us(lambda k, i: bw(k, 1, 1, 1), n_sets),
    }
    assert int(st.item()) == 0, f"status word {int(st.item())} on {name}"
    flop = 2.0 * M_keep * C_in * C_out
    tf, bw_ = pk["bf16_tflops_sustained"] * 1e12, pk["hbm_gbs"] * 1e9
    by = {   # algorithmic HBM bytes of each call
        "sample": 4.0 * M_keep + 4 * (B + 1),
        "cache": 2.0 * M_keep * C_in * es + 4 * M_keep,
        "db": M_keep * C_out * es + 4.0 * M_keep,
        "dW": M_keep * (C_in + C_out) * es + 4.0 * C_in * C_out,
        "dX": M_keep * C_out * es + C_in * C_out * es + M * C_in * es,
    }
    by["bwd"] = M_keep * (C_in + C_out) * es + C_in * C_out * es + 4.0 * C_in * C_out + M * C_in * es + 4 * C_out
    by["dW+dX"] = by["bwd"] - 4 * C_out
    fl = {"sample": 0.0, "cache": 0.0, "db": 0.0, "dW": flop, "dX": flop, "dW+dX": 2 * flop, "bwd": 2 * flop}
    tmin = {k: max(fl[k] / tf, by[k] / bw_) * 1e6 for k in t}
    bound = {k: ("tensor" if fl[k] / tf > by[k] / bw_ else "hbm") for k in t}
    del sets
    torch.cuda.empty_cache()
    return dict(name=name, M=M, M_keep=M_keep, t=t, tmin=tmin, bound=bound, flop=flop, bytes=by)


def mlp_block(bench, B, H, W_, d, h, r):
    """Backward of a two-layer block d -> h -> d (a ViT MLP, a ConvNeXt block's point-wise pair; upper layer first)
    with the same keep set on both layers: the gradient between the layers scattered to all rows and gathered
    again, against kept packed (Eq. 9)."""
    M = B * H * W_
    cap = B * sbp.sbp_keep_count(0, H, W_, r)
    gen = torch.Generator(device="cuda").manual_seed(99)
    rn = lambda *sh: torch.randn(*sh, device="cuda", generator=gen)
    n_sets = 3
    sets = []
    for _ in range(n_sets):
        sets.append(dict(X0k=rn(cap, d).bfloat16(), X1k=rn(cap, h).bfloat16(), dY=(rn(M, d) * 0.01).bfloat16(),
                         W1=(rn(d, h) * 0.02).bfloat16(), W2=(rn(h, d) * 0.02).bfloat16(),
                         dW1=torch.zeros(d, h, device="cuda"), db1=torch.zeros(h, device="cuda"),
                         dW2=torch.zeros(h, d, device="cuda"), db2=torch.zeros(d, device="cuda"),
                         dX1=torch.zeros(M, h, device="cuda", dtype=torch.bfloat16),
                         dX0=torch.zeros(M, d, device="cuda", dtype=torch.bfloat16),
                         rows=torch.zeros(cap, dtype=torch.int32, device="cuda"),
                         offs=torch.zeros(B + 1, dtype=torch.int32, device="cuda")))
    nb = max(sbp.sbp_linear_backward_workspace_bytes(sbp.SBP_BF16, M, cap, d, h),
             sbp.sbp_linear_backward_workspace_bytes(sbp.SBP_BF16, M, cap, h, d))
    ws = torch.empty(nb, dtype=torch.uint8, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    with torch.cuda.stream(bench.stream):
        for s in sets:
            sbp.sbp_sample_keep(0, B, H, W_, r, 0, 0, 0, 0, s["rows"], s["offs"], stream=bench.sid)
    bench.stream.synchronize()

    def block(k, packed):
        s = sets[k]
        up, low = (sbp.SBP_FLAG_DX_COMPACT, sbp.SBP_FLAG_DY_COMPACT) if packed else (0, 0)
        sbp.sbp_linear_backward(sbp.SBP_BF16, s["X1k"], s["dY"], s["W2"], s["rows"], None, M, cap, h, d, s["dW2"], s["db2"],
                                s["dX1"], up, ws, nb, st, stream=bench.sid)
        sbp.sbp_linear_backward(sbp.SBP_BF16, s["X0k"], s["dX1"], s["W1"], s["rows"], None, M, cap, d, h, s["dW1"], s["db1"],
                                s["dX0"], low, ws, nb, st, stream=bench.sid)

    t_scatter = bench.time_us(lambda k, i: block(k, False), n_sets)
    t_packed = bench.time_us(lambda k, i: block(k, True), n_sets)
    assert int(st.item()) == 0
    flop = 8.0 * cap * d * h
    return cap, t_scatter, t_packed, flop


def forward_layers(bench, pk):
    """sbp_linear_forward with the cache fused in, against the forward alone followed by sbp_forward_cache."""
    rows = []
    for name, B, H, W_, C_in, C_out, r in (("vit_b16 fc1 B=64", 64, 14, 14, 768, 3072, 0.5), ("vit_b16 fc2 B=64", 64, 14, 14, 3072, 768, 0.5),
                                           ("vit_b16 fc1 B=128", 128, 14, 14, 768, 3072, 0.5), ("vit_b16 qkv B=128", 128, 14, 14, 768, 2304, 0.5),
                                           ("convnext_b s1 pw1", 64, 56, 56, 128, 512, 0.5), ("convnext_b s1 pw2", 64, 56, 56, 512, 128, 0.5),
                                           ("convnext_b s3 pw1", 64, 14, 14, 512, 2048, 0.5)):
        M = B * H * W_
        cap = B * sbp.sbp_keep_count(0, H, W_, r)
        gen = torch.Generator(device="cuda").manual_seed(7)
        set_bytes = (M * C_in + M * C_out + C_in * C_out + cap * C_in) * 2
        n_sets = max(3, int(400e6 // set_bytes) + 1)
        sets = [dict(X=torch.randn(M, C_in, device="cuda", generator=gen).bfloat16(),
                     W=(torch.randn(C_in, C_out, device="cuda", generator=gen) * 0.02).bfloat16(),
                     b=torch.randn(C_out, device="cuda", generator=gen), Y=torch.zeros(M, C_out, device="cuda", dtype=torch.bfloat16),
                     Xk=torch.zeros(cap, C_in, device="cuda", dtype=torch.bfloat16), rows=torch.zeros(cap, dtype=torch.int32, device="cuda"),
                     offs=torch.zeros(B + 1, dtype=torch.int32, device="cuda")) for _ in range(n_sets)]
        torch.cuda.synchronize()
        with torch.cuda.stream(bench.stream):
            for s in sets:
                sbp.sbp_sample_keep(0, B, H, W_, r, 0, 0, 0, 0, s["rows"], s["offs"], stream=bench.sid)
        bench.stream.synchronize()

        def fused(k, i):
            s = sets[k]
            sbp.sbp_linear_forward(sbp.SBP_BF16, s["X"], s["W"], s["b"], M, C_in, C_out, s["Y"], s["rows"], None, cap, s["Xk"],
                                   stream=bench.sid)

        def separate(k, i):
            s = sets[k]
            sbp.sbp_linear_forward(sbp.SBP_BF16, s["X"], s["W"], s["b"], M, C_in, C_out, s["Y"], stream=bench.sid)
            sbp.sbp_forward_cache(sbp.SBP_BF16, s["X"], M, C_in, s["rows"], None, cap, s["Xk"], stream=bench.sid)

        tf, ts = bench.time_us(fused, n_sets), bench.time_us(separate, n_sets)
        flop = 2.0 * M * C_in * C_out
        by = (M * C_in + C_in * C_out + M * C_out + cap * C_in) * 2.0
        tmin = max(flop / (pk["bf16_tflops_sustained"] * 1e12), by / (pk["hbm_gbs"] * 1e9)) * 1e6
        rows.append((name, M, tf, ts, tmin, flop / tf / 1e6))
        del sets
        torch.cuda.empty_cache()
    return rows


def attention_layers(bench, pk):
    """sbp_attention_backward on ViT-B/16 heads (12 heads of 64, 196 tokens, B = 128): Drop QKV at three keep ratios,
    Drop Query only, and ordinary attention backward (keep ratio 1.0) through the same kernel."""
    B, H, W_, heads, d = 128, 14, 14, 12, 64
    N, M, C = H * W_, B * H * W_, heads * d
    gen = torch.Generator(device="cuda").manual_seed(5)
    n_sets = 3
    sets = [dict(qkv=torch.randn(M, 3 * C, device="cuda", generator=gen).bfloat16(),
                 dA=(torch.randn(M, C, device="cuda", generator=gen) * 0.01).bfloat16(),
                 out=torch.zeros(M, 3 * C, device="cuda", dtype=torch.bfloat16),
                 rows=torch.zeros(M, dtype=torch.int32, device="cuda"), offs=torch.zeros(B + 1, dtype=torch.int32, device="cuda"))
            for _ in range(n_sets)]
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    out_rows = []
    for name, r, flags, lists in (("Drop QKV r=0.25", 0.25, 0, True), ("Drop QKV r=0.5", 0.5, 0, True), ("Drop QKV r=0.75", 0.75, 0, True),
                                  ("Drop QKV r=0.5, kept rows only (no zero rows written)", 0.5, sbp.SBP_FLAG_ATTN_KEPT_ROWS_ONLY, True),
                                  ("Drop Query only r=0.5", 0.5, sbp.SBP_FLAG_ATTN_ALL_KEYS, True),
                                  ("all tokens (keep ratio 1.0)", 1.0, sbp.SBP_FLAG_ATTN_ALL_KEYS, False)):
        cap = sbp.sbp_keep_count(0, H, W_, r)
        torch.cuda.synchronize()
        with torch.cuda.stream(bench.stream):
            for s_ in sets:
                sbp.sbp_sample_keep(0, B, H, W_, r, 0, 0, 0, 0, s_["rows"], s_["offs"], stream=bench.sid)
        bench.stream.synchronize()

        def call(k, i):
            s_ = sets[k]
            q, o = s_["qkv"], s_["out"]
            sbp.sbp_attention_backward(sbp.SBP_BF16, q[:, :C], q[:, C:2 * C], q[:, 2 * C:], 3 * C, s_["dA"], C,
                                       s_["rows"] if lists else None, s_["offs"] if lists else None, None, None, B, N, heads, d,
                                       cap if lists else 0, o[:, :C], o[:, C:2 * C], o[:, 2 * C:], 3 * C, flags, st, stream=bench.sid)
        us = bench.time_us(call, n_sets)
        nq = cap if lists else N
        nk = N if (flags & sbp.SBP_FLAG_ATTN_ALL_KEYS) else cap
        flop = 10.0 * nq * nk * d * B * heads
        # kept rows of Q and dA, of K and V read; kept rows of dQ, dK, dV written, zeros in all their other rows
        by = (2.0 * nq + 2.0 * nk) * B * C * 2 + (3.0 * M * C * 2 if not (flags & sbp.SBP_FLAG_ATTN_KEPT_ROWS_ONLY) else (nq + 2.0 * nk) * B * C * 2)
        tmin = max(flop / (pk["bf16_tflops_sustained"] * 1e12), by / (pk["hbm_gbs"] * 1e9)) * 1e6
        out_rows.append((name, nq, nk, us, tmin, flop / us / 1e6, by / us / 1e3))
    assert int(st.item()) == 0
    return out_rows


def sampler_stress(bench, pk):
    """Sampler alone on a shape whose index stream is large enough to read as bandwidth."""
    rows = []
    for B, H, W_, r in ((4096, 56, 56, 0.5), (4096, 14, 14, 0.5), (2, 200, 334, 0.5)):
        cap = B * sbp.sbp_keep_count(0, H, W_, r)
        bufs = [(torch.zeros(cap, dtype=torch.int32, device="cuda"), torch.zeros(B + 1, dtype=torch.int32, device="cuda"))
                for _ in range(3)]
        torch.cuda.synchronize()
        us = bench.time_us(lambda k, i: sbp.sbp_sample_keep(0, B, H, W_, r, 0, i, 0, 0, bufs[k][0], bufs[k][1],
                                                            stream=bench.sid), 3)
        rows.append((B, H, W_, cap, us, 4.0 * cap / us / 1e3, B * H * W_ / us / 1e3))
    return rows


def run_sweep(args):
    global torch, sbp
    import torch
    import paper_2210_00129_b200 as sbp
    from paper_2210_00129_b200 import build as sbp_build
    sbp_build.build()
    sbp.load_library()
    pk, kind = load_peaks()
    pk.setdefault("bf16_tflops_sustained", pk["bf16_tflops"])
    bench = GraphTimer(args.iters)
    args.group = args.sweep
    print(f"peaks ({kind}): bf16 {pk['bf16_tflops_sustained']:.0f} TFLOP/s sustained, HBM {pk['hbm_gbs']:.0f} GB/s; "
          f"{args.iters} graph-replayed launches per figure, rotating buffer sets larger than L2\n")
    if args.group not in ("sampler", "blocks", "forward", "attention"):
        if args.compact:
            print("us (t_min / t) per call; bound of the whole backward in the last column\n")
            print("| layer | M_keep | sample | cache | db | dW | dX | dW+dX (one launch) | backward (dW+db+dX) | TFLOP/s | bound |")
            print("|---|---|---|---|---|---|---|---|---|---|---|")
        else:
            print("| layer | M_keep | call | us | t_min us | t_min/t | bound | achieved |")
            print("|---|---|---|---|---|---|---|---|")
        full = {}
        res = []
        for spec in sweep_layers(args.group):
            m = measure_layer(bench, spec, pk)
            res.append((spec, m))
            if args.compact:
                cells = " | ".join(f"{m['t'][k]:.1f} ({m['tmin'][k] / m['t'][k]:.2f})" for k in ("cache", "db", "dW", "dX", "dW+dX", "bwd"))
                print(f"| {m['name']} | {m['M_keep']} | {m['t']['sample']:.1f} | {cells} | "
                      f"{2 * m['flop'] / m['t']['bwd'] / 1e6:.0f} | {m['bound']['bwd']} |")
            for k in (() if args.compact else ("sample", "cache", "db", "dW", "dX", "dW+dX", "bwd")):
                us = m["t"][k]
                if k in ("dW", "dX", "dW+dX", "bwd"):
                    ach = f"{(2 if k in ('bwd', 'dW+dX') else 1) * m['flop'] / us / 1e6:.0f} TFLOP/s"
                else:
                    ach = f"{m['bytes'][k] / us / 1e3:.0f} GB/s"
                print(f"| {m['name']} | {m['M_keep']} | {k} | {us:.1f} | {m['tmin'][k]:.1f} | {m['tmin'][k] / us:.2f} | "
                      f"{m['bound'][k]} | {ach} |")
            sys.stdout.flush()
            if spec[6] == 1.0:
                full[(spec[1], spec[2], spec[3], spec[4], spec[5], spec[7])] = m["t"]["bwd"]
        lines = []
        for spec, m in res:
            key = (spec[1], spec[2], spec[3], spec[4], spec[5], spec[7])
            if key in full and spec[6] != 1.0:
                lines.append(f"| {m['name']} | {spec[6]} | {m['t']['bwd']:.1f} | {full[key]:.1f} | {full[key] / m['t']['bwd']:.2f} | {1 / spec[6]:.2f} |")
        if lines:
            print("\n| layer | keep ratio | backward us | at keep 1.0 us | speed-up | 1/r |")
            print("|---|---|---|---|---|---|")
            print("\n".join(lines))
    if args.group in ("forward", "all"):
        print("\n| forward Y = XW + b with the cache (sbp_linear_forward) | M | fused us | forward + sbp_forward_cache us | "
              "t_min us | t_min/t | TFLOP/s |")
        print("|---|---|---|---|---|---|---|")
        for name, M, tf, ts, tmin, tfl in forward_layers(bench, pk):
            print(f"| {name} | {M} | {tf:.1f} | {ts:.1f} | {tmin:.1f} | {tmin / tf:.2f} | {tfl:.0f} |")
    if args.group in ("blocks", "all"):
        print("\n| two-layer block backward, d -> 4d -> d (both layers, dW + db + dX each) | M_keep | gradient between "
              "the layers scattered, us | packed, us | gain | packed TFLOP/s |")
        print("|---|---|---|---|---|---|")
        blocks = [("vit_b16 MLP B=64 r=0.5", 64, 14, 14, 768, 0.5), ("vit_b16 MLP B=128 r=0.25", 128, 14, 14, 768, 0.25),
                  ("vit_b16 MLP B=128 r=0.5", 128, 14, 14, 768, 0.5), ("vit_b16 MLP B=128 r=0.75", 128, 14, 14, 768, 0.75),
                  ("convnext_b s1 block", 64, 56, 56, 128, 0.5), ("convnext_b s2 block", 64, 28, 28, 256, 0.5),
                  ("convnext_b s3 block", 64, 14, 14, 512, 0.5), ("detection 200x334 block", 2, 200, 334, 128, 0.5)]
        for nm, B, H, W_, d, r in blocks:
            cap, ts, tp, flop = mlp_block(bench, B, H, W_, d, 4 * d, r)
            print(f"| {nm} | {cap} | {ts:.1f} | {tp:.1f} | {ts / tp:.2f} | {flop / tp / 1e6:.0f} |")
    if args.group in ("attention", "all"):
        print("\n| sbp_attention_backward, ViT-B/16 heads (B=128, 12 x 64, 196 tokens) | queries | keys | us | t_min us | t_min/t | TFLOP/s | GB/s |")
        print("|---|---|---|---|---|---|---|---|")
        rows = attention_layers(bench, pk)
        for name, nq, nk, us, tmin, tf, gbs in rows:
            print(f"| {name} | {nq} | {nk} | {us:.1f} | {tmin:.1f} | {tmin / us:.2f} | {tf:.0f} | {gbs:.0f} |")
        full = rows[-1][3]
        print("\nspeed-up against keep ratio 1.0: " + ", ".join(f"{name}: {full / us:.2f}x" for name, _, _, us, _, _, _ in rows[:-1]))
    if args.group in ("sampler", "all"):
        print("\n| sampler shape | kept ids | us | index stream GB/s | positions per ns |")
        print("|---|---|---|---|---|")
        for B, H, W_, cap, us, gbs, pos in sampler_stress(bench, pk):
            print(f"| B={B}, {H}x{W_} | {cap} | {us:.1f} | {gbs:.1f} | {pos:.2f} |")



def run_probes(args):
    """Tables of the two diagnostic probes of the library: what the cp.async gather path sustains, and what a
    tcgen05.mma of a given width costs."""
    import torch
    import paper_2210_00129_b200 as sbp
    from paper_2210_00129_b200 import build as sbp_build
    sbp_build.build()
    sbp.load_library()
    st = torch.zeros(1, dtype=torch.int32, device="cuda")

    def time_us(fn, reps=5):
        best = 1e30
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record(); torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1) * 1e3)
        return best

    print("| gather of random rows (every other row kept) | source | rows x bytes | blocks | copy threads | ring | us | GB/s | GB/s per SM |")
    print("|---|---|---|---|---|---|---|---|---|")
    gen = torch.Generator(device="cuda").manual_seed(3)
    # lists long enough (about 800 000 rows) for runs of 100 us and more: with five tiles per block the launch and the
    # fill of the ring are half of the time
    for source, M, rb, reps in (("DRAM (616 MB of 6 KB rows)", 100352, 6144, 16), ("DRAM / L2 (205 MB of 1 KB rows)", 200704, 1024, 8),
                                ("DRAM / L2 (51 MB of 256-byte rows)", 200704, 256, 8), ("L2 (24 MB)", 24576, 1024, 64)):
        src = torch.ones(M * rb, dtype=torch.uint8, device="cuda")
        lists = [torch.nonzero(torch.rand(M, device="cuda", generator=gen) < 0.5).flatten().to(torch.int32) for _ in range(reps)]
        rows = torch.cat(lists).contiguous()
        n = int(rows.numel())
        for blocks in (148, 74, 37):
            for threads, stages in ((64, 6), (128, 6), (256, 12)):
                us = time_us(lambda: sbp.sbp_probe_gather_ring(src, rb, rows, n, threads, stages, blocks, st))
                gbs = n * rb / us / 1e3
                print(f"| | {source} | {n} x {rb} | {blocks} | {threads} | {stages} x 16 KB | {us:.1f} | {gbs:.0f} | {gbs / blocks:.1f} |")
        del src
    print("\n| operand feed per stage (gathered rows x 128 B + TMA boxes of 16 KB; sources L2-resident unless noted) | blocks | ring | us | "
          "GB/s gathered | GB/s by TMA | GB/s per SM | clocks per stage at 1.9 GHz |")
    print("|---|---|---|---|---|---|---|---|")
    M, rb = 24576, 1024
    src = torch.ones(M * rb, dtype=torch.uint8, device="cuda")
    rows = torch.cat([torch.nonzero(torch.rand(M, device="cuda", generator=gen) < 0.5).flatten().to(torch.int32) for _ in range(4)]).contiguous()
    dense = torch.ones(6144, 2048, dtype=torch.bfloat16, device="cuda")          # 24 MB
    big_src = torch.ones(200704 * rb, dtype=torch.uint8, device="cuda")          # 205 MB: the gathered rows come from DRAM
    big_rows = torch.nonzero(torch.rand(200704, device="cuda", generator=gen) < 0.5).flatten().to(torch.int32).contiguous()
    steps = 512
    for label, g_src, g_rows in (("", src, rows), (", gathered rows from DRAM", big_src, big_rows)):
        for g, boxes in ((128, 0), (0, 1), (0, 2), (0, 3), (128, 2), (128, 1), (64, 2), (64, 3)):
            if label and g == 0:
                continue
            stage = g * 128 + boxes * 16384
            stages = min(12, (192 * 1024) // stage)
            for blocks in (148, 74):
                us = time_us(lambda: sbp.sbp_probe_operand_feed(g_src, rb, g_rows, int(g_rows.numel()), g, dense, 6144, 2048, boxes, stages, steps, blocks, st))
                gg, gt = blocks * steps * g * 128 / us / 1e3, blocks * steps * boxes * 16384 / us / 1e3
                print(f"| {g} rows + {boxes} boxes{label} | {blocks} | {stages} x {stage // 1024} KB | {us:.1f} | {gg:.0f} | {gt:.0f} | {(gg + gt) / blocks:.1f} | {us * 1e-6 / steps * 1.9e9:.0f} |")
    del src, dense, big_src

    print("\n| tcgen05.mma, M = 128, K = 16, bf16 | operands | N | accumulators | clocks per instruction | clocks per 64-deep k-block | ideal (4096 MAC/clk) | fraction |")
    print("|---|---|---|---|---|---|---|---|")
    cyc = torch.zeros(1, dtype=torch.int64, device="cuda")
    iters = 2000
    for blocks in (1, 148):
        for mn in (0, 1):
            for acc in (1, 2):
                for N in (16, 32, 64, 128, 192, 256):
                    sbp.sbp_probe_mma_rate(N, mn, acc, iters, blocks, cyc, st)
                    sbp.sbp_probe_mma_rate(N, mn, acc, iters, blocks, cyc, st)
                    torch.cuda.synchronize()
                    c = int(cyc.item())
                    per_kb = c / iters / acc                      # per accumulator chain and k-block
                    ideal = 128.0 * N * 64 / 4096.0
                    print(f"| {blocks} block(s) | {'MN-major' if mn else 'K-major'} | {N} | {acc} | {c / (iters * 4 * acc):.1f} | {per_kb:.0f} | {ideal:.0f} | {ideal / per_kb:.2f} |")
    print("\n| tcgen05.mma.cta_group::2, M = 256 over two SMs, K = 16, bf16 | operands | N | clocks per instruction | ideal per SM (4096 MAC/clk) | fraction |")
    print("|---|---|---|---|---|---|")
    for pairs in (1, 74):
        for mn in (0, 1):
            for N in (64, 128, 256):
                sbp.sbp_probe_mma_pair_rate(N, mn, iters, pairs, cyc, st)
                sbp.sbp_probe_mma_pair_rate(N, mn, iters, pairs, cyc, st)
                torch.cuda.synchronize()
                c = int(cyc.item()) / (iters * 4)
                ideal = 128.0 * N * 16 / 4096.0
                print(f"| {pairs} pair(s) | {'MN-major' if mn else 'K-major'} | {N} | {c:.1f} | {ideal:.0f} | {ideal / c:.2f} |")
    assert int(st.item()) == 0, "device status word set by a probe"


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--launch", default="graph", choices=["graph", "calls"],
                    help="timed steps: replay of captured steps (default) or direct C-ABI calls from Python")
    ap.add_argument("--allreduce", action="store_true",
                    help="also time the steps followed by the all-reduce of dW / db when started under a launcher with one rank")
    ap.add_argument("--sweep", default=None, choices=["vit", "convnext", "detection", "forward", "blocks", "attention", "sampler", "all"],
                    help="print per-call timing tables of every layer shape of a group instead of the JSON line")
    ap.add_argument("--iters", type=int, default=24, help="--sweep: launches per figure")
    ap.add_argument("--compact", action="store_true", help="--sweep: one table row per layer, us (t_min / t) per call")
    ap.add_argument("--probe", action="store_true", help="print the tables of the library's diagnostic probes (gather ring, tcgen05.mma rate)")
    args = ap.parse_args()
    if args.probe:
        run_probes(args)
        return
    if args.sweep:
        run_sweep(args)
        return
    w = WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w, args.workload)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(respawn_under_torchrun(args.gpus))
    else:
        run_cuda(args, w, args.workload)


if __name__ == "__main__":
    main()
