#!/usr/bin/env python
"""Benchmark of one SPA block (forward + backward) on synthetic data.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config I] [--impl ours|reference]

A step is one pass of the whole block over one batch: gate, select/pack, QKV, segment-masked
attention, output projection, unpack, then the backward pass, issued by the library's two block calls.
The metric is selected tokens per second (N_p of the batch / step time), whole job over all GPUs.  At
N > 1 every rank runs the same independent replica on its own GPU (images are independent; the block has
no exchange step); with --gpus N and no launcher environment the script starts the N ranks itself.

The headline workload is the largest one (ViT-B/16 at 384^2); the same run also times the whole step of
the other four workloads and reports them under `per_config`.

Timing: CUDA events on the launching stream, max over ranks, several buffer sets rotated so the
working set exceeds L2.  One JSON line is printed by rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "selected_tokens_per_sec_spa_block_fwd_bwd"
UNIT = "tokens/s"
L2_BYTES = 126e6
HEADLINE_CONFIG = 4
UNIT_REPLAYS = 200          # replays of every per-unit graph (median and minimum are reported)


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            m = json.load(f)
        return dict(hbm=float(m["hbm_gbs"]), tensor=float(m["bf16_tflops"]), source="measured")
    return dict(hbm=6650.0, tensor=1590.0, source="fallback")


def measured_traffic(workload, unit):
    """DRAM bytes per launch of `unit` from the committed ncu summary, or None when there is no figure
    or the kernel's source has changed since the counters were taken."""
    import hashlib
    path = os.path.join(ROOT, "profiles", f"traffic_{workload}.txt")
    if not os.path.exists(path):
        return None
    for line in open(path):
        parts = line.split()
        if len(parts) == 4 and parts[0] == unit:
            src = os.path.join(ROOT, "paper_2410_23608_b200", "csrc", parts[2])
            if os.path.exists(src) and hashlib.sha256(open(src, "rb").read()).hexdigest()[:16] == parts[3]:
                return int(parts[1])
    return None


# ----------------------------------------------------------------------------- work model
def work_model(cfg, cu):
    """Algorithmic bytes, FLOPs (2 x MACs) and exponentials of every call for the realised selection."""
    n = np.diff(np.asarray(cu, np.int64))
    Np, S2 = int(n.sum()), int((n * n).sum())
    B, N, C, H, es = cfg.B, cfg.N, cfg.C, cfg.H, cfg.elem_size
    BN = B * N
    w = {}
    w["gate"] = dict(bytes=BN * C * es + 5 * BN, flops=2 * BN * C)
    w["select_pack"] = dict(bytes=BN + 2 * Np * C * es + 4 * Np + 4 * BN, flops=0)
    # gate, selection and packing in one pass over x: x read once, the selected rows written once
    w["gate_pack"] = dict(bytes=BN * C * es + Np * C * es + 9 * BN + 4 * Np, flops=2 * BN * C)
    w["qkv"] = dict(bytes=(Np * C + 3 * C * C + 3 * Np * C) * es, flops=2 * Np * C * 3 * C)
    # one exponential per (query, key) pair and head, forward and backward alike
    w["attn_fwd"] = dict(bytes=4 * Np * C * es + 4 * H * Np, flops=4 * C * S2, exps=H * S2)
    w["proj"] = dict(bytes=(2 * Np * C + C * C) * es, flops=2 * Np * C * C)
    w["unpack"] = dict(bytes=2 * BN * C * es + 4 * BN, flops=0)
    w["unpack_bwd"] = dict(bytes=2 * BN * C * es + 4 * BN, flops=0)
    w["attn_bwd"] = dict(bytes=(3 + 1 + 1 + 3) * Np * C * es + 4 * H * Np, flops=10 * C * S2, exps=H * S2)
    for name, n_out in (("proj_bwd", C), ("qkv_bwd", 3 * C)):
        w[name + ".da"] = dict(bytes=(Np * n_out + n_out * C + Np * C) * es, flops=2 * Np * C * n_out)
        w[name + ".dW"] = dict(bytes=(Np * n_out + Np * C) * es + 4 * n_out * C + 4 * n_out,
                               flops=2 * Np * C * n_out + Np * n_out)   # dW and db
    w["pack_bwd"] = dict(bytes=2 * Np * C * es + 4 * Np, flops=0)
    # fused unpack: the gate also writes y = x; the projection writes to the tokens (idx read per row)
    w["gate_prefill"] = dict(bytes=2 * BN * C * es + 5 * BN, flops=2 * BN * C)
    w["gate_pack_prefill"] = dict(bytes=2 * BN * C * es + Np * C * es + 9 * BN + 4 * Np, flops=2 * BN * C)
    w["proj_scatter"] = dict(bytes=(2 * Np * C + C * C) * es + 4 * Np, flops=2 * Np * C * C)
    return w, Np, S2


def timing_units(L, blk, d, b_g):
    """The block's calls as (name, thunk) pairs with the linear-layer gradients split the way the step issues them:
    the input gradient, and the weight gradient together with the bias gradient (column sums taken from the tiles
    that stream through the weight-gradient product; split-K product plus its fixed-order reduction)."""
    p, C = blk.p, blk.C
    fused = blk.fused
    units = []
    if blk.one_pass:
        units.append(("gate_pack", lambda: L.spa_gate_select_pack(p, d["x"], d["w_g"], b_g, None, blk.scores, blk.mask,
                                                                  blk.y if fused else None, blk.xp, blk.idx, blk.inv,
                                                                  blk.cu, blk.pack_state, blk.status)))
    else:
        if fused:
            units.append(("gate", lambda: L.spa_gate_prefill(p, d["x"], d["w_g"], b_g, None, blk.scores, blk.mask, blk.y)))
        else:
            units.append(("gate", lambda: L.spa_gate(p, d["x"], d["w_g"], b_g, None, blk.scores, blk.mask)))
        units.append(("select_pack", lambda: L.spa_select_pack(p, d["x"], blk.mask, blk.scores, blk.xp, blk.idx, blk.inv,
                                                               blk.cu, blk.status)))
    units += [
        ("qkv", lambda: L.spa_packed_qkv(p, blk.xp, d["W_qkv"], d["b_qkv"], blk.cu, blk.qkv, blk.status)),
        ("attn_fwd", lambda: L.spa_packed_attention_fwd(p, blk.qkv, blk.cu, blk.B, blk.ao, blk.lse, blk.status)),
    ]
    if fused:
        units.append(("proj_scatter", lambda: L.spa_packed_proj_scatter(p, blk.ao, d["W_o"], d["b_o"], blk.idx, blk.cu,
                                                                        blk.y, blk.status)))
    else:
        units += [("proj", lambda: L.spa_packed_proj(p, blk.ao, d["W_o"], d["b_o"], blk.cu, blk.z, blk.status)),
                  ("unpack", lambda: L.spa_unpack_scatter(p, blk.z, d["x"], blk.idx, blk.inv, blk.cu, blk.y, blk.status))]
    units.append(("unpack_bwd", lambda: L.spa_unpack_scatter_bwd(p, d["dY"], blk.idx, blk.inv, blk.cu, blk.dz, blk.dX)))
    units.append(("attn_bwd", lambda: L.spa_packed_attention_bwd(p, blk.qkv, blk.ao, blk.lse, blk.dao, blk.cu, blk.B,
                                                                 blk.dqkv, blk.workspace, blk.status)))

    def lin(a, W, dout, n_out, da, dW, db):
        return lambda: L.spa_packed_linear_bwd(p, a, W, dout, C, n_out, blk.cu, da, dW, db, blk.workspace, blk.status)

    units += [
        ("proj_bwd.da", lin(blk.ao, d["W_o"], blk.dz, C, blk.dao, None, None)),
        ("proj_bwd.dW", lin(blk.ao, d["W_o"], blk.dz, C, None, blk.dW_o, blk.db_o)),
        ("qkv_bwd.da", (lambda: L.spa_packed_linear_bwd_scatter(p, blk.xp, d["W_qkv"], blk.dqkv, C, 3 * C, blk.idx, blk.cu,
                                                                 blk.dX, None, None, None, blk.status))
         if fused else lin(blk.xp, d["W_qkv"], blk.dqkv, 3 * C, blk.dxp, None, None)),
        ("qkv_bwd.dW", lin(blk.xp, d["W_qkv"], blk.dqkv, 3 * C, None, blk.dW_qkv, blk.db_qkv)),
    ]
    if not fused:
        units.append(("pack_bwd", lambda: L.spa_select_pack_bwd(p, blk.dxp, d["dY"], blk.idx, blk.cu, blk.dX)))
    return units


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in out.strip().splitlines():
            parts = [s.strip() for s in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


# ----------------------------------------------------------------------------- oracle timing
def oracle_step(O, inp, cfg):
    fwd = O.block_fwd(inp.x, inp.w_g, inp.b_g, inp.tau, inp.W_qkv, inp.b_qkv, inp.W_o, inp.b_o, cfg.H)
    O.block_bwd(fwd, inp.dY, inp.x, inp.W_qkv, inp.W_o, cfg.H)
    return int(fwd["cu_seqlens"][-1])


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def time_oracle(inp, cfg, budget_s, max_reps=200, min_reps=1):
    from oracle import spa_oracle as O
    Np = oracle_step(O, inp, cfg)  # untimed first pass (page-in)
    times = []
    t_end = time.perf_counter() + budget_s
    while len(times) < min_reps or (time.perf_counter() < t_end and len(times) < max_reps):
        t0 = time.perf_counter()
        oracle_step(O, inp, cfg)
        times.append(time.perf_counter() - t0)
    return Np, times


def cpu_baseline(cfg, inp, make_inputs, scaled_config):
    """The oracle as it stands on the host cores: every core the BLAS uses on the whole batch, and one thread on a
    slice of the batch (a bounded sample: about 10 s of CPU work each)."""
    Np_o, times = time_oracle(inp, cfg, budget_s=10.0)
    out = {"value": Np_o / float(np.mean(times)), "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
           "sample": f"whole {cfg.name} batch, forward+backward, {len(times)} repetitions "
                     f"({sum(times):.1f} s of CPU work)"}
    try:
        from threadpoolctl import threadpool_limits
        Bs = max(2, min(cfg.B, 4))
        small = scaled_config(cfg, B=Bs)
        inp_s = make_inputs(small)
        with threadpool_limits(limits=1):
            Np_s, t_s = time_oracle(inp_s, small, budget_s=8.0, max_reps=20)
        out["single_thread"] = {"value": Np_s / float(np.mean(t_s)), "unit": UNIT, "cores": 1,
                                "sample": f"first {Bs} images of {cfg.name}, forward+backward, {len(t_s)} repetitions "
                                          f"({sum(t_s):.1f} s of CPU work)"}
    except Exception as e:  # threadpoolctl missing: report the threaded figure alone
        out["single_thread"] = {"unavailable": str(e)}
    return out


def run_reference(args):
    """The reference arm: the fp64 oracle, as it stands, on the host cores.  Each step is a bounded sample of the
    workload (the first images of the batch) so that the whole run ends within minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from spa_workloads import get_config, make_inputs, scaled_config
    from oracle import spa_oracle as O
    full = get_config(args.config)
    Bs = min(full.B, 8)
    cfg = scaled_config(full, B=Bs)
    inp = make_inputs(cfg)
    Np = 0
    for _ in range(args.warmup):
        Np = oracle_step(O, inp, cfg)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        Np = oracle_step(O, inp, cfg)
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    val = Np / dt
    cores = blas_threads()
    sample = f"first {Bs} of {full.B} images of {full.name}, forward+backward, {args.steps} timed repetitions"
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": full.name, "B": full.B, "N": full.N, "C": full.C, "H": full.H,
                   "sample": sample, "selected_tokens_in_sample": Np},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------- one workload on this GPU
class Workload:
    """Rotating buffer sets of one workload, its whole-step graphs and its per-unit timings."""

    def __init__(self, torch, L, cfg, no_fuse=False, sets=0, one_pass=False, overlap=True, flags=0):
        from paper_2410_23608_b200.block import SpaBlock
        from spa_workloads import make_inputs, scaled_config
        self.torch, self.L, self.cfg, self.overlap = torch, L, cfg, overlap
        x_bytes = cfg.B * cfg.N * cfg.C * cfg.elem_size
        # enough sets that even the smallest single tensor a call streams (x) exceeds L2 over one rotation
        self.n_sets = sets if sets > 0 else min(24, max(3, int(np.ceil(1.3 * L2_BYTES / x_bytes))))
        self.x_bytes = x_bytes
        names = ("x", "w_g", "W_qkv", "b_qkv", "W_o", "b_o", "dY")
        self.inps, self.sets = [], []
        for s in range(self.n_sets):
            inp = make_inputs(scaled_config(cfg, seed=cfg.seed + 1000 * s)) if s < 2 else self.inps[s % 2]
            self.inps.append(inp)
            d = {n: inp.torch(n, "cuda") for n in names}
            blk = SpaBlock(cfg.B, cfg.N, cfg.C, cfg.H, cfg.dtype, tau=cfg.tau, flags=flags, fused=False if no_fuse else None, one_pass=one_pass)
            self.sets.append((inp, d, blk))
        self.stream = torch.cuda.current_stream()
        for s in range(self.n_sets):     # eager pass: first-use set-up (attributes, tensor maps) outside capture
            self.step_fn(s, True)()
        torch.cuda.synchronize()
        self.step_graphs, self.launches_per_step = [], 0
        for s in range(self.n_sets):
            g, n = self.capture([self.step_fn(s, True)])
            self.step_graphs.append(g)
            self.launches_per_step = n

    def step_fn(self, s, backward, container_len=0):
        inp, d, blk = self.sets[s]
        overlap = self.overlap

        def run():
            blk.forward(d["x"], d["w_g"], inp.b_g, d["W_qkv"], d["b_qkv"], d["W_o"], d["b_o"], container_len=container_len)
            if backward:
                blk.backward(d["dY"], overlap=overlap)
        return run

    def capture(self, fns):
        """One CUDA graph holding the given library calls in order; returns (graph, kernels launched)."""
        torch, L = self.torch, self.L
        g = torch.cuda.CUDAGraph()
        n_before = L.spa_launch_count()
        with torch.cuda.graph(g):
            for fn in fns:
                fn()
        return g, L.spa_launch_count() - n_before

    def step(self, i):
        self.step_graphs[i % self.n_sets].replay()

    def warm(self, n):
        for i in range(n):
            self.step(i)
        self.torch.cuda.synchronize()
        self.Np_sets = [int(b.cu[-1].item()) for _, _, b in self.sets]
        statuses = [b.read_status() for _, _, b in self.sets]
        assert all(st == 0 for st in statuses), f"device status after warm-up: {statuses}"

    def tokens_per_step(self, steps):
        return float(np.mean([self.Np_sets[i % self.n_sets] for i in range(steps)]))

    def time_steps(self, steps):
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(self.stream)
        for i in range(steps):
            self.step(i)
        e1.record(self.stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    def time_graph(self, g, calls_per_replay, replays):
        """Per-call device time over `replays` replays of g, each bracketed by its own events: (median, min) in ms."""
        torch = self.torch
        for _ in range(3):
            g.replay()
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(replays + 1)]
        ev[0].record(self.stream)
        for r in range(replays):
            g.replay()
            ev[r + 1].record(self.stream)
        torch.cuda.synchronize()
        t = [ev[r].elapsed_time(ev[r + 1]) / calls_per_replay for r in range(replays)]
        return statistics.median(t), min(t)

    def containers_ms(self, container_len, replays):
        """Whole step (forward + backward) with the paper's own batching: attention limited to containers of
        `container_len` tokens, their cuts built on the device inside the step.  Median per step in ms."""
        fns = [self.step_fn(s, True, container_len=container_len) for s in range(self.n_sets)]
        for f in fns:
            f()
        self.torch.cuda.synchronize()
        g, _ = self.capture(fns)
        return self.time_graph(g, self.n_sets, max(20, replays // 4))[0]

    def forward_only_ms(self, replays):
        fns = [self.step_fn(s, False) for s in range(self.n_sets)]
        g, _ = self.capture(fns)
        return self.time_graph(g, self.n_sets, max(20, replays // 4))[0]

    def per_call(self, pk, exp_rate, replays=UNIT_REPLAYS):
        """Every unit alone (one graph holding the unit once per buffer set), against the roofline that bounds it:
        the slowest of FLOPs / tensor peak, bytes / HBM peak and, for attention, exponentials / measured rate."""
        L, cfg = self.L, self.cfg
        per_set = [dict(timing_units(L, blk, d, inp.b_g)) for inp, d, blk in self.sets]
        work, Np0, S2 = work_model(cfg, self.sets[0][2].cu.cpu().numpy())
        if self.sets[0][2].fused:
            work["gate"] = work["gate_prefill"]
            work["gate_pack"] = work["gate_pack_prefill"]
        out = {}
        for name in per_set[0]:
            g, n_l = self.capture([u[name] for u in per_set])
            med, mn = self.time_graph(g, self.n_sets, replays)
            wk = work[name]
            t = {"hbm": wk["bytes"] / (pk["hbm"] * 1e9)}
            if cfg.dtype == "bf16":
                t["tensor"] = wk["flops"] / (pk["tensor"] * 1e12)
                if wk.get("exps") and exp_rate:
                    t["alu"] = wk["exps"] / exp_rate
            bound = max(t, key=t.get)
            if bound == "tensor":
                ach, peak, unit = wk["flops"] / (med * 1e-3) / 1e12, pk["tensor"], "TFLOP/s"
            elif bound == "alu":
                ach, peak, unit = wk["exps"] / (med * 1e-3) / 1e9, exp_rate / 1e9, "Gexp/s"
            else:
                ach, peak, unit = wk["bytes"] / (med * 1e-3) / 1e9, pk["hbm"], "GB/s"
            out[name] = dict(us=round(med * 1e3, 2), us_min=round(mn * 1e3, 2), bound=bound, achieved=round(ach, 2),
                             peak=round(peak, 1), unit=unit, frac=round(ach / peak, 4), roofline_us=round(t[bound] * 1e6, 2),
                             kernels=n_l // self.n_sets)
        return out, work, Np0, S2


def roofline_of(cfg, per_call, work, pk):
    top = max(per_call, key=lambda k: per_call[k]["us"])
    tr = per_call[top]
    r = {"kernel": top, "bound": tr["bound"], "achieved": tr["achieved"], "peak": tr["peak"], "unit": tr["unit"],
         "frac": tr["frac"], "traffic": measured_traffic(cfg.name, top), "algorithmic_bytes": work[top]["bytes"],
         "algorithmic_flops": work[top]["flops"], "peak_source": pk["source"], "us_per_launch": tr["us"],
         "us_per_launch_min": tr["us_min"], "replays": UNIT_REPLAYS}
    if tr["bound"] == "alu":
        r["alu_kind"] = "base-2 exponentials (ex2.approx), peak measured in this run by spa_probe_exp2"
        r["algorithmic_exps"] = work[top]["exps"]
    return r


def measure_exp_rate(torch, L):
    """Exponentials per second of the whole GPU with every SM busy (the softmax instruction, 8 independent chains
    per thread), best of three launches."""
    sink = torch.zeros(4096, dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n_sm = torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count
    best = 0.0
    for _ in range(4):
        e0.record(stream)
        n = L.spa_probe_exp2(n_sm * 4, 2048, sink)
        e1.record(stream)
        torch.cuda.synchronize()
        best = max(best, n / (e0.elapsed_time(e1) * 1e-3))
    return best


def spawn_ranks(args):
    """--gpus N without a launcher: start the N ranks (one process per GPU) and pass rank 0's line through."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


# ----------------------------------------------------------------------------- main arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--config", type=int, default=HEADLINE_CONFIG,
                    help="headline workload 1..5 (default 4, ViT-B/16 at 384^2, the largest)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sets", type=int, default=0, help="rotating buffer sets (0 = enough to exceed L2)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="time the headline workload only")
    ap.add_argument("--no-fuse", action="store_true", help="separate projection / scatter kernels instead of the fused calls")
    ap.add_argument("--one-pass-pack", action="store_true", help="gate, selection and packing as one kernel (spa_gate_select_pack) instead of two")
    ap.add_argument("--one-pass-bwd", action="store_true", help="attention backward: one-pass kernel for segments of at most 128 rows (SPA_FLAG_ONE_PASS_BWD)")
    ap.add_argument("--no-overlap", action="store_true", help="weight gradients on the main stream too (no second stream)")
    ap.add_argument("--train", action="store_true", help="also time the trainable-selection calls (loss, gated pack backward, gate backward)")
    ap.add_argument("--layer", action="store_true", help="also time the whole pre-norm block (LayerNorm, SPA, feed-forward) and its new calls")
    args = ap.parse_args()
    if args.impl == "reference":
        if args.steps == 1000 and args.warmup == 50:
            args.steps, args.warmup = 3, 1
        return run_reference(args)
    if args.gpus > 1 and "RANK" not in os.environ:
        sys.exit(spawn_ranks(args))

    import torch
    from paper_2410_23608_b200 import build as spa_build
    from paper_2410_23608_b200 import binding as L
    from spa_workloads import get_config, make_inputs, scaled_config

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the SPA library has no CPU path")
    from paper_2410_23608_b200 import replicas
    rank, local, world = replicas.world()
    torch.cuda.set_device(local)
    replicas.init("nccl", torch.device("cuda", local))
    if rank == 0:
        spa_build.build()
    replicas.barrier()
    L.lib()
    args.warmup = max(args.warmup, 3)

    cfg = get_config(args.config)
    wl = Workload(torch, L, cfg, no_fuse=args.no_fuse, sets=args.sets, one_pass=args.one_pass_pack, overlap=not args.no_overlap, flags=64 if args.one_pass_bwd else 0)
    stream = wl.stream
    n_sets = wl.n_sets
    wl.warm(args.warmup)
    tokens_per_step = wl.tokens_per_step(args.steps)

    def barrier():
        replicas.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing of exactly K steps
    sampler = ClockSampler(local) if rank == 0 else None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for i in range(args.steps):
        wl.step(i)
    e1.record(stream)
    barrier()
    launches = wl.launches_per_step * args.steps
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop() if sampler else None
    # whole job = every rank's tokens over the slowest rank's time
    value, ms_total = replicas.whole_job_rate(tokens_per_step * args.steps, ms, "cuda")
    ms_per_step = ms_total / args.steps

    # ---- end to end: pinned host inputs in, results out, every step.  A three-stage pipeline over the rotating
    # buffer sets: the inputs of a step are copied in on one stream while the previous step computes on the main
    # stream and the step before that is copied out on a third (PCIe carries both directions at once); every
    # step still pays for all four copies, and the timed region ends when the last result has reached the host.
    hx = [inp.torch("x").pin_memory() for inp in wl.inps[:2]]
    hdy = [inp.torch("dY").pin_memory() for inp in wl.inps[:2]]
    hy = [torch.empty_like(hx[0]).pin_memory() for _ in range(2)]
    hdx = [torch.empty_like(hx[0]).pin_memory() for _ in range(2)]
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(n_sets)]
    ev_done = [torch.cuda.Event() for _ in range(n_sets)]
    ev_out = [torch.cuda.Event() for _ in range(n_sets)]

    def e2e_step(i):
        k = i % n_sets
        inp, d, blk = wl.sets[k]
        with torch.cuda.stream(s_in):
            s_in.wait_event(ev_out[k])               # the set's previous results have left the device (no-op at first use)
            d["x"].copy_(hx[k % 2], non_blocking=True)
            d["dY"].copy_(hdy[k % 2], non_blocking=True)
            ev_in[k].record(s_in)
        stream.wait_event(ev_in[k])
        wl.step(i)
        ev_done[k].record(stream)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_done[k])
            hy[i % 2].copy_(blk.y, non_blocking=True)
            hdx[i % 2].copy_(blk.dX, non_blocking=True)
            ev_out[k].record(s_out)

    e2e_steps = min(args.steps, 300)
    for i in range(min(3, n_sets)):
        e2e_step(i)
    torch.cuda.synchronize()
    barrier()
    e0.record(stream)
    for i in range(e2e_steps):
        e2e_step(i)
    stream.wait_stream(s_out)
    e1.record(stream)
    barrier()
    e2e_value, e2e_total = replicas.whole_job_rate(wl.tokens_per_step(e2e_steps) * e2e_steps, e0.elapsed_time(e1), "cuda")
    e2e_ms = e2e_total / e2e_steps
    bytes_io = cfg.B * cfg.N * cfg.C * cfg.elem_size

    if rank != 0:
        replicas.shutdown()
        return

    # ---- per-kernel device times and the roofline of the dominant one
    pk = peaks()
    exp_rate = measure_exp_rate(torch, L)
    per_call, work, Np0, S2 = wl.per_call(pk, exp_rate)
    roofline = roofline_of(cfg, per_call, work, pk)
    fwd_ms = wl.forward_only_ms(UNIT_REPLAYS)
    cont_ms = wl.containers_ms(49, UNIT_REPLAYS) if (args.config in (3, 4) and cfg.dtype == "bf16") else None
    reps = 50

    train = None
    if args.train:
        # trainable selection (Eq. 4-5, Eq. 10): timed like the other units, reported beside them
        BN = cfg.B * cfg.N
        extra = []
        for inp_, d_, blk_ in wl.sets:
            t = dict(ds=torch.zeros(BN, dtype=torch.float32, device="cuda"), ds_up=torch.empty(BN, dtype=torch.float32, device="cuda"),
                     dw=torch.empty(cfg.C, dtype=torch.float32, device="cuda"), db=torch.empty(1, dtype=torch.float32, device="cuda"),
                     loss=torch.empty(1, dtype=torch.float32, device="cuda"),
                     lab=(torch.rand(BN, device="cuda") < 0.4).to(torch.uint8),
                     ws=torch.empty(max(L.spa_train_workspace_bytes(blk_.p), 256), dtype=torch.uint8, device="cuda"))
            extra.append(t)

        def train_units(k):
            inp_, d_, blk_ = wl.sets[k]; t = extra[k]; p_ = blk_.p
            return {
                "select_loss": lambda: L.spa_select_loss(p_, blk_.scores, t["lab"], 0.5, t["ds"], t["loss"], t["ws"]),
                "pack_bwd_gated": lambda: L.spa_select_pack_bwd_gated(p_, blk_.dxp, d_["x"], blk_.scores, d_["dY"], blk_.idx,
                                                                      blk_.cu, blk_.dX, t["ds"]),
                "gate_bwd": lambda: L.spa_gate_bwd(p_, d_["x"], d_["w_g"], blk_.scores, None, t["ds"], blk_.dX, t["dw"],
                                                   t["db"], t["ds_up"], t["ws"]),
            }
        tu = [train_units(k) for k in range(n_sets)]
        es_ = cfg.elem_size
        tw = {"select_loss": 9 * BN, "pack_bwd_gated": 3 * Np0 * cfg.C * es_ + 12 * Np0, "gate_bwd": 3 * BN * cfg.C * es_ + 12 * BN}
        train = {}
        for name in ("select_loss", "pack_bwd_gated", "gate_bwd"):
            for u in tu:
                u[name]()
            g, n_l = wl.capture([u[name] for u in tu])
            ms_c, _ = wl.time_graph(g, n_sets, reps)
            ach = tw[name] / (ms_c * 1e-3) / 1e9
            train[name] = dict(us=round(ms_c * 1e3, 2), bound="hbm", achieved=round(ach, 2), frac=round(ach / pk["hbm"], 4),
                               kernels=n_l // n_sets)
    layer = None
    if args.layer:
        # the pre-norm block around SPA: whole forward + backward as one graph per buffer set, and its new calls alone
        from paper_2410_23608_b200.layer import SpaLayer
        n_l = min(n_sets, 6)
        Hd = 4 * cfg.C
        lays = []
        for k in range(n_l):
            inp_, d_, blk_ = wl.sets[k]
            rp = lambda *sh: (torch.randn(*sh, device="cuda") * 0.05).to(blk_.tdtype)
            prm = dict(g1=(1 + rp(cfg.C)), be1=rp(cfg.C), g2=(1 + rp(cfg.C)), be2=rp(cfg.C), W1=rp(Hd, cfg.C), b1=rp(Hd),
                       W2=rp(cfg.C, Hd), b2=rp(cfg.C), w_g=d_["w_g"], b_g=0.0, W_qkv=d_["W_qkv"], b_qkv=d_["b_qkv"],
                       W_o=d_["W_o"], b_o=d_["b_o"])
            lays.append((SpaLayer(cfg.B, cfg.N, cfg.C, cfg.H, cfg.dtype), prm, d_))

        def timed(fns):
            for f_ in fns:
                f_()
            torch.cuda.synchronize()
            g_, n_k = wl.capture(fns)
            return wl.time_graph(g_, len(fns), reps)[0], n_k // len(fns)

        def whole(k):
            lay, prm, d_ = lays[k]

            def run():
                lay.forward(d_["x"], prm)
                lay.backward(d_["dY"])
            return run
        ms_l, k_l = timed([whole(k) for k in range(n_l)])
        BNr, es_ = cfg.B * cfg.N, cfg.elem_size
        units = {
            "layer_norm": (lambda lay, prm, d_: (lambda: L.spa_layer_norm(lay.p, d_["x"], prm["g1"], prm["be1"], 1e-5, lay.z, lay.m1, lay.r1)),
                           2 * BNr * cfg.C * es_, 0),
            "layer_norm_bwd": (lambda lay, prm, d_: (lambda: L.spa_layer_norm_bwd(lay.p, lay.dt, lay.y1, prm["g2"], lay.m2, lay.r2, d_["dY"], lay.dy1,
                                                                                    lay.dg2, lay.dbe2, lay.workspace)), 4 * BNr * cfg.C * es_, 0),
            "gelu": (lambda lay, prm, d_: (lambda: L.spa_gelu(lay.p, lay.u, Hd, lay.h)), 2 * BNr * Hd * es_, 0),
            "gelu_bwd": (lambda lay, prm, d_: (lambda: L.spa_gelu_bwd(lay.p, lay.dh, lay.u, Hd, lay.dh)), 3 * BNr * Hd * es_, 0),
            "ffn1": (lambda lay, prm, d_: (lambda: L.spa_packed_linear(lay.p, lay.t, prm["W1"], prm["b1"], cfg.C, Hd, lay.cu_all, lay.u, False,
                                                                        lay.blk.status)), (BNr * cfg.C + Hd * cfg.C + BNr * Hd) * es_, 2 * BNr * cfg.C * Hd),
            "ffn2": (lambda lay, prm, d_: (lambda: L.spa_packed_linear(lay.p, lay.h, prm["W2"], prm["b2"], Hd, cfg.C, lay.cu_all, lay.out, True,
                                                                        lay.blk.status)), (BNr * Hd + Hd * cfg.C + 2 * BNr * cfg.C) * es_, 2 * BNr * cfg.C * Hd),
        }
        layer = {"ms_per_step": ms_l, "kernels_per_step": k_l, "tokens_per_s": cfg.B * cfg.N / (ms_l * 1e-3), "per_call": {}}
        for name, (mk, nbytes, nflops) in units.items():
            ms_c, n_k = timed([mk(*lays[k]) for k in range(n_l)])
            t_b, t_f = nbytes / (pk["hbm"] * 1e9), nflops / (pk["tensor"] * 1e12)
            bound = "tensor" if (t_f > t_b and cfg.dtype == "bf16") else "hbm"
            ach = nflops / (ms_c * 1e-3) / 1e12 if bound == "tensor" else nbytes / (ms_c * 1e-3) / 1e9
            layer["per_call"][name] = dict(us=round(ms_c * 1e3, 2), bound=bound, achieved=round(ach, 2), frac=round(ach / pk[bound], 4),
                                           kernels=n_k)

    cpu = None
    if not args.no_cpu_baseline:
        cpu = cpu_baseline(cfg, wl.inps[0], make_inputs, scaled_config)

    flop_units = ("gate_pack" if wl.sets[0][2].one_pass else "gate", "qkv", "attn_fwd", "proj", "attn_bwd", "proj_bwd.da", "proj_bwd.dW",
                  "qkv_bwd.da", "qkv_bwd.dW")
    useful_flops = sum(work[k]["flops"] for k in flop_units)
    Np_head = wl.Np_sets[0]
    fused_head = wl.sets[0][2].fused

    # ---- the other workloads: whole step, forward only and the dominant unit, same protocol, fewer steps
    per_config = {}
    summary = dict(ms_per_step=ms_per_step, tokens_per_s=value / world, forward_only_ms=fwd_ms,
                   forward_only_tokens_per_s=Np_head / (fwd_ms * 1e-3), selected_tokens=Np_head,
                   kernels_per_step=wl.launches_per_step, dominant_unit=roofline["kernel"],
                   dominant_bound=roofline["bound"], dominant_us=roofline["us_per_launch"], dominant_frac=roofline["frac"],
                   traffic=roofline["traffic"], useful_tflops=useful_flops / (ms_per_step * 1e-3) / 1e12)
    if cont_ms is not None:   # the paper's containers of L = 7 x 7 tokens (cost linear in N, Eq. 9)
        summary["containers_L49_ms_per_step"] = cont_ms
    per_config[cfg.name] = summary
    if not args.no_per_config:
        del wl
        torch.cuda.empty_cache()
        for ci in range(1, 6):
            if ci == args.config:
                continue
            c2 = get_config(ci)
            w2 = Workload(torch, L, c2, no_fuse=args.no_fuse, one_pass=args.one_pass_pack, overlap=not args.no_overlap, flags=64 if args.one_pass_bwd else 0)
            w2.warm(20)
            steps2 = 200
            ms2 = w2.time_steps(steps2) / steps2
            pc2, work2, Np2, _ = w2.per_call(pk, exp_rate)
            r2 = roofline_of(c2, pc2, work2, pk)
            f2 = w2.forward_only_ms(UNIT_REPLAYS)
            uf2 = sum(work2[k]["flops"] for k in flop_units)
            c2_ms = w2.containers_ms(49, UNIT_REPLAYS) if ci in (3, 4) else None
            per_config[c2.name] = dict(
                ms_per_step=ms2, tokens_per_s=w2.tokens_per_step(steps2) / (ms2 * 1e-3), forward_only_ms=f2,
                forward_only_tokens_per_s=w2.Np_sets[0] / (f2 * 1e-3), selected_tokens=w2.Np_sets[0],
                kernels_per_step=w2.launches_per_step, dominant_unit=r2["kernel"], dominant_bound=r2["bound"],
                dominant_us=r2["us_per_launch"], dominant_frac=r2["frac"], traffic=r2["traffic"],
                useful_tflops=uf2 / (ms2 * 1e-3) / 1e12, steps=steps2,
                per_call={k: dict(us=v["us"], bound=v["bound"], frac=v["frac"]) for k, v in pc2.items()})
            if c2_ms is not None:
                per_config[c2.name]["containers_L49_ms_per_step"] = c2_ms
            del w2
            torch.cuda.empty_cache()

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if cfg.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": cfg.name, "B": cfg.B, "N": cfg.N, "C": cfg.C, "H": cfg.H,
                   "selected_tokens": Np_head, "sum_nb_squared": S2, "pass": "forward+backward",
                   "l2_policy": f"{n_sets} rotating buffer sets (x alone {cfg.B * cfg.N * cfg.C * cfg.elem_size * n_sets / 1e6:.0f} MB > L2)",
                   "launch": "one CUDA graph per step (spa_block_fwd + spa_block_bwd)",
                   "unpack": "scatter fused into the projection / input-gradient epilogues" if fused_head
                             else "separate scatter kernels",
                   "replicas": world},
        "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": e2e_ms, "steps": e2e_steps,
                "h2d_bytes_per_step": 2 * bytes_io, "d2h_bytes_per_step": 2 * bytes_io},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": roofline,
        "cpu_baseline": cpu,
        "forward_only": {"ms_per_step": fwd_ms, "value": Np_head / (fwd_ms * 1e-3), "unit": UNIT},
        "useful_tflops": useful_flops / (ms_per_step * 1e-3) / 1e12,
        "exp2_rate_gexp_per_s": round(exp_rate / 1e9, 1),
        "per_call": per_call,
        "per_config": per_config,
    }
    if train is not None:
        line["trainable_selection"] = train
    if layer is not None:
        line["pre_norm_block"] = layer
    print(json.dumps(line))
    replicas.shutdown()


if __name__ == "__main__":
    main()
