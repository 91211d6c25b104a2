#!/usr/bin/env python
"""Throughput of the W4A8-dINT quantized linear path on B200.

One step = one pass of the hot path over the four linears of an OPT-6.7B-shaped decoder
block at M = 2048 tokens: for each linear, the token-wise INT8 activation quantizer followed
by the tensor-core linear (weights are packed once, before timing, as the method does
offline).  Inputs are seeded synthetic tensors (see paper_2311_05161_b200/synth.py).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  `value` is TOPS (2*M*N*K per linear) with inputs resident in HBM;
`e2e` is the same metric with host buffers and the copies inside the timed region;
`roofline` describes the tensor-core kernel; `decode` gives the M = 1 weight-streaming
GB/s of the same block; `cpu_baseline` is the CPU checker timed on a bounded sample.
With --impl reference the CPU checker itself is the timed program.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

CONFIG = 2            # OPT-6.7B-shaped block
# DRAM bytes per launch of the dominant kernel from one ncu capture of this command (see
# profiles/); set to None whenever that kernel changes until the counters are taken again.
NCU_TRAFFIC_BYTES_PER_LAUNCH = 54.7e6
M_PREFILL = 2048
M_DECODE = 1
CPU_SAMPLE_TOKENS = 48


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_burst": p["bf16_tflops"],
                "bf16_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0,
            "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.perf_counter(), line.strip()))

    def wait_first(self, timeout=5.0):
        t0 = time.perf_counter()
        while self.proc is not None and not self.lines and time.perf_counter() - t0 < timeout:
            time.sleep(0.01)

    def mark(self):
        """Samples taken before this moment are dropped."""
        self.t_mark = time.perf_counter()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, line in self.lines:
            if ts < getattr(self, "t_mark", 0.0):
                continue
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm),
                "reasons": sorted(reasons)}


def cpu_sample_time(layers_host, tokens):
    """CPU checker on the first `tokens` tokens of every linear: seconds and op count."""
    import oracle
    ops = 0
    t0 = time.perf_counter()
    for lay in layers_host:
        X = lay["X"][:tokens]
        codes, scales, zeros = lay["oracle_pack"]
        Xq, tok = oracle.quantize_act(X, lay["inv_s"])
        oracle.linear(Xq, tok, codes, scales, zeros, lay["bias"], lay["group"])
        ops += 2 * X.shape[0] * lay["W"].shape[0] * lay["W"].shape[1]
    return time.perf_counter() - t0, ops


def host_layers(M, with_oracle_pack=False):
    from paper_2311_05161_b200 import synth
    wl = synth.WORKLOADS[CONFIG]
    out = []
    for i, (K, N, label) in enumerate(wl.shapes):
        lay = synth.workload_layer(CONFIG, i, M)
        lay.update(K=K, N=N, label=label, group=wl.group)
        if with_oracle_pack:
            import oracle
            lay["oracle_pack"] = oracle.pack_weights(lay["W"], lay["s"], wl.group)
        out.append(lay)
    return out


def run_reference(args):
    """The CPU checker as the timed program (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    layers = host_layers(CPU_SAMPLE_TOKENS, with_oracle_pack=True)
    for _ in range(min(args.warmup, 1)):
        cpu_sample_time(layers, CPU_SAMPLE_TOKENS)
    total_t, total_ops = 0.0, 0
    for _ in range(args.steps):
        t, ops = cpu_sample_time(layers, CPU_SAMPLE_TOKENS)
        total_t += t
        total_ops += ops
    tops = total_ops / total_t / 1e12
    sample = f"first {CPU_SAMPLE_TOKENS} of {M_PREFILL} tokens of each of the 4 linears per step"
    line = {
        "impl": "reference", "metric": "w4a8_dint_linear_tops", "value": tops, "unit": "TOPS",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * total_t / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": "opt-6.7b block linears (qkv 4096->12288, out 4096->4096, "
                               "fc1 4096->16384, fc2 16384->4096), M=2048 prefill, per-channel dINT4",
                   "step": "CPU oracle on a bounded sample of the same step", "sample": sample},
        "cpu_baseline": {"value": tops, "unit": "TOPS", "cores": oracle.get_threads(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": tops, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def max_over_ranks(ms: float, world: int, device=None) -> float:
    """Slowest rank's time: replicas run independently, the job ends when the last one does."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_throughput(ops_per_step: float, world: int, ms_per_step: float) -> float:
    """Whole-job TOPS of `world` independent replicas that each do `ops_per_step` per step."""
    return world * ops_per_step / (ms_per_step * 1e-3) / 1e12


def run_case(args):
    """One linear shape: quantize_act + linear, each timed with its own CUDA events.
    Rotates over enough copies of the weights and activations to exceed L2."""
    import torch

    import __graft_entry__ as entry
    entry.build()
    import paper_2311_05161_b200 as w4a8
    from paper_2311_05161_b200 import synth

    vals = [int(v) for v in args.case.split(",")]
    K, N, M, group = vals[:4]
    tok_tile = vals[4] if len(vals) > 4 else 0
    split_k = vals[5] if len(vals) > 5 else 0
    dw = vals[6] if len(vals) > 6 else 0
    if tok_tile < 0:            # the weight-streaming kernel on request; dw = warps of a row-slab CTA
        opts = w4a8.make_opts(w4a8.PATH_GEMV, 0, 0, dw)
    else:
        opts = w4a8.make_opts(w4a8.PATH_TCGEN05, split_k, tok_tile, dw) if (tok_tile or split_k or dw) else None
    torch.cuda.set_device(0)
    peaks = read_peaks()
    lay = synth.make_layer(K, N, M, seed=7, dist="normal", outliers=0.001, mult=60.0)
    d = {k: torch.from_numpy(lay[k]).cuda() for k in ("W", "X", "s", "inv_s", "bias")}
    packed = w4a8.pack_weights(d["W"], d["s"], group)
    del d["W"]
    per_copy = packed.numel() + M * K * 3 + M * N * 2
    copies = max(1, min(8, -(-(256 << 20) // per_copy)))
    packs = [packed] + [packed.clone() for _ in range(copies - 1)]
    Xs = [d["X"]] + [d["X"].clone() for _ in range(copies - 1)]
    Xq = [torch.empty((M, K), dtype=torch.int8, device="cuda") for _ in range(copies)]
    tok = [torch.empty((M,), dtype=torch.float32, device="cuda") for _ in range(copies)]
    Y = [torch.empty((M, N), dtype=torch.bfloat16, device="cuda") for _ in range(copies)]
    ws = w4a8.new_workspace(M, N, K, group, opts)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]

    def one(it, e=None):
        c = it % copies
        if e:
            e[0].record()
        w4a8.quantize_act(Xs[c], d["inv_s"], out=(Xq[c], tok[c]))
        if e:
            e[1].record()
        w4a8.linear(Xq[c], tok[c], packs[c], d["bias"], N, group, ws, opts, out=Y[c])
        if e:
            e[2].record()

    for it in range(max(args.warmup, 3)):
        one(it)
    torch.cuda.synchronize()
    w4a8.check_status(ws)
    for it in range(args.steps):
        one(it, ev[it])
    torch.cuda.synchronize()
    w4a8.check_status(ws)
    q_ms_ev = statistics.median(e[0].elapsed_time(e[1]) for e in ev)
    l_ms_ev = statistics.median(e[1].elapsed_time(e[2]) for e in ev)
    q_ms, l_ms = q_ms_ev, l_ms_ev
    if not args.no_graph:
        # Short kernels are launch-bound from Python: replay the same launches from a CUDA
        # graph so that the device runs them back to back, and time the replay.
        def graph_ms(fn):
            g = torch.cuda.CUDAGraph()
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                with torch.cuda.graph(g, stream=side):
                    for it in range(args.steps):
                        fn(it)
            torch.cuda.synchronize()
            g.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            g.replay()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / args.steps

        q_ms = graph_ms(lambda it: w4a8.quantize_act(Xs[it % copies], d["inv_s"],
                                                     out=(Xq[it % copies], tok[it % copies])))
        l_ms = graph_ms(lambda it: w4a8.linear(Xq[it % copies], tok[it % copies], packs[it % copies],
                                               d["bias"], N, group, ws, opts, out=Y[it % copies]))
        w4a8.check_status(ws)
    G = K // group if group else 1
    ops = 2.0 * M * N * K
    lin_bytes = N * K / 2 + 5 * N * G + M * K + 4 * M + 2 * M * N + 4 * N
    q_bytes = 3.0 * M * K + 4 * M
    line = {
        "case": {"K": K, "N": N, "M": M, "group": group, "tok_tile": tok_tile, "split_k": split_k,
                 "decode_warps": dw, "copies": copies},
        "linear_ms": l_ms, "linear_tops": ops / l_ms / 1e9, "linear_gbs": lin_bytes / l_ms / 1e6,
        "linear_frac_tensor": ops / l_ms / 1e9 / (2 * peaks["bf16_burst"]),
        "linear_frac_hbm": lin_bytes / l_ms / 1e6 / peaks["hbm_gbs"],
        "quant_ms": q_ms, "quant_gbs": q_bytes / q_ms / 1e6,
        "quant_frac_hbm": q_bytes / q_ms / 1e6 / peaks["hbm_gbs"],
        "linear_ms_events": l_ms_ev, "quant_ms_events": q_ms_ev,
        "timing": "events per launch" if args.no_graph else "CUDA graph replay of `steps` launches",
        "peaks": peaks, "steps": args.steps,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true",
                    help="--case only: time with per-launch events, no CUDA graph replay")
    ap.add_argument("--case", default=None,
                    help="K,N,M,group[,tok_tile[,split_k[,decode_warps]]]: time one linear shape instead of "
                         "(tok_tile -1: the weight-streaming kernel, decode_warps = warps per CTA) "
                         "the block (profiling and sweeps); prints its own JSON line")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.case:
        run_case(args)
        return

    import numpy as np
    import torch
    import torch.distributed as dist

    import __graft_entry__ as entry
    entry.build()
    import paper_2311_05161_b200 as w4a8

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dev = torch.device("cuda", local_rank)
    peaks = read_peaks()
    warmup = max(args.warmup, 3)

    # ------------------------------------------------------------------ set-up (untimed)
    layers = host_layers(M_PREFILL, with_oracle_pack=(rank == 0 and not args.no_cpu_baseline))
    group = layers[0]["group"]
    L = []
    for lay in layers:
        K, N = lay["K"], lay["N"]
        d = {k: torch.from_numpy(lay[k]).to(dev) for k in ("W", "X", "s", "inv_s", "bias")}
        d["packed"] = w4a8.pack_weights(d["W"], d["s"], group)
        del d["W"]
        d["Xq"] = torch.empty((M_PREFILL, K), dtype=torch.int8, device=dev)
        d["tok"] = torch.empty((M_PREFILL,), dtype=torch.float32, device=dev)
        d["Y"] = torch.empty((M_PREFILL, N), dtype=torch.bfloat16, device=dev)
        d["ws"] = w4a8.new_workspace(M_PREFILL, N, K, group)
        d["tz"] = torch.empty((M_PREFILL,), dtype=torch.int32, device=dev)
        d["rowsum"] = w4a8.weight_rowsum(d["packed"], N, K, group)[0].contiguous()
        d["K"], d["N"] = K, N
        d["X_host"] = torch.from_numpy(lay["X"]).pin_memory()
        d["Y_host"] = torch.empty((M_PREFILL, N), dtype=torch.bfloat16).pin_memory()
        # decode (M = 1): three rotating blob copies so that every launch streams from HBM
        d["packed_rot"] = [d["packed"]] + [d["packed"].clone() for _ in range(2)]
        d["X1"] = d["X"][:M_DECODE].contiguous()
        d["Xq1"] = torch.empty((M_DECODE, K), dtype=torch.int8, device=dev)
        d["tok1"] = torch.empty((M_DECODE,), dtype=torch.float32, device=dev)
        d["Y1"] = torch.empty((M_DECODE, N), dtype=torch.bfloat16, device=dev)
        d["ws1"] = w4a8.new_workspace(M_DECODE, N, K, group)
        d["wsf"] = w4a8.new_quantize_linear_workspace(M_DECODE, N, K, group)
        L.append(d)
    ops_per_step = sum(2 * M_PREFILL * d["K"] * d["N"] for d in L)

    def step(record=None):
        for i, d in enumerate(L):
            w4a8.quantize_act(d["X"], d["inv_s"], out=(d["Xq"], d["tok"]))
            if record is not None:
                record[i][0].record()
            w4a8.linear(d["Xq"], d["tok"], d["packed"], d["bias"], d["N"], group, d["ws"],
                        out=d["Y"])
            if record is not None:
                record[i][1].record()

    # End to end: inputs start in pinned host memory, results end there.  Three streams, as a
    # caller would do it: uploads, kernels and downloads of different layers overlap (the two copy
    # engines run in both directions at once); events carry the per-layer dependencies.
    s_up, s_down = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    ev_up = [torch.cuda.Event() for _ in L]
    ev_done = [torch.cuda.Event() for _ in L]
    ev_down = [torch.cuda.Event() for _ in L]

    def step_e2e():
        main = torch.cuda.current_stream()
        for i, d in enumerate(L):
            with torch.cuda.stream(s_up):
                s_up.wait_event(ev_done[i])          # the previous step's kernels have read X
                d["X"].copy_(d["X_host"], non_blocking=True)
                ev_up[i].record(s_up)
            main.wait_event(ev_up[i])
            main.wait_event(ev_down[i])              # the previous step's download has read Y
            w4a8.quantize_act(d["X"], d["inv_s"], out=(d["Xq"], d["tok"]))
            w4a8.linear(d["Xq"], d["tok"], d["packed"], d["bias"], d["N"], group, d["ws"],
                        out=d["Y"])
            ev_done[i].record(main)
            with torch.cuda.stream(s_down):
                s_down.wait_event(ev_done[i])
                d["Y_host"].copy_(d["Y"], non_blocking=True)
                ev_down[i].record(s_down)

    def step_asym(it=None):
        # the same block with the paper's asymmetric token-wise activation quantizer
        for d in L:
            w4a8.quantize_act_asym(d["X"], d["inv_s"], out=(d["Xq"], d["tok"], d["tz"]))
            w4a8.linear_asym(d["Xq"], d["tok"], d["tz"], d["packed"], d["rowsum"], d["bias"],
                             d["N"], d["ws"], out=d["Y"])

    def step_decode(it):
        for d in L:
            w4a8.quantize_act(d["X1"], d["inv_s"], out=(d["Xq1"], d["tok1"]))
            w4a8.linear(d["Xq1"], d["tok1"], d["packed_rot"][it % 3], d["bias"], d["N"], group,
                        d["ws1"], out=d["Y1"])

    def step_decode_fused(it):
        # the same decode step with the quantizer inside the weight-streaming kernel: one launch per linear
        for d in L:
            w4a8.quantize_linear(d["X1"], d["inv_s"], d["packed_rot"][it % 3], d["bias"], d["N"], group,
                                 d["wsf"], out=d["Y1"])

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        for it in range(steps):
            fn(it)
        e1.record()
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), world, dev)

    # ------------------------------------------------------------------ prefill, resident
    for _ in range(warmup):
        step()
    for d in L:
        w4a8.check_status(d["ws"])
    records = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                for _ in L] for _ in range(args.steps)]
    sampler = ClockSampler(local_rank)
    sampler.start()
    sampler.wait_first()
    for _ in range(warmup):
        step()
    sampler.mark()
    ms = timed(lambda it: step(records[it]), args.steps)
    clocks = sampler.stop()
    lin_ms = [statistics.mean(records[it][i][0].elapsed_time(records[it][i][1])
                              for it in range(args.steps)) for i in range(len(L))]
    ms_per_step = ms / args.steps
    tops = replica_throughput(ops_per_step, world, ms_per_step)
    lin_tops = ops_per_step / (sum(lin_ms) * 1e-3) / 1e12
    peak_tops = 2.0 * peaks["bf16_sustained"]        # INT8 dense = 2 x BF16 dense (nominal ratio)

    # ------------------------------------------------------------------ prefill, host buffers
    for _ in range(3):
        step_e2e()
    e2e_steps = max(3, min(args.steps, 10))
    def e2e_run(it):
        step_e2e()
        if it == e2e_steps - 1:                      # the timed region ends when the last result is on the host
            torch.cuda.current_stream().wait_stream(s_down)
            torch.cuda.current_stream().wait_stream(s_up)
    ms_e2e = timed(e2e_run, e2e_steps) / e2e_steps
    h2d = sum(d["X_host"].numel() * 2 for d in L)
    d2h = sum(d["Y_host"].numel() * 2 for d in L)

    # ------------------------------------------------------------------ asymmetric activations
    for _ in range(3):
        step_asym()
    asym_steps = max(3, min(args.steps, 50))
    ms_asym = timed(step_asym, asym_steps) / asym_steps

    # ------------------------------------------------------------------ special value step / 4
    fmt_opts = w4a8.make_opts(level_shift=2)
    for d, lay in zip(L, layers):
        W = torch.from_numpy(lay["W"]).to(dev)
        d["packed_fmt"] = w4a8.pack_weights(W, d["s"], group, level_shift=2)
        del W

    def step_fmt(it=None):
        for d in L:
            w4a8.quantize_act(d["X"], d["inv_s"], out=(d["Xq"], d["tok"]))
            w4a8.linear(d["Xq"], d["tok"], d["packed_fmt"], d["bias"], d["N"], group, d["ws"],
                        fmt_opts, out=d["Y"])

    for _ in range(3):
        step_fmt()
    ms_fmt = timed(step_fmt, asym_steps) / asym_steps
    for d in L:
        w4a8.check_status(d["ws"])
        del d["packed_fmt"]

    # ------------------------------------------------------------------ decode (M = 1)
    # The eight launches of a decode step take a few microseconds each: from Python they would
    # be launch-bound, so the steps are captured once into a CUDA graph and the replay is timed.
    dec_steps = 60

    def graph_ms(step_fn):
        for it in range(6):
            step_fn(it)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                for it in range(dec_steps):
                    step_fn(it)
        torch.cuda.synchronize()
        graph.replay()
        return timed(lambda it: graph.replay(), 3) / (3 * dec_steps)

    ms_dec = graph_ms(step_decode)
    ms_dec_fused = graph_ms(step_decode_fused)
    dec_bytes = sum(d["K"] * d["N"] // 2 + 5 * d["N"] + M_DECODE * (d["K"] + 4) + 2 * M_DECODE * d["N"]
                    + 4 * d["N"] for d in L)
    dec_gbs = dec_bytes / (ms_dec * 1e-3) / 1e9
    for d in L:
        w4a8.check_status(d["ws"])
        w4a8.check_status(d["ws1"])
        w4a8.check_status(d["wsf"])

    # ------------------------------------------------------------------ decode, one large layer
    # OPT-66B-shaped fc1 (9216 -> 36864, 170 MB of codes) at M = 1: the weight stream without the
    # fixed cost that dominates the 8-34 MB layers of the block above.  Two blob copies (> L2).
    from paper_2311_05161_b200 import synth
    for d in L:
        for k in ("packed_rot", "packed", "X", "Xq", "Y", "X_host", "Y_host"):
            d.pop(k, None)
    torch.cuda.empty_cache()
    big = synth.workload_layer(4, 0, M_DECODE)
    bK, bN = big["W"].shape[1], big["W"].shape[0]
    bd = {k: torch.from_numpy(big[k]).to(dev) for k in ("W", "X", "s", "inv_s", "bias")}
    bpacked = [w4a8.pack_weights(bd["W"], bd["s"], 0)]
    del bd["W"]
    bpacked.append(bpacked[0].clone())
    bws = w4a8.new_workspace(M_DECODE, bN, bK, 0)
    bY = torch.empty((M_DECODE, bN), dtype=torch.bfloat16, device=dev)
    bXq = torch.empty((M_DECODE, bK), dtype=torch.int8, device=dev)
    btok = torch.empty((M_DECODE,), dtype=torch.float32, device=dev)

    def step_big(it):
        # two calls: on a matrix this large every CTA of the one-launch form would repeat the
        # quantizer for several waves of CTAs (measured 38 us against 35 us)
        w4a8.quantize_act(bd["X"], bd["inv_s"], out=(bXq, btok))
        w4a8.linear(bXq, btok, bpacked[it % 2], bd["bias"], bN, 0, bws, out=bY)

    dec_steps = 40
    ms_big = graph_ms(step_big)
    w4a8.check_status(bws)
    big_bytes = bK * bN // 2 + 5 * bN + M_DECODE * (bK + 4) + 2 * M_DECODE * bN + 4 * bN   # as for the block above
    big_gbs = big_bytes / (ms_big * 1e-3) / 1e9
    del bpacked, big

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    cpu = None
    if not args.no_cpu_baseline:
        import oracle
        t, ops = cpu_sample_time(layers, CPU_SAMPLE_TOKENS)
        cpu = {"value": ops / t / 1e12, "unit": "TOPS", "cores": oracle.get_threads(),
               "kind": "oracle", "seconds": t,
               "sample": f"first {CPU_SAMPLE_TOKENS} of {M_PREFILL} tokens of each of the 4 linears"}

    line = {
        "metric": "w4a8_dint_linear_tops", "value": tops, "unit": "TOPS", "n_gpus": world,
        "steps": args.steps, "warmup": warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8",
        "data": "synthetic",
        "config": {"workload": "opt-6.7b block linears (qkv 4096->12288, out 4096->4096, "
                               "fc1 4096->16384, fc2 16384->4096), M=2048 prefill, per-channel dINT4",
                   "step": "4 x (quantize_act + linear); weights packed once before timing",
                   "l2": "inputs larger than L2 (about 400 MB touched per step)",
                   "parallelism": "replicas" if world > 1 else "single"},
        "clocks": clocks,
        "e2e": {"value": replica_throughput(ops_per_step, world, ms_e2e), "unit": "TOPS",
                "ms_per_step": ms_e2e, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": 2 * len(L) * args.steps,
        "roofline": {"bound": "tensor", "kernel": "linear_tcgen05_kernel<256,false>",
                     "achieved": lin_tops, "peak": peak_tops, "unit": "TOPS",
                     "frac": lin_tops / peak_tops,
                     "peak_source": f"2 x {peaks['source']} sustained bf16 cuBLAS TFLOP/s",
                     "frac_of_nominal_4500": lin_tops / 4500.0,
                     "per_linear_ms": dict(zip([lay["label"] for lay in layers], lin_ms)),
                     "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH,
                     "traffic_source": "ncu dram__bytes_read.sum + dram__bytes_write.sum, mean over the "
                                       "four launches of a step (profiles/bench_opt6.7b_block_launch_list.md)",
                     "algorithmic_bytes_per_launch": sum(
                         lay["N"] * lay["K"] // 2 + 5 * lay["N"] + M_PREFILL * lay["K"] + 4 * M_PREFILL
                         + 2 * M_PREFILL * lay["N"] + 4 * lay["N"] for lay in layers) / len(layers)},
        "decode": {"metric": "w4a8_dint_linear_hbm_gbs", "value": dec_gbs, "unit": "GB/s", "M": M_DECODE,
                   "ms_per_step": ms_dec, "bytes_per_step": dec_bytes,
                   "frac_of_measured_copy": dec_gbs / peaks["hbm_gbs"],
                   "frac_of_nominal_8000": dec_gbs / 8000.0,
                   "note": "quantize_act + linear per shape, 3 rotating blob copies (> L2), CUDA graph replay",
                   "one_launch": {"value": dec_bytes / (ms_dec_fused * 1e-3) / 1e9, "unit": "GB/s",
                                  "ms_per_step": ms_dec_fused,
                                  "frac_of_measured_copy": dec_bytes / (ms_dec_fused * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                  "note": "the same step through quantize_linear: the quantizer runs inside "
                                          "the weight-streaming kernel, one launch per linear"},
                   "large_layer": {"workload": "opt-66b fc1 9216->36864, M=1, per-channel dINT4 (quantize_act + linear)",
                                   "value": big_gbs, "unit": "GB/s", "ms_per_step": ms_big,
                                   "bytes_per_step": big_bytes,
                                   "frac_of_measured_copy": big_gbs / peaks["hbm_gbs"],
                                   "frac_of_nominal_8000": big_gbs / 8000.0,
                                   "note": "2 rotating blob copies (> L2), CUDA graph replay"}},
        "asym": {"metric": "w4a8_dint_linear_tops", "value": replica_throughput(ops_per_step, world, ms_asym),
                 "unit": "TOPS", "ms_per_step": ms_asym,
                 "note": "same block and step with asymmetric token-wise activations "
                         "(quantize_act_asym + linear_asym)"},
        "special_value_quarter_step": {"metric": "w4a8_dint_linear_tops",
                                       "value": replica_throughput(ops_per_step, world, ms_fmt),
                                       "unit": "TOPS", "ms_per_step": ms_fmt,
                                       "note": "same block and step with weights packed for the special "
                                               "value step/4 (pack_weights_fmt, level_shift 2)"},
        "cpu_baseline": cpu,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
