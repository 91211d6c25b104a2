#!/usr/bin/env python
"""Throughput of the W4A8-dINT quantized linear path on B200.

One pass of the hot path = the four linears of an OPT-66B-shaped decoder block (hidden 9216,
FFN 36864) at M = 2048 tokens: for each linear, the token-wise INT8 activation quantizer
followed by the tensor-core linear.  Weights are packed once, before timing, as the method
does offline.  Inputs are seeded synthetic tensors (paper_2311_05161_b200/synth.py).  A timed
"step" is a fixed number of back-to-back passes, chosen so that `--steps` steps keep the GPU
busy for about a second: the clock samples then describe the region the number comes from.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  `value` is TOPS (2*M*N*K per linear) with inputs resident in HBM; `e2e`
is the same metric with pinned host buffers and the copies inside the timed region; `roofline`
describes the tensor-core kernel of the headline; the other keys are legs on the other
workloads (OPT-6.7B block, group-128 LLaMA-7B block and token sweep, M = 16 and M = 1 decode
shapes, asymmetric activations, special value step/4); `cpu_baseline` is the CPU checker timed
on a bounded sample.  With --impl reference the CPU checker itself is the timed program.
With --gpus N > 1 outside a torchrun launch the script starts the N replica processes itself.
"""
from __future__ import annotations

import argparse
import importlib.util
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

HEADLINE_CONFIG = 4
HEADLINE_SHAPES = (2, 3, 0, 1)      # qkv, out, fc1, fc2 of the OPT-66B-shaped block
HEADLINE_NAME = ("opt-66b block linears (qkv 9216->27648, out 9216->9216, fc1 9216->36864, "
                 "fc2 36864->9216), M=2048 prefill, per-channel dINT4")
M_PREFILL = 2048
MIN_REGION_S = 1.2                  # length of the headline's timed region
SUSTAINED_FROM_S = 1.0              # regions at least this long are compared with the sustained peak
# DRAM bytes per launch of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum, mean
# over the four linears of the headline block, from the ncu launch list of this program); None
# while the kernel has changed since the counters were taken.
NCU_TRAFFIC_BYTES_PER_LAUNCH = 292.0e6
CPU_SAMPLE_TOKENS = 48
CPU_SAMPLE_ROWS = 4096
NOMINAL_INT8_TOPS = 4500.0
NOMINAL_HBM_GBS = 8000.0


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


def load_synth():
    """The input generators, by file: importing the package would load the CUDA library,
    which the CPU-only arm must not need."""
    spec = importlib.util.spec_from_file_location(
        "w4a8_synth", os.path.join(ROOT, "paper_2311_05161_b200", "synth.py"))
    mod = importlib.util.module_from_spec(spec)
    sys.modules["w4a8_synth"] = mod
    spec.loader.exec_module(mod)
    return mod


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap,power.draw")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []
        self.t_mark = 0.0
        self.t_end = float("inf")

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

    def mark_end(self):
        """Samples taken after this moment are dropped."""
        self.t_end = time.perf_counter()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, watts, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, line in self.lines:
            if ts < self.t_mark or ts > self.t_end:
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
            if len(parts) > 6:
                try:
                    watts.append(float(parts[6]))
                except ValueError:
                    pass
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_min_mhz": min(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm),
                "power_w_max": max(watts) if watts else None,
                "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------- host inputs
def host_layers(synth, config, shape_indices, M):
    wl = synth.WORKLOADS[config]
    out = []
    for i in shape_indices:
        K, N, label = wl.shapes[i]
        lay = synth.workload_layer(config, i, M)
        lay.update(K=K, N=N, label=label, group=wl.group)
        out.append(lay)
    return out


def cpu_sample(layers):
    """What the CPU checker is timed on: the first tokens and output rows of every linear,
    weights of those rows packed beforehand (quantization is per output row)."""
    import oracle
    sample = []
    for lay in layers:
        rows = min(CPU_SAMPLE_ROWS, lay["N"])
        toks = min(CPU_SAMPLE_TOKENS, lay["X"].shape[0])
        pack = oracle.pack_weights(lay["W"][:rows], lay["s"], lay["group"])
        sample.append({"X": lay["X"][:toks], "inv_s": lay["inv_s"], "pack": pack,
                       "bias": lay["bias"][:rows], "group": lay["group"],
                       "ops": 2 * toks * rows * lay["K"]})
    return sample


def cpu_sample_text(n):
    return (f"first {CPU_SAMPLE_TOKENS} of {M_PREFILL} tokens x first {CPU_SAMPLE_ROWS} output rows "
            f"of each of the {n} linears (activation quantizer + linear)")


def cpu_sample_time(sample):
    import oracle
    t0 = time.perf_counter()
    ops = 0
    for s in sample:
        codes, scales, zeros = s["pack"]
        Xq, tok = oracle.quantize_act(s["X"], s["inv_s"])
        oracle.linear(Xq, tok, codes, scales, zeros, s["bias"], s["group"])
        ops += s["ops"]
    return time.perf_counter() - t0, ops


def run_reference(args):
    """The CPU checker as the timed program (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    oracle.build()
    synth = load_synth()
    # only what the sample needs is drawn: the first rows of each weight matrix (the values the
    # full matrix has there) and the first tokens; the Eq. 1 scale comes from those
    wl = synth.WORKLOADS[HEADLINE_CONFIG]
    layers = []
    for i in HEADLINE_SHAPES:
        K, N, label = wl.shapes[i]
        W = synth.make_weights(N, K, wl.seed(i), n_rows=CPU_SAMPLE_ROWS)
        X = synth.make_activations(CPU_SAMPLE_TOKENS, K, wl.seed(i), wl.act_dist, wl.outlier_channels,
                                   wl.outlier_mult)
        s, inv = synth.make_channel_scales(X, W)
        layers.append({"W": W, "X": X, "s": s, "inv_s": inv, "bias": synth.make_bias(N, wl.seed(i)),
                       "K": K, "N": W.shape[0], "label": label, "group": wl.group})
    sample = cpu_sample(layers)
    for _ in range(min(args.warmup, 1)):
        cpu_sample_time(sample)
    total_t, total_ops = 0.0, 0
    for _ in range(args.steps):
        t, ops = cpu_sample_time(sample)
        total_t += t
        total_ops += ops
    tops = total_ops / total_t / 1e12
    text = cpu_sample_text(len(layers)) + " per step"
    line = {
        "impl": "reference", "metric": "w4a8_dint_linear_tops", "value": tops, "unit": "TOPS",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * total_t / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": HEADLINE_NAME,
                   "step": "CPU oracle on a bounded sample of the same pass", "sample": text},
        "cpu_baseline": {"value": tops, "unit": "TOPS", "cores": oracle.get_threads(),
                         "kind": "oracle", "sample": text},
        "e2e": {"value": tops, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- multi-GPU plumbing
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


def launch_mode(gpus: int, env) -> str:
    """How `--gpus` relates to the process environment: "single" (one process, one GPU),
    "rank" (this process is one of `gpus` ranks started by a launcher), "spawn" (no launcher
    started us although several GPUs were asked for: start the ranks ourselves).  A launcher
    whose world size differs from --gpus is an error."""
    if gpus < 1:
        raise SystemExit("--gpus must be at least 1")
    ws = env.get("WORLD_SIZE")
    if ws is None:
        return "single" if gpus == 1 else "spawn"
    if int(ws) != gpus:
        raise SystemExit(f"--gpus {gpus} does not match WORLD_SIZE={ws}: launch one rank per GPU, "
                         f"or run `python bench.py --gpus {gpus}` without a launcher")
    return "single" if gpus == 1 else "rank"


def spawn_command(gpus: int, argv, port: int):
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
            f"--nproc-per-node={gpus}", "--master-addr", "127.0.0.1", "--master-port", str(port),
            os.path.join(ROOT, "bench.py"), *argv]


# ----------------------------------------------------------------------------- single shapes
def run_case(args):
    """One linear shape: quantize_act + linear, each timed with its own CUDA events.
    Rotates over enough copies of the weights and activations to exceed L2."""
    import torch

    import __graft_entry__ as entry
    entry.build()
    import paper_2311_05161_b200 as w4a8
    from paper_2311_05161_b200 import synth

    vals = [int(v) for v in args.case.split(",")] + [0] * 7
    K, N, M, group, tok_tile, split_k, dw, cluster, offset_tables, tok_run, bits = vals[:11]
    plan_given = bool(tok_tile or split_k or dw or cluster or offset_tables or tok_run)
    if tok_tile < 0:            # the weight-streaming kernel on request; dw = warps of a row-slab CTA
        opts = w4a8.make_opts(w4a8.PATH_GEMV, 0, 0, dw)
    elif plan_given or bits:
        opts = w4a8.make_opts(w4a8.PATH_TCGEN05 if plan_given else w4a8.PATH_AUTO, split_k, tok_tile, dw,
                              cluster=cluster, offset_tables=offset_tables, tok_run=tok_run, bits=bits)
    else:
        opts = None
    torch.cuda.set_device(0)
    peaks = read_peaks()
    lay = synth.make_layer(K, N, M, seed=7, dist="normal", outliers=0.001, mult=60.0)
    d = {k: torch.from_numpy(lay[k]).cuda() for k in ("W", "X", "s", "inv_s", "bias")}
    packed = w4a8.pack_weights(d["W"], d["s"], group, bits=bits) if bits else w4a8.pack_weights(d["W"], d["s"], group)
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
                 "decode_warps": dw, "copies": copies, "plan": w4a8.linear_plan(M, N, K, group, opts)},
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


def linear_bytes(K, N, M, group):
    """Algorithmic bytes of one linear call: codes, steps and zero-points, INT8 tokens and their
    steps, BF16 output, FP32 bias."""
    G = K // group if group else 1
    return N * K // 2 + 5 * N * G + M * K + 4 * M + 2 * M * N + 4 * N


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-legs", action="store_true",
                    help="only the headline workload (resident and host-buffer timings)")
    ap.add_argument("--plan", default=None,
                    help="tok_tile,split_k,decode_warps,cluster[,offset_tables[,tok_run]] for the tensor-core kernel of the headline "
                         "instead of the library's own choice (sweeps)")
    ap.add_argument("--no-graph", action="store_true",
                    help="--case only: time with per-launch events, no CUDA graph replay")
    ap.add_argument("--case", default=None,
                    help="K,N,M,group[,tok_tile[,split_k[,decode_warps[,cluster[,offset_tables[,tok_run[,bits]]]]]]]: time one linear shape instead of "
                         "(tok_tile -1: the weight-streaming kernel, decode_warps = warps per CTA) "
                         "the block (profiling and sweeps); prints its own JSON line")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.case:
        run_case(args)
        return
    mode = launch_mode(args.gpus, os.environ)
    if mode == "spawn":
        port = 29000 + os.getpid() % 2000
        raise SystemExit(subprocess.call(spawn_command(args.gpus, sys.argv[1:], port)))

    import torch
    import torch.distributed as dist

    import __graft_entry__ as entry
    entry.build()
    import paper_2311_05161_b200 as w4a8
    from paper_2311_05161_b200 import synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dev = torch.device("cuda", local_rank)
    peaks = read_peaks()
    warmup = max(args.warmup, 3)
    legs_on = world == 1 and not args.no_legs

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        """Milliseconds of `steps` calls of fn(it): device events, barrier and synchronize on
        both sides, the slowest rank's time."""
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        for it in range(steps):
            fn(it)
        e1.record()
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), world, dev)

    plan_opts = None
    if args.plan:
        pv = [int(v) for v in args.plan.split(",")] + [0, 0]
        pt, ps, pd, pc, po, pr = pv[:6]
        plan_opts = w4a8.make_opts(w4a8.PATH_TCGEN05, ps, pt, pd, cluster=pc, offset_tables=po, tok_run=pr)

    def device_block(layers, M, rot=1, host_buffers=False, asym=False, opts=None):
        """Device tensors of a list of layers: packed weights (rot rotating copies), inputs,
        outputs, workspaces."""
        L = []
        for lay in layers:
            K, N, group = lay["K"], lay["N"], lay["group"]
            d = {k: torch.from_numpy(lay[k]).to(dev) for k in ("W", "X", "s", "inv_s", "bias")}
            d["packed"] = w4a8.pack_weights(d["W"], d["s"], group)
            del d["W"]
            d["packed_rot"] = [d["packed"]] + [d["packed"].clone() for _ in range(rot - 1)]
            d["Xq"] = torch.empty((M, K), dtype=torch.int8, device=dev)
            d["tok"] = torch.empty((M,), dtype=torch.float32, device=dev)
            d["Y"] = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
            d["ws"] = w4a8.new_workspace(M, N, K, group, opts)
            d.update(K=K, N=N, M=M, group=group, label=lay["label"], opts=opts)
            if host_buffers:
                d["X_host"] = torch.from_numpy(lay["X"]).pin_memory()
                d["Y_host"] = torch.empty((M, N), dtype=torch.bfloat16).pin_memory()
            if asym:
                d["tz"] = torch.empty((M,), dtype=torch.int32, device=dev)
                d["rowsum"] = w4a8.weight_rowsum(d["packed"], N, K, group)[0].contiguous()
            L.append(d)
        return L

    def block_pass(L, record=None, it=0):
        for i, d in enumerate(L):
            w4a8.quantize_act(d["X"], d["inv_s"], out=(d["Xq"], d["tok"]))
            if record is not None:
                record[i][0].record()
            w4a8.linear(d["Xq"], d["tok"], d["packed_rot"][it % len(d["packed_rot"])], d["bias"],
                        d["N"], d["group"], d["ws"], d["opts"], out=d["Y"])
            if record is not None:
                record[i][1].record()

    def passes_for(L, steps, seconds):
        """Passes per step so that `steps` steps last about `seconds`."""
        ms = timed(lambda it: block_pass(L), 3) / 3
        return max(1, int(-(-seconds * 1e3 // (steps * ms))))

    def time_block(L, steps, seconds, sampler=None):
        """(ms per pass, per-linear ms, passes per step, region seconds): `steps` steps of
        back-to-back passes with an event pair around every linear launch."""
        for _ in range(warmup):
            block_pass(L)
        for d in L:
            w4a8.check_status(d["ws"])
        passes = passes_for(L, steps, seconds)
        total = steps * passes
        records = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                    for _ in L] for _ in range(total)]
        if sampler is not None:
            sampler.mark()
        ms = timed(lambda it: [block_pass(L, records[it * passes + j]) for j in range(passes)], steps)
        if sampler is not None:
            sampler.mark_end()
        for d in L:
            w4a8.check_status(d["ws"])
        lin_ms = [statistics.mean(records[p][i][0].elapsed_time(records[p][i][1])
                                  for p in range(total)) for i in range(len(L))]
        return ms / total, lin_ms, passes, ms * 1e-3

    def graph_ms(step_fn, steps_in_graph, replays=3):
        """Milliseconds per step of a CUDA graph holding `steps_in_graph` steps (short launches
        would be launch-bound from Python)."""
        for it in range(4):
            step_fn(it)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                for it in range(steps_in_graph):
                    step_fn(it)
        torch.cuda.synchronize()
        graph.replay()
        return timed(lambda it: graph.replay(), replays) / (replays * steps_in_graph)

    def tensor_fracs(tops, region_s):
        burst, sus = 2.0 * peaks["bf16_burst"], 2.0 * peaks["bf16_sustained"]
        long_region = region_s >= SUSTAINED_FROM_S
        return {"frac": tops / (sus if long_region else burst),
                "peak": sus if long_region else burst,
                "peak_source": (f"2 x {peaks['source']} bf16 cuBLAS TFLOP/s (nominal INT8:BF16 ratio), "
                                + ("sustained: the timed region lasts %.2f s" % region_s if long_region
                                   else "burst: the timed region lasts %.3f s" % region_s)),
                "frac_burst": tops / burst, "frac_sustained": tops / sus,
                "frac_of_nominal_4500": tops / NOMINAL_INT8_TOPS}

    # ------------------------------------------------------------------ headline: set-up (untimed)
    layers = host_layers(synth, HEADLINE_CONFIG, HEADLINE_SHAPES, M_PREFILL)
    L = device_block(layers, M_PREFILL, host_buffers=True, opts=plan_opts)
    ops_per_pass = sum(2 * M_PREFILL * d["K"] * d["N"] for d in L)

    # ------------------------------------------------------------------ headline: resident inputs
    sampler = ClockSampler(local_rank)
    sampler.start()
    sampler.wait_first()
    ms_pass, lin_ms, passes, region_s = time_block(L, args.steps, MIN_REGION_S, sampler)
    clocks = sampler.stop()
    ms_per_step = ms_pass * passes
    tops = replica_throughput(ops_per_pass, world, ms_pass)
    lin_tops = ops_per_pass / (sum(lin_ms) * 1e-3) / 1e12

    # ------------------------------------------------------------------ headline: host buffers
    # Inputs start in pinned host memory, results end there.  Three streams, as a caller would do
    # it: uploads, kernels and downloads of different layers overlap (the two copy engines run in
    # both directions at once); events carry the per-layer dependencies.
    s_up, s_down = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    ev_up = [torch.cuda.Event() for _ in L]
    ev_done = [torch.cuda.Event() for _ in L]
    ev_down = [torch.cuda.Event() for _ in L]

    def pass_e2e():
        main_stream = torch.cuda.current_stream()
        for i, d in enumerate(L):
            with torch.cuda.stream(s_up):
                s_up.wait_event(ev_done[i])          # the previous pass's kernels have read X
                d["X"].copy_(d["X_host"], non_blocking=True)
                ev_up[i].record(s_up)
            main_stream.wait_event(ev_up[i])
            main_stream.wait_event(ev_down[i])       # the previous pass's download has read Y
            w4a8.quantize_act(d["X"], d["inv_s"], out=(d["Xq"], d["tok"]))
            w4a8.linear(d["Xq"], d["tok"], d["packed"], d["bias"], d["N"], d["group"], d["ws"],
                        d["opts"], out=d["Y"])
            ev_done[i].record(main_stream)
            with torch.cuda.stream(s_down):
                s_down.wait_event(ev_done[i])
                d["Y_host"].copy_(d["Y"], non_blocking=True)
                ev_down[i].record(s_down)

    for _ in range(3):
        pass_e2e()
    e2e_steps = max(3, min(args.steps, 10))

    def e2e_run(it):
        pass_e2e()
        if it == e2e_steps - 1:                      # the region ends when the last result is on the host
            torch.cuda.current_stream().wait_stream(s_down)
            torch.cuda.current_stream().wait_stream(s_up)
    ms_e2e = timed(e2e_run, e2e_steps) / e2e_steps
    h2d = sum(d["X_host"].numel() * 2 for d in L)
    d2h = sum(d["Y_host"].numel() * 2 for d in L)
    for d in L:
        w4a8.check_status(d["ws"])
        for k in ("X_host", "Y_host"):
            d.pop(k)

    legs = {}
    if legs_on:
        fc1 = L[2]          # 9216 -> 36864, kept for the decode legs below
        # -------------------------------------------------------------- M = 16 decode, large layers
        def decode_point(d, M, rot, steps_in_graph=20):
            """quantize_act + linear on the first M tokens, rotating blob copies, graph replay."""
            K, N, group = d["K"], d["N"], d["group"]
            X = d["X"][:M].contiguous()
            Xq = torch.empty((M, K), dtype=torch.int8, device=dev)
            tok = torch.empty((M,), dtype=torch.float32, device=dev)
            Y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
            ws = w4a8.new_workspace(M, N, K, group)
            while len(d["packed_rot"]) < rot:
                d["packed_rot"].append(d["packed"].clone())

            def fn(it):
                w4a8.quantize_act(X, d["inv_s"], out=(Xq, tok))
                w4a8.linear(Xq, tok, d["packed_rot"][it % rot], d["bias"], N, group, ws, out=Y)
            ms = graph_ms(fn, steps_in_graph)
            w4a8.check_status(ws)
            nbytes = linear_bytes(K, N, M, group)
            gbs = nbytes / (ms * 1e-3) / 1e9
            tops_pt = 2.0 * M * N * K / (ms * 1e-3) / 1e12
            return {"shape": f"{K}->{N}", "M": M, "group": group, "ms": ms, "gbs": gbs, "tops": tops_pt,
                    "frac_of_measured_copy": gbs / peaks["hbm_gbs"],
                    "frac_of_nominal_8000": gbs / NOMINAL_HBM_GBS,
                    "frac_of_burst_tensor": tops_pt / (2.0 * peaks["bf16_burst"]),
                    "plan": w4a8.linear_plan(M, N, K, group)}

        m16 = [decode_point(fc1, 16, 2)]
        big1 = decode_point(fc1, 1, 2, steps_in_graph=40)
        for d in L:
            d.clear()
        L.clear()
        torch.cuda.empty_cache()
        down65 = device_block(host_layers(synth, 4, (5,), 16), 16, rot=3)       # 22016 -> 8192
        m16.append(decode_point(down65[0], 16, 3))
        del down65
        torch.cuda.empty_cache()
        legs["decode_m16"] = {"metric": "w4a8_dint_linear_hbm_gbs", "unit": "GB/s", "points": m16,
                              "note": "quantize_act + linear per step at M = 16, per-channel dINT4, "
                                      "rotating blob copies (> L2), CUDA graph replay"}

        # -------------------------------------------------------------- OPT-6.7B block, M = 2048 and M = 1
        layers2 = host_layers(synth, 2, (0, 1, 2, 3), M_PREFILL)
        L2 = device_block(layers2, M_PREFILL, rot=3, asym=True)
        ops2 = sum(2 * M_PREFILL * d["K"] * d["N"] for d in L2)
        ms2, lin2, passes2, region2 = time_block(L2, 10, 0.3)
        lin2_tops = ops2 / (sum(lin2) * 1e-3) / 1e12
        legs["opt6.7b_block"] = {
            "workload": "opt-6.7b block linears (qkv 4096->12288, out 4096->4096, fc1 4096->16384, "
                        "fc2 16384->4096), M=2048 prefill, per-channel dINT4",
            "metric": "w4a8_dint_linear_tops", "value": ops2 / (ms2 * 1e-3) / 1e12, "unit": "TOPS",
            "ms_per_pass": ms2, "region_s": region2, "linear_only_tops": lin2_tops,
            **{k: v for k, v in tensor_fracs(lin2_tops, region2).items() if k.startswith("frac")},
            "per_linear_ms": dict(zip([d["label"] for d in L2], lin2))}

        def pass_asym(it=None):
            for d in L2:
                w4a8.quantize_act_asym(d["X"], d["inv_s"], out=(d["Xq"], d["tok"], d["tz"]))
                w4a8.linear_asym(d["Xq"], d["tok"], d["tz"], d["packed"], d["rowsum"], d["bias"],
                                 d["N"], d["ws"], out=d["Y"])
        for _ in range(3):
            pass_asym()
        ms_asym = timed(pass_asym, 100) / 100
        legs["asym"] = {"metric": "w4a8_dint_linear_tops", "value": ops2 / (ms_asym * 1e-3) / 1e12,
                        "unit": "TOPS", "ms_per_pass": ms_asym,
                        "note": "opt-6.7b block, M=2048, asymmetric token-wise activations "
                                "(quantize_act_asym + linear_asym)"}

        fmt_opts = w4a8.make_opts(level_shift=2)
        for d, lay in zip(L2, layers2):
            W = torch.from_numpy(lay["W"]).to(dev)
            d["packed_fmt"] = w4a8.pack_weights(W, d["s"], d["group"], level_shift=2)
            del W

        def pass_fmt(it=None):
            for d in L2:
                w4a8.quantize_act(d["X"], d["inv_s"], out=(d["Xq"], d["tok"]))
                w4a8.linear(d["Xq"], d["tok"], d["packed_fmt"], d["bias"], d["N"], d["group"], d["ws"],
                            fmt_opts, out=d["Y"])
        for _ in range(3):
            pass_fmt()
        ms_fmt = timed(pass_fmt, 100) / 100
        legs["special_value_quarter_step"] = {
            "metric": "w4a8_dint_linear_tops", "value": ops2 / (ms_fmt * 1e-3) / 1e12, "unit": "TOPS",
            "ms_per_pass": ms_fmt,
            "note": "opt-6.7b block, M=2048, weights packed for the special value step/4 "
                    "(pack_weights_fmt, level_shift 2)"}
        for d in L2:
            w4a8.check_status(d["ws"])
            del d["packed_fmt"]

        # 3-bit dINT (p = 5 steps; Tables 10-11): the same block from 0.375-byte-per-weight blobs
        opts3 = w4a8.make_opts(bits=3)
        for d, lay in zip(L2, layers2):
            W = torch.from_numpy(lay["W"]).to(dev)
            d["packed3"] = [w4a8.pack_weights(W, d["s"], d["group"], bits=3)]
            d["packed3"] += [d["packed3"][0].clone() for _ in range(2)]
            d["ws3"] = w4a8.new_workspace(M_PREFILL, d["N"], d["K"], d["group"], opts3)
            d["ws3_1"] = w4a8.new_workspace(1, d["N"], d["K"], d["group"], opts3)
            del W

        def pass_dint3(it=None):
            for d in L2:
                w4a8.quantize_act(d["X"], d["inv_s"], out=(d["Xq"], d["tok"]))
                w4a8.linear(d["Xq"], d["tok"], d["packed3"][0], d["bias"], d["N"], d["group"], d["ws3"],
                            opts3, out=d["Y"])
        for _ in range(3):
            pass_dint3()
        ms_d3 = timed(pass_dint3, 100) / 100
        Xq1 = {id(d): torch.empty((1, d["K"]), dtype=torch.int8, device=dev) for d in L2}
        tok1 = torch.empty((1,), dtype=torch.float32, device=dev)
        Y1 = {id(d): torch.empty((1, d["N"]), dtype=torch.bfloat16, device=dev) for d in L2}

        def step_dint3_decode(it):
            for d in L2:
                w4a8.quantize_act(d["X"][:1], d["inv_s"], out=(Xq1[id(d)], tok1))
                w4a8.linear(Xq1[id(d)], tok1, d["packed3"][it % 3], d["bias"], d["N"], d["group"],
                            d["ws3_1"], opts3, out=Y1[id(d)])
        ms_d3_dec = graph_ms(step_dint3_decode, 60)
        bytes3 = sum(3 * d["K"] * d["N"] // 8 + 5 * d["N"] + d["K"] + 4 + 2 * d["N"] + 4 * d["N"] for d in L2)
        for d in L2:
            w4a8.check_status(d["ws3"])
            w4a8.check_status(d["ws3_1"])
            for k in ("packed3", "ws3", "ws3_1"):
                del d[k]
        legs["dint3"] = {
            "workload": "opt-6.7b block linears, 3-bit dINT weights (0.375 byte per weight), per-channel",
            "prefill": {"metric": "w4a8_dint_linear_tops", "M": M_PREFILL,
                        "value": ops2 / (ms_d3 * 1e-3) / 1e12, "unit": "TOPS", "ms_per_pass": ms_d3},
            "decode": {"metric": "w4a8_dint_linear_hbm_gbs", "M": 1, "value": bytes3 / (ms_d3_dec * 1e-3) / 1e9,
                       "unit": "GB/s", "ms_per_step": ms_d3_dec, "bytes_per_step": bytes3,
                       "frac_of_measured_copy": bytes3 / (ms_d3_dec * 1e-3) / 1e9 / peaks["hbm_gbs"],
                       "note": "quantize_act + linear per shape (weight-streaming kernel, row slabs, 3-bit "
                               "tiles), 3 rotating blob copies, CUDA graph replay"}}

        # decode, M = 1: eight launches of a few microseconds per step, timed from a CUDA graph
        for d in L2:
            d["X1"] = d["X"][:1].contiguous()
            d["Xq1"] = torch.empty((1, d["K"]), dtype=torch.int8, device=dev)
            d["tok1"] = torch.empty((1,), dtype=torch.float32, device=dev)
            d["Y1"] = torch.empty((1, d["N"]), dtype=torch.bfloat16, device=dev)
            d["ws1"] = w4a8.new_workspace(1, d["N"], d["K"], d["group"])
            d["wsf"] = w4a8.new_quantize_linear_workspace(1, d["N"], d["K"], d["group"])

        def step_decode(it):
            for d in L2:
                w4a8.quantize_act(d["X1"], d["inv_s"], out=(d["Xq1"], d["tok1"]))
                w4a8.linear(d["Xq1"], d["tok1"], d["packed_rot"][it % 3], d["bias"], d["N"], d["group"],
                            d["ws1"], out=d["Y1"])

        def step_decode_fused(it):
            for d in L2:
                w4a8.quantize_linear(d["X1"], d["inv_s"], d["packed_rot"][it % 3], d["bias"], d["N"],
                                     d["group"], d["wsf"], out=d["Y1"])
        ms_dec = graph_ms(step_decode, 60)
        ms_dec_fused = graph_ms(step_decode_fused, 60)
        for d in L2:
            w4a8.check_status(d["ws1"])
            w4a8.check_status(d["wsf"])
        dec_bytes = sum(linear_bytes(d["K"], d["N"], 1, d["group"]) for d in L2)
        dec_gbs = dec_bytes / (ms_dec * 1e-3) / 1e9
        fused_gbs = dec_bytes / (ms_dec_fused * 1e-3) / 1e9
        legs["decode"] = {
            "metric": "w4a8_dint_linear_hbm_gbs", "value": dec_gbs, "unit": "GB/s", "M": 1,
            "workload": "opt-6.7b block linears, M=1", "ms_per_step": ms_dec, "bytes_per_step": dec_bytes,
            "frac_of_measured_copy": dec_gbs / peaks["hbm_gbs"],
            "frac_of_nominal_8000": dec_gbs / NOMINAL_HBM_GBS,
            "note": "quantize_act + linear per shape, 3 rotating blob copies (> L2), CUDA graph replay",
            "one_launch": {"value": fused_gbs, "unit": "GB/s", "ms_per_step": ms_dec_fused,
                           "frac_of_measured_copy": fused_gbs / peaks["hbm_gbs"],
                           "note": "the same step through quantize_linear: the quantizer runs inside "
                                   "the weight-streaming kernel, one launch per linear"},
            "large_layer": {"workload": "opt-66b fc1 9216->36864, M=1, per-channel dINT4 (quantize_act + linear)",
                            "value": big1["gbs"], "unit": "GB/s", "ms_per_step": big1["ms"],
                            "frac_of_measured_copy": big1["frac_of_measured_copy"],
                            "frac_of_nominal_8000": big1["frac_of_nominal_8000"],
                            "note": "2 rotating blob copies (> L2), CUDA graph replay"}}
        # the activation quantizer with the normalisation in front of it fused in (the Eq. 1 scale
        # lives in the normalisation's weight): one pass over X instead of norm + quantizer
        nq = {}
        for name, K in (("hidden_4096", 4096), ("hidden_16384", 16384)):
            d = next(x for x in L2 if x["K"] == K)
            gamma = (1.0 / d["s"]).contiguous()
            beta = torch.zeros_like(gamma)
            for kind, code, bias_t in (("rms", w4a8.NORM_RMS, None), ("layer", w4a8.NORM_LAYER, beta)):
                fn = lambda it, d=d, code=code, bias_t=bias_t: w4a8.norm_quantize_act(
                    d["X"], gamma, bias_t, code, 1e-5, out=(d["Xq"], d["tok"]))
                ms_n = graph_ms(fn, 20)
                gbs = (3.0 * M_PREFILL * K + 4 * M_PREFILL) / (ms_n * 1e-3) / 1e9
                nq[f"{name}_{kind}"] = {"ms": ms_n, "gbs": gbs, "frac_of_measured_copy": gbs / peaks["hbm_gbs"]}
            ms_p = graph_ms(lambda it, d=d: w4a8.quantize_act(d["X"], d["inv_s"], out=(d["Xq"], d["tok"])), 20)
            gbs = (3.0 * M_PREFILL * K + 4 * M_PREFILL) / (ms_p * 1e-3) / 1e9
            nq[f"{name}_plain_quantizer"] = {"ms": ms_p, "gbs": gbs, "frac_of_measured_copy": gbs / peaks["hbm_gbs"]}
        legs["norm_fused_act_quant"] = {
            "metric": "hbm_gbs", "unit": "GB/s", "tokens": M_PREFILL, **nq,
            "note": "w4a8_norm_quantize_act (RMSNorm; LayerNorm with bias) against w4a8_quantize_act, "
                    "3 bytes per element, CUDA graph replay of 20 launches on the same tensor (L2-warm "
                    "for 4096, larger than L2 with its output for 16384)"}
        for d in L2:
            d.clear()
        del L2, layers2
        torch.cuda.empty_cache()

        # -------------------------------------------------------------- group-128: LLaMA-7B block and token sweep
        layers3 = host_layers(synth, 3, (0, 1, 2, 3), M_PREFILL)
        L3 = device_block(layers3, M_PREFILL)
        ops3 = sum(2 * M_PREFILL * d["K"] * d["N"] for d in L3)
        ms3, lin3, passes3, region3 = time_block(L3, 10, 0.3)
        lin3_tops = ops3 / (sum(lin3) * 1e-3) / 1e12
        group_leg = {
            "workload": "llama-7b block linears (gate 4096->11008, up 4096->11008, down 11008->4096, "
                        "qkv 4096->12288), M=2048 prefill, group-128 dINT4",
            "metric": "w4a8_dint_linear_tops", "value": ops3 / (ms3 * 1e-3) / 1e12, "unit": "TOPS",
            "ms_per_pass": ms3, "region_s": region3, "linear_only_tops": lin3_tops,
            **{k: v for k, v in tensor_fracs(lin3_tops, region3).items() if k.startswith("frac")},
            "per_linear_ms": dict(zip([d["label"] for d in L3], lin3)),
            "per_linear_tops": {d["label"]: 2.0 * M_PREFILL * d["K"] * d["N"] / (t * 1e-3) / 1e12
                                for d, t in zip(L3, lin3)}}
        # the gated feed-forward block as two launches per matmul stage: gate and up rows interleaved
        # in one blob, silu(gate) * up in the epilogue (binary16), quantizer, down projection
        gate, up, down_l = L3[0], L3[1], L3[2]
        Wgu = w4a8.interleave_gate_up(torch.from_numpy(layers3[0]["W"]).to(dev), torch.from_numpy(layers3[1]["W"]).to(dev))
        F3, K3 = gate["N"], gate["K"]
        packed_gu = w4a8.pack_weights(Wgu, gate["s"], 128)
        del Wgu
        ws_gu = w4a8.new_linear_swiglu_workspace(M_PREFILL, F3, K3, 128)
        Hbuf = torch.empty((M_PREFILL, F3), dtype=torch.float16, device=dev)

        def pass_mlp(it=None):
            w4a8.quantize_act(gate["X"], gate["inv_s"], out=(gate["Xq"], gate["tok"]))
            w4a8.linear_swiglu(gate["Xq"], gate["tok"], packed_gu, None, F3, 128, ws_gu, out=Hbuf)
            w4a8.quantize_act(Hbuf, down_l["inv_s"], out=(down_l["Xq"], down_l["tok"]))
            w4a8.linear(down_l["Xq"], down_l["tok"], down_l["packed"], down_l["bias"], down_l["N"], 128,
                        down_l["ws"], out=down_l["Y"])
        for _ in range(3):
            pass_mlp()
        ms_mlp = timed(pass_mlp, 50) / 50
        w4a8.check_status(ws_gu)
        ops_mlp = 2.0 * M_PREFILL * K3 * F3 * 3
        group_leg["gated_mlp_fused"] = {
            "metric": "w4a8_dint_linear_tops", "value": ops_mlp / (ms_mlp * 1e-3) / 1e12, "unit": "TOPS",
            "ms_per_pass": ms_mlp,
            "unfused_linears_ms": lin3[0] + lin3[1] + lin3[2],
            "note": "llama-7b feed-forward block at M=2048, group-128: quantize_act, linear_swiglu "
                    "(4096 -> 2 x 11008 with silu(gate) * up in the epilogue), quantize_act, linear "
                    "(11008 -> 4096); unfused_linears_ms is the sum of the three separate tensor-core "
                    "launches of the block above (without the unit and without the quantizers)"}
        del packed_gu, ws_gu, Hbuf
        for d in L3:
            d.clear()
        del L3, layers3
        torch.cuda.empty_cache()
        # the down projection over token counts: weight-streaming kernel, tensor-core kernel with
        # narrow tiles and K split, full tiles (the library picks; `plan` says what it picked)
        sweep = []
        big_m = 16384
        down = device_block(host_layers(synth, 5, (0,), big_m), big_m, rot=1)[0]
        for M in (1, 16, 256, 4096, 16384):
            rot = max(1, min(6, (300 << 20) // linear_bytes(down["K"], down["N"], M, 128)))
            sweep.append(decode_point(down, M, rot, steps_in_graph=20 if M <= 4096 else 5))
        group_leg["token_sweep_down_11008_4096"] = sweep
        legs["group128"] = group_leg
        down.clear()
        torch.cuda.empty_cache()

    if legs_on:
        # -------------------------------------------------------------- attention value path (W4A8V4)
        Hh, Dh = 32, 128
        gen = torch.Generator(device=dev)
        gen.manual_seed(5005)
        pv = {}
        for name, T, S in (("prefill_T2048_S2048", 2048, 2048), ("decode_T1_S4096", 1, 4096)):
            V = torch.randn((S, Hh, Dh), generator=gen, device=dev, dtype=torch.float16)
            P = torch.softmax(2.0 * torch.randn((Hh, T, S), generator=gen, device=dev, dtype=torch.float32), -1).half()
            blobs = [w4a8.pack_value(V)]
            blobs += [blobs[0].clone() for _ in range(3)]
            Pq = torch.empty((Hh * T, S), dtype=torch.int8, device=dev)
            ps = torch.empty((Hh * T,), dtype=torch.float32, device=dev)
            O = torch.empty((T, Hh, Dh), dtype=torch.bfloat16, device=dev)
            wsv = w4a8.new_attn_pv_workspace(T, S, Hh, Dh)

            def fn(it, P=P, Pq=Pq, ps=ps, blobs=blobs, O=O, wsv=wsv, T=T, S=S):
                w4a8.quantize_act(P.view(Hh * T, S), None, out=(Pq, ps))
                w4a8.attn_pv(Pq.view(Hh, T, S), ps.view(Hh, T), blobs[it % 4], Dh, wsv, out=O)
            ms_pv = graph_ms(fn, 20)
            w4a8.check_status(wsv)
            ops_pv = 2.0 * T * S * Hh * Dh
            bytes_pv = S * Hh * Dh // 2 + 5 * Hh * Dh + Hh * T * (S + 4) + 2 * T * Hh * Dh
            pv[name] = {"ms": ms_pv, "tops": ops_pv / (ms_pv * 1e-3) / 1e12,
                        "gbs": bytes_pv / (ms_pv * 1e-3) / 1e9,
                        "frac_of_burst_tensor": ops_pv / (ms_pv * 1e-3) / 1e12 / (2.0 * peaks["bf16_burst"]),
                        "frac_of_measured_copy": bytes_pv / (ms_pv * 1e-3) / 1e9 / peaks["hbm_gbs"]}
            del V, P, blobs, Pq, ps, O, wsv
        torch.cuda.empty_cache()
        legs["attn_pv_value4"] = {
            "workload": "attention map x values, 32 heads of dimension 128, channel-wise dINT4 values "
                        "(W4A8V4), token-wise INT8 attention map", **pv,
            "note": "per step: quantize_act on the FP16 attention map + attn_pv (all heads in one "
                    "launch of the tensor-core kernel); random map and values drawn on the device; "
                    "CUDA graph replay of 20 steps"}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    cpu = None
    if not args.no_cpu_baseline:
        import oracle
        sample = cpu_sample(layers)
        t, ops = cpu_sample_time(sample)
        cpu = {"value": ops / t / 1e12, "unit": "TOPS", "cores": oracle.get_threads(),
               "kind": "oracle", "seconds": t, "sample": cpu_sample_text(len(layers))}

    line = {
        "metric": "w4a8_dint_linear_tops", "value": tops, "unit": "TOPS", "n_gpus": world,
        "steps": args.steps, "warmup": warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8",
        "data": "synthetic",
        "config": {"workload": HEADLINE_NAME,
                   "pass": "4 x (quantize_act + linear); weights packed once before timing",
                   "passes_per_step": passes, "ms_per_pass": ms_pass, "timed_region_s": region_s,
                   "l2": "inputs larger than L2 (about 1.3 GB touched per pass)",
                   "plan": w4a8.linear_plan(M_PREFILL, layers[2]["N"], layers[2]["K"], layers[2]["group"], plan_opts),
                   "parallelism": "replicas" if world > 1 else "single"},
        "clocks": clocks,
        "e2e": {"value": replica_throughput(ops_per_pass, world, ms_e2e), "unit": "TOPS",
                "ms_per_pass": ms_e2e, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "note": "one pass per step: pinned host inputs up, results down, copies inside the region"},
        "gpu_launches": 2 * len(layers) * passes * args.steps,
        "roofline": {"bound": "tensor", "kernel": "linear_tcgen05_kernel (256-token tile, per-channel)",
                     "achieved": lin_tops, "unit": "TOPS", **tensor_fracs(lin_tops, region_s),
                     "per_linear_ms": dict(zip([lay["label"] for lay in layers], lin_ms)),
                     "per_linear_tops": {lay["label"]: 2.0 * M_PREFILL * lay["K"] * lay["N"] / (t * 1e-3) / 1e12
                                         for lay, t in zip(layers, lin_ms)},
                     "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH,
                     "algorithmic_bytes_per_launch": sum(
                         linear_bytes(lay["K"], lay["N"], M_PREFILL, lay["group"]) for lay in layers) / len(layers)},
        **legs,
        "cpu_baseline": cpu,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
