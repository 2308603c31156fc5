#!/usr/bin/env python
"""Benchmark of the BCQ linear-layer hot path on B200.

Headline: a step is one AlphaTuning adaptation pass over a GPT-2-XL-shaped stack -- for each of
the 48 layers and each of its four quantized linears (1600->4800, 1600->1600, 1600->6400,
6400->1600; q = 4, group-wise alpha with g = 128) the forward (Eq. 2), the scale gradient
(Eq. 4) and the input gradient (Eq. 3) on 4096 tokens.  The weights are quantized once before
the timed region (the paper's post-training step).  Reported beside it: the GPT-2-medium stack
(q = 3, row-wise alpha, 2048 tokens), the single 1024 x 1024 layer, the decode GEMV table
(OPT-6.7B shapes) and the quantizer's throughput.

    python bench.py --gpus N --steps K --warmup W            # this library
    python bench.py --impl reference --gpus N --steps K ...  # the fp64 CPU oracle on a sample

With N > 1 (torchrun) every rank runs the same per-GPU workload on its own tokens (weak scaling)
and the scale gradients, which live in one flat buffer, are all-reduced once per step.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "bcq_linear_fwd_bwd_tflops"
UNIT = "TFLOP/s"


def block(hidden, ffn):
    return [("att_qkv", hidden, 3 * hidden), ("att_out", hidden, hidden), ("ffn_h_4h", hidden, ffn),
            ("ffn_4h_h", ffn, hidden)]


STACKS = {
    "gpt2-xl": dict(workload="gpt2-xl-block x48, q=4, g=128, 4096 tokens, fwd+dalpha+dX", layers=48, tokens=4096,
                    q=4, g=128, linears=block(1600, 6400)),
    "gpt2-medium": dict(workload="gpt2-medium-block x24, q=3 row-wise alpha, 2048 tokens, fwd+dalpha+dX", layers=24,
                        tokens=2048, q=3, g=None, linears=block(1024, 4096)),
    "single-1024": dict(workload="one 1024->1024 linear, q=3 row-wise alpha, 512 tokens, fwd+dalpha+dX", layers=1,
                        tokens=512, q=3, g=None, linears=[("lin", 1024, 1024)]),
}
HEADLINE = "gpt2-xl"

# DRAM bytes (read + write) of one forward call and its pre-pass, from the ncu capture of the FFN
# shape 1600 -> 6400 with 4096 tokens (profiles/expand_gemm_gpt2xl.md): pre-pass 14.5 MB read, GEMM
# 20.0 MB read + 3.9 MB written.  The fp16 copy of X and most of Y are still in L2 when the kernels
# end, which is why this is below the call's algorithmic bytes.
TRAFFIC_BYTES_PER_LAUNCH = 38.4e6


def step_flops(cfg):
    return 3 * sum(2.0 * cfg["tokens"] * di * do for _, di, do in cfg["linears"]) * cfg["layers"]


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        burst = float(p.get("bf16_tflops", 1590.0))
        return {"burst": burst, "sustained": float(p.get("bf16_tflops_sustained", burst)),
                "hbm_gbs": float(p.get("hbm_gbs", 6650.0)), "source": "measured"}
    return {"burst": 1590.0, "sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
        sm = sorted(int(r[0]) for r in self.rows if r and r[0].isdigit())
        mx = [int(r[1]) for r in self.rows if len(r) > 1 and r[1].isdigit()]
        reasons = set()
        for r in self.rows:
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------ oracle arm

ORACLE_SAMPLE = "att_out 1600->1600, q=4, g=128, 256 of 4096 tokens, fwd+dalpha+dX, fp64"


def oracle_sample(steps, warmup):
    """Times the oracle, as it stands, on a bounded sample of the headline workload: one att_out
    linear (1600 -> 1600, q = 4, g = 128) with 256 of the 4096 tokens, forward + dalpha + dX."""
    import oracle
    from paper_2210_03858_b200 import synth
    n, d_in, d_out, q, g = 256, 1600, 1600, 4, 128
    key = (2, 0, 1)
    W = synth.weights(d_out, d_in, key)
    X = synth.activations(n, d_in, key, synth.ROLE_X)
    dY = synth.activations(n, d_out, key, synth.ROLE_DY)
    bits, alpha, _, _ = oracle.quantize(W, q, g)
    flops = 3 * 2.0 * n * d_in * d_out

    def step():
        oracle.fwd(X, bits, alpha, d_in, g)
        oracle.bwd_alpha(dY, X, bits, d_in, g)
        oracle.bwd_x(dY, bits, alpha, d_in, g)

    for _ in range(max(0, warmup)):
        step()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    dt = (time.perf_counter() - t0) / steps
    return {"value": flops / dt / 1e12, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": ORACLE_SAMPLE, "ms_per_step": dt * 1e3}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps = max(1, min(args.steps, 5))
    cb = oracle_sample(steps, min(args.warmup, 1))
    line = {"impl": "reference", "metric": METRIC, "value": cb["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": cb["ms_per_step"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": STACKS[HEADLINE]["workload"], "sample": cb["sample"]},
            "cpu_baseline": {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": cb["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------ GPU arm

class Stack:
    """The linears of one workload on one GPU: quantized weights, inputs, outputs, workspaces, and
    the step enqueued on (operation, chain) streams, optionally captured as one CUDA graph."""

    OPS = ("fwd", "bwd_alpha", "bwd_x")

    def __init__(self, cfg, torch, bcq, dev, rank, chains, out_bf16, seed_base, prepared=True):
        from paper_2210_03858_b200.dist import AlphaBucket
        self.cfg, self.torch, self.bcq, self.dev = cfg, torch, bcq, dev
        self.chains = max(1, chains)
        self.prepared = prepared and hasattr(bcq, "prepare_planes")
        q, n = cfg["q"], cfg["tokens"]
        gen = torch.Generator(device=dev)
        self.layers = []
        shapes = []
        for layer in range(cfg["layers"]):
            for li, (_, d_in, d_out) in enumerate(cfg["linears"]):
                g = cfg["g"] or d_in
                gen.manual_seed(seed_base + 1000003 * rank + 4099 * layer + li)
                W = torch.randn((d_out, d_in), generator=gen, device=dev, dtype=torch.float32) * 0.02
                bits, alpha, _ = bcq.quantize(W, q, g)
                del W
                # B is frozen from here on: its planes are regrouped once for the forward and for dX
                planes_fwd = bcq.prepare_planes(bcq.OP_FWD, bits, d_in, g) if self.prepared else bits
                planes_dx = bcq.prepare_planes(bcq.OP_BWD_X, bits, d_in, g) if self.prepared else bits
                X = torch.randn((n, d_in), generator=gen, device=dev, dtype=torch.float32).bfloat16()
                dY = torch.randn((n, d_out), generator=gen, device=dev, dtype=torch.float32).bfloat16()
                self.layers.append(dict(d_in=d_in, d_out=d_out, g=g, bits=bits, alpha=alpha, X=X, dY=dY,
                                        planes_fwd=planes_fwd, planes_dx=planes_dx,
                                        chain=len(self.layers) % self.chains))
                shapes.append((q, d_out, bcq.num_groups(d_in, g)))
        # the scale gradients of all linears: views of one flat buffer (one all-reduce for N > 1)
        self.bucket = AlphaBucket(shapes, dev)
        for i, l in enumerate(self.layers):
            l["dalpha"] = self.bucket[i]
        out_dtype = torch.bfloat16 if out_bf16 else torch.float32
        self.bufs = {}
        for _, d_in, d_out in cfg["linears"]:
            g = cfg["g"] or d_in

            def ws(op):
                return torch.empty(max(16, bcq.workspace_bytes(op, d_out, d_in, q, g, n)), dtype=torch.uint8, device=dev)
            for c in range(self.chains):
                self.bufs[(d_in, d_out, c)] = dict(Y=torch.empty((n, d_out), device=dev, dtype=out_dtype),
                                                   dX=torch.empty((n, d_in), device=dev, dtype=out_dtype),
                                                   ws_fwd=ws(bcq.OP_FWD), ws_dx=ws(bcq.OP_BWD_X),
                                                   ws_da=ws(bcq.OP_BWD_ALPHA))
        # one stream per (operation, chain); the dX chains are the longest, so theirs get the higher priority
        self.streams = {(name, c): torch.cuda.Stream(device=dev, priority=-1 if name == "bwd_x" else 0)
                        for name in self.OPS for c in range(self.chains)}
        self.graph = None
        self.launches_per_step = 0

    def op(self, name, l):
        bcq = self.bcq
        b = self.bufs[(l["d_in"], l["d_out"], l["chain"])]
        if name == "fwd":
            bcq.linear_fwd(l["X"], l["planes_fwd"], l["alpha"], l["d_in"], l["g"], out=b["Y"], ws=b["ws_fwd"])
        elif name == "bwd_alpha":
            bcq.linear_bwd_alpha(l["dY"], l["X"], l["bits"], l["d_in"], l["g"], out=l["dalpha"], ws=b["ws_da"])
        else:
            bcq.linear_bwd_x(l["dY"], l["planes_dx"], l["alpha"], l["d_in"], l["g"], out=b["dX"], ws=b["ws_dx"])

    def linear_step(self, l):
        for name in self.OPS:
            self.op(name, l)

    def enqueue_step(self):
        # the linears are independent problems, and within one linear dalpha and dX only share their
        # inputs: forward, dalpha and dX of the linears of a chain are three queues on three streams
        torch = self.torch
        cur = torch.cuda.current_stream()
        for s_ in self.streams.values():
            s_.wait_stream(cur)
        for name in self.OPS:
            for c in range(self.chains):
                with torch.cuda.stream(self.streams[(name, c)]):
                    for l in self.layers:
                        if l["chain"] == c:
                            self.op(name, l)
        for s_ in self.streams.values():
            cur.wait_stream(s_)

    def prepare(self, main, use_graph):
        """Warm-up outside capture (resolves lazy CUDA state), then one step captured as a graph."""
        torch, bcq = self.torch, self.bcq
        with torch.cuda.stream(main):
            self.enqueue_step()
            torch.cuda.synchronize()
            c0 = bcq.kernel_launches()
            if use_graph:
                self.graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(self.graph, stream=main):
                    self.enqueue_step()
            else:
                self.enqueue_step()
            self.launches_per_step = bcq.kernel_launches() - c0
        torch.cuda.synchronize()

    def step(self):
        if self.graph is not None:
            self.graph.replay()
        else:
            self.enqueue_step()

    def per_op(self, main):
        """GPU time of each operation alone: its calls back to back on one stream (a graph, so
        host launch time stays out).  Three untimed replays bring the clocks to where they settle
        under load, then five replays are timed as one region and averaged: a single replay after an
        idle gap runs at boost clocks and its time moves by tens of percent from run to run."""
        torch = self.torch
        res = {}
        for name in self.OPS:
            g_ = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g_, stream=main):
                for l in self.layers:
                    self.op(name, l)
            for _ in range(3):
                g_.replay()
            torch.cuda.synchronize()
            a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(5):
                g_.replay()
            b_.record()
            torch.cuda.synchronize()
            best = a.elapsed_time(b_) / 5.0
            flops = sum(2.0 * self.cfg["tokens"] * l["d_in"] * l["d_out"] for l in self.layers)
            res[name] = (best, flops, len(self.layers))
            del g_
        return res


def timed_region(torch, dist, world, dev, step, steps):
    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
    sync_all()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    sync_all()
    ms = torch.tensor([e0.elapsed_time(e1)], device=dev)
    if world > 1:
        dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    return float(ms.item()) / steps


def run_gpu(args):
    import torch
    import torch.distributed as dist
    import paper_2210_03858_b200 as bcq
    from paper_2210_03858_b200 import build as bcq_build
    from paper_2210_03858_b200.dist import allreduce_dalpha

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        bcq_build.build_library()
    if world > 1:
        dist.barrier()
    bcq.lib()

    cfg = STACKS[args.stack]
    flops = step_flops(cfg)
    stack = Stack(cfg, torch, bcq, dev, rank, args.chains, args.out_bf16, 221003858, prepared=args.prepared)
    main = torch.cuda.Stream(device=dev)
    stack.prepare(main, args.graph)
    torch.cuda.set_stream(main)

    def step():
        stack.step()
        if world > 1:  # data parallel: the scale gradients are summed over ranks once per step
            allreduce_dalpha(stack.bucket)

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()  # nvidia-smi needs a moment to come up: start it before the warm-up
    warmup = max(3, args.warmup)
    for _ in range(warmup):
        step()
    c0 = bcq.kernel_launches()
    ms_per_step = timed_region(torch, dist, world, dev, step, args.steps)
    launches = stack.launches_per_step * args.steps if stack.graph is not None else bcq.kernel_launches() - c0
    assert bcq.device_timeout_flag() == 0, "a kernel reported an expired wait"
    value = world * flops / (ms_per_step * 1e-3) / 1e12
    if args.timed_only:
        if rank == 0:
            sampler.stop()
            print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                              "ms_per_step": ms_per_step, "gpu_launches": int(launches), "note": "timed steps only"}))
        if world > 1:
            dist.destroy_process_group()
        return
    # the same region four more times: how much one sample moves
    regions = [ms_per_step] + [timed_region(torch, dist, world, dev, step, args.steps) for _ in range(4)]
    clocks = sampler.stop() if rank == 0 else None

    per_op = stack.per_op(main)

    # ---- end to end: the inputs of every linear come from pinned host memory every step and its
    # scale gradient is read back; Y and dX stay on the device (they feed the neighbouring layers)
    e2e_steps = max(1, min(args.steps, 2))
    host = {}
    for l in stack.layers:
        k = (l["d_in"], l["d_out"])
        if k not in host:  # one pinned source per shape: the bytes that cross PCIe are the same
            host[k] = (l["X"].cpu().pin_memory(), l["dY"].cpu().pin_memory(),
                       torch.empty(l["dalpha"].shape, dtype=torch.float32).pin_memory())
    h2d = sum(l["X"].numel() * 2 + l["dY"].numel() * 2 for l in stack.layers)
    d2h = sum(l["dalpha"].numel() * 4 for l in stack.layers)
    h2d_s, d2h_s = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)

    def e2e_step():
        cur = torch.cuda.current_stream()
        h2d_s.wait_stream(cur)  # the previous step's kernels have read the inputs about to be overwritten
        for l in stack.layers:
            hX, hdY, hdA = host[(l["d_in"], l["d_out"])]
            with torch.cuda.stream(h2d_s):
                l["X"].copy_(hX, non_blocking=True)
                l["dY"].copy_(hdY, non_blocking=True)
                arrived = torch.cuda.Event()
                arrived.record(h2d_s)
            cur.wait_event(arrived)
            stack.linear_step(l)
            computed = torch.cuda.Event()
            computed.record(cur)
            with torch.cuda.stream(d2h_s):
                d2h_s.wait_event(computed)
                hdA.copy_(l["dalpha"], non_blocking=True)
        cur.wait_stream(h2d_s)
        cur.wait_stream(d2h_s)
        if world > 1:
            allreduce_dalpha(stack.bucket)
    e2e_step()
    e2e_ms = timed_region(torch, dist, world, dev, e2e_step, e2e_steps)
    e2e = {"value": world * flops / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": d2h, "steps": e2e_steps,
           "note": "through the C-ABI calls of the Python binding: X and dY of every linear copied from pinned host "
                   "memory and its dalpha copied back, every step (one pinned source per layer shape); copies on their "
                   "own streams overlap the neighbouring linears' kernels; Y and dX stay on the device"}
    del host

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    # dominant kernel: the expansion GEMM (forward and dX calls, their pre-pass included)
    t_exp = per_op["fwd"][0] + per_op["bwd_x"][0]
    f_exp = per_op["fwd"][1] + per_op["bwd_x"][1]
    n_exp = per_op["fwd"][2] + per_op["bwd_x"][2]
    achieved = f_exp / (t_exp * 1e-3) / 1e12
    roofline = {"bound": "tensor",
                "kernel": "expand_gemm_kernel (bcq_linear_fwd / bcq_linear_bwd_x calls, pre-pass included), one stream",
                "achieved": achieved, "peak": peaks["burst"], "unit": "TFLOP/s", "frac": achieved / peaks["burst"],
                "peak_source": "of %s (burst bf16/fp16 dense; each operation's calls are timed alone)" % peaks["source"],
                "frac_of_sustained": achieved / peaks["sustained"],
                "traffic": TRAFFIC_BYTES_PER_LAUNCH if args.stack == HEADLINE else None,
                "flops_per_launch": f_exp / n_exp, "avg_launch_ms": t_exp / n_exp,
                "step": {"tflops": value, "frac_of_burst": value / world / peaks["burst"],
                         "frac_of_sustained": value / world / peaks["sustained"]},
                "per_op_tflops": {k: v[1] / (v[0] * 1e-3) / 1e12 for k, v in per_op.items()},
                "per_op_share": {k: v[0] / sum(x[0] for x in per_op.values()) for k, v in per_op.items()}}

    cb = oracle_sample(3, 1)
    cpu_baseline = {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")}
    inputs_gb = sum(l["X"].numel() * 2 + l["dY"].numel() * 2 + l["bits"].numel() * 4 + l["alpha"].numel() * 4
                    for l in stack.layers) / 1e9
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f16", "data": "synthetic",
            "config": {"workload": cfg["workload"], "layers": cfg["layers"], "tokens_per_gpu": cfg["tokens"],
                       "q": cfg["q"], "g": cfg["g"] or "d_in",
                       "l2": "a step touches %.1f GB of distinct inputs, far more than the 126 MB L2" % inputs_gb,
                       "outputs": "bf16" if args.out_bf16 else "fp32",
                       "planes": "regrouped once per layer (bcq_prepare_planes), B being frozen" if stack.prepared
                                 else "canonical planes, regrouped by every call",
                       "launch": ("one CUDA graph per step, " if args.graph else "") +
                                 "forward / dalpha / dX on %d streams (dX at high priority)" % (3 * stack.chains),
                       "parallelism": "dp%d" % world},
            "repeats": {"regions": len(regions), "ms_per_step_median": statistics.median(regions),
                        "ms_per_step_min": min(regions), "ms_per_step_max": max(regions)},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
            "cpu_baseline": cpu_baseline}
    del stack
    torch.cuda.empty_cache()
    if args.extras:
        for name in ("gpt2-medium", "single-1024"):
            if name != args.stack:
                line[name] = small_stack_numbers(name, torch, bcq, dev, rank, args, peaks)
        line["decode"] = decode_numbers(bcq, torch, dev, peaks)
        line["quantize"] = quantize_numbers(bcq, torch, dev, peaks)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def small_stack_numbers(name, torch, bcq, dev, rank, args, peaks):
    """The other fwd+dalpha+dX workloads, timed the same way (one graph per step, 10 steps)."""
    cfg = STACKS[name]
    st = Stack(cfg, torch, bcq, dev, rank, args.chains, args.out_bf16, 221003858 + 17, prepared=args.prepared)
    main = torch.cuda.current_stream()
    st.prepare(main, True)
    for _ in range(3):
        st.step()
    ms = timed_region(torch, None, 1, dev, st.step, 10)
    per_op = st.per_op(main)
    tf = step_flops(cfg) / (ms * 1e-3) / 1e12
    return {"workload": cfg["workload"], "tflops": tf, "ms_per_step": ms, "frac_of_burst": tf / peaks["burst"],
            "per_op_tflops": {k: v[1] / (v[0] * 1e-3) / 1e12 for k, v in per_op.items()}}


def decode_numbers(bcq, torch, dev, peaks):
    """Decode GEMV of OPT-6.7B-shaped linears (q in {3, 4}, g = 128, 1 / 4 / 16 tokens) from packs
    (bcq_linear_decode_packed), rotating over about 1 GB of distinct layers so that the weights
    come from HBM; one CUDA graph of the rotation, best of five replays; GB/s on the
    algorithmic bytes q d_out d_in / 8 + 4 q d_out G + 2 n d_in + 4 n d_out."""
    out = {}
    g = 128
    for q in (3, 4):
        for name, d_in, d_out in (("att_qkv", 4096, 12288), ("ffn_h_4h", 4096, 16384), ("ffn_4h_h", 16384, 4096)):
            per = bcq.bits_bytes(d_out, d_in, q) + bcq.alpha_count(d_out, d_in, q, g) * 4
            L = int(1.0e9 // per) + 1
            gen = torch.Generator(device=dev)
            gen.manual_seed(7 + d_in + d_out + q)
            packs = []
            for _ in range(L):
                bits = torch.randint(-2 ** 31, 2 ** 31 - 1, (q, d_out, bcq.pitch_words(d_in)), generator=gen,
                                     dtype=torch.int32, device=dev)
                alpha = torch.rand((q, d_out, d_in // g), generator=gen, device=dev) * 0.02
                packs.append(bcq.decode_pack(bits, alpha, d_in, g))
                del bits, alpha
            for n in (1, 4, 16):
                X = torch.randn((n, d_in), generator=gen, device=dev).bfloat16()
                Y = torch.empty((n, d_out), device=dev)
                ws = torch.empty(max(16, bcq.workspace_bytes(bcq.OP_DECODE_PACKED, d_out, d_in, q, g, n)),
                                 dtype=torch.uint8, device=dev)
                s = torch.cuda.Stream(device=dev)
                with torch.cuda.stream(s):
                    for l in range(L):
                        bcq.linear_decode_packed(X, packs[l], d_out, d_in, q, g, out=Y, ws=ws)
                    torch.cuda.synchronize()
                    gr = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(gr, stream=s):
                        for l in range(L):
                            bcq.linear_decode_packed(X, packs[l], d_out, d_in, q, g, out=Y, ws=ws)
                    gr.replay()
                    torch.cuda.synchronize()
                    best = None
                    for _ in range(5):
                        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        e0.record()
                        gr.replay()
                        e1.record()
                        torch.cuda.synchronize()
                        best = e0.elapsed_time(e1) if best is None else min(best, e0.elapsed_time(e1))
                us = best * 1e3 / L
                byt = per + 2 * n * d_in + 4 * n * d_out
                gbs = byt / us / 1e3
                out["%s_q%d_n%d" % (name, q, n)] = {"us": us, "GB/s": gbs, "frac_of_hbm": gbs / peaks["hbm_gbs"]}
                del gr
            del packs
    return out


def quantize_numbers(bcq, torch, dev, peaks):
    """bcq_quantize throughput: greedy on the four GPT-2-XL shapes (q = 4, g = 128) and greedy + 5
    alternating rounds on one OPT-13B-shaped layer (5120 -> 15360, 0.1 % outliers x 20) per q.
    20 launches back to back over weight buffers larger than L2, CUDA-event timed; GB/s on the
    algorithmic bytes 4 + q/8 + 4q/g per weight."""
    out = {}
    gen = torch.Generator(device=dev)

    def run(tag, d_in, d_out, q, g, alt, outliers, launches):
        gen.manual_seed(99 + d_in + d_out + q)
        nbuf = max(1, int(300e6 // (d_in * d_out * 4)) + 1)  # rotate over > 126 MB of weights
        Ws = []
        for _ in range(nbuf):
            W = torch.randn((d_out, d_in), generator=gen, device=dev) * 0.02
            if outliers:
                W = torch.where(torch.rand((d_out, d_in), generator=gen, device=dev) < 1e-3, W * 20.0, W)
            Ws.append(W)
        for i in range(2):
            bcq.quantize(Ws[i % nbuf], q, g, alt)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(launches):
            bcq.quantize(Ws[i % nbuf], q, g, alt)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / launches
        weights = float(d_in) * d_out
        gbs = weights * (4 + q / 8 + 4 * q / g) / (ms * 1e-3) / 1e9
        out[tag] = {"ms": ms, "Gweights/s": weights / (ms * 1e-3) / 1e9, "GB/s": gbs,
                    "frac_of_hbm": gbs / peaks["hbm_gbs"],
                    "bound": "hbm" if alt == 0 else "fp64 alu (the alternating rounds), not memory"}
        del Ws

    for name, d_in, d_out in block(1600, 6400):
        run("greedy_gpt2xl_%s_q4" % name, d_in, d_out, 4, 128, 0, False, 20)
    for q in (2, 3, 4):
        run("alt5_opt13b_att_qkv_q%d" % q, 5120, 15360, q, 128, 5, True, 20)
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=("ours", "reference"))
    ap.add_argument("--stack", default=HEADLINE, choices=sorted(STACKS), help="workload of the headline line")
    ap.add_argument("--no-extras", dest="extras", action="store_false",
                    help="skip the other stacks, the decode table and the quantizer numbers")
    ap.add_argument("--unprepared", dest="prepared", action="store_false",
                    help="pass the canonical planes to every call instead of planes prepared once")
    ap.add_argument("--no-graph", dest="graph", action="store_false", help="launch every kernel from the host each step")
    ap.add_argument("--out-fp32", dest="out_bf16", action="store_false", help="fp32 Y and dX instead of bf16")
    ap.add_argument("--chains", type=int, default=3,
                    help="independent chains per operation: the linears of a step are dealt round-robin to this many "
                         "streams (each with its own outputs and workspaces) for each of forward, dalpha and dX")
    ap.add_argument("--timed-only", action="store_true",
                    help="warm-up and timed steps only (no per-operation, end-to-end, CPU or extra legs): the command to profile")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
