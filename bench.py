#!/usr/bin/env python
"""Benchmark of the BCQ linear-layer hot path on B200.

A step is one AlphaTuning adaptation pass over a GPT-2-medium-shaped stack: for each of the
24 layers and each of its four quantized linears (1024->3072, 1024->1024, 1024->4096,
4096->1024; q = 3, row-wise alpha) the forward (Eq. 2), the scale gradient (Eq. 4) and the input
gradient (Eq. 3) on 2048 tokens.  The weights are quantized once before the timed region (the
paper's post-training step); its time, and the decode numbers, are reported as extra fields.

    python bench.py --gpus N --steps K --warmup W            # this library
    python bench.py --impl reference --gpus N --steps K ...  # the fp64 CPU oracle on a sample

With N > 1 (torchrun) every rank runs the same per-GPU workload on its own tokens (weak scaling)
and the scale gradients are all-reduced once per step.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "bcq_linear_fwd_bwd_tflops"
UNIT = "TFLOP/s"
WORKLOAD = "gpt2-medium-block x24, q=3 row-wise alpha, 2048 tokens, fwd+dalpha+dX"
LAYERS, TOKENS, Q = 24, 2048, 3
LINEARS = [("att_qkv", 1024, 3072), ("att_out", 1024, 1024), ("ffn_h_4h", 1024, 4096), ("ffn_4h_h", 4096, 1024)]
STEP_FLOPS = 3 * sum(2.0 * TOKENS * di * do for _, di, do in LINEARS) * LAYERS


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"tflops": float(p.get("bf16_tflops_sustained", p.get("bf16_tflops", 1400.0))),
                "hbm_gbs": float(p.get("hbm_gbs", 6650.0)), "source": "measured"}
    return {"tflops": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


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

def oracle_sample(steps, warmup):
    """Times the oracle, as it stands, on a bounded sample of the workload: one att_out linear
    (1024 -> 1024, q = 3, row-wise) with 256 of the 2048 tokens, forward + dalpha + dX."""
    import numpy as np
    import oracle
    from paper_2210_03858_b200 import synth
    n, d_in, d_out = 256, 1024, 1024
    key = (1, 0, 1)
    W = synth.weights(d_out, d_in, key)
    X = synth.activations(n, d_in, key, synth.ROLE_X)
    dY = synth.activations(n, d_out, key, synth.ROLE_DY)
    bits, alpha, _, _ = oracle.quantize(W, Q, d_in)
    flops = 3 * 2.0 * n * d_in * d_out

    def step():
        oracle.fwd(X, bits, alpha, d_in, d_in)
        oracle.bwd_alpha(dY, X, bits, d_in, d_in)
        oracle.bwd_x(dY, bits, alpha, d_in, d_in)

    for _ in range(max(0, warmup)):
        step()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    dt = (time.perf_counter() - t0) / steps
    return {"value": flops / dt / 1e12, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": "att_out 1024->1024, q=3 row-wise, 256 of 2048 tokens, fwd+dalpha+dX, fp64",
            "ms_per_step": dt * 1e3}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps = max(1, min(args.steps, 5))
    cb = oracle_sample(steps, min(args.warmup, 1))
    line = {"impl": "reference", "metric": METRIC, "value": cb["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": cb["ms_per_step"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": WORKLOAD, "sample": cb["sample"]},
            "cpu_baseline": {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": cb["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------ GPU arm

def run_gpu(args):
    import torch
    import torch.distributed as dist
    import paper_2210_03858_b200 as bcq
    from paper_2210_03858_b200 import build as bcq_build

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

    # ---- synthetic inputs (seeded per rank, layer, linear) and the one-off quantization
    layers = []
    gen = torch.Generator(device=dev)
    quant_ms = 0.0
    for layer in range(LAYERS):
        for li, (name, d_in, d_out) in enumerate(LINEARS):
            gen.manual_seed(221003858 + 1000003 * rank + 4099 * layer + li)
            W = torch.randn((d_out, d_in), generator=gen, device=dev, dtype=torch.float32) * 0.02
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            bits, alpha, _ = bcq.quantize(W, Q, d_in)
            e1.record()
            torch.cuda.synchronize()
            quant_ms += e0.elapsed_time(e1)
            del W
            X = torch.randn((TOKENS, d_in), generator=gen, device=dev, dtype=torch.float32).bfloat16()
            dY = torch.randn((TOKENS, d_out), generator=gen, device=dev, dtype=torch.float32).bfloat16()
            layers.append(dict(d_in=d_in, d_out=d_out, bits=bits, alpha=alpha, X=X, dY=dY,
                               dalpha=torch.zeros_like(alpha)))
    # outputs and workspaces: one set per shape, per operation and per chain, so that the operations
    # of a step can run on several streams at once
    chains = max(1, args.chains)
    for i, l in enumerate(layers):
        l["chain"] = i % chains
    bufs = {}
    out_dtype = torch.bfloat16 if args.out_bf16 else torch.float32
    for _, d_in, d_out in LINEARS:
        def ws(op):
            return torch.empty(max(16, bcq.workspace_bytes(op, d_out, d_in, Q, d_in, TOKENS)), dtype=torch.uint8, device=dev)
        for c in range(chains):
            bufs[(d_in, d_out, c)] = dict(Y=torch.empty((TOKENS, d_out), device=dev, dtype=out_dtype),
                                          dX=torch.empty((TOKENS, d_in), device=dev, dtype=out_dtype),
                                          ws_fwd=ws(bcq.OP_FWD), ws_dx=ws(bcq.OP_BWD_X), ws_da=ws(bcq.OP_BWD_ALPHA))
    flat_dalpha = torch.zeros(sum(l["dalpha"].numel() for l in layers), device=dev) if world > 1 else None

    def op_fwd(l):
        b = bufs[(l["d_in"], l["d_out"], l["chain"])]
        bcq.linear_fwd(l["X"], l["bits"], l["alpha"], l["d_in"], l["d_in"], out=b["Y"], ws=b["ws_fwd"])

    def op_da(l):
        b = bufs[(l["d_in"], l["d_out"], l["chain"])]
        bcq.linear_bwd_alpha(l["dY"], l["X"], l["bits"], l["d_in"], l["d_in"], out=l["dalpha"], ws=b["ws_da"])

    def op_dx(l):
        b = bufs[(l["d_in"], l["d_out"], l["chain"])]
        bcq.linear_bwd_x(l["dY"], l["bits"], l["alpha"], l["d_in"], l["d_in"], out=b["dX"], ws=b["ws_dx"])

    OPS = (("fwd", op_fwd), ("bwd_alpha", op_da), ("bwd_x", op_dx))

    def linear_step(l):
        for _, fn in OPS:
            fn(l)

    # one stream per (operation, chain); the dX chains are the longest, so theirs get the higher priority
    streams = {}
    for name, _ in OPS:
        for c in range(chains):
            streams[(name, c)] = torch.cuda.Stream(device=dev, priority=-1 if name == "bwd_x" else 0)

    def enqueue_step():
        # the linears are independent problems, and within one linear dalpha and dX only share their
        # inputs: forward, dalpha and dX of the linears of a chain are three queues on three streams
        cur = torch.cuda.current_stream()
        for s_ in streams.values():
            s_.wait_stream(cur)
        for name, fn in OPS:
            for c in range(chains):
                with torch.cuda.stream(streams[(name, c)]):
                    for l in layers:
                        if l["chain"] == c:
                            fn(l)
        for s_ in streams.values():
            cur.wait_stream(s_)

    # warm up outside capture (also resolves lazy CUDA state), then capture one step as a CUDA graph
    main = torch.cuda.Stream(device=dev)
    torch.cuda.synchronize()
    graph = None
    launches_per_step = 0
    with torch.cuda.stream(main):
        enqueue_step()
        torch.cuda.synchronize()
        c0 = bcq.kernel_launches()
        if args.graph:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=main):
                enqueue_step()
        else:
            enqueue_step()
        launches_per_step = bcq.kernel_launches() - c0
    torch.cuda.synchronize()
    torch.cuda.set_stream(main)

    def step():
        if graph is not None:
            graph.replay()
        else:
            enqueue_step()
        if world > 1:  # data parallel: the scale gradients are summed over ranks once per step
            torch.cat([l["dalpha"].reshape(-1) for l in layers], out=flat_dalpha)
            dist.all_reduce(flat_dalpha)

    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()  # nvidia-smi needs a moment to come up: start it before the warm-up
    for _ in range(max(3, args.warmup)):
        step()
    sync_all()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    sync_all()
    launches = launches_per_step * args.steps
    ms = torch.tensor([e0.elapsed_time(e1)], device=dev)
    if world > 1:
        dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    ms_per_step = float(ms.item()) / args.steps
    assert bcq.device_timeout_flag() == 0, "a kernel reported an expired wait"
    if args.timed_only:
        if rank == 0:
            sampler.stop()
            print(json.dumps({"metric": METRIC, "value": world * STEP_FLOPS / (ms_per_step * 1e-3) / 1e12, "unit": UNIT,
                              "n_gpus": world, "steps": args.steps, "ms_per_step": ms_per_step,
                              "gpu_launches": int(launches), "note": "timed steps only"}))
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- per-operation GPU time for the roofline: all 96 calls of one operation back to back on
    # one stream (captured as a graph so that host launch time stays out), CUDA-event timed
    per_op = {}
    for name, fn in OPS:
        g_ = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_, stream=main):
            for l in layers:
                fn(l)
        g_.replay()
        torch.cuda.synchronize()
        best = None
        for _ in range(3):
            a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            g_.replay()
            b_.record()
            torch.cuda.synchronize()
            best = a.elapsed_time(b_) if best is None else min(best, a.elapsed_time(b_))
        per_op[name] = (best, sum(2.0 * TOKENS * l["d_in"] * l["d_out"] for l in layers), len(layers))
        del g_

    # ---- end to end: inputs in pinned host memory, H2D every step, dalpha read back every step
    e2e = None
    if rank == 0 or world > 1:
        hX = [l["X"].cpu().pin_memory() for l in layers]
        hdY = [l["dY"].cpu().pin_memory() for l in layers]
        hdA = [torch.empty(l["dalpha"].shape, dtype=torch.float32).pin_memory() for l in layers]
        h2d = sum(t.numel() * 2 for t in hX) + sum(t.numel() * 2 for t in hdY)
        d2h = sum(t.numel() * 4 for t in hdA)
        e2e_steps = max(1, min(args.steps, 3))

        # the copies run on streams of their own, so that the inputs of the next linear arrive and the
        # result of the previous one leaves while the current one computes
        h2d_s, d2h_s = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)

        def e2e_step():
            cur = torch.cuda.current_stream()
            h2d_s.wait_stream(cur)  # the previous step's kernels have read the inputs about to be overwritten
            for i, l in enumerate(layers):
                with torch.cuda.stream(h2d_s):
                    l["X"].copy_(hX[i], non_blocking=True)
                    l["dY"].copy_(hdY[i], non_blocking=True)
                    arrived = torch.cuda.Event()
                    arrived.record(h2d_s)
                cur.wait_event(arrived)
                linear_step(l)
                computed = torch.cuda.Event()
                computed.record(cur)
                with torch.cuda.stream(d2h_s):
                    d2h_s.wait_event(computed)
                    hdA[i].copy_(l["dalpha"], non_blocking=True)
            cur.wait_stream(h2d_s)
            cur.wait_stream(d2h_s)
        e2e_step()
        sync_all()
        a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(e2e_steps):
            e2e_step()
        b_.record()
        sync_all()
        t = torch.tensor([a.elapsed_time(b_)], device=dev)
        if world > 1:
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e = {"value": world * STEP_FLOPS / (float(t.item()) / e2e_steps * 1e-3) / 1e12, "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
               "note": "X and dY copied from pinned host memory and dalpha copied back, every linear, every step; "
                       "copies on their own streams overlap the kernels of the neighbouring linears"}

    clocks = sampler.stop() if rank == 0 else None
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    # the expansion GEMM (forward and dX calls) is where most of the step goes
    t_exp = per_op["fwd"][0] + per_op["bwd_x"][0]
    f_exp = per_op["fwd"][1] + per_op["bwd_x"][1]
    n_exp = per_op["fwd"][2] + per_op["bwd_x"][2]
    achieved = f_exp / (t_exp * 1e-3) / 1e12
    roofline = {"bound": "tensor", "kernel": "expand_gemm_kernel (bcq_linear_fwd / bcq_linear_bwd_x calls, fp16 pre-pass included)",
                "achieved": achieved, "peak": peaks["tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["tflops"],
                "peak_source": "of %s (sustained bf16/fp16 dense)" % peaks["source"], "traffic": None,
                "flops_per_launch": f_exp / n_exp, "avg_launch_ms": t_exp / n_exp,
                "per_op_tflops": {k: v[1] / (v[0] * 1e-3) / 1e12 for k, v in per_op.items()},
                "per_op_share": {k: v[0] / sum(x[0] for x in per_op.values()) for k, v in per_op.items()}}

    cb = oracle_sample(3, 1)
    cpu_baseline = {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")}

    extra = decode_numbers(bcq, torch, dev, peaks) if args.decode else None
    value = world * STEP_FLOPS / (ms_per_step * 1e-3) / 1e12
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "layers": LAYERS, "tokens_per_gpu": TOKENS, "q": Q, "g": "d_in",
                       "l2": "a step touches ~1.5 GB of distinct inputs, far more than the 126 MB L2",
                       "outputs": "bf16" if args.out_bf16 else "fp32",
                       "launch": ("one CUDA graph per step, " if args.graph else "") + "forward / dalpha / dX on %d streams (dX at high priority)" % (3 * chains),
                       "parallelism": "dp%d" % world, "quantize_ms_once": quant_ms},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
            "cpu_baseline": cpu_baseline}
    if extra is not None:
        line["decode"] = extra
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def decode_numbers(bcq, torch, dev, peaks):
    """Decode GEMV of OPT-6.7B-shaped linears (q = 4, g = 128), rotating over enough distinct
    layers that the planes come from HBM; GB/s on the algorithmic bytes."""
    out = {}
    q, g = 4, 128
    for name, d_in, d_out in (("att_qkv", 4096, 12288), ("ffn_h_4h", 4096, 16384), ("ffn_4h_h", 16384, 4096)):
        per = bcq.bits_bytes(d_out, d_in, q) + bcq.alpha_count(d_out, d_in, q, g) * 4
        L = int(0.6e9 // per) + 1
        gen = torch.Generator(device=dev)
        gen.manual_seed(7 + d_in + d_out)
        bits = [torch.randint(-2 ** 31, 2 ** 31 - 1, (q, d_out, bcq.pitch_words(d_in)), generator=gen,
                              dtype=torch.int32, device=dev) for _ in range(L)]
        alphas = [torch.rand((q, d_out, d_in // g), generator=gen, device=dev) * 0.02 for _ in range(L)]
        for n in (1, 16):
            X = torch.randn((n, d_in), generator=gen, device=dev).bfloat16()
            Y = torch.empty((n, d_out), device=dev)
            ws = torch.empty(max(16, bcq.workspace_bytes(bcq.OP_DECODE, d_out, d_in, q, g, n)), dtype=torch.uint8, device=dev)
            for _ in range(2):
                for l in range(L):
                    bcq.linear_decode(X, bits[l], alphas[l], d_in, g, out=Y, ws=ws)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for l in range(L):
                bcq.linear_decode(X, bits[l], alphas[l], d_in, g, out=Y, ws=ws)
            e1.record()
            torch.cuda.synchronize()
            us = e0.elapsed_time(e1) * 1e3 / L
            byt = per + 2 * n * d_in + 4 * n * d_out
            gbs = byt / us / 1e3
            out["%s_n%d" % (name, n)] = {"us": us, "GB/s": gbs, "frac_of_hbm": gbs / peaks["hbm_gbs"]}
        del bits, alphas
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=("ours", "reference"))
    ap.add_argument("--no-decode", dest="decode", action="store_false")
    ap.add_argument("--no-graph", dest="graph", action="store_false", help="launch every kernel from the host each step")
    ap.add_argument("--out-fp32", dest="out_bf16", action="store_false", help="fp32 Y and dX instead of bf16")
    ap.add_argument("--chains", type=int, default=3,
                    help="independent chains per operation: the linears of a step are dealt round-robin to this many "
                         "streams (each with its own outputs and workspaces) for each of forward, dalpha and dX")
    ap.add_argument("--timed-only", action="store_true",
                    help="warm-up and timed steps only (no per-operation, end-to-end, CPU or decode legs): the command to profile")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
