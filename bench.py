#!/usr/bin/env python
"""Benchmark of the MoE expert step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--no-study]

Headline workload (N = 1): the Mixtral-8x7B-shaped single-layer decode configuration -- d_model 4096,
8 experts, top-2, SwiGLU d_ff 14336, bf16 weights, batch of 16 tokens, router logits drawn from a
Zipf(1.1) expert popularity, every expert resident in the HBM slot cache.  A step is one pass of the
whole path through the library's single call saem_moe_step (gate -> repack -> expert FFN -> merge).
The layer's weights (2.8 GB) are far larger than L2, so consecutive steps cannot reuse them from cache.

Prints one JSON line (rank 0): the headline value, its spread over ten blocks of steps, the roofline
of the expert FFN, the end-to-end figure from host buffers, a CPU-oracle baseline, and (N = 1) a
`study` list with the same measurements on the other configurations (fine-grained layer at 32 and
2048 tokens, Qwen-MoE-shaped layer at 1 / 8 / 64 tokens under skewed and uniform routing, the
Qwen3-shaped layer at 1 / 8 tokens, a 64-step slice of the partially resident 32-layer stack).
N > 1 runs N independent replicas, one per GPU (the path has no exchange step), and reports the
aggregate.  `--impl reference` times the CPU oracle instead.

Other modes (one JSON line each): `--workload W [--tokens T] [--routing R]` times one configuration
as the headline; `--segments` sweeps the expert FFN over segment sizes of one expert; `--segment-classes`
splits a prefill call's time by segment-size class.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "MoE-layer decode tokens/sec"
UNIT = "tokens/s"
WORKLOADS = {
    "c2": "c2: Mixtral-8x7B-shaped layer decode, d_model=4096, 8 experts top-2, d_ff=14336",
    "c3": "c3: fine-grained layer, d_model=2048, 64 experts top-6 + 2 shared, d_ff=1408",
    "c4": "c4: Qwen-MoE-shaped layer, d_model=2048, 60 experts top-4 + shared d_ff=5632, routed d_ff=1408",
    "qwen3": "Qwen3-30B-A3B-shaped layer, d_model=2048, 128 experts top-8, d_ff=768",
    "ernie": "ERNIE-4.5-21B-A3B-shaped layer, d_model=2560, 64 experts top-6 + 2 shared, d_ff=1536",
}
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
# DRAM bytes (read + write) of the two expert-FFN kernels of one step of workload c2 at 16 tokens with all
# 8 experts active, from an ncu capture (not measured by this run)
NCU_FFN_TRAFFIC = {("c2", 16): (2831072592, "profiles/ffn_prefill_c2_decode.md (ncu capture, dram__bytes_read.sum + dram__bytes_write.sum)")}
STUDY = [("c3", 32, None), ("c3", 2048, None), ("c4", 1, None), ("c4", 8, None), ("c4", 64, None), ("c4", 8, "uniform"),
         ("c4", 64, "uniform"), ("qwen3", 1, None), ("qwen3", 8, None)]


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as fh:
            return json.load(fh), "measured"
    except Exception:
        return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": FALLBACK_BF16_TFLOPS}, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed regions run."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.t0 = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t0 = time.perf_counter()
        except Exception:
            self.proc = None

    def alive_s(self):
        return 0.0 if self.t0 is None else time.perf_counter() - self.t0

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
                pw.append(float(parts[2]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        # samples taken while the GPU was drawing power under load describe the timed regions best
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "power_w_max": max(pw) if pw else None, "reasons": sorted(reasons)}


def max_over_ranks(values, device):
    """Element-wise maximum of `values` over all ranks (identity when not distributed): the
    time of a multi-replica run is the slowest replica's."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(values, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def aggregate_tokens_per_s(world, tokens_per_step, steps, slowest_ms):
    """Whole-job throughput of `world` independent replicas timed by the slowest one."""
    return world * tokens_per_step * steps / (slowest_ms * 1e-3)


def percentile(v, q):
    s = sorted(v)
    if not s:
        return None
    pos = (len(s) - 1) * q
    lo, hi = int(np.floor(pos)), int(np.ceil(pos))
    return s[lo] + (s[hi] - s[lo]) * (pos - lo)


def cpu_model():
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("model name"):
                return line.split(":", 1)[1].strip()
    except Exception:
        pass
    return "unknown"


def workload_name(name, cfg):
    return "%s, %d token%s per step, %s routing" % (WORKLOADS[name], cfg.tokens, "" if cfg.tokens == 1 else "s", cfg.routing)


# ------------------------------------------------------------------------------- one configuration
class LayerBench:
    """One layer configuration resident on the GPU, with a few routing draws of the same stage."""

    def __init__(self, name, tokens, routing, distinct, device, ffn_path=0):
        import torch
        from paper_2608_21614_b200 import inputs as gen
        from paper_2608_21614_b200.layer import MoELayer
        self.torch, self.name, self.device = torch, name, device
        self.cfg = cfg = gen.layer_config(name, tokens=tokens, routing=routing)
        self.li = li = gen.layer_inputs(cfg, n_distinct_experts=distinct)
        T, E = cfg.tokens, cfg.n_experts
        self.layer = MoELayer(cfg.d_model, cfg.d_ff, E, cfg.top_k, T, cfg.d_ff_shared, device=device, ffn_path=ffn_path)
        self.layer.load_all(li.gate, li.up, li.down, li.shared)
        self.layer.drop_host_copies()
        # The headline workload streams 2.8 GB of weights per step from one routing draw.  Smaller layers
        # rotate over eight routing draws of the same stage (different active experts step to step, as
        # consecutive tokens would), so that a step cannot find its weights in L2.
        self.n_draws = 1 if (name == "c2" and T <= 64) else 8
        rng = np.random.default_rng(np.random.SeedSequence([cfg.seed, 4242]))
        pop = gen.zipf_popularity(li.ranking, cfg.zipf_s) if cfg.routing == "zipf" else None
        draws = [li.logits] + [gen.router_logits(rng, T, E, cfg.routing, pop) for _ in range(self.n_draws - 1)]
        self.logits = [torch.from_numpy(lg).to(device) for lg in draws]
        self.x = torch.from_numpy(li.x).to(device)
        self.out = torch.empty((T, cfg.d_model), dtype=torch.float32, device=device)
        self.active = []
        for lg in self.logits:                          # active experts of every draw (and first-call set-up)
            self.layer.step(lg, self.x, T)
            torch.cuda.synchronize()
            self.active.append(int((self.layer.counts.cpu().numpy()[:E] > 0).sum()))
        for lg in self.logits:
            self.layer.step_fused_call(lg, self.x, T, self.out)
        torch.cuda.synchronize()
        self.weight_bytes = 3 * cfg.d_model * cfg.d_ff * 2
        self.shared_bytes = 3 * cfg.d_model * cfg.d_ff_shared * 2
        self.graph = None

    def step(self, i):
        self.layer.step_fused_call(self.logits[i % self.n_draws], self.x, self.cfg.tokens, self.out)

    def capture(self):
        """All routing draws' steps recorded once as ONE CUDA graph (as a decoder records all its layers)."""
        torch = self.torch
        side = torch.cuda.Stream(device=self.device)
        side.wait_stream(torch.cuda.current_stream(self.device))
        with torch.cuda.stream(side):
            for i in range(self.n_draws):
                self.step(i)
            side.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                for i in range(self.n_draws):
                    self.step(i)
        torch.cuda.current_stream(self.device).wait_stream(side)
        self.graph = graph

    def run_steps(self, k):
        """Enqueues k steps (k a multiple of n_draws when replaying the graph)."""
        if self.graph is not None:
            for _ in range(k // self.n_draws):
                self.graph.replay()
        else:
            for i in range(k):
                self.step(i)

    def timed_steps(self, k):
        torch = self.torch
        stream = torch.cuda.current_stream(self.device)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        self.run_steps(k)
        b.record(stream)
        return a, b

    def mean_active_bytes(self):
        return sum(self.active) / len(self.active) * self.weight_bytes + self.shared_bytes

    def ffn_pass(self, k):
        """k steps through the four separate calls with CUDA events around the expert-FFN call(s):
        the dominant kernels' duration for the roofline.  Returns per-step FFN milliseconds."""
        torch, layer, T = self.torch, self.layer, self.cfg.tokens
        stream = torch.cuda.current_stream(self.device)
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(k)]
        for i in range(k):
            layer.route(self.logits[i % self.n_draws], T)
            layer.repack(self.x, T)
            ev[i][0].record(stream)
            layer.expert_ffn(T)
            if layer.shared is not None:
                layer.shared_ffn(self.x, T)
            ev[i][1].record(stream)
            layer.combine(T)
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in ev]

    def ffn_back_to_back(self, k):
        """The expert-FFN call(s) of the last routing issued k times back to back (each call's set-up overlaps the
        previous call's tail, as it overlaps the repack's inside a graph-replayed step): milliseconds per call."""
        torch, layer, T = self.torch, self.layer, self.cfg.tokens
        stream = torch.cuda.current_stream(self.device)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(k):
            layer.expert_ffn(T)
            if layer.shared is not None:
                layer.shared_ffn(self.x, T)
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / k

    def close(self):
        self.layer.close()
        self.graph = None
        self.logits = self.x = self.out = None
        self.torch.cuda.empty_cache()


def roofline_of(lb, step_ms, ffn_ms, peaks, which):
    """Roofline of the dominant kernel(s).  Decode-sized batches: expert-weight bytes of the experts with rows
    (each read once) over the expert-FFN call's time, against the measured copy bandwidth.  Prefill-sized
    batches (more than 64 tokens): the call's flops against the measured bf16 tensor peak.  The one-launch
    decode step has no separate FFN call: its weight bytes are set against the WHOLE step's time."""
    cfg = lb.cfg
    T, d, f = cfg.tokens, cfg.d_model, cfg.d_ff
    if T > 64:
        flops = 6.0 * T * d * (cfg.top_k * f + cfg.d_ff_shared)
        achieved = flops / (ffn_ms * 1e-3) / 1e12
        peak = float(peaks.get("bf16_tflops", FALLBACK_BF16_TFLOPS))
        roof = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                "traffic": None, "algorithmic_flops": flops, "avg_ms": ffn_ms,
                "frac_of_sustained": achieved / float(peaks.get("bf16_tflops_sustained", 1400.0)),
                "kernel": "saem_expert_ffn (ffn_prefill_kernel<0/1>: tiled tcgen05 gate/up + down)"}
    else:
        n0 = lb.layer.launches()                 # does saem_moe_step take its one-launch form here?  Count its launches
        lb.step(0)
        single = T <= 8 and lb.layer.launches() - n0 <= 2
        ms = step_ms if single else ffn_ms
        nbytes = lb.mean_active_bytes()
        achieved = nbytes / (ms * 1e-3) / 1e9
        peak = float(peaks["hbm_gbs"])
        traffic = NCU_FFN_TRAFFIC.get((lb.name, T)) if all(a == cfg.n_experts for a in lb.active) else None
        roof = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": traffic[0] if traffic else None, "traffic_source": traffic[1] if traffic else None,
                "algorithmic_bytes": nbytes, "avg_ms": ms, "frac_of_nominal_8000": achieved / 8000.0,
                "kernel": "decode_step_kernel (whole step: gate, repack indices, gate/up, down, merge in one launch)" if single
                else "saem_expert_ffn (%s gate/up + down kernels%s)" % (
                    "ffn_gemv_kernel<0/1>: matrix-vector" if T <= 8 else "ffn_prefill_kernel<0/1>: tiled tcgen05",
                    ", second call for the shared expert" if lb.layer.shared is not None else "")}
    roof["peak_source"] = which
    return roof


def study_row(name, tokens, routing, distinct, device, peaks, which, min_block_ms=30.0):
    """One study configuration: ten blocks of graph-replayed steps (median, p10, p90) and the roofline."""
    import torch
    lb = LayerBench(name, tokens, routing, distinct, device)
    cfg = lb.cfg
    if cfg.tokens <= 64:
        lb.capture()
    lb.run_steps(lb.n_draws * 3)
    torch.cuda.synchronize()
    a, b = lb.timed_steps(lb.n_draws * 2)
    torch.cuda.synchronize()
    est = a.elapsed_time(b) / (lb.n_draws * 2)
    k = max(lb.n_draws, int(min_block_ms / est) // lb.n_draws * lb.n_draws)
    blocks = []
    for _ in range(10):
        a, b = lb.timed_steps(k)
        torch.cuda.synchronize()
        blocks.append(a.elapsed_time(b) / k)
    n_ffn = max(lb.n_draws * 4, 24)
    ffn = lb.ffn_pass(n_ffn)
    bb_ms = lb.ffn_back_to_back(n_ffn)
    med = statistics.median(blocks)
    ffn_ms = statistics.median(ffn)
    row = {"workload": workload_name(name, cfg), "tokens_per_step": cfg.tokens, "value": cfg.tokens / (med * 1e-3), "unit": UNIT,
           "ms_per_step": {"median": med, "p10": percentile(blocks, 0.1), "p90": percentile(blocks, 0.9),
                           "blocks": len(blocks), "steps_per_block": k},
           "active_experts": sum(lb.active) / len(lb.active), "routing_draws": lb.n_draws,
           "launch": "CUDA-graph replay of the draws' steps" if lb.graph is not None else "one host call per step",
           "gpu_launches_per_step": None, "roofline": roofline_of(lb, med, ffn_ms, peaks, which),
           "device_status": lb.layer.device_status()}
    roof = row["roofline"]
    if "decode_step_kernel" not in roof["kernel"]:
        if roof["bound"] == "hbm":      # bytes of the draw that call ran on (the last one of the instrumented pass)
            bb = (lb.active[(n_ffn - 1) % lb.n_draws] * lb.weight_bytes + lb.shared_bytes) / (bb_ms * 1e-3) / 1e9
        else:
            bb = roof["achieved"] * ffn_ms / bb_ms
        roof["back_to_back"] = {"avg_ms": bb_ms, "achieved": bb, "frac": bb / roof["peak"],
                                "note": "the same saem_expert_ffn call issued back to back on one routing draw"}
    n0 = lb.layer.launches()
    lb.step(0)
    row["gpu_launches_per_step"] = lb.layer.launches() - n0
    lb.close()
    return row


def stack_slice(steps, device):
    """A slice of the fifth configuration: 32 Mixtral-shaped layers, 4 of 8 experts per layer resident (+ 4
    temporary slots), the first `steps` steps of the 4096-step stage trace at batch 1; misses are copied
    from pinned host memory on a side stream.  Bound by the host link."""
    import torch
    from paper_2608_21614_b200 import inputs as gen
    from paper_2608_21614_b200.stack import StackRunner
    cfg = gen.layer_config("c5")
    L, E, k, d, f, C = 32, cfg.n_experts, cfg.top_k, cfg.d_model, cfg.d_ff, 4
    trace = gen.stage_trace(4096, L, E, cfg.zipf_s, 0)
    rng = np.random.default_rng(np.random.SeedSequence([0, 77]))
    weights = [gen.expert_weights(rng, d, f) for _ in range(4)]
    run = StackRunner(d, f, E, k, L, C, 4, 1, weights, device=device)
    run.warm([list(np.argsort(trace.rankings[0, l])[:C]) for l in range(L)])
    run.copy.synchronize()
    bounds = set(int(b) for b in trace.boundaries[1:])
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for t in range(steps):
        if t in bounds:
            run.boundary()
        lg = np.stack([gen.trace_logits(trace, t, l, 1) for l in range(L)])
        x = gen.trace_activations(trace, t, 1, d)
        run.step(torch.from_numpy(lg).to(device, non_blocking=True), torch.from_numpy(x).to(device, non_blocking=True), keep_out=False)
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    from paper_2608_21614_b200 import binding as B
    st = run.stats
    row = {"workload": "c5 slice: Mixtral-8x7B-shaped 32-layer stack decode, batch 1, cache 50 %% of the experts per layer, "
                       "first %d steps of the 4096-step stage trace" % steps,
           "tokens_per_step": 1, "value": steps / dt, "unit": UNIT, "ms_per_step": {"median": dt / steps * 1e3, "blocks": 1, "steps_per_block": steps},
           "chr_distinct": st.chr(), "demand_loads": st.demand_loads, "boundary_loads": st.boundary_loads,
           "roofline": {"bound": "host link", "achieved": run.h2d_bytes() / dt / 1e9, "unit": "GB/s", "peak": None, "frac": None,
                        "algorithmic_bytes": run.h2d_bytes() / max(steps, 1),
                        "note": "bytes of missed experts copied host -> HBM per wall-clock second; 32 layer-steps of weight streaming ride on top"},
           "gpu_launches_per_step": B.saem_launch_count(run.h) / max(steps, 1), "device_status": B.saem_last_device_status(run.h)}
    run.close()
    del run
    torch.cuda.empty_cache()
    return row


# ----------------------------------------------------------------------------------------- ours
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2608_21614_b200 import binding as B          # raises if the CUDA library is missing

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    device = "cuda:%d" % local
    peaks, which = measured_peaks()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()                                  # before warm-up: samples cover every timed region
    lb = LayerBench(args.workload, args.tokens, args.routing, args.distinct, device,
                    ffn_path={"auto": 0, "tensor": 2}[args.ffn_path])
    cfg = lb.cfg
    T, E, d = cfg.tokens, cfg.n_experts, cfg.d_model
    if args.graph:
        lb.capture()
    K = args.steps if not args.graph else max(lb.n_draws, args.steps // lb.n_draws * lb.n_draws)
    W = max(args.warmup, 3)
    lb.run_steps(W if not args.graph else max(lb.n_draws, W // lb.n_draws * lb.n_draws))
    torch.cuda.synchronize()

    # timed region 1: exactly K steps, nothing between the kernels of a step -> the headline value
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    launches0 = lb.layer.launches()
    ev0, ev1 = lb.timed_steps(K)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    total_ms = ev0.elapsed_time(ev1)
    if args.graph:
        n0 = lb.layer.launches()
        lb.step(0)
        launches = (lb.layer.launches() - n0) * K
        torch.cuda.synchronize()
    else:
        launches = lb.layer.launches() - launches0
    # spread: ten blocks of steps, each long enough (about 0.1 s) that the clock sampler sees the GPU under load
    kb = max(K, int(100.0 / (total_ms / K)))
    if args.graph:
        kb = max(lb.n_draws, kb // lb.n_draws * lb.n_draws)
    blocks = []
    for _ in range(10):
        a, b = lb.timed_steps(kb)
        torch.cuda.synchronize()
        blocks.append(a.elapsed_time(b) / kb)
    # timed region 2: steps with CUDA events around the saem_expert_ffn call(s) -> the dominant kernels' duration
    ffn_ms = lb.ffn_pass(max(K, 24))
    # the same call issued back to back on the last routing (its set-up overlaps the previous call's tail)
    ffn_bb_ms = lb.ffn_back_to_back(min(max(K, 24), 200))
    status = lb.layer.device_status()

    # end to end through the host-buffer call: H2D of logits and x, the kernels, D2H of out
    lh = torch.from_numpy(lb.li.logits).pin_memory()
    xh = torch.from_numpy(lb.li.x).pin_memory()
    oh = torch.empty((T, d), dtype=torch.float32).pin_memory()
    for _ in range(3):
        lb.layer.step_host(lh, xh, T, oh)
    Ks = max(K // 4, 10)                                 # one synchronous call at a time: the latency of a step
    t0 = time.perf_counter()
    for _ in range(Ks):
        lb.layer.step_host(lh, xh, T, oh)
    e2e_sync_s = (time.perf_counter() - t0) / Ks
    # throughput: the asynchronous form of the same call, every step with its own copies in and its own copy out (four
    # pinned result buffers in rotation), the stream synchronised once at the end of the timed region
    ohs = [torch.empty((T, d), dtype=torch.float32).pin_memory() for _ in range(4)]
    for i in range(4):
        lb.layer.step_host_async(lh, xh, T, ohs[i])
    torch.cuda.synchronize()
    Ke = max(K, 20)
    t0 = time.perf_counter()
    for i in range(Ke):
        lb.layer.step_host_async(lh, xh, T, ohs[i % 4])
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    if rank == 0:
        while sampler.alive_s() < 1.5:                   # keep the GPU under load until the sampler has something to show
            lb.run_steps(kb)
            torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None

    total_ms, e2e_step_s = max_over_ranks([total_ms, e2e_s / Ke], device)
    line = None
    if rank == 0:
        ffn_med = statistics.median(ffn_ms)
        roof = roofline_of(lb, total_ms / K, ffn_med, peaks, which)
        last_active = lb.active[(max(K, 24) - 1) % lb.n_draws]
        if roof["bound"] == "hbm":
            bb = (last_active * lb.weight_bytes + lb.shared_bytes) / (ffn_bb_ms * 1e-3) / 1e9
        else:
            bb = roof["achieved"] * ffn_med / ffn_bb_ms
        roof["back_to_back"] = {"avg_ms": ffn_bb_ms, "achieved": bb, "frac": bb / roof["peak"],
                                "note": "the same saem_expert_ffn call issued back to back on one routing draw"}
        roof.update({"routing_draws": lb.n_draws, "ffn_ms": {"median": ffn_med, "p10": percentile(ffn_ms, 0.1),
                                                             "p90": percentile(ffn_ms, 0.9), "calls": len(ffn_ms)}})
        weight_gb = (E * lb.weight_bytes + lb.shared_bytes) / 1e9
        line = {
            "metric": METRIC, "value": aggregate_tokens_per_s(world, T, K, total_ms), "unit": UNIT, "n_gpus": world,
            "steps": K, "warmup": W, "ms_per_step": total_ms / K, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": workload_name(args.workload, cfg), "tokens_per_step": T,
                       "active_experts": sum(lb.active) / len(lb.active),
                       "routing": "%s popularity + Gumbel, seed 0" % cfg.routing, "cache": "all experts resident in HBM",
                       "l2": "layer weights %.2f GB vs 126 MB L2: inputs larger than L2, no flush" % weight_gb,
                       "distinct_weight_sets": args.distinct, "replicas": world,
                       "ffn_path": args.ffn_path,
                       "launch": "CUDA-graph replay of the draws' steps" if args.graph else "one saem_moe_step call per step",
                       "timing": "value: K steps back to back; spread: ten more blocks; roofline: steps with events around the FFN call"},
            "spread": {"median_ms": statistics.median(blocks), "p10_ms": percentile(blocks, 0.1), "p90_ms": percentile(blocks, 0.9),
                       "blocks": len(blocks), "steps_per_block": kb},
            "roofline": roof,
            "e2e": {"value": world * T / e2e_step_s, "unit": UNIT, "h2d_bytes_per_step": T * E * 4 + T * d * 2,
                    "d2h_bytes_per_step": T * d * 4, "ms_per_step": e2e_step_s * 1e3,
                    "call": "saem_moe_step_host_async per step (copies in, kernels, copy out on one stream; pinned host "
                            "buffers, four result buffers in rotation), one synchronisation at the end",
                    "synchronous_call_ms": e2e_sync_s * 1e3},
            "gpu_launches": launches, "clocks": clocks, "device_status": status,
        }
    li, cfg0 = lb.li, lb.cfg
    lb.close()
    if rank == 0:
        if not args.no_study and world == 1 and args.workload == "c2" and args.tokens is None:
            study = []
            for name, tokens, routing in STUDY:
                study.append(study_row(name, tokens, routing, min(args.distinct, 4), device, peaks, which))
            study.append(stack_slice(64, device))
            line["study"] = study
        if not args.no_cpu and world == 1:
            line["cpu_baseline"] = cpu_baseline(li, cfg0, budget_s=12.0)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# -------------------------------------------------------------------------- segment-size studies
def run_segments(args):
    """Expert-FFN throughput by segment size: one expert, one segment of N rows, N from decode-sized to
    prefill-sized; the expert sits in several slots used in rotation so that small N stream from HBM."""
    import torch
    from paper_2608_21614_b200 import binding as B
    from paper_2608_21614_b200 import inputs as gen
    d, f, copies = args.d_model, args.d_ff, args.copies
    rng = np.random.default_rng(0)
    w = gen.expert_weights(rng, d, f)
    peaks, which = measured_peaks()
    rows = []
    for n in [int(s) for s in args.sizes.split(",")]:
        cfg = B.make_config(d, f, 1, 1, n, n_layers=copies, slots_per_layer=1)
        ctx = B.Context(cfg)
        packed = ctx.pack(*w)
        for layer in range(copies):
            B.saem_cache_load(ctx.handle, layer, 0, 0, packed)
        x = torch.from_numpy(gen.activations(rng, n, d)).cuda()
        y = torch.empty((n, d), dtype=torch.float32, device="cuda")
        for i in range(copies):
            B.saem_expert_ffn(ctx.handle, i, x, None, n, None, y)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        steps = min(args.steps, 40)
        a.record()
        for i in range(steps):
            B.saem_expert_ffn(ctx.handle, i % copies, x, None, n, None, y)
        b.record()
        torch.cuda.synchronize()
        us = a.elapsed_time(b) / steps * 1e3
        rows.append({"rows": n, "us": us, "weight_gbs": 3 * d * f * 2 / us / 1e3, "tflops": 6.0 * n * d * f / us / 1e6,
                     "status": B.saem_last_device_status(ctx.handle)})
        ctx.close()
    print(json.dumps({"mode": "segments", "d_model": d, "d_ff": f, "copies": copies, "peak_source": which,
                      "peaks": {k: peaks.get(k) for k in ("hbm_gbs", "bf16_tflops", "bf16_tflops_sustained")}, "rows": rows}))


def run_segment_classes(args):
    """Where a prefill-sized expert-FFN call spends its time: saem_expert_ffn restricted (expert_subset) to the
    experts whose segments fall in a size class.  The classes do not add up to the whole call."""
    import torch
    from paper_2608_21614_b200 import inputs as gen
    from paper_2608_21614_b200.layer import MoELayer
    cfg = gen.layer_config(args.workload, tokens=args.tokens or 2048)
    li = gen.layer_inputs(cfg, n_distinct_experts=min(args.distinct, 4))
    T = cfg.tokens
    layer = MoELayer(cfg.d_model, cfg.d_ff, cfg.n_experts, cfg.top_k, T, cfg.d_ff_shared)
    layer.load_all(li.gate, li.up, li.down, li.shared)
    layer.route(torch.from_numpy(li.logits).cuda(), T)
    layer.repack(torch.from_numpy(li.x).cuda(), T)
    torch.cuda.synchronize()
    counts = layer.counts.cpu().numpy()
    ids = np.arange(len(counts))

    def timeit(subset, name):
        for _ in range(3):
            layer.expert_ffn(T, 0, subset)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(20):
            layer.expert_ffn(T, 0, subset)
        b.record()
        torch.cuda.synchronize()
        us = a.elapsed_time(b) / 20 * 1e3
        rows = int(counts.sum()) if subset is None else int(counts[subset].sum())
        ne = len(counts) if subset is None else len(subset)
        return {"class": name, "experts": ne, "rows": rows, "us": us, "tflops": 6.0 * rows * cfg.d_model * cfg.d_ff / us / 1e6,
                "weight_gbs": ne * 3 * cfg.d_model * cfg.d_ff * 2 / us / 1e3}

    out = [timeit(None, "all"), timeit([int(e) for e in ids if counts[e] > 256], "more than 256 rows"),
           timeit([int(e) for e in ids if 64 < counts[e] <= 256], "65..256 rows"),
           timeit([int(e) for e in ids if 0 < counts[e] <= 64], "at most 64 rows")]
    print(json.dumps({"mode": "segment-classes", "workload": workload_name(args.workload, cfg),
                      "segments_sorted": sorted(counts.tolist(), reverse=True), "classes": out,
                      "device_status": layer.device_status()}))
    layer.close()


# -------------------------------------------------------------------------------------- oracle
def oracle_tokens_per_s(li, cfg, n_tokens, reps=1):
    """Times the CPU oracle's whole step on the first n_tokens tokens of the workload."""
    from oracle import saem_oracle
    lg, x = li.logits[:n_tokens], li.x[:n_tokens]
    t0 = time.perf_counter()
    for _ in range(reps):
        saem_oracle.moe_step(lg, x, cfg.top_k, li.gate, li.up, li.down, shared=li.shared)
    return n_tokens * reps / (time.perf_counter() - t0)


def one_thread_tokens_per_s(cfg_name):
    """The oracle restricted to one thread (OMP_NUM_THREADS=1 in a child process), one token of the workload."""
    code = ("import sys, json; sys.path.insert(0, %r); import bench; from paper_2608_21614_b200 import inputs as gen;"
            "from oracle import saem_oracle; saem_oracle.build(); cfg = gen.layer_config(%r);"
            "li = gen.layer_inputs(cfg, n_distinct_experts=2); bench.oracle_tokens_per_s(li, cfg, 1);"
            "print(json.dumps(bench.oracle_tokens_per_s(li, cfg, 1, reps=2)))") % (ROOT, cfg_name)
    try:
        env = dict(os.environ, OMP_NUM_THREADS="1")
        out = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=180)
        return float(out.stdout.strip().splitlines()[-1])
    except Exception:
        return None


def cpu_baseline(li, cfg, budget_s):
    """The oracle as it stands on the host cores: whole-step passes over the workload's tokens
    until about `budget_s` seconds of CPU work have been timed."""
    from oracle import saem_oracle
    saem_oracle.build()
    one = oracle_tokens_per_s(li, cfg, 1)                      # warms the pages; sizes the sample
    n = int(max(1, min(cfg.tokens, budget_s * one)))
    t0 = time.perf_counter()
    passes = 0
    while True:
        saem_oracle.moe_step(li.logits[:n], li.x[:n], cfg.top_k, li.gate, li.up, li.down, shared=li.shared)
        passes += 1
        dt = time.perf_counter() - t0
        if dt >= budget_s or passes >= 200:
            break
    return {"value": n * passes / dt, "unit": UNIT, "cores": saem_oracle.max_threads(), "kind": "oracle",
            "cpu": cpu_model(), "one_thread_value": one_thread_tokens_per_s(cfg.name) if cfg.name in ("c1", "c2") else None,
            "sample": "the first %d of the step's %d tokens, whole path, %d passes in %.1f s" % (n, cfg.tokens, passes, dt)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import saem_oracle
    from paper_2608_21614_b200 import inputs as gen
    saem_oracle.build()
    cfg = gen.layer_config(args.workload, tokens=args.tokens, routing=args.routing)
    li = gen.layer_inputs(cfg, n_distinct_experts=args.distinct)
    one = oracle_tokens_per_s(li, cfg, 1)
    total_steps = args.steps + args.warmup
    per_step_budget = 150.0 / max(total_steps, 1)
    n = int(max(1, min(cfg.tokens, per_step_budget * one)))
    for _ in range(args.warmup):
        oracle_tokens_per_s(li, cfg, n)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_tokens_per_s(li, cfg, n)
    dt = time.perf_counter() - t0
    v = n * args.steps / dt
    sample = "each step = the first %d of the workload's %d tokens, whole path" % (n, cfg.tokens)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(args.workload, cfg), "tokens_per_step": cfg.tokens, "oracle_tokens_per_step": n,
                   "distinct_weight_sets": args.distinct},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": saem_oracle.max_threads(), "kind": "oracle", "cpu": cpu_model(),
                         "sample": sample},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--distinct", type=int, default=8, help="distinct expert weight sets to generate (1..8)")
    ap.add_argument("--no-cpu", action="store_true", help="skip the cpu_baseline leg")
    ap.add_argument("--no-study", action="store_true", help="skip the study list of the other configurations")
    ap.add_argument("--graph", action="store_true", help="time CUDA-graph replays of the step (for steps of a few tens of us)")
    ap.add_argument("--workload", default="c2", choices=sorted(WORKLOADS), help="c2 is the benchmark; the others for study")
    ap.add_argument("--tokens", type=int, default=None, help="override the batch of the workload")
    ap.add_argument("--routing", default=None, choices=["zipf", "uniform", "normal"])
    ap.add_argument("--ffn-path", default="auto", choices=["auto", "tensor"],
                    help="tensor: the tcgen05 weight-streaming kernels up to 64 rows per segment (SAEM_FFN_TENSOR), for comparison")
    ap.add_argument("--segments", action="store_true", help="expert-FFN throughput by segment size of one expert")
    ap.add_argument("--segment-classes", action="store_true", help="a prefill call's time by segment-size class")
    ap.add_argument("--d-model", type=int, default=2048)
    ap.add_argument("--d-ff", type=int, default=1408)
    ap.add_argument("--copies", type=int, default=8)
    ap.add_argument("--sizes", type=str, default="1,8,16,32,64,128,256,512,1024,2048,4096,8192")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.segments:
        run_segments(args)
    elif args.segment_classes:
        run_segment_classes(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
