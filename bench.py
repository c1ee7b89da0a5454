#!/usr/bin/env python
"""Benchmark of the MoE expert step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Workload (N = 1): the Mixtral-8x7B-shaped single-layer decode configuration -- d_model 4096,
8 experts, top-2, SwiGLU d_ff 14336, bf16 weights, batch of 16 tokens, router logits drawn from a
Zipf(1.1) expert popularity, every expert resident in the HBM slot cache.  A step is one pass of
the whole path: saem_route -> saem_repack -> saem_expert_ffn -> saem_combine.  The layer's
weights (2.8 GB) are far larger than L2, so consecutive steps cannot reuse them from cache.

Prints one JSON line (rank 0).  N > 1 runs N independent replicas, one per GPU (the path has no
exchange step), and reports the aggregate.  `--impl reference` times the CPU oracle instead.
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
    "c2": "c2: Mixtral-8x7B-shaped layer decode, d_model=4096, 8 experts top-2, d_ff=14336, batch 16",
    "c3": "c3: fine-grained layer, d_model=2048, 64 experts top-6 + 2 shared, d_ff=1408",
    "c4": "c4: Qwen-MoE-shaped layer, d_model=2048, 60 experts top-4 + shared d_ff=5632, routed d_ff=1408",
    "qwen3": "Qwen3-30B-A3B-shaped layer, d_model=2048, 128 experts top-8, d_ff=768",
    "ernie": "ERNIE-4.5-21B-A3B-shaped layer, d_model=2560, 64 experts top-6 + 2 shared, d_ff=1536",
}
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of the two FFN kernels of one step of workload c2
# with all 8 experts active, from the ncu capture summarised in profiles/ffn_tensor_c2_decode.md
NCU_FFN_TRAFFIC_BYTES = {"c2": 2844872000}


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as fh:
            return json.load(fh), "measured"
    except Exception:
        return {"hbm_gbs": FALLBACK_HBM_GBS}, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


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


def build_inputs(args):
    from paper_2608_21614_b200 import inputs as gen
    cfg = gen.layer_config(args.workload, tokens=args.tokens, routing=args.routing)
    return cfg, gen.layer_inputs(cfg, n_distinct_experts=args.distinct)


# ----------------------------------------------------------------------------------------- ours
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2608_21614_b200 import binding as B          # raises if the CUDA library is missing
    from paper_2608_21614_b200.layer import MoELayer

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    device = "cuda:%d" % local

    cfg, li = build_inputs(args)
    T, k, E, d, f = cfg.tokens, cfg.top_k, cfg.n_experts, cfg.d_model, cfg.d_ff
    layer = MoELayer(d, f, E, k, T, cfg.d_ff_shared, device=device)
    layer.load_all(li.gate, li.up, li.down, li.shared)
    layer.drop_host_copies()
    # The benchmark workload (c2) streams 2.8 GB of weights per step, far more than L2, from one
    # routing draw.  The study workloads are smaller, so they rotate over eight routing draws of the
    # same stage (different active experts step to step, as consecutive tokens would).
    from paper_2608_21614_b200 import inputs as gen
    n_draws = 1 if args.workload == "c2" else 8
    rng = np.random.default_rng(np.random.SeedSequence([cfg.seed, 4242]))
    pop = gen.zipf_popularity(li.ranking, cfg.zipf_s) if cfg.routing == "zipf" else None
    draws = [li.logits] + [gen.router_logits(rng, T, E, cfg.routing, pop) for _ in range(n_draws - 1)]
    logits_all = [torch.from_numpy(lg).to(device) for lg in draws]
    logits = logits_all[0]
    x = torch.from_numpy(li.x).to(device)
    stream = torch.cuda.current_stream()

    active = []
    for i in range(max(args.warmup, 3, n_draws)):
        layer.step(logits_all[i % n_draws], x, T)
        if i < n_draws:
            torch.cuda.synchronize()
            active.append(int((layer.counts.cpu().numpy()[:E] > 0).sum()))
    torch.cuda.synchronize()
    n_active = sum(active) / len(active)
    # algorithmic: weights of the active experts (and the always-on shared expert), each read once
    ffn_bytes = n_active * 3 * d * f * 2 + 3 * d * cfg.d_ff_shared * 2
    weight_gb = (E * 3 * d * f * 2 + 3 * d * cfg.d_ff_shared * 2) / 1e9

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    K = args.steps
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = layer.launches()
    # timed region 1: exactly K steps, nothing between the kernels of a step (an event recorded
    # between two launches would forbid their programmatic overlap) -> the headline value
    if args.graph:      # the step of every routing draw recorded once; the timed loop replays them
        graphs = [layer.capture_step(lg, x, T) for lg in logits_all]
        per_step = (layer.launches() - launches0) // (2 * n_draws)      # capture_step runs the step twice
        torch.cuda.synchronize()
        ev0.record(stream)
        for i in range(K):
            graphs[i % n_draws].replay()
        ev1.record(stream)
    else:
        ev0.record(stream)
        for i in range(K):
            layer.step(logits_all[i % n_draws], x, T)
        ev1.record(stream)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    launches = per_step * K if args.graph else layer.launches() - launches0
    total_ms = ev0.elapsed_time(ev1)
    # timed region 2: the same K steps with CUDA events around the saem_expert_ffn call(s) -> the
    # dominant kernel's duration for the roofline
    ffn_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    for i in range(K):
        layer.route(logits_all[i % n_draws], T)
        layer.repack(x, T)
        ffn_ev[i][0].record(stream)
        layer.expert_ffn(T)
        if layer.shared is not None:
            layer.shared_ffn(x, T)
        ffn_ev[i][1].record(stream)
        layer.combine(T)
    torch.cuda.synchronize()
    ffn_ms = [a.elapsed_time(b) for a, b in ffn_ev]
    # the same call issued back to back on the last routing (its set-up overlaps the previous call's tail,
    # as it overlaps the repack's inside a step): two events around the whole batch
    bb0, bb1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    Kb = min(K, 200)
    bb0.record(stream)
    for _ in range(Kb):
        layer.expert_ffn(T)
        if layer.shared is not None:
            layer.shared_ffn(x, T)
    bb1.record(stream)
    torch.cuda.synchronize()
    ffn_bb_ms = bb0.elapsed_time(bb1) / Kb
    clocks = sampler.stop() if rank == 0 else None
    status = layer.device_status()

    # end to end through the host-buffer call: H2D of logits and x, the kernels, D2H of out
    lh = torch.from_numpy(li.logits).pin_memory()
    xh = torch.from_numpy(li.x).pin_memory()
    oh = torch.empty((T, d), dtype=torch.float32).pin_memory()
    for _ in range(3):
        layer.step_host(lh, xh, T, oh)
    Ke = max(K // 4, 10)
    t0 = time.perf_counter()
    for _ in range(Ke):
        layer.step_host(lh, xh, T, oh)
    e2e_s = time.perf_counter() - t0

    total_ms, e2e_step_s = max_over_ranks([total_ms, e2e_s / Ke], device)
    if rank == 0:
        peaks, which = measured_peaks()
        ffn_avg_ms = sum(ffn_ms) / len(ffn_ms)
        if T > 64:      # prefill-sized segments are a dense contraction: judged against the tensor peak
            ffn_flops = 6.0 * T * d * (cfg.top_k * f + cfg.d_ff_shared)
            achieved = ffn_flops / (ffn_avg_ms * 1e-3) / 1e12
            peak = float(peaks.get("bf16_tflops", 1590.0))
            roof = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                    "traffic": None, "algorithmic_flops": ffn_flops,
                    "frac_of_sustained": achieved / float(peaks.get("bf16_tflops_sustained", 1400.0))}
        else:
            achieved = ffn_bytes / (ffn_avg_ms * 1e-3) / 1e9
            peak = float(peaks["hbm_gbs"])
            roof = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                    "traffic": NCU_FFN_TRAFFIC_BYTES.get(args.workload) if (args.tokens is None and n_active == E) else None,
                    "algorithmic_bytes": ffn_bytes, "frac_of_nominal_8000": achieved / 8000.0}
        if T > 64:
            bb_achieved = roof["achieved"] * ffn_avg_ms / ffn_bb_ms
        else:       # bytes of the draw that call ran on (the last one of the instrumented pass)
            bb_bytes = active[(K - 1) % n_draws] * 3 * d * f * 2 + 3 * d * cfg.d_ff_shared * 2
            bb_achieved = bb_bytes / (ffn_bb_ms * 1e-3) / 1e9
        roof["back_to_back"] = {"avg_ms": ffn_bb_ms, "achieved": bb_achieved, "frac": bb_achieved / roof["peak"],
                                "note": "the same call issued back to back on one routing draw"}
        roof.update({"peak_source": which, "routing_draws": n_draws, "avg_ms": ffn_avg_ms,
                     "kernel": "saem_expert_ffn (gate/up + down kernels%s)" % (
                         ", second call for the shared expert" if layer.shared is not None else "")})
        line = {
            "metric": METRIC, "value": aggregate_tokens_per_s(world, T, K, total_ms), "unit": UNIT, "n_gpus": world,
            "steps": K, "warmup": max(args.warmup, 3), "ms_per_step": total_ms / K, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOADS[args.workload], "tokens_per_step": T, "active_experts": n_active,
                       "routing": "%s popularity + Gumbel, seed 0" % cfg.routing, "cache": "all experts resident in HBM",
                       "l2": "layer weights %.2f GB vs 126 MB L2: inputs larger than L2, no flush" % weight_gb,
                       "distinct_weight_sets": args.distinct, "replicas": world,
                       "launch": "CUDA-graph replay of the step" if args.graph else "one host call per kernel group",
                       "timing": "value: K steps back to back; roofline: a second pass of K steps with events around the FFN call"},
            "roofline": roof,
            "e2e": {"value": world * T / e2e_step_s, "unit": UNIT, "h2d_bytes_per_step": T * E * 4 + T * d * 2,
                    "d2h_bytes_per_step": T * d * 4, "ms_per_step": e2e_step_s * 1e3},
            "gpu_launches": launches, "clocks": clocks, "device_status": status,
        }
        if not args.no_cpu and world == 1:
            line["cpu_baseline"] = cpu_baseline(li, cfg, budget_s=12.0)
        print(json.dumps(line))
    layer.close()
    if world > 1:
        dist.destroy_process_group()


# -------------------------------------------------------------------------------------- oracle
def oracle_tokens_per_s(li, cfg, n_tokens, reps=1):
    """Times the CPU oracle's whole step on the first n_tokens tokens of the workload."""
    from oracle import saem_oracle
    lg, x = li.logits[:n_tokens], li.x[:n_tokens]
    t0 = time.perf_counter()
    for _ in range(reps):
        saem_oracle.moe_step(lg, x, cfg.top_k, li.gate, li.up, li.down, shared=li.shared)
    return n_tokens * reps / (time.perf_counter() - t0)


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
            "sample": "the first %d of the step's %d tokens, whole path, %d passes in %.1f s" % (n, cfg.tokens, passes, dt)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import saem_oracle
    saem_oracle.build()
    cfg, li = build_inputs(args)
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
        "config": {"workload": WORKLOADS[args.workload], "tokens_per_step": n, "distinct_weight_sets": args.distinct},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": saem_oracle.max_threads(), "kind": "oracle", "sample": sample},
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
    ap.add_argument("--graph", action="store_true", help="time CUDA-graph replays of the step (for steps of a few tens of us)")
    ap.add_argument("--workload", default="c2", choices=sorted(WORKLOADS), help="c2 is the benchmark; c3/c4 for study")
    ap.add_argument("--tokens", type=int, default=None, help="override the batch of the workload")
    ap.add_argument("--routing", default=None, choices=["zipf", "uniform", "normal"])
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
