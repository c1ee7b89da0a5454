"""Measurement of the partially resident 32-layer stack (the fifth benchmark configuration):

    python -m paper_2608_21614_b200.stack_bench [--steps 512] [--batch 1] [--ecr 0.5] [--independent]

Mixtral-8x7B-shaped layers (d_model 4096, d_ff 14336, 8 experts, top-2), a stage-structured
routing trace (geometric stage lengths of mean 200, per-stage Zipf(1.2) ranking), an HBM cache of
`ecr * 8` fixed slots per layer plus temporary slots; misses are copied from pinned host memory
with cudaMemcpyAsync on a side stream.  Prints one JSON line with tokens/s, hit ratios, bytes over
the host link and the achieved host-link bandwidth.
"""
from __future__ import annotations

import argparse
import json
import time

import numpy as np
import torch

from . import inputs as gen
from .stack import StackRunner, tc_seq


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--steps", type=int, default=512)
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--ecr", type=float, default=0.5, help="expert cache ratio: resident / routed experts per layer")
    ap.add_argument("--temp-slots", type=int, default=4)
    ap.add_argument("--distinct", type=int, default=8, help="distinct host weight sets shared by the (layer, expert) pairs")
    ap.add_argument("--independent", action="store_true", help="independent ranking per stage (stress trace)")
    ap.add_argument("--trace-steps", type=int, default=4096)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--host-reads", action="store_true",
                    help="missed experts are read in place from mapped pinned host memory instead of being copied to a temporary slot")
    ap.add_argument("--no-readback", action="store_true",
                    help="with --ecr 1.0: do not read the routing counts back (no host sync per layer; no statistics)")
    args = ap.parse_args()

    cfg = gen.layer_config("c5")
    L, E, k, d, f = args.layers, cfg.n_experts, cfg.top_k, cfg.d_model, cfg.d_ff
    C = max(1, int(round(args.ecr * E)))
    trace = gen.stage_trace(args.trace_steps, L, E, cfg.zipf_s, args.seed,
                            reshuffled=None if args.independent else 3.2)
    rng = np.random.default_rng(np.random.SeedSequence([args.seed, 77]))
    weights = [gen.expert_weights(rng, d, f) for _ in range(args.distinct)]
    run = StackRunner(d, f, E, k, L, C, args.temp_slots if C < E else 0, args.batch, weights,
                      read_counts=not args.no_readback, miss_mode="host" if args.host_reads else "temp")
    run.warm([list(np.argsort(trace.rankings[0, l])[:C]) for l in range(L)])
    run.copy.synchronize()
    bounds = set(int(b) for b in trace.boundaries[1:])
    stage_counts = np.zeros((len(trace.boundaries), L, E))

    # logits for all steps up front on the host (the runner reads layer l's only when it gets there)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for t in range(args.steps):
        if t in bounds:
            run.boundary()
        lg = np.stack([gen.trace_logits(trace, t, l, args.batch) for l in range(L)])
        x = gen.trace_activations(trace, t, args.batch, d)
        log_before = run.log.copy()
        run.step(torch.from_numpy(lg).cuda(non_blocking=True), torch.from_numpy(x).cuda(non_blocking=True),
                 keep_out=False)
        stage_counts[trace.stage_of(t)] += run.log - log_before
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    st = run.stats
    n_stages_seen = trace.stage_of(args.steps - 1) + 1
    from . import binding as B
    line = {
        "workload": "c5: Mixtral-8x7B-shaped %d-layer stack decode, stage-coherent routing, ECR %.3f" % (L, C / E),
        "steps": args.steps, "batch": args.batch, "tokens_per_s": args.steps * args.batch / dt,
        "ms_per_token_step": dt / args.steps * 1e3,
        "trace": {"stages_seen": n_stages_seen, "tc_seq": tc_seq(stage_counts[:n_stages_seen]),
                  "kind": "independent" if args.independent else "coherent (3.2 ranks reshuffled per boundary)"},
        "chr_distinct": st.chr(), "chr_pair_weighted": st.pair_chr(), "temp_hits": st.temp_hits,
        "demand_loads": st.demand_loads, "host_reads": st.host_reads, "miss_mode": run.miss_mode, "boundary_loads": st.boundary_loads, "boundaries": st.boundaries,
        "h2d_bytes": run.h2d_bytes(), "h2d_gbs_over_wall_time": run.h2d_bytes() / dt / 1e9,
        "slot_bytes": run.slot_bytes, "slots_per_layer": C, "temp_slots": run.cfg.temp_slots,
        "distinct_host_weight_sets": args.distinct, "device_status": B.saem_last_device_status(run.h),
        "gpu_launches": B.saem_launch_count(run.h),
    }
    print(json.dumps(line))
    run.close()


if __name__ == "__main__":
    main()
