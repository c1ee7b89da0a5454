"""Replay study of the cache policy on a synthetic stage trace (the paper's prediction-oracle
protocol, Sec. VI-D, Eq. 2):

    python -m paper_2608_21614_b200.policy_study [--steps 384] [--batch 1] [--ecr 0.5,0.25]

1. one fully resident run records the per-stage expert activation counts EAP_s;
2. the same trace is replayed under the online policy (plan stage s from EAP_{s-1}), the
   clairvoyant policy (plan from EAP_s) and a token-level LRU baseline, at each cache ratio;
3. prints hit ratios, tokens/s, bytes over the host link and the efficiencies
   eta_CHR = CHR_online / CHR_clairvoyant, eta_TP = T_online / T_clairvoyant.
Routing does not depend on placement, so one recorded trace serves every ratio and policy.
"""
from __future__ import annotations

import argparse
import json
import time

import numpy as np
import torch

from . import inputs as gen
from .stack import StackRunner, tc_seq


def run(trace, weights, shape, C, temp, batch, steps, policy, eap=None):
    L, E, k, d, f = shape
    r = StackRunner(d, f, E, k, L, C, temp, batch, weights, policy=policy, recorded_eap=eap)
    r.warm([list(np.argsort(trace.rankings[0, l])[:C]) for l in range(L)])
    r.copy.synchronize()
    bounds = set(int(b) for b in trace.boundaries[1:])
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for t in range(steps):
        if t in bounds:
            r.boundary()
        lg = np.stack([gen.trace_logits(trace, t, l, batch) for l in range(L)])
        x = gen.trace_activations(trace, t, batch, d)
        r.step(torch.from_numpy(lg).cuda(non_blocking=True), torch.from_numpy(x).cuda(non_blocking=True), keep_out=False)
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    eap_out = r.finish()
    st = r.stats
    res = {"policy": policy, "slots_per_layer": C, "tokens_per_s": steps * batch / dt, "chr": st.chr(),
           "chr_pair_weighted": st.pair_chr(), "demand_loads": st.demand_loads, "boundary_loads": st.boundary_loads,
           "h2d_gb": r.h2d_bytes() / 1e9}
    r.close()
    return res, eap_out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--steps", type=int, default=384)
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--ecr", type=str, default="0.5,0.25")
    ap.add_argument("--distinct", type=int, default=4)
    ap.add_argument("--mean-stage-len", type=float, default=64.0,
                    help="shorter than the benchmark's 200 so that a short replay still crosses several boundaries")
    ap.add_argument("--seed", type=int, default=0)
    args = ap.parse_args()
    cfg = gen.layer_config("c5")
    shape = (args.layers, cfg.n_experts, cfg.top_k, cfg.d_model, cfg.d_ff)
    trace = gen.stage_trace(args.steps, args.layers, cfg.n_experts, cfg.zipf_s, args.seed,
                            mean_stage_len=args.mean_stage_len)
    rng = np.random.default_rng(np.random.SeedSequence([args.seed, 77]))
    weights = [gen.expert_weights(rng, cfg.d_model, cfg.d_ff) for _ in range(args.distinct)]
    full, eap = run(trace, weights, shape, cfg.n_experts, 0, args.batch, args.steps, "stage")
    out = {"steps": args.steps, "batch": args.batch, "layers": args.layers, "stages": int(len(trace.boundaries)),
           "mean_stage_len": args.mean_stage_len, "tc_seq": tc_seq(eap),
           "full_gpu_tokens_per_s": full["tokens_per_s"], "runs": []}
    for ecr in [float(v) for v in args.ecr.split(",")]:
        C = max(1, int(round(ecr * cfg.n_experts)))
        temp = max(4, min(cfg.n_experts - C, args.batch * cfg.top_k))
        rows = {}
        for policy in ("stage", "oracle", "lru"):
            if policy == "lru" and C < min(cfg.n_experts, args.batch * cfg.top_k):
                continue                       # an LRU slot set smaller than one step's active experts cannot hold them
            rows[policy], _ = run(trace, weights, shape, C, temp, args.batch, args.steps, policy, eap)
            rows[policy]["ecr"] = C / cfg.n_experts
            out["runs"].append(rows[policy])
        out["runs"].append({"ecr": C / cfg.n_experts, "eta_chr": rows["stage"]["chr"] / rows["oracle"]["chr"],
                            "eta_tp": rows["stage"]["tokens_per_s"] / rows["oracle"]["tokens_per_s"]})
    print(json.dumps(out))
    for r in out["runs"]:
        print("# " + "  ".join("%s=%s" % (k, ("%.4g" % v) if isinstance(v, float) else v) for k, v in r.items()))


if __name__ == "__main__":
    main()
