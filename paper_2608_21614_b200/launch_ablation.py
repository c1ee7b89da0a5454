"""Launch-granularity ablation on one layer: the paper's token repacking runs "each expert in a
single batched kernel launch" over its contiguous segment (Sec. IV-E); this library runs ALL
segments of the layer in one grouped launch per GEMM.  This script measures both on the same
repacked batch:

    python -m paper_2608_21614_b200.launch_ablation [--workload c4] [--tokens 8]

  grouped     one saem_expert_ffn call for the whole layer (2 kernel launches)
  per-expert  one saem_expert_ffn call per active expert with expert_subset = [e]
              (2 launches per active expert; the host must first read the counts back)

Outputs of the two modes are compared: identical bits on the matrix-vector path (no k-split), and
equal up to fp32 summation order on the streaming path, whose k-split points depend on how many
experts share the launch.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import inputs as gen
from .layer import MoELayer


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c4")
    ap.add_argument("--tokens", type=int, default=8)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--distinct", type=int, default=4)
    args = ap.parse_args()
    cfg = gen.layer_config(args.workload, tokens=args.tokens)
    li = gen.layer_inputs(cfg, n_distinct_experts=args.distinct)
    T = cfg.tokens
    layer = MoELayer(cfg.d_model, cfg.d_ff, cfg.n_experts, cfg.top_k, T, cfg.d_ff_shared)
    layer.load_all(li.gate, li.up, li.down, li.shared)
    logits, x = torch.from_numpy(li.logits).cuda(), torch.from_numpy(li.x).cuda()
    layer.route(logits, T)
    layer.repack(x, T)
    torch.cuda.synchronize()
    counts = layer.counts.cpu().numpy()
    active = [int(e) for e in np.nonzero(counts)[0]]

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n0 = layer.launches()
        a.record()
        for _ in range(args.steps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / args.steps * 1e3, (layer.launches() - n0) / args.steps

    def per_expert():
        for e in active:
            layer.expert_ffn(T, 0, [e])

    t_group, l_group = timed(lambda: layer.expert_ffn(T))
    y_group = layer.y_packed.clone()
    layer.y_packed.zero_()
    t_each, l_each = timed(per_expert)
    same = bool(torch.equal(y_group, layer.y_packed))
    max_diff = float((y_group - layer.y_packed).abs().max())
    out = {"workload": args.workload, "tokens": T, "active_experts": len(active),
           "grouped": {"us": t_group, "launches": l_group}, "per_expert": {"us": t_each, "launches": l_each},
           "speedup_of_grouping": t_each / t_group, "outputs_bit_identical": same, "max_abs_difference": max_diff,
           "device_status": layer.device_status()}
    print(json.dumps(out))
    layer.close()


if __name__ == "__main__":
    main()
