"""Where a prefill-sized expert-FFN call spends its time, by segment size.

    python -m paper_2608_21614_b200.segment_class_bench [--workload c3] [--tokens 2048]

Routes and repacks one batch, then times ``saem_expert_ffn`` with its ``expert_subset`` argument
restricted to the experts whose segments fall in a size class (CUDA events, 20 calls each).  The
classes do not add up to the whole call: each launch pays its own fixed cost and wave quantisation.
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
    ap.add_argument("--workload", default="c3")
    ap.add_argument("--tokens", type=int, default=2048)
    ap.add_argument("--distinct", type=int, default=4)
    args = ap.parse_args()
    cfg = gen.layer_config(args.workload, tokens=args.tokens)
    li = gen.layer_inputs(cfg, n_distinct_experts=args.distinct)
    T = args.tokens
    layer = MoELayer(cfg.d_model, cfg.d_ff, cfg.n_experts, cfg.top_k, T, cfg.d_ff_shared)
    layer.load_all(li.gate, li.up, li.down, li.shared)
    layer.route(torch.from_numpy(li.logits).cuda(), T)
    layer.repack(torch.from_numpy(li.x).cuda(), T)
    torch.cuda.synchronize()
    counts = layer.counts.cpu().numpy()
    n_all = len(counts)

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
        ne = n_all if subset is None else len(subset)
        row = {"class": name, "experts": ne, "rows": rows, "us": us,
               "tflops": 6.0 * rows * cfg.d_model * cfg.d_ff / us / 1e6,
               "weight_gbs": ne * 3 * cfg.d_model * cfg.d_ff * 2 / us / 1e3}
        print("# %-28s experts %3d  rows %6d  %8.1f us  %7.0f TFLOP/s  %6.0f GB/s on their weights"
              % (name, ne, rows, us, row["tflops"], row["weight_gbs"]))
        return row

    ids = np.arange(n_all)
    E = cfg.n_experts
    out = [timeit(None, "all"),
           timeit([int(e) for e in ids if counts[e] > 256], "more than 256 rows"),
           timeit([int(e) for e in ids if 64 < counts[e] <= 256], "65..256 rows"),
           timeit([int(e) for e in ids if 0 < counts[e] <= 64], "at most 64 rows")]
    if n_all > E:
        out.append(timeit([int(e) for e in ids if e >= E], "shared experts only"))
        out.append(timeit([int(e) for e in ids if e < E], "routed experts only"))
    print(json.dumps({"workload": args.workload, "tokens": T, "segments_sorted": sorted(counts.tolist(), reverse=True),
                      "classes": out, "device_status": layer.device_status()}))
    layer.close()


if __name__ == "__main__":
    main()
