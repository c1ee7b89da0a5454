"""Expert-FFN throughput by segment size: one expert, one segment of N rows, N swept from
decode-sized to prefill-sized.

    python -m paper_2608_21614_b200.segment_bench [--d-model 2048] [--d-ff 1408] [--copies 8]

For each N it times saem_expert_ffn (gate/up + down kernels) with CUDA events and prints the
achieved GB/s on the expert's weight bytes and the achieved TFLOP/s, which shows where the path
changes from HBM-bound (small N) to tensor-bound (large N) and which kernels serve which sizes.
The expert's weights are loaded into `copies` different slots that are used in rotation, so that
small-N timings stream weights from HBM instead of re-reading one expert from L2.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding as B
from . import inputs as gen


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--d-model", type=int, default=2048)
    ap.add_argument("--d-ff", type=int, default=1408)
    ap.add_argument("--copies", type=int, default=8)
    ap.add_argument("--sizes", type=str, default="1,8,16,32,64,128,256,512,1024,2048,4096,8192")
    ap.add_argument("--steps", type=int, default=40)
    args = ap.parse_args()
    d, f = args.d_model, args.d_ff
    sizes = [int(s) for s in args.sizes.split(",")]
    rng = np.random.default_rng(0)
    w = gen.expert_weights(rng, d, f)
    peaks = {}
    try:
        import os
        peaks = json.load(open(os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))),
                                            "MEASURED_PEAKS.json")))
    except Exception:
        pass
    rows = []
    for n in sizes:
        # `copies` layers, one slot each: the same expert at different HBM addresses
        cfg = B.make_config(d, f, 1, 1, n, n_layers=args.copies, slots_per_layer=1)
        ctx = B.Context(cfg)
        packed = ctx.pack(*w)
        for layer in range(args.copies):
            B.saem_cache_load(ctx.handle, layer, 0, 0, packed)
        x = torch.from_numpy(gen.activations(rng, n, d)).cuda()
        y = torch.empty((n, d), dtype=torch.float32, device="cuda")
        for i in range(args.copies):
            B.saem_expert_ffn(ctx.handle, i, x, None, n, None, y)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(args.steps):
            B.saem_expert_ffn(ctx.handle, i % args.copies, x, None, n, None, y)
        b.record()
        torch.cuda.synchronize()
        us = a.elapsed_time(b) / args.steps * 1e3
        status = B.saem_last_device_status(ctx.handle)
        rows.append({"rows": n, "us": us, "weight_gbs": 3 * d * f * 2 / us / 1e3, "tflops": 6.0 * n * d * f / us / 1e6,
                     "kernels": ("tiled tcgen05 on CTA pairs (tokens as M)" if n >= 1536 and d >= 4096 and d % 256 == 0
                                 else "tiled tcgen05 (tokens as M)" if n > 64
                                 else "streaming tcgen05 (weights as M)" if n > 8
                                 else "matrix-vector (mma.sync)"), "status": status})
        ctx.close()
    print(json.dumps({"d_model": d, "d_ff": f, "copies": args.copies, "peaks": {k: peaks.get(k) for k in
                      ("hbm_gbs", "bf16_tflops", "bf16_tflops_sustained")}, "rows": rows}))
    for r in rows:
        print("# rows %5d  %8.1f us  %7.0f GB/s on weights  %7.1f TFLOP/s  %s" % (
            r["rows"], r["us"], r["weight_gbs"], r["tflops"], r["kernels"]))


if __name__ == "__main__":
    main()
