"""Launch-granularity ablation on one layer: the paper's token repacking runs "each expert in a
single batched kernel launch" over its contiguous segment (Sec. IV-E); this library runs ALL
segments of the layer in one grouped launch per GEMM.  This script measures both on the same
repacked batch:

    python -m paper_2608_21614_b200.launch_ablation [--workload c4] [--tokens 8]

  grouped     one saem_expert_ffn call for the whole layer (2 kernel launches)
  per-expert  one saem_expert_ffn call per active expert with expert_subset = [e]
              (2 launches per active expert; the host must first read the counts back)

Outputs of the two modes are compared: identical bits on the matrix-vector path (no k-split), and
equal up to fp32 summation order on the streaming path (ffn_path TENSOR), whose k-split points depend on how many
experts share the launch.

With --bookkeeping the whole step is also run the way the paper describes its starting point
(Sec. III "bookkeeping": a mask per expert, a gather of that expert's tokens, the expert's dense
execution, a scatter-add of the weighted result): per active expert one `nonzero` on the routing
mask (a host synchronisation), one row gather, one FFN call on the gathered rows, one `index_add_`.
The mask, gather and scatter-add are library (torch) operations here, as they are in the paper's
PyTorch baseline; only the expert FFN runs in this library's kernels (a second context that holds
every expert as a one-expert "layer").  It is a measurement harness, not a product path.
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
    ap.add_argument("--bookkeeping", action="store_true", help="also time the whole step with per-expert mask / gather / scatter-add")
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
    if args.bookkeeping:
        out["bookkeeping"] = bookkeeping_step(cfg, li, layer, logits, x, args.steps)
    print(json.dumps(out))
    layer.close()


class BookkeepingStep:
    """The step done the way the paper describes its starting point (Sec. III, "bookkeeping"): route,
    then per expert a mask over the routing, a gather of that expert's tokens, the expert's dense
    execution on the gathered rows and a scatter-add of the weighted result.  Mask, gather and
    scatter-add are torch operations; the gate and every expert FFN run in this library's kernels
    (`one` holds every expert, and every d_ff-wide part of the shared expert, as a one-expert layer)."""

    def __init__(self, cfg, li, layer: MoELayer):
        self.cfg, self.layer = cfg, layer
        T, E, d = cfg.tokens, cfg.n_experts, cfg.d_model
        self.n_sh = cfg.d_ff_shared // cfg.d_ff if cfg.d_ff_shared else 0
        assert cfg.d_ff_shared == self.n_sh * cfg.d_ff, "shared width must be a multiple of d_ff here"
        self.one = MoELayer(d, cfg.d_ff, 1, 1, T, 0, n_layers=E + self.n_sh, slots_per_layer=1)
        for e in range(E):
            self.one.load_expert(e, 0, 0, li.gate[e], li.up[e], li.down[e])
        for s_ in range(self.n_sh):
            rows = slice(s_ * cfg.d_ff, (s_ + 1) * cfg.d_ff)
            self.one.load_expert(E + s_, 0, 0, li.shared[0][rows], li.shared[1][rows],
                                 np.ascontiguousarray(li.shared[2][:, rows]))
        self.one.drop_host_copies()
        self.xg = torch.empty((T, d), dtype=torch.uint16, device="cuda")
        self.yg = torch.empty((T, d), dtype=torch.float32, device="cuda")
        self.out = torch.zeros((T, d), dtype=torch.float32, device="cuda")
        self.ffn_calls = 0

    def run(self, logits: torch.Tensor, x: torch.Tensor) -> torch.Tensor:
        from . import binding as B
        T, E = self.cfg.tokens, self.cfg.n_experts
        layer, one, xg, yg, out = self.layer, self.one, self.xg, self.yg, self.out
        layer.route(logits, T)
        out.zero_()
        idx, w = layer.topk_idx[:T].to(torch.int64), layer.topk_w[:T]
        for e in range(E):
            tok, slot = (idx == e).nonzero(as_tuple=True)           # mask -> indices: synchronises with the host
            n = int(tok.numel())
            if n == 0:
                continue
            xg.view(torch.int16)[:n] = x.view(torch.int16)[tok]      # gather (bit patterns)
            B.saem_expert_ffn(one.ctx.handle, e, xg, None, n, None, yg)
            out.index_add_(0, tok, yg[:n] * w[tok, slot].unsqueeze(1))      # scatter-add
            self.ffn_calls += 1
        for s_ in range(self.n_sh):                                 # shared expert: every token, weight 1
            B.saem_expert_ffn(one.ctx.handle, E + s_, x, None, T, None, yg)
            out.add_(yg[:T])
            self.ffn_calls += 1
        return out

    def close(self):
        self.one.close()


def bookkeeping_step(cfg, li, layer, logits, x, steps):
    """Whole step, grouped (route, repack, grouped FFN, combine) against per-expert bookkeeping."""
    T = cfg.tokens
    book = BookkeepingStep(cfg, li, layer)

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(steps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / steps * 1e3

    t_g = timed(lambda: layer.step(logits, x, T))
    ref = layer.out[:T].clone()
    book.ffn_calls = 0
    t_b = timed(lambda: book.run(logits, x))
    res = {"grouped_step_us": t_g, "bookkeeping_step_us": t_b, "ffn_calls_per_step": book.ffn_calls / (steps + 3),
           "speedup": t_b / t_g, "max_abs_difference": float((ref - book.out).abs().max()),
           "device_status": book.one.device_status()}
    book.close()
    return res


if __name__ == "__main__":
    main()
