"""Memory and call plumbing for one MoE layer (or a stack of identical layers) on one GPU.

Allocates the slot region, workspace and step tensors with torch, packs and loads expert weights
through ``saem_pack_expert_host`` / ``saem_cache_load``, and chains the four C-ABI calls.  No
arithmetic of the method lives here: every step runs in libsaem's kernels.
"""
from __future__ import annotations

from typing import Optional, Sequence

import numpy as np
import torch

from . import binding as B


class MoELayer:
    def __init__(self, d_model: int, d_ff: int, n_experts: int, top_k: int, max_tokens: int, d_ff_shared: int = 0,
                 n_layers: int = 1, slots_per_layer: Optional[int] = None, temp_slots: int = 0, renorm: int = 1,
                 out_dtype: int = B.SAEM_OUT_F32, ffn_path: int = B.SAEM_FFN_AUTO, device: str = "cuda:0",
                 merge_shared: bool = True):
        self.device = torch.device(device)
        self.d, self.f, self.E, self.k, self.max_T = d_model, d_ff, n_experts, top_k, max_tokens
        # A shared expert whose width is a multiple of d_ff runs inside the layer's grouped launch
        # as S always-on experts of width d_ff; any other width gets a context of its own.
        S = d_ff_shared // d_ff if (merge_shared and d_ff_shared and d_ff_shared % d_ff == 0) else 0
        if S > 16 or n_experts + S > B.SAEM_MAX_EXPERTS:
            S = 0
        self.S = S
        self.cfg = B.make_config(d_model, d_ff, n_experts, top_k, max_tokens, n_layers,
                                 None if slots_per_layer is None else slots_per_layer + S, temp_slots, renorm,
                                 out_dtype, ffn_path, n_shared=S)
        self.ctx = B.Context(self.cfg, device)
        self.shared: Optional[B.Context] = None
        if d_ff_shared and S == 0:
            scfg = B.make_config(d_model, d_ff_shared, 1, 1, max_tokens, n_layers, 1, 0, 1, B.SAEM_OUT_F32, ffn_path)
            self.shared = B.Context(scfg, device)
        self.copy_stream = torch.cuda.Stream(device=self.device)
        P = max_tokens * top_k
        R = max_tokens * (top_k + S)                 # packed rows: pairs, then T rows per in-layer shared expert
        dev = self.device
        self.topk_idx = torch.empty((max_tokens, top_k), dtype=torch.int32, device=dev)
        self.topk_w = torch.empty((max_tokens, top_k), dtype=torch.float32, device=dev)
        self.counts = torch.empty(n_experts + S, dtype=torch.int32, device=dev)
        self.offsets = torch.empty(n_experts + S + 1, dtype=torch.int32, device=dev)
        self.perm = torch.empty(P, dtype=torch.int32, device=dev)
        self.inv_perm = torch.empty(P, dtype=torch.int32, device=dev)
        self.x_packed = torch.empty((R, d_model), dtype=torch.uint16, device=dev)
        self.y_packed = torch.empty((R, d_model), dtype=torch.float32, device=dev)
        self.shared_y = torch.empty((max_tokens, d_model), dtype=torch.float32, device=dev) if self.shared else None
        self.out = torch.empty((max_tokens, d_model),
                               dtype=torch.float32 if out_dtype == B.SAEM_OUT_F32 else torch.uint16, device=dev)
        self._pinned = []          # keep packed host buffers alive while copies may be in flight

    # ------------------------------------------------------------------ weights
    def load_expert(self, layer: int, expert: int, slot: int, gate: np.ndarray, up: np.ndarray, down: np.ndarray):
        packed = self.ctx.pack(gate, up, down)
        self._pinned.append(packed)
        B.saem_cache_load(self.ctx.handle, layer, expert, slot, packed, self.copy_stream)
        return packed

    def load_all(self, gate: Sequence[np.ndarray], up: Sequence[np.ndarray], down: Sequence[np.ndarray],
                 shared=None, layer: int = 0):
        """Every routed expert e into slot e of `layer` (needs slots_per_layer == n_experts)."""
        cache = {}
        for e in range(self.E):
            key = id(gate[e])
            if key not in cache:
                cache[key] = self.ctx.pack(gate[e], up[e], down[e])
                self._pinned.append(cache[key])
            B.saem_cache_load(self.ctx.handle, layer, e, e, cache[key], self.copy_stream)
        if shared is not None and self.S:
            sg, su, sd = shared
            for s in range(self.S):                  # hidden units [s f, (s+1) f) of the wide shared expert
                rows = slice(s * self.f, (s + 1) * self.f)
                packed = self.ctx.pack(sg[rows], su[rows], np.ascontiguousarray(sd[:, rows]))
                self._pinned.append(packed)
                B.saem_cache_load(self.ctx.handle, layer, self.E + s, self.E + s, packed, self.copy_stream)
        elif shared is not None:
            packed = self.shared.pack(*shared)
            self._pinned.append(packed)
            B.saem_cache_load(self.shared.handle, layer, 0, 0, packed, self.copy_stream)

    def drop_host_copies(self):
        self.copy_stream.synchronize()
        self._pinned.clear()

    # ------------------------------------------------------------------ the four calls
    def route(self, logits: torch.Tensor, T: int, stream=None):
        B.saem_route(self.ctx.handle, logits, T, self.topk_idx, self.topk_w, stream)

    def repack(self, x: torch.Tensor, T: int, stream=None):
        B.saem_repack(self.ctx.handle, self.topk_idx, x, T, self.counts, self.offsets, self.perm, self.inv_perm,
                      self.x_packed, stream)

    def expert_ffn(self, T: int, layer: int = 0, subset=None, stream=None):
        B.saem_expert_ffn(self.ctx.handle, layer, self.x_packed, self.offsets, T * (self.k + self.S), subset,
                          self.y_packed, stream)

    def shared_ffn(self, x: torch.Tensor, T: int, layer: int = 0, stream=None):
        B.saem_expert_ffn(self.shared.handle, layer, x, None, T, None, self.shared_y, stream)

    def combine(self, T: int, stream=None):
        B.saem_combine(self.ctx.handle, self.y_packed, self.inv_perm, self.topk_w, T, self.shared_y, self.out, stream)

    def step(self, logits: torch.Tensor, x: torch.Tensor, T: int, layer: int = 0, stream=None) -> torch.Tensor:
        """route -> repack -> expert FFN (-> shared FFN) -> combine, as four (five) C-ABI calls."""
        self.route(logits, T, stream)
        self.repack(x, T, stream)
        self.expert_ffn(T, layer, None, stream)
        if self.shared is not None:
            self.shared_ffn(x, T, layer, stream)
        self.combine(T, stream)
        return self.out[:T]

    def capture_step(self, logits: torch.Tensor, x: torch.Tensor, T: int, layer: int = 0) -> "torch.cuda.CUDAGraph":
        """The same five launches recorded once as a CUDA graph (every call of the library only
        enqueues on the stream it is given, so a step can be captured).  `replay()` re-runs the step
        on the current contents of `logits` and `x`; at batch 1 a step is short enough that issuing
        five launches from the host costs more than running them."""
        side = torch.cuda.Stream(device=self.device)
        side.wait_stream(torch.cuda.current_stream(self.device))
        with torch.cuda.stream(side):
            self.step(logits, x, T, layer)          # warm-up outside the capture (first-call set-up, tensor maps)
            side.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                self.step(logits, x, T, layer)
        torch.cuda.current_stream(self.device).wait_stream(side)
        return graph

    def step_fused_call(self, logits: torch.Tensor, x: torch.Tensor, T: int, out: torch.Tensor, layer: int = 0,
                        stream=None):
        """The same step through the single saem_moe_step call (intermediates in the workspace)."""
        B.saem_moe_step(self.ctx.handle, self.shared.handle if self.shared else None, layer, logits, x, T, out, stream)

    def step_host(self, logits_host: torch.Tensor, x_host: torch.Tensor, T: int, out_host: torch.Tensor,
                  layer: int = 0, stream=None):
        """The step from host buffers: H2D of logits and x, the kernels, D2H of out, synchronised."""
        B.saem_moe_step_host(self.ctx.handle, self.shared.handle if self.shared else None, layer, logits_host, x_host,
                             T, out_host, stream)

    def step_host_async(self, logits_host: torch.Tensor, x_host: torch.Tensor, T: int, out_host: torch.Tensor,
                        layer: int = 0, stream=None):
        """step_host without the final synchronisation: out_host is valid once the stream has passed the call."""
        B.saem_moe_step_host_async(self.ctx.handle, self.shared.handle if self.shared else None, layer, logits_host,
                                   x_host, T, out_host, stream)

    def device_status(self) -> int:
        s = B.saem_last_device_status(self.ctx.handle)
        if self.shared is not None:
            s = s or B.saem_last_device_status(self.shared.handle)
        return s

    def launches(self) -> int:
        n = B.saem_launch_count(self.ctx.handle)
        if self.shared is not None:
            n += B.saem_launch_count(self.shared.handle)
        return n

    def close(self):
        self.ctx.close()
        if self.shared is not None:
            self.shared.close()
