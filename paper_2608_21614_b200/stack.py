"""Host-side driver of an L-layer MoE stack whose expert cache holds only part of the experts
(Sec. IV-C of the paper: fixed per-layer cache slots, a residency map, a live activation log,
a residency planner run at stage boundaries, asynchronous prefetch overlapped with compute; and
the ablation's on-demand loads through reserved temporary slots, since this build has no CPU
expert path).

Everything numerical runs in libsaem's kernels; this module holds the policy (which expert lives
in which slot, what to load when) and the bookkeeping (hit ratio, bytes moved).
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch

from . import binding as B


def plan_layer(counts: Sequence[int], slot_expert: Sequence[int]) -> List[Tuple[int, int, int]]:
    """Residency planner for one layer at a stage boundary (Sec. IV-C "Dynamic Expert Placement").

    counts[e]: activations of expert e in the stage that just ended; slot_expert[s]: the expert in
    fixed slot s (-1 = empty).  Experts are ranked by count; the least-used residents give way to
    more-used non-residents, the newcomer taking the victim's slot (the slot layout is fixed).
    A swap happens only while the newcomer's count is strictly larger; ties go to the lower id.
    Returns [(victim or -1, newcomer, slot)] in the order the loads should be issued.
    """
    E = len(counts)
    resident = [e for e in slot_expert if e >= 0]
    res_set = set(resident)
    worst_first = sorted(resident, key=lambda e: (counts[e], -e))
    best_first = sorted((e for e in range(E) if e not in res_set), key=lambda e: (-counts[e], e))
    moves = []
    empty = [s for s, e in enumerate(slot_expert) if e < 0]
    bi = 0
    for s in empty:                                     # free slots first: nothing to evict
        if bi < len(best_first) and counts[best_first[bi]] > 0:
            moves.append((-1, best_first[bi], s))
            bi += 1
    for victim in worst_first:
        if bi >= len(best_first) or counts[best_first[bi]] <= counts[victim]:
            break
        moves.append((victim, best_first[bi], list(slot_expert).index(victim)))
        bi += 1
    return moves


class ExpertStore:
    """Packed experts in pinned host memory.  (layer, expert) maps onto `n_distinct` buffers so
    that a 32-layer Mixtral-shaped stack (90 GB of experts) fits in host RAM; traffic per load is
    unchanged.  `weights(i)` gives the canonical matrices of buffer i (for the oracle)."""

    def __init__(self, ctx: B.Context, canonical: Sequence[Tuple[np.ndarray, np.ndarray, np.ndarray]]):
        self.canonical = list(canonical)
        self.packed = [ctx.pack(*w) for w in self.canonical]
        self.n = len(self.packed)

    def index(self, layer: int, expert: int) -> int:
        return (layer * 7 + expert * 13 + (layer // 3)) % self.n

    def get(self, layer: int, expert: int) -> torch.Tensor:
        return self.packed[self.index(layer, expert)]

    def weights(self, layer: int, expert: int):
        return self.canonical[self.index(layer, expert)]


@dataclasses.dataclass
class StackStats:
    layer_steps: int = 0
    active: int = 0            # distinct active experts over all layer-steps
    hits: int = 0              # ... of which in the residency map (fixed slots) when routing was known
    temp_hits: int = 0         # ... not resident but still bound to a temporary slot (no transfer)
    pair_total: int = 0
    pair_hits: int = 0
    demand_loads: int = 0
    host_reads: int = 0        # missed experts read in place from mapped host memory
    boundary_loads: int = 0
    boundaries: int = 0

    def chr(self) -> float:
        return self.hits / max(self.active, 1)

    def pair_chr(self) -> float:
        return self.pair_hits / max(self.pair_total, 1)


class StackRunner:
    def __init__(self, d_model: int, d_ff: int, n_experts: int, top_k: int, n_layers: int, slots_per_layer: int,
                 temp_slots: int, batch: int, store_weights, device: str = "cuda:0",
                 ffn_path: int = B.SAEM_FFN_AUTO, policy: str = "stage", recorded_eap: Optional[np.ndarray] = None,
                 read_counts: bool = True, miss_mode: str = "temp"):
        """policy: "stage" -- at a boundary re-plan from the counts of the stage that just ended
        (the paper's online policy); "oracle" -- re-plan from `recorded_eap[s]`, the counts of the
        stage that is about to start, recorded in an earlier run of the same trace (the paper's
        clairvoyant replay, Sec. VI-D); "lru" -- no stage logic: every miss evicts the layer's least
        recently used resident expert and takes its slot (token-level baseline)."""
        assert policy in ("stage", "oracle", "lru")
        # miss_mode: "temp" -- a missed expert is copied into a temporary slot first (the ablation's on-demand
        # transfer); "host" -- it is bound to its pinned host buffer and the matrix-vector kernels read the
        # weights in place over the host link (batches of at most 8 tokens): no HBM write + read, no slot.
        assert miss_mode in ("temp", "host") and (miss_mode == "temp" or batch <= 8)
        self.miss_mode = miss_mode
        # With every expert resident nothing on the host depends on the routing; read_counts=False
        # then skips the per-layer read-back (and with it the activation log and the hit statistics).
        self.read_counts = read_counts or slots_per_layer < n_experts
        self.policy, self.recorded_eap, self.stage = policy, recorded_eap, 0
        self.d, self.f, self.E, self.k, self.L, self.C = d_model, d_ff, n_experts, top_k, n_layers, slots_per_layer
        self.batch = batch
        self.device = torch.device(device)
        self.cfg = B.make_config(d_model, d_ff, n_experts, top_k, batch, n_layers, slots_per_layer, temp_slots,
                                 ffn_path=ffn_path)
        self.ctx = B.Context(self.cfg, device)
        self.store = ExpertStore(self.ctx, store_weights)
        self.h = self.ctx.handle
        self.compute = torch.cuda.current_stream(self.device)
        self.copy = torch.cuda.Stream(device=self.device)
        dev, P = self.device, batch * top_k
        self.topk_idx = torch.empty((batch, top_k), dtype=torch.int32, device=dev)
        self.topk_w = torch.empty((batch, top_k), dtype=torch.float32, device=dev)
        self.counts = torch.empty(n_experts, dtype=torch.int32, device=dev)
        self.offsets = torch.empty(n_experts + 1, dtype=torch.int32, device=dev)
        self.perm = torch.empty(P, dtype=torch.int32, device=dev)
        self.inv_perm = torch.empty(P, dtype=torch.int32, device=dev)
        self.x_packed = torch.empty((P, d_model), dtype=torch.uint16, device=dev)
        self.y_packed = torch.empty((P, d_model), dtype=torch.float32, device=dev)
        self.out = torch.empty((n_layers, batch, d_model), dtype=torch.float32, device=dev)
        self.counts_host = torch.empty(n_experts, dtype=torch.int32).pin_memory()
        self.counts_ready = torch.cuda.Event()
        # host mirrors of the policy state
        self.slot_expert = [[-1] * slots_per_layer for _ in range(n_layers)]     # fixed slot layout
        self.log = np.zeros((n_layers, n_experts), np.int64)                      # live activation log
        self.eap: List[np.ndarray] = []                                           # counts of every finished stage
        self.last_use = np.zeros((n_layers, n_experts), np.int64)                 # LRU clock per expert
        self.clock = 0
        self.stats = StackStats()
        self.slot_bytes = self.ctx.slot_bytes

    # ------------------------------------------------------------------ residency
    def warm(self, resident: Sequence[Sequence[int]]):
        """Initial placement: resident[l] lists the experts preloaded into layer l's slots."""
        for l, experts in enumerate(resident):
            for s, e in enumerate(experts[: self.C]):
                B.saem_cache_load(self.h, l, e, s, self.store.get(l, e), self.copy)
                self.slot_expert[l][s] = e

    def is_resident(self, layer: int, expert: int) -> bool:
        return expert in self.slot_expert[layer]

    def boundary(self):
        """Stage boundary: re-plan every layer from the activation log, enqueue the transfers on
        the copy stream (they overlap with the following decode steps), clear the log."""
        self.stats.boundaries += 1
        self.eap.append(self.log.copy())
        self.stage += 1
        if self.policy == "lru":
            self.log[:] = 0
            return
        profile = self.log
        if self.policy == "oracle":
            profile = self.recorded_eap[min(self.stage, len(self.recorded_eap) - 1)]
        for l in range(self.L):
            for victim, newcomer, s in plan_layer(profile[l], self.slot_expert[l]):
                if victim >= 0:
                    B.saem_cache_evict(self.h, l, victim)
                if B.saem_cache_query(self.h, l, newcomer)[0] >= 0:   # bound to a temporary slot: release it
                    B.saem_cache_evict(self.h, l, newcomer)
                B.saem_cache_load(self.h, l, newcomer, s, self.store.get(l, newcomer), self.copy)
                self.slot_expert[l][s] = newcomer
                self.stats.boundary_loads += 1
        self.log[:] = 0

    def finish(self):
        """Call after the last step: closes the last stage's record."""
        self.eap.append(self.log.copy())
        return np.stack(self.eap)

    def _lru_load(self, layer: int, expert: int):
        """Token-level LRU: the miss takes the slot of the layer's least recently used resident."""
        slots = self.slot_expert[layer]
        s = min(range(self.C), key=lambda i: (-1 if slots[i] < 0 else self.last_use[layer, slots[i]], i))
        if slots[s] >= 0:
            B.saem_cache_evict(self.h, layer, slots[s])
        B.saem_cache_load(self.h, layer, expert, s, self.store.get(layer, expert), self.copy)
        slots[s] = expert
        self.stats.demand_loads += 1

    def _demand_load(self, layer: int, expert: int):
        """Miss without a CPU path: copy the expert into the next temporary slot (round-robin);
        whatever that slot held loses its binding.  The residency map is unchanged."""
        B.saem_cache_load(self.h, layer, expert, B.SAEM_TEMP, self.store.get(layer, expert), self.copy)
        self.stats.demand_loads += 1

    # ------------------------------------------------------------------ one decode step
    def step(self, logits_all: torch.Tensor, x: torch.Tensor, keep_out: bool = True):
        """logits_all[L, B, E] fp32 and x[B, d] bf16 on the device.  Runs the L layers in order;
        layer l's routing is read back (counts only) before its misses can be loaded -- nothing
        about a later layer or step is looked at earlier."""
        Bt, k = self.batch, self.k
        st = self.stats
        for l in range(self.L):
            if not self.read_counts:                   # nothing on the host depends on the routing: the single call
                B.saem_moe_step(self.h, None, l, logits_all[l], x, Bt, self.out[l] if keep_out else self.out[0])
                continue
            B.saem_route(self.h, logits_all[l], Bt, self.topk_idx, self.topk_w)
            B.saem_repack(self.h, self.topk_idx, x, Bt, self.counts, self.offsets, self.perm, self.inv_perm,
                          self.x_packed)
            self.counts_host.copy_(self.counts, non_blocking=True)
            self.counts_ready.record(self.compute)
            self.counts_ready.synchronize()
            counts = self.counts_host.numpy()
            active = [int(e) for e in np.nonzero(counts)[0]]
            st.layer_steps += 1
            need = []
            for e in active:
                st.active += 1
                st.pair_total += int(counts[e])
                if self.is_resident(l, e):
                    st.hits += 1
                    st.pair_hits += int(counts[e])
                else:
                    need.append(e)
                    if B.saem_cache_query(self.h, l, e)[0] >= 0:      # still bound to a temporary slot
                        st.temp_hits += 1
            self.clock += 1
            for e in active:
                self.last_use[l, e] = self.clock
            if self.policy == "lru":
                for e in need:                         # needs slots_per_layer >= active experts of a step
                    self._lru_load(l, e)
                need = []
            mapped = []
            if self.miss_mode == "host":
                for e in need:
                    if B.saem_cache_query(self.h, l, e)[0] < 0:
                        B.saem_cache_map_host(self.h, l, e, self.store.get(l, e))
                        mapped.append(e)
                        st.host_reads += 1
            else:
                # every non-resident active expert must hold a temporary slot when the FFN is enqueued;
                # a load may recycle the slot of another one of them, so repeat until all are bound
                for _ in range(self.cfg.temp_slots + 1):
                    missing = [e for e in need if B.saem_cache_query(self.h, l, e)[0] < 0]
                    if not missing:
                        break
                    for e in missing:
                        self._demand_load(l, e)
            self.log[l] += counts
            B.saem_expert_ffn(self.h, l, self.x_packed, self.offsets, Bt * k, active, self.y_packed)
            for e in mapped:                           # the binding was consumed at enqueue; the host buffer stays valid
                B.saem_cache_evict(self.h, l, e)
            B.saem_combine(self.h, self.y_packed, self.inv_perm, self.topk_w, Bt, None,
                           self.out[l] if keep_out else self.out[0])
        return self.out

    def h2d_bytes(self) -> int:
        return (self.stats.demand_loads + self.stats.boundary_loads + self.stats.host_reads) * self.slot_bytes

    def close(self):
        self.ctx.close()


def tc_seq(stage_counts: np.ndarray) -> float:
    """Sequence-level temporal coherence (Eq. 1): stage_counts[p, l, e] = tokens of stage p routed
    to expert e in layer l.  R^p is the row-normalised matrix; the result is the mean over
    consecutive stage pairs of the layer-averaged cosine similarity of R^p and R^{p+1}."""
    c = np.asarray(stage_counts, np.float64)
    if c.shape[0] < 2:
        return 1.0
    r = c / np.maximum(c.sum(axis=2, keepdims=True), 1e-300)
    a, b = r[:-1], r[1:]
    cos = (a * b).sum(2) / np.maximum(np.linalg.norm(a, axis=2) * np.linalg.norm(b, axis=2), 1e-300)
    return float(cos.mean(axis=1).mean())
