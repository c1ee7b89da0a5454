"""Seeded synthetic inputs for the MoE expert step.

This module only *draws data*: weights, activations, router logits and stage
traces with the shapes and distributions of the paper's workloads (Table of
evaluated models; skewed, stage-coherent expert popularity, Motivation 1-2).
It holds none of the method's arithmetic (no gating, repacking, FFN or combine)
so that both the CPU oracle's tests and the CUDA path's tests can take their
inputs from here without sharing any code of the method itself.

All floating-point tensors that the method consumes in bf16 are returned as
``numpy.uint16`` bit patterns (round-to-nearest-even from float32), so that
every consumer widens exactly the same bits.
"""
from __future__ import annotations

import dataclasses
from typing import Optional

import numpy as np


# --------------------------------------------------------------------------- bf16 bits
def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 array -> uint16 bf16 bit patterns, round-to-nearest-even."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32)
    rounded = bits + np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns -> float32 (exact widening)."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------- configs
@dataclasses.dataclass(frozen=True)
class LayerConfig:
    """One MoE layer workload (one entry of the benchmark's configuration list)."""
    name: str
    d_model: int
    d_ff: int
    n_experts: int
    top_k: int
    tokens: int
    d_ff_shared: int = 0          # 0 = no shared expert; two shared experts of width f are one of width 2f
    routing: str = "normal"       # "normal" | "zipf" | "uniform"
    zipf_s: float = 1.1
    seed: int = 0
    n_layers: int = 1


def layer_config(name: str, tokens: Optional[int] = None, routing: Optional[str] = None) -> LayerConfig:
    """The five benchmark configurations, by short name.

    c1 tiny; c2 Mixtral-8x7B-shaped decode; c3 fine-grained (64 routed top-6 + 2 shared);
    c4 Qwen-MoE-shaped (60 routed top-4 + one wide shared expert); c5 the Mixtral-shaped
    32-layer stack (per-layer shape only; the trace comes from :func:`stage_trace`).
    "qwen3" / "ernie": layers shaped like the paper's two models (Qwen3-30B-A3B, ERNIE-4.5-21B-A3B).
    """
    table = {
        "c1": LayerConfig("c1", 512, 1024, 8, 2, 64, 0, "normal"),
        "c2": LayerConfig("c2", 4096, 14336, 8, 2, 16, 0, "zipf", 1.1),
        "c3": LayerConfig("c3", 2048, 1408, 64, 6, 32, 2 * 1408, "zipf", 1.1),
        "c4": LayerConfig("c4", 2048, 1408, 60, 4, 8, 5632, "zipf", 1.1),
        "c5": LayerConfig("c5", 4096, 14336, 8, 2, 1, 0, "zipf", 1.2, 0, 32),
        # the paper's two evaluated models (model table): 128 routed experts top-8, no shared expert,
        # 4.72 M parameters per expert; 64 routed top-6 + 2 shared experts
        "qwen3": LayerConfig("qwen3", 2048, 768, 128, 8, 8, 0, "zipf", 1.1, 0, 48),
        "ernie": LayerConfig("ernie", 2560, 1536, 64, 6, 8, 2 * 1536, "zipf", 1.1, 0, 28),
    }
    cfg = table[name]
    if tokens is not None:
        cfg = dataclasses.replace(cfg, tokens=int(tokens))
    if routing is not None:
        cfg = dataclasses.replace(cfg, routing=routing)
    return cfg


def _streams(seed: int):
    """Independent child generators in a fixed order: weights, x, ranking, gumbel, lengths, subsample."""
    kids = np.random.SeedSequence(seed).spawn(6)
    names = ("w", "x", "rank", "gum", "len", "sub")
    return {n: np.random.default_rng(k) for n, k in zip(names, kids)}


# --------------------------------------------------------------------------- tensors
def expert_weights(rng: np.random.Generator, d_model: int, d_ff: int):
    """One expert: gate[f,d], up[f,d] ~ N(0,1/d); down[d,f] ~ N(0,1/f); bf16 bits."""
    g = to_bf16_bits(rng.standard_normal((d_ff, d_model), dtype=np.float32) * np.float32(d_model ** -0.5))
    u = to_bf16_bits(rng.standard_normal((d_ff, d_model), dtype=np.float32) * np.float32(d_model ** -0.5))
    dn = to_bf16_bits(rng.standard_normal((d_model, d_ff), dtype=np.float32) * np.float32(d_ff ** -0.5))
    return g, u, dn


def activations(rng: np.random.Generator, tokens: int, d_model: int) -> np.ndarray:
    """x[T,d] ~ N(0,1) as bf16 bits."""
    return to_bf16_bits(rng.standard_normal((tokens, d_model), dtype=np.float32))


def router_weights(rng: np.random.Generator, n_experts: int, d_model: int) -> np.ndarray:
    """w_router[E, d] ~ N(0, 1/d) as bf16 bits: with x ~ N(0,1) the logits are about N(0,1)."""
    return to_bf16_bits(rng.standard_normal((n_experts, d_model), dtype=np.float32) * np.float32(d_model ** -0.5))


def zipf_popularity(ranking: np.ndarray, s: float) -> np.ndarray:
    """p(e) proportional to rank(e)^-s, where ranking[e] in 1..E."""
    p = ranking.astype(np.float64) ** (-float(s))
    return p / p.sum()


def router_logits(rng: np.random.Generator, tokens: int, n_experts: int, routing: str,
                  popularity: Optional[np.ndarray] = None) -> np.ndarray:
    """fp32 logits[T,E].

    "normal": iid N(0,1).  "zipf"/"uniform": ln p(e) + Gumbel(0,1) noise, so that the top-k
    of a row is a draw of k experts without replacement with probability proportional to p.
    """
    if routing == "normal":
        return rng.standard_normal((tokens, n_experts)).astype(np.float32)
    if routing == "uniform" or popularity is None:
        popularity = np.full(n_experts, 1.0 / n_experts)
    gum = rng.gumbel(0.0, 1.0, size=(tokens, n_experts))
    return (np.log(popularity)[None, :] + gum).astype(np.float32)


@dataclasses.dataclass
class LayerInputs:
    cfg: LayerConfig
    gate: list            # per expert uint16[f,d]
    up: list
    down: list            # per expert uint16[d,f]
    shared: Optional[tuple]  # (gate[fs,d], up[fs,d], down[d,fs]) or None
    x: np.ndarray         # uint16[T,d]
    logits: np.ndarray    # float32[T,E]
    ranking: np.ndarray   # int[E], 1 = most popular


def layer_inputs(cfg: LayerConfig, n_distinct_experts: Optional[int] = None) -> LayerInputs:
    """All tensors of one layer workload, from cfg.seed.

    ``n_distinct_experts`` (default: all) lets very large layers reuse a few distinct
    weight sets: expert e gets set e mod n -- traffic is unchanged, host memory is not.
    """
    st = _streams(cfg.seed)
    n = cfg.n_experts if n_distinct_experts is None else min(cfg.n_experts, n_distinct_experts)
    sets = [expert_weights(st["w"], cfg.d_model, cfg.d_ff) for _ in range(n)]
    gate = [sets[e % n][0] for e in range(cfg.n_experts)]
    up = [sets[e % n][1] for e in range(cfg.n_experts)]
    down = [sets[e % n][2] for e in range(cfg.n_experts)]
    shared = expert_weights(st["w"], cfg.d_model, cfg.d_ff_shared) if cfg.d_ff_shared else None
    x = activations(st["x"], cfg.tokens, cfg.d_model)
    ranking = st["rank"].permutation(cfg.n_experts) + 1
    pop = zipf_popularity(ranking, cfg.zipf_s) if cfg.routing == "zipf" else None
    logits = router_logits(st["gum"], cfg.tokens, cfg.n_experts, cfg.routing, pop)
    return LayerInputs(cfg, gate, up, down, shared, x, logits, ranking)


# --------------------------------------------------------------------------- stage traces (c5)
@dataclasses.dataclass
class StageTrace:
    """Piecewise-stationary routing for an L-layer stack.

    boundaries[s] is the first step of stage s (boundaries[0] == 0); rankings[s, l, e] is the
    popularity rank (1 = hottest) of expert e in layer l during stage s.
    """
    n_steps: int
    boundaries: np.ndarray
    rankings: np.ndarray
    zipf_s: float
    seed: int
    reshuffled: float

    def stage_of(self, step: int) -> int:
        return int(np.searchsorted(self.boundaries, step, side="right") - 1)


def stage_trace(n_steps: int, n_layers: int, n_experts: int, zipf_s: float, seed: int,
                mean_stage_len: float = 200.0, reshuffled: Optional[float] = 3.2) -> StageTrace:
    """Stage lengths iid Geometric(1/mean) until n_steps; per layer, stage 0 has a uniform
    random ranking and every later stage re-draws the ranks of ``reshuffled`` randomly chosen
    experts among themselves (a fractional value m + p means m or m + 1 experts with probability
    1 - p and p; ``None``: an independent fresh ranking per stage).  The default 3.2 gives a
    measured adjacent-stage coherence (Eq. 1 of the paper) of about 0.89 for 8 experts, top-2,
    Zipf exponent 1.2 -- the paper's reported mean."""
    st = _streams(seed)
    lens = []
    while sum(lens) < n_steps:
        lens.append(int(st["len"].geometric(1.0 / mean_stage_len)))
    bounds = np.concatenate([[0], np.cumsum(lens)[:-1]]).astype(np.int64)
    bounds = bounds[bounds < n_steps]
    n_stages = len(bounds)
    rk = np.empty((n_stages, n_layers, n_experts), dtype=np.int64)
    for l in range(n_layers):
        rk[0, l] = st["rank"].permutation(n_experts) + 1
        for s in range(1, n_stages):
            if reshuffled is None:
                rk[s, l] = st["rank"].permutation(n_experts) + 1
            else:
                cur = rk[s - 1, l].copy()
                m = int(np.floor(reshuffled)) + int(st["rank"].random() < (reshuffled - np.floor(reshuffled)))
                pos = st["rank"].choice(n_experts, size=min(m, n_experts), replace=False)
                cur[pos] = cur[st["rank"].permutation(pos)]
                rk[s, l] = cur
    return StageTrace(n_steps, bounds, rk, zipf_s, seed, -1.0 if reshuffled is None else float(reshuffled))


def trace_logits(trace: StageTrace, step: int, layer: int, batch: int) -> np.ndarray:
    """fp32 logits[batch, E] of one (step, layer): ln p_stage + Gumbel, from a counter-based
    seed so that any (step, layer) can be drawn alone and in any order."""
    s = trace.stage_of(step)
    rng = np.random.default_rng(np.random.SeedSequence([trace.seed, 0x5AE3, step, layer]))
    pop = zipf_popularity(trace.rankings[s, layer], trace.zipf_s)
    return router_logits(rng, batch, trace.rankings.shape[2], "zipf", pop)


def trace_activations(trace: StageTrace, step: int, batch: int, d_model: int) -> np.ndarray:
    """bf16 bits x[batch, d] of one step (the same token activation feeds every layer)."""
    rng = np.random.default_rng(np.random.SeedSequence([trace.seed, 0xAC71, step]))
    return activations(rng, batch, d_model)
