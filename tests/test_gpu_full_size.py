"""Parity at the benchmark's full sizes (configs 2, 3, 4), in the launch configuration bench.py
times (default context), and the stack configuration at its own layer shape.  Decode sizes and the
2048-token fine-grained prefill are compared in full; the Mixtral-shaped 1024-token prefill on
packed rows around every tile boundary, which the oracle computes one by one, with the integer
outputs and the combine checked in full."""
import numpy as np
import pytest
import torch

from paper_2608_21614_b200 import inputs as gen

pytestmark = pytest.mark.gpu
TENSOR = 0      # SAEM_FFN_AUTO: the path bench.py times (matrix-vector kernels up to 8 rows, tiled tcgen05 beyond)
STREAMING = 2   # SAEM_FFN_TENSOR: the weight-streaming tcgen05 kernels up to 64 rows per segment


@pytest.mark.parametrize("path", [TENSOR, STREAMING], ids=["auto-tiled", "streaming"])
def test_c2_mixtral_shaped_decode_full(oracle, path):
    import gpu_util as g
    li = gen.layer_inputs(gen.layer_config("c2"))
    layer = g.make_layer(li, path)
    ref, stats = g.run_stepwise_and_compare(layer, li, oracle)
    assert int((ref["counts"] > 0).sum()) >= 6
    layer.close()


@pytest.mark.parametrize("name,T,routing", [("c3", 32, "zipf"), ("c4", 1, "zipf"), ("c4", 8, "zipf"),
                                            ("c4", 8, "uniform"), ("c4", 64, "zipf"), ("c4", 64, "uniform"),
                                            ("qwen3", 1, "zipf"), ("qwen3", 8, "zipf"), ("qwen3", 200, "zipf"),
                                            ("ernie", 8, "zipf")])
def test_fine_grained_decode_full(oracle, name, T, routing):
    import gpu_util as g
    li = gen.layer_inputs(gen.layer_config(name, tokens=T, routing=routing))
    layer = g.make_layer(li, TENSOR)
    ref, _ = g.run_stepwise_and_compare(layer, li, oracle)
    layer.close()
    if 8 < T <= 64:        # the streaming kernels at the same full size (SAEM_FFN_AUTO takes the tiled ones here)
        layer = g.make_layer(li, STREAMING)
        g.run_stepwise_and_compare(layer, li, oracle, ref=ref)
        layer.close()


@pytest.mark.parametrize("name,T", [("c4", 1), ("c4", 4), ("c4", 8), ("qwen3", 1), ("qwen3", 4), ("qwen3", 8),
                                    ("ernie", 1), ("ernie", 8), ("c5", 1), ("c5", 4), ("c5", 8)])
def test_single_launch_decode_step_full_shapes(oracle, name, T):
    """The two-launch decode step (saem_moe_step, at most 8 tokens) on the layer shapes of the
    benchmark configurations and of the paper's two models."""
    import gpu_util as g
    li = gen.layer_inputs(gen.layer_config(name, tokens=T), n_distinct_experts=4)
    layer = g.make_layer(li, 4)                     # SAEM_FFN_DECODE_FUSED: the one-launch form up to 8 tokens
    n0 = layer.launches()
    g.run_single_call_and_compare(layer, li, oracle)
    assert layer.launches() - n0 in (1, 2)      # one cooperative launch, or two where that is not available
    layer.close()


@pytest.mark.parametrize("name,T,one_launch", [("qwen3", 8, True), ("c4", 6, True), ("ernie", 8, False), ("c5", 8, False),
                                               ("qwen3", 9, False), ("c5", 4, True)])
def test_default_path_one_launch_range(oracle, name, T, one_launch):
    """SAEM_FFN_AUTO: saem_moe_step is one launch up to 4 tokens on every layer, and up to 8 tokens on
    layers of many small experts (at most 20 MB each); five launches otherwise.  Either way the step
    agrees with the oracle."""
    import gpu_util as g
    li = gen.layer_inputs(gen.layer_config(name, tokens=T), n_distinct_experts=4)
    layer = g.make_layer(li, 0)
    n0 = layer.launches()
    g.run_single_call_and_compare(layer, li, oracle)
    n = layer.launches() - n0
    assert (n in (1, 2)) if one_launch else n >= 5
    layer.close()


PAIRS = 3       # SAEM_FFN_TENSOR_PAIRS: the CTA-pair form of the tiled kernels wherever the shape allows


@pytest.mark.parametrize("T", [1, 8])
def test_c5_layer_shape_matrix_vector_kernels(oracle, T):
    """One layer of the 32-layer stack configuration (d_model 4096, d_ff 14336, 8 experts, top-2,
    Zipf 1.2) at the batch sizes the stack is decoded with: these run on the matrix-vector kernels
    (224 k-chunks per 16-row group in the down projection)."""
    import gpu_util as g
    li = gen.layer_inputs(gen.layer_config("c5", tokens=T), n_distinct_experts=4)
    layer = g.make_layer(li, TENSOR)
    g.run_stepwise_and_compare(layer, li, oracle)
    layer.close()


@pytest.mark.parametrize("batch", [1, 8])
def test_c5_full_shape_partially_resident_stack_subsample(oracle, batch):
    """The stack configuration at its own layer shape with half of the experts resident: 4 layers,
    4 fixed slots per layer + 4 temporary slots, the first 4096-step trace's opening 16 steps and the
    16 steps around its first stage boundary.  Every kept layer-step's output is compared with the
    oracle under the same (layer, expert) -> weight-set mapping, and the hit / load counters with an
    independent host simulation of the policy."""
    import gpu_util as g
    L, E, k, d, f, C, temp = 4, 8, 2, 4096, 14336, 4, 4
    trace = gen.stage_trace(4096, L, E, 1.2, seed=0)
    b1 = int(trace.boundaries[1])
    keep = sorted(set(range(16)) | set(range(max(b1 - 8, 0), b1 + 8)))
    steps = keep[-1] + 1
    rng = np.random.default_rng(np.random.SeedSequence([0, 77]))
    weights = [gen.expert_weights(rng, d, f) for _ in range(4)]
    outs, st, final, run = g.run_stack(trace, weights, L, E, k, d, f, C, temp, batch, steps, set(keep))
    sim, sim_final = g.simulate_stack(trace, oracle, L, E, k, C, temp, batch, steps)
    assert (st.active, st.hits, st.temp_hits) == (sim["active"], sim["hits"], sim["temp_hits"])
    assert (st.pair_total, st.pair_hits) == (sim["pair_total"], sim["pair_hits"])
    assert st.demand_loads == sim["demand"] and st.boundary_loads == sim["boundary"]
    assert [sorted(x) for x in final] == sim_final
    assert st.demand_loads > 0 and st.boundaries >= 1
    for t, out in zip(keep, outs):
        x = gen.trace_activations(trace, t, batch, d)
        for l in range(L):
            ws = [run.store.weights(l, e) for e in range(E)]
            ref = oracle.moe_step(gen.trace_logits(trace, t, l, batch), x, k, [w[0] for w in ws],
                                  [w[1] for w in ws], [w[2] for w in ws])
            g.assert_close(g.host(out[l]), ref["out"], "step %d layer %d" % (t, l))
    run.close()


def _check_integer_outputs(g, layer, li, oracle):
    cfg = li.cfg
    E, k = cfg.n_experts, cfg.top_k
    P = cfg.tokens * k
    ridx, rw = oracle.route(li.logits, k)
    rc, ro, rp, ri, rx = oracle.repack(ridx, li.x, E)
    assert np.array_equal(g.host(layer.topk_idx), ridx)
    assert np.abs(g.host(layer.topk_w).astype(np.float64) - rw).max() <= g.W_TOL
    assert np.array_equal(g.host(layer.counts)[:E], rc) and np.array_equal(g.host(layer.offsets)[:E + 1], ro)
    assert np.array_equal(g.host(layer.perm), rp) and np.array_equal(g.host(layer.inv_perm), ri)
    assert np.array_equal(g.host(layer.x_packed[:P]), rx)
    return ro, ri, rx


_C3_PREFILL_REF = {}


@pytest.mark.parametrize("path", [TENSOR, PAIRS], ids=["one-cta-tiles", "cta-pairs"])
def test_c3_prefill_2048_in_full(oracle, path):
    """The fine-grained layer at 2048 tokens (12 288 pair rows + 2 x 2048 shared rows) through the tiled
    kernels, one CTA per tile (the default for this shape) and CTA pairs (forced): every packed row
    and every output element against the oracle."""
    import gpu_util as g
    cfg = gen.layer_config("c3", tokens=2048)
    li = gen.layer_inputs(cfg)
    if "ref" not in _C3_PREFILL_REF:
        _C3_PREFILL_REF["ref"] = oracle.moe_step(li.logits, li.x, cfg.top_k, li.gate, li.up, li.down, shared=li.shared)
    layer = g.make_layer(li, path)
    g.run_stepwise_and_compare(layer, li, oracle, ref=_C3_PREFILL_REF["ref"])
    layer.close()


def test_c2_prefill_1024_every_tile_boundary(oracle):
    """The Mixtral-shaped layer at 1024 tokens (2048 packed rows: CTA pairs by the default rule).  The
    oracle computes, one by one, the first and last row of every segment and the rows on both sides
    of every 128-row boundary inside it (each 256-token item is split between the two CTAs of a pair
    at row 128), plus a few random rows; integer outputs and the combine are checked in full."""
    import gpu_util as g
    cfg = gen.layer_config("c2", tokens=1024)
    li = gen.layer_inputs(cfg)
    T, k, E = cfg.tokens, cfg.top_k, cfg.n_experts
    P = T * k
    layer = g.make_layer(li, TENSOR)
    out = layer.step(g.dev(li.logits), g.dev(li.x), T)
    torch.cuda.synchronize()
    assert layer.device_status() == 0
    ro, ri, rx = _check_integer_outputs(g, layer, li, oracle)
    rng = np.random.default_rng(0)
    rows = []
    for e in range(E):
        lo, hi = int(ro[e]), int(ro[e + 1])
        if hi > lo:
            cand = {lo, hi - 1} | {int(r) for r in rng.integers(lo, hi, 3)}
            for edge in range(lo + 128, hi, 128):
                cand |= {edge - 1, edge, min(edge + 1, hi - 1)}
            rows += sorted(cand)
    rows = np.array(rows)
    sub_off = np.searchsorted(rows, ro).astype(np.int32)            # rows are sorted, so per-expert ranges
    y_ref = oracle.expert_ffn(rx[rows], sub_off, li.gate, li.up, li.down)
    y_gpu = g.host(layer.y_packed[:P])
    g.assert_close(y_gpu[rows], y_ref, "sampled y_packed rows")
    assert np.isfinite(y_gpu).all()
    # combine: in full, from the GPU's own FFN outputs (isolates the merge)
    c_ref = oracle.combine(y_gpu.astype(np.float64), ri, g.host(layer.topk_w).astype(np.float64), None)
    assert np.abs(g.host(out).astype(np.float64) - c_ref).max() <= 1e-4
    o = g.host(out)
    assert np.isfinite(o).all() and 0.3 < o.std() < 3.0
    layer.close()
