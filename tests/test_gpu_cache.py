"""Expert-slot cache on the GPU: load / evict / query / wait semantics, ordering of loads against
enqueued FFNs, and the partially resident stack (50 % of the experts per layer in fixed slots,
misses through temporary slots, planner at stage boundaries) against full residency and against
an independent host simulation of the same policy."""
import numpy as np
import pytest
import torch

from paper_2608_21614_b200 import inputs as gen

pytestmark = pytest.mark.gpu


def _small_experts(n, d, f, seed):
    rng = np.random.default_rng(seed)
    return [gen.expert_weights(rng, d, f) for _ in range(n)]


def test_cache_api_semantics():
    import gpu_util as g
    from paper_2608_21614_b200 import binding as B
    d, f, E = 128, 128, 4
    ws = _small_experts(E, d, f, 1)
    cfg = B.make_config(d, f, E, 2, 8, n_layers=2, slots_per_layer=2, temp_slots=2)
    ctx = B.Context(cfg)
    h = ctx.handle
    packed = [ctx.pack(*w) for w in ws]
    cs = torch.cuda.Stream()
    assert B.saem_cache_query(h, 0, 0) == (-1, 0)
    B.saem_cache_load(h, 0, 0, 0, packed[0], cs)
    slot, _ = B.saem_cache_query(h, 0, 0)
    assert slot == 0
    cs.synchronize()
    assert B.saem_cache_query(h, 0, 0) == (0, 1)
    assert B.saem_cache_load(h, 0, 1, 0, packed[1], cs, check=False) == B.SAEM_ERR_SLOT_BUSY
    assert B.saem_cache_load(h, 0, 0, 1, packed[0], cs, check=False) == B.SAEM_ERR_INVALID_ARG      # already resident
    B.saem_cache_load(h, 1, 3, 1, packed[3], cs)                       # layer 1, slot 1 -> global slot 3
    assert B.saem_cache_query(h, 1, 3)[0] == 3
    # temporary slots: round-robin over the pool (global slots 4, 5), old bindings dropped
    B.saem_cache_load(h, 0, 2, B.SAEM_TEMP, packed[2], cs)
    B.saem_cache_load(h, 1, 0, B.SAEM_TEMP, packed[0], cs)
    assert B.saem_cache_query(h, 0, 2)[0] == 4 and B.saem_cache_query(h, 1, 0)[0] == 5
    B.saem_cache_load(h, 1, 1, B.SAEM_TEMP, packed[1], cs)             # recycles pool slot 0
    assert B.saem_cache_query(h, 0, 2)[0] == -1 and B.saem_cache_query(h, 1, 1)[0] == 4
    assert B.saem_cache_load(h, 0, 0, B.SAEM_TEMP, packed[0], cs, check=False) == B.SAEM_ERR_INVALID_ARG
    B.saem_cache_evict(h, 0, 0)
    assert B.saem_cache_query(h, 0, 0) == (-1, 0)
    assert B.saem_cache_evict(h, 0, 0, check=False) == B.SAEM_ERR_NOT_RESIDENT
    assert B.saem_cache_wait(h, 0, 0, None, check=False) == B.SAEM_ERR_NOT_RESIDENT
    assert B.saem_cache_wait(h, 1, 3, None, check=False) == B.SAEM_OK
    torch.cuda.synchronize()
    ctx.close()


def test_load_is_ordered_after_enqueued_reads_and_before_later_ones(oracle):
    """Swap the expert in a slot right after enqueuing an FFN that reads it: the first result
    uses the old weights, the next one the new weights."""
    import gpu_util as g
    from paper_2608_21614_b200 import binding as B
    d, f, T = 256, 256, 24
    wa, wb = _small_experts(2, d, f, 5)
    cfg = B.make_config(d, f, 2, 1, T, slots_per_layer=1, temp_slots=1)
    ctx = B.Context(cfg)
    h = ctx.handle
    pa, pb = ctx.pack(*wa), ctx.pack(*wb)
    cs = torch.cuda.Stream()
    rng = np.random.default_rng(2)
    x = gen.activations(rng, T, d)
    xd = g.dev(x)
    off0 = g.dev(np.array([0, T, T], np.int32))          # every row belongs to expert 0
    off1 = g.dev(np.array([0, 0, T], np.int32))          # ... to expert 1
    y0 = torch.zeros((T, d), dtype=torch.float32, device="cuda:0")
    y1 = torch.zeros((T, d), dtype=torch.float32, device="cuda:0")
    B.saem_cache_load(h, 0, 0, 0, pa, cs)
    for _ in range(3):                                     # a queue of reads of the slot
        B.saem_expert_ffn(h, 0, xd, off0, T, [0], y0)
    B.saem_cache_evict(h, 0, 0)
    B.saem_cache_load(h, 0, 1, 0, pb, cs)                  # same slot, other expert, no host sync in between
    assert B.saem_expert_ffn(h, 0, xd, off0, T, [0], y0, check=False) == B.SAEM_ERR_NOT_RESIDENT
    B.saem_expert_ffn(h, 0, xd, off1, T, [1], y1)
    torch.cuda.synchronize()
    seg = np.array([0, T], np.int32)
    g.assert_close(g.host(y0), oracle.expert_ffn(x, seg, [wa[0]], [wa[1]], [wa[2]]), "old expert")
    g.assert_close(g.host(y1), oracle.expert_ffn(x, seg, [wb[0]], [wb[1]], [wb[2]]), "new expert")
    assert B.saem_last_device_status(h) == 0
    ctx.close()


def test_half_resident_stack_equals_full_residency_and_simulation(oracle):
    import gpu_util as g
    L, E, k, d, f, batch, steps = 3, 8, 2, 256, 256, 4, 40
    trace = gen.stage_trace(steps, L, E, 1.2, seed=11, mean_stage_len=8.0)
    assert len(trace.boundaries) >= 3
    weights = _small_experts(6, d, f, 3)                     # 24 (layer, expert) pairs share 6 weight sets
    keep = set(range(steps))
    full, st_full, _, run_full = g.run_stack(trace, weights, L, E, k, d, f, E, 0, batch, steps, keep)
    half, st_half, final_half, run_half = g.run_stack(trace, weights, L, E, k, d, f, E // 2, 4, batch, steps, keep)
    # routing does not depend on placement: identical bits under 50 % and 100 % residency
    for a, b in zip(full, half):
        assert torch.equal(a, b)
    assert st_full.chr() == 1.0 and st_full.demand_loads == 0 and st_full.boundary_loads == 0
    # the policy bookkeeping equals an independent simulation, number for number
    sim, sim_final = g.simulate_stack(trace, oracle, L, E, k, E // 2, 4, batch, steps)
    assert (st_half.active, st_half.hits, st_half.temp_hits) == (sim["active"], sim["hits"], sim["temp_hits"])
    assert (st_half.pair_total, st_half.pair_hits) == (sim["pair_total"], sim["pair_hits"])
    assert st_half.demand_loads == sim["demand"] and st_half.boundary_loads == sim["boundary"]
    assert [sorted(s) for s in final_half] == sim_final
    assert 0.3 < st_half.chr() < 1.0 and st_half.demand_loads > 0 and st_half.boundary_loads > 0
    # floating-point parity of sampled layer-steps against the oracle (same weight mapping)
    for t in (0, int(trace.boundaries[1]), steps - 1):
        x = gen.trace_activations(trace, t, batch, d)
        for l in range(L):
            ws = [run_half.store.weights(l, e) for e in range(E)]
            ref = oracle.moe_step(gen.trace_logits(trace, t, l, batch), x, k, [w[0] for w in ws],
                                  [w[1] for w in ws], [w[2] for w in ws])
            g.assert_close(g.host(half[t][l]), ref["out"], "step %d layer %d" % (t, l))
    run_full.close()
    run_half.close()


def test_replay_policies_share_bits_and_oracle_is_no_worse(oracle):
    """The prediction-oracle replay (Sec. VI-D): the same trace under the online policy, the
    clairvoyant policy fed with the recorded per-stage counts, and token-level LRU.  Routing is
    independent of placement, so every policy yields the same output bits; the clairvoyant
    planner never has fewer hits at a boundary than the lag-one planner on this trace."""
    import gpu_util as g
    L, E, k, d, f, batch, steps = 2, 8, 2, 128, 128, 2, 48
    trace = gen.stage_trace(steps, L, E, 1.2, seed=5, mean_stage_len=8.0, reshuffled=None)   # independent stages
    weights = _small_experts(4, d, f, 9)
    keep = {steps - 1}
    ref, st_full, _, run0 = g.run_stack(trace, weights, L, E, k, d, f, E, 0, batch, steps, keep)
    eap = run0.finish()
    # the recorded EAP equals routing counts from the oracle, stage by stage
    bounds = list(trace.boundaries) + [steps]
    for s in range(len(bounds) - 1):
        cnt = np.zeros((L, E), np.int64)
        for t in range(int(bounds[s]), int(bounds[s + 1])):
            for l in range(L):
                idx, _ = oracle.route(gen.trace_logits(trace, t, l, batch), k)
                cnt[l] += np.bincount(idx.ravel(), minlength=E)
        assert np.array_equal(eap[s], cnt)
    res = {}
    for policy in ("stage", "oracle", "lru"):
        outs, st, _, run = g.run_stack(trace, weights, L, E, k, d, f, 4, 4, batch, steps, keep, policy, eap)
        assert torch.equal(outs[0], ref[0]), policy
        res[policy] = st
        run.close()
    assert res["oracle"].hits >= res["stage"].hits
    assert res["lru"].boundary_loads == 0 and res["lru"].demand_loads > 0
    run0.close()


def test_missed_experts_read_in_place_from_mapped_host_memory(oracle):
    """saem_cache_map_host: an expert without a slot is bound to its packed copy in pinned host memory and
    the matrix-vector kernels read it over the host link.  API semantics, the FFN against the oracle with
    one expert in HBM and one in host memory, and the half-resident stack with this miss mode: identical
    bits to full residency, the same hits as the temporary-slot mode, no on-demand copies."""
    import gpu_util as g
    from paper_2608_21614_b200 import binding as B
    d, f, T = 256, 384, 6
    wa, wb = _small_experts(2, d, f, 15)
    ctx = B.Context(B.make_config(d, f, 2, 1, T, slots_per_layer=1, temp_slots=1))
    h = ctx.handle
    pa, pb = ctx.pack(*wa), ctx.pack(*wb)
    B.saem_cache_load(h, 0, 0, 0, pa)
    assert B.saem_cache_map_host(h, 0, 0, pb, check=False) == B.SAEM_ERR_INVALID_ARG         # has a slot
    assert B.saem_cache_map_host(h, 0, 1, torch.empty(16, dtype=torch.uint8), check=False) == B.SAEM_ERR_INVALID_ARG   # not pinned
    B.saem_cache_map_host(h, 0, 1, pb)
    assert B.saem_cache_query(h, 0, 1) == (B.SAEM_HOST_MAPPED, 1)
    rng = np.random.default_rng(4)
    x = gen.activations(rng, T, d)
    off = np.array([0, 2, T], np.int32)                   # rows 0..1 -> expert 0 (HBM slot), rows 2..5 -> expert 1 (host)
    y = torch.full((T, d), float("nan"), dtype=torch.float32, device="cuda:0")
    B.saem_expert_ffn(h, 0, g.dev(x), g.dev(off), T, None, y)
    torch.cuda.synchronize()
    ref = oracle.expert_ffn(x, off, [wa[0], wb[0]], [wa[1], wb[1]], [wa[2], wb[2]])
    g.assert_close(g.host(y), ref, "one expert in HBM, one read from host memory")
    B.saem_cache_evict(h, 0, 1)
    assert B.saem_cache_query(h, 0, 1) == (-1, 0)
    assert B.saem_expert_ffn(h, 0, g.dev(x), g.dev(off), T, [1], y, check=False) == B.SAEM_ERR_NOT_RESIDENT
    assert B.saem_last_device_status(h) == 0
    ctx.close()

    L, E, k, batch, steps = 3, 8, 2, 4, 40
    d, f = 256, 256
    trace = gen.stage_trace(steps, L, E, 1.2, seed=11, mean_stage_len=8.0)
    weights = _small_experts(6, d, f, 3)
    keep = set(range(steps))
    full, _, _, run_full = g.run_stack(trace, weights, L, E, k, d, f, E, 0, batch, steps, keep)
    temp, st_temp, _, run_temp = g.run_stack(trace, weights, L, E, k, d, f, E // 2, 4, batch, steps, keep)
    host, st_host, _, run_host = g.run_stack(trace, weights, L, E, k, d, f, E // 2, 4, batch, steps, keep, miss_mode="host")
    for a, b in zip(full, host):
        assert torch.equal(a, b)
    assert (st_host.active, st_host.hits, st_host.boundary_loads) == (st_temp.active, st_temp.hits, st_temp.boundary_loads)
    assert st_host.demand_loads == 0 and st_host.host_reads == st_host.active - st_host.hits > 0
    for r in (run_full, run_temp, run_host):
        r.close()


@pytest.mark.parametrize("batch", [2, 12])
def test_fully_resident_stack_without_readback_uses_the_single_call(oracle, batch):
    """With every expert resident nothing on the host depends on the routing: read_counts=False drives each
    layer through the single saem_moe_step call (the one-launch decode step at batch 2), with no host
    synchronisation per layer.  Every layer-step against the oracle."""
    import gpu_util as g
    from paper_2608_21614_b200.stack import StackRunner
    L, E, k, d, f, steps = 3, 8, 2, 256, 384, 5
    trace = gen.stage_trace(steps, L, E, 1.2, seed=21, mean_stage_len=3.0)
    weights = _small_experts(5, d, f, 8)
    run = StackRunner(d, f, E, k, L, E, 0, batch, weights, read_counts=False)
    assert not run.read_counts
    run.warm([list(range(E)) for _ in range(L)])
    for t in range(steps):
        lg = np.stack([gen.trace_logits(trace, t, l, batch) for l in range(L)])
        x = gen.trace_activations(trace, t, batch, d)
        out = run.step(torch.from_numpy(lg).cuda(), torch.from_numpy(x).cuda())
        torch.cuda.synchronize()
        for l in range(L):
            ws = [run.store.weights(l, e) for e in range(E)]
            ref = oracle.moe_step(lg[l], x, k, [w[0] for w in ws], [w[1] for w in ws], [w[2] for w in ws])
            g.assert_close(g.host(out[l]), ref["out"], "step %d layer %d" % (t, l))
    from paper_2608_21614_b200 import binding as B
    assert B.saem_last_device_status(run.h) == 0
    assert run.stats.layer_steps == 0                     # no read-back, hence no statistics
    run.close()
