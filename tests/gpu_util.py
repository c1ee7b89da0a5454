"""Helpers shared by the GPU parity tests: upload seeded inputs, run the C-ABI calls, compare with
the oracle.  Tolerances are the ones the benchmark contract states: indices bit-exact, gate weights
1e-6, FFN / combine outputs max-abs <= 2e-2 and relative L2 <= 1e-2."""
import numpy as np
import torch

from paper_2608_21614_b200 import inputs as gen

MAX_ABS = 2e-2
REL_L2 = 1e-2
W_TOL = 1e-6


def dev(a, device="cuda:0"):
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


def host(t):
    return t.detach().cpu().numpy()


def assert_close(got, ref, what=""):
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    assert np.isfinite(got).all(), what + ": non-finite values"
    err = np.abs(got - ref)
    worst = np.unravel_index(np.argmax(err), err.shape) if err.size else ()
    max_abs = float(err.max()) if err.size else 0.0
    denom = float(np.linalg.norm(ref))
    rel = float(np.linalg.norm(got - ref)) / denom if denom > 0 else float(np.linalg.norm(got - ref))
    assert max_abs <= MAX_ABS, "%s: max-abs %.3e at %s (got %r ref %r)" % (what, max_abs, worst, got[worst], ref[worst])
    assert rel <= REL_L2, "%s: rel-L2 %.3e" % (what, rel)
    return max_abs, rel


def make_layer(li, ffn_path, max_tokens=None, **kw):
    """MoELayer with every expert of LayerInputs `li` resident."""
    from paper_2608_21614_b200.layer import MoELayer
    c = li.cfg
    layer = MoELayer(c.d_model, c.d_ff, c.n_experts, c.top_k, max_tokens or c.tokens, c.d_ff_shared,
                     ffn_path=ffn_path, **kw)
    layer.load_all(li.gate, li.up, li.down, li.shared)
    return layer


def shared_rows(layer, T):
    """Output of the shared expert(s) of the last step, [T, d] fp32: the sum of the in-layer shared
    experts' rows of y_packed, or the separate shared context's output."""
    if layer.S:
        P = T * layer.k
        return layer.y_packed[P:P + layer.S * T].view(layer.S, T, layer.d).sum(0)
    return layer.shared_y[:T]


def run_stepwise_and_compare(layer, li, oracle, ref=None):
    """Runs the four calls one by one and compares every output with the oracle's."""
    c = li.cfg
    T, k = c.tokens, c.top_k
    P = T * k
    if ref is None:
        ref = oracle.moe_step(li.logits, li.x, k, li.gate, li.up, li.down, shared=li.shared)
    logits, x = dev(li.logits), dev(li.x)
    out = layer.step(logits, x, T)
    torch.cuda.synchronize()
    assert layer.device_status() == 0
    assert np.array_equal(host(layer.topk_idx[:T]), ref["topk_idx"]), "topk_idx"
    assert np.abs(host(layer.topk_w[:T]).astype(np.float64) - ref["topk_w"]).max() <= W_TOL, "topk_w"
    E = c.n_experts
    assert np.array_equal(host(layer.counts)[:E], ref["counts"]), "counts"
    assert np.array_equal(host(layer.offsets)[:E + 1], ref["offsets"]), "offsets"
    if layer.S:                                      # in-layer shared experts: one segment of T rows each
        assert np.all(host(layer.counts)[E:] == T), "shared counts"
        assert np.array_equal(host(layer.offsets)[E:], P + T * np.arange(layer.S + 1)), "shared offsets"
        assert np.array_equal(host(layer.x_packed[P:P + layer.S * T]), np.tile(li.x, (layer.S, 1))), "shared x rows"
    assert np.array_equal(host(layer.perm[:P]), ref["perm"]), "perm"
    assert np.array_equal(host(layer.inv_perm[:P]), ref["inv_perm"]), "inv_perm"
    assert np.array_equal(host(layer.x_packed[:P]), ref["x_packed"]), "x_packed"
    stats = {"y_packed": assert_close(host(layer.y_packed[:P]), ref["y_packed"], "y_packed")}
    if li.shared is not None:
        stats["shared_y"] = assert_close(host(shared_rows(layer, T)), ref["shared_y"], "shared_y")
    stats["out"] = assert_close(host(out), ref["out"], "out")
    return ref, stats


def run_single_call_and_compare(layer, li, oracle, ref=None):
    """The whole step through saem_moe_step (for at most 8 tokens: the two-launch decode path) against
    the oracle: the index outputs left in the workspace bit-exact, the layer output within tolerance."""
    c = li.cfg
    T, k, E = c.tokens, c.top_k, c.n_experts
    P, ES = T * k, c.n_experts + layer.S
    if ref is None:
        ref = oracle.moe_step(li.logits, li.x, k, li.gate, li.up, li.down, shared=li.shared)
    out = torch.full((T, c.d_model), float("nan"), dtype=torch.float32, device=layer.device)
    layer.step_fused_call(dev(li.logits), dev(li.x), T, out)
    torch.cuda.synchronize()
    assert layer.device_status() == 0
    ctx = layer.ctx
    assert np.array_equal(host(ctx.step_tensor(0, (T, k), torch.int32)), ref["topk_idx"]), "topk_idx"
    assert np.abs(host(ctx.step_tensor(1, (T, k), torch.float32)).astype(np.float64) - ref["topk_w"]).max() <= W_TOL
    counts, offsets = host(ctx.step_tensor(2, (ES,), torch.int32)), host(ctx.step_tensor(3, (ES + 1,), torch.int32))
    assert np.array_equal(counts[:E], ref["counts"]) and np.array_equal(offsets[:E + 1], ref["offsets"])
    if layer.S:
        assert np.all(counts[E:] == T) and np.array_equal(offsets[E:], P + T * np.arange(layer.S + 1))
    assert np.array_equal(host(ctx.step_tensor(4, (P,), torch.int32)), ref["perm"]), "perm"
    assert np.array_equal(host(ctx.step_tensor(5, (P,), torch.int32)), ref["inv_perm"]), "inv_perm"
    return ref, assert_close(host(out), ref["out"], "out of the single-call step")


# ------------------------------------------------------------------ partially resident stacks
def run_stack(trace, weights, L, E, k, d, f, C, temp, batch, steps, keep, policy="stage", eap=None, miss_mode="temp"):
    from paper_2608_21614_b200.stack import StackRunner
    run = StackRunner(d, f, E, k, L, C, temp, batch, weights, policy=policy, recorded_eap=eap, miss_mode=miss_mode)
    # warm set: the C most popular experts of stage 0 (stand-in for the calibration warm-up)
    run.warm([list(np.argsort(trace.rankings[0, l])[:C]) for l in range(L)])
    outs = []
    bounds = set(int(b) for b in trace.boundaries[1:])
    for t in range(steps):
        if t in bounds:
            run.boundary()
        lg = np.stack([gen.trace_logits(trace, t, l, batch) for l in range(L)])
        x = gen.trace_activations(trace, t, batch, d)
        out = run.step(torch.from_numpy(lg).cuda(), torch.from_numpy(x).cuda())
        if t in keep:
            torch.cuda.synchronize()
            outs.append(out.clone())
    torch.cuda.synchronize()
    from paper_2608_21614_b200 import binding as B
    assert B.saem_last_device_status(run.h) == 0
    stats = run.stats
    final = [list(s) for s in run.slot_expert]
    store = run.store
    return outs, stats, final, run


def simulate_stack(trace, oracle, L, E, k, C, temp, batch, steps):
    """Independent host simulation of the policy: residency sets, a ring of temporary slots,
    the pairwise-swap planner at boundaries; routing from the oracle."""
    res = [set(int(e) for e in np.argsort(trace.rankings[0, l])[:C]) for l in range(L)]
    ring = [None] * temp
    nxt = 0
    log = np.zeros((L, E), np.int64)
    st = dict(active=0, hits=0, temp_hits=0, demand=0, boundary=0, pair_total=0, pair_hits=0)
    bounds = set(int(b) for b in trace.boundaries[1:])
    for t in range(steps):
        if t in bounds:
            for l in range(L):
                while True:
                    non = [e for e in range(E) if e not in res[l]]
                    best = min(non, key=lambda e: (-log[l, e], e))
                    worst = min(res[l], key=lambda e: (log[l, e], -e))
                    if log[l, best] <= log[l, worst]:
                        break
                    res[l].remove(worst)
                    res[l].add(best)
                    st["boundary"] += 1
                    ring = [None if r == (l, best) else r for r in ring]
            log[:] = 0
        for l in range(L):
            idx, _ = oracle.route(gen.trace_logits(trace, t, l, batch), k)
            cnt = np.bincount(idx.ravel(), minlength=E)
            need = []
            for e in np.nonzero(cnt)[0]:
                e = int(e)
                st["active"] += 1
                st["pair_total"] += int(cnt[e])
                if e in res[l]:
                    st["hits"] += 1
                    st["pair_hits"] += int(cnt[e])
                else:
                    need.append(e)
                    if (l, e) in ring:
                        st["temp_hits"] += 1
            while True:
                missing = [e for e in need if (l, e) not in ring]
                if not missing:
                    break
                for e in missing:
                    ring[nxt] = (l, e)
                    nxt = (nxt + 1) % temp
                    st["demand"] += 1
            log[l] += cnt
    return st, [sorted(r) for r in res]
