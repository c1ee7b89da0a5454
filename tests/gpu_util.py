"""Helpers shared by the GPU parity tests: upload seeded inputs, run the C-ABI calls, compare with
the oracle.  Tolerances are the ones the benchmark contract states: indices bit-exact, gate weights
1e-6, FFN / combine outputs max-abs <= 2e-2 and relative L2 <= 1e-2."""
import numpy as np
import torch

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
        stats["shared_y"] = assert_close(host(layer.shared_rows(T)), ref["shared_y"], "shared_y")
    stats["out"] = assert_close(host(out), ref["out"], "out")
    return ref, stats
