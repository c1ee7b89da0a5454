"""Pins of the oracle's expert FFN and combine: library float64 dense SwiGLU, the odd-part
identity of SiLU, zeroed experts, routing independence, equivariances, dense mixture at k = E."""
import numpy as np
import pytest
import torch

from paper_2608_21614_b200 import inputs as gen


def _f64(bits):
    return torch.from_numpy(gen.bf16_bits_to_f32(bits).astype(np.float64))


def _dense(xb, g, u, dn):
    x = _f64(xb)
    return (torch.nn.functional.silu(x @ _f64(g).T) * (x @ _f64(u).T)) @ _f64(dn).T


def test_single_expert_equals_library_dense_swiglu(oracle):
    rng = np.random.default_rng(0)
    d, f, T = 48, 80, 7                         # d != f: a transposed operand cannot pass
    g, u, dn = gen.expert_weights(rng, d, f)
    x = gen.activations(rng, T, d)
    r = oracle.moe_step(np.zeros((T, 1), np.float32), x, 1, [g], [u], [dn])
    assert np.array_equal(r["topk_idx"], np.zeros((T, 1)))
    assert np.all(r["topk_w"] == 1.0)
    ref = _dense(x, g, u, dn).numpy()
    assert np.allclose(r["out"], ref, rtol=1e-12, atol=1e-12)
    assert np.allclose(r["y_packed"], ref, rtol=1e-12, atol=1e-12)


def test_silu_closed_forms(oracle):
    """silu(0) = 0, and silu(z) - silu(-z) = z because sigma(z) + sigma(-z) = 1."""
    z = np.array([0.0, 0.5, -1.25, 3.0, 7.5], np.float32)           # exactly representable in bf16
    x = gen.to_bf16_bits(np.stack([z, np.ones_like(z)], 1))          # d = 2: x = (z, 1)
    g = gen.to_bf16_bits(np.array([[1.0, 0.0], [-1.0, 0.0]], np.float32))   # hidden 0: +z, hidden 1: -z
    u = gen.to_bf16_bits(np.array([[0.0, 1.0], [0.0, 1.0]], np.float32))    # up = 1 for both
    dn = gen.to_bf16_bits(np.array([[1.0, -1.0], [0.0, 0.0]], np.float32))
    y = oracle.expert_ffn(x, np.array([0, len(z)], np.int32), [g], [u], [dn])
    assert np.allclose(y[:, 0], z.astype(np.float64), rtol=0, atol=1e-15)
    assert np.all(y[:, 1] == 0.0)
    dn_plus = gen.to_bf16_bits(np.array([[1.0, 0.0], [0.0, 0.0]], np.float32))
    y0 = oracle.expert_ffn(x[:1], np.array([0, 1], np.int32), [g], [u], [dn_plus])
    assert y0[0, 0] == 0.0
    # large |z|: silu(z) -> z and silu(-z) -> -0 without overflow
    big = gen.to_bf16_bits(np.array([[800.0, 1.0]], np.float32))
    yb = oracle.expert_ffn(big, np.array([0, 1], np.int32), [g], [u], [dn_plus])
    assert yb[0, 0] == 800.0


def test_zeroed_down_projection_contributes_nothing(oracle):
    cfg = gen.LayerConfig("t", 32, 64, 4, 2, 12, seed=4)
    li = gen.layer_inputs(cfg)
    li.down[1] = np.zeros_like(li.down[1])
    r = oracle.moe_step(li.logits, li.x, 2, li.gate, li.up, li.down)
    seg = slice(r["offsets"][1], r["offsets"][2])
    assert r["counts"][1] > 0 and np.all(r["y_packed"][seg] == 0.0)


def test_identical_experts_make_routing_irrelevant(oracle):
    """All experts equal and gate weights summing to 1 -> the layer is the dense FFN, whatever the
    routing: pins sum(w) = 1 together with the un-permute."""
    cfg = gen.LayerConfig("t", 40, 24, 6, 3, 17, seed=9)
    li = gen.layer_inputs(cfg, n_distinct_experts=1)
    r = oracle.moe_step(li.logits, li.x, 3, li.gate, li.up, li.down)
    ref = _dense(li.x, li.gate[0], li.up[0], li.down[0]).numpy()
    assert np.allclose(r["out"], ref, rtol=1e-12, atol=1e-12)


def test_k_equals_E_is_dense_softmax_mixture(oracle):
    cfg = gen.LayerConfig("t", 24, 40, 5, 5, 6, seed=2)
    li = gen.layer_inputs(cfg)
    r = oracle.moe_step(li.logits, li.x, 5, li.gate, li.up, li.down)
    p = torch.softmax(torch.from_numpy(li.logits.astype(np.float64)), 1)
    ref = sum(p[:, e:e + 1] * _dense(li.x, li.gate[e], li.up[e], li.down[e]) for e in range(5)).numpy()
    assert np.allclose(r["out"], ref, rtol=1e-11, atol=1e-12)


def test_topk_mixture_against_library_ops(oracle):
    """General case re-expressed with library top-k / softmax / dense ops (no repacking at all)."""
    cfg = gen.LayerConfig("t", 32, 48, 8, 2, 21, d_ff_shared=16, seed=6)
    li = gen.layer_inputs(cfg)
    r = oracle.moe_step(li.logits, li.x, 2, li.gate, li.up, li.down, shared=li.shared)
    lg = torch.from_numpy(li.logits.astype(np.float64))
    val, idx = torch.topk(lg, 2, dim=1)
    w = torch.softmax(val, 1)
    ref = _dense(li.x, *li.shared)
    for e in range(8):
        ye = _dense(li.x, li.gate[e], li.up[e], li.down[e])
        for j in range(2):
            ref = ref + (idx[:, j] == e).double()[:, None] * w[:, j:j + 1] * ye
    assert np.allclose(r["out"], ref.numpy(), rtol=1e-11, atol=1e-12)
    assert np.allclose(r["shared_y"], _dense(li.x, *li.shared).numpy(), rtol=1e-12, atol=1e-12)


def test_token_permutation_and_expert_relabel_equivariance(oracle):
    cfg = gen.LayerConfig("t", 32, 32, 7, 3, 10, seed=8)
    li = gen.layer_inputs(cfg)
    base = oracle.moe_step(li.logits, li.x, 3, li.gate, li.up, li.down)["out"]
    rng = np.random.default_rng(1)
    tp = rng.permutation(10)
    out_tp = oracle.moe_step(li.logits[tp], li.x[tp], 3, li.gate, li.up, li.down)["out"]
    assert np.array_equal(out_tp, base[tp])
    ep = rng.permutation(7)                                  # new id n holds old expert ep[n]
    out_ep = oracle.moe_step(li.logits[:, ep], li.x, 3, [li.gate[e] for e in ep], [li.up[e] for e in ep],
                             [li.down[e] for e in ep])["out"]
    assert np.array_equal(out_ep, base)                      # slot order is by logit, not by id


def test_fp32_accumulation_is_far_inside_tolerance(oracle):
    cfg = gen.layer_config("c1")
    li = gen.layer_inputs(cfg)
    a = oracle.moe_step(li.logits, li.x, cfg.top_k, li.gate, li.up, li.down)["out"]
    b = oracle.moe_step(li.logits, li.x, cfg.top_k, li.gate, li.up, li.down, acc_fp32=True)["out"]
    assert np.abs(a - b).max() < 2e-4                       # two orders below the 2e-2 bound
    assert np.linalg.norm(a - b) / np.linalg.norm(a) < 1e-4
    assert 0.2 < a.std() < 1.0                               # the regime the error budget assumes


def test_combine_alone_matches_definition_on_integers(oracle):
    y = np.arange(12, dtype=np.float64).reshape(6, 2)         # 3 tokens, k = 2
    inv = np.array([3, 0, 1, 5, 4, 2], np.int32)
    w = np.array([[0.5, 0.25], [1.0, 0.0], [2.0, 3.0]])
    sh = np.full((3, 2), 100.0)
    out = oracle.combine(y, inv, w, sh)
    exp = [[0.5 * 6 + 0.25 * 0 + 100, 0.5 * 7 + 0.25 * 1 + 100],
           [2 + 100, 3 + 100],
           [2 * 8 + 3 * 4 + 100, 2 * 9 + 3 * 5 + 100]]
    assert out.tolist() == exp
