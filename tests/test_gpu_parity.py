"""GPU parity: every C-ABI call against the CPU oracle on the same seeded inputs."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2608_21614_b200 import inputs as gen

pytestmark = pytest.mark.gpu

AUTO, SCALAR, TENSOR, PAIRS, FUSED = 0, 1, 2, 3, 4


@pytest.fixture(scope="module")
def B():
    from paper_2608_21614_b200 import binding
    return binding


def _g():
    import gpu_util
    return gpu_util


@pytest.mark.parametrize("path", [SCALAR, TENSOR], ids=["scalar", "tensor"])
def test_c1_every_call(oracle, path):
    g = _g()
    li = gen.layer_inputs(gen.layer_config("c1"))
    layer = g.make_layer(li, path)
    ref, stats = g.run_stepwise_and_compare(layer, li, oracle)
    # run twice: bit-identical outputs (no atomics decide any order)
    y1, o1 = layer.y_packed.clone(), layer.out.clone()
    layer.step(g.dev(li.logits), g.dev(li.x), li.cfg.tokens)
    torch.cuda.synchronize()
    assert torch.equal(y1, layer.y_packed) and torch.equal(o1, layer.out)
    layer.close()


@pytest.mark.parametrize("T,E,k,d,f,fs", [(1, 1, 1, 128, 128, 0), (1, 60, 4, 256, 384, 256), (1, 60, 4, 256, 384, 384),
                                          (8, 8, 8, 128, 256, 0), (5, 120, 8, 256, 128, 128), (8, 8, 2, 512, 1024, 0),
                                          (3, 16, 2, 2048, 1408, 2816)])
def test_tiny_batches_matrix_vector_path(oracle, T, E, k, d, f, fs):
    """Batches of at most 8 tokens take the row-split matrix-vector kernels (ffn_path AUTO)."""
    g = _g()
    cfg = gen.LayerConfig("t", d, f, E, k, T, fs, "zipf", 1.1, seed=100 + T + E)
    li = gen.layer_inputs(cfg, n_distinct_experts=min(E, 6))
    layer = g.make_layer(li, AUTO)
    g.run_stepwise_and_compare(layer, li, oracle)
    y1 = layer.y_packed.clone()
    layer.step(g.dev(li.logits), g.dev(li.x), T)
    torch.cuda.synchronize()
    assert torch.equal(y1, layer.y_packed)                 # deterministic
    layer.close()


@pytest.mark.parametrize("T,E,k,d,f,fs", [(1, 1, 1, 128, 128, 0), (1, 60, 4, 256, 384, 384), (8, 8, 8, 128, 256, 0),
                                          (5, 120, 8, 256, 128, 128), (8, 8, 2, 512, 1024, 0), (7, 33, 5, 384, 640, 0),
                                          (3, 16, 2, 2048, 1408, 2816), (8, 12, 1, 256, 128, 2048), (2, 8, 2, 2432, 256, 0)])
def test_single_launch_decode_step(oracle, T, E, k, d, f, fs):
    """saem_moe_step for at most 8 tokens (top-k at most 8): gate, repack indices, gate/up, down
    projection and merge in one launch.  Index outputs bit-exact, output within tolerance, run to
    run bit-identical, and (bf16 hidden activations, fp32 sums on both sides) close to the four
    separate calls."""
    g = _g()
    cfg = gen.LayerConfig("t", d, f, E, k, T, fs, "zipf", 1.1, seed=200 + T + E)
    li = gen.layer_inputs(cfg, n_distinct_experts=min(E, 6))
    layer = g.make_layer(li, FUSED)
    assert layer.shared is None
    n0 = layer.launches()
    ref, _ = g.run_single_call_and_compare(layer, li, oracle)
    assert layer.launches() - n0 in (1, 2)      # one cooperative launch, or two where that is not available
    logits, x = g.dev(li.logits), g.dev(li.x)
    o1 = torch.empty((T, d), dtype=torch.float32, device="cuda:0")
    o2 = torch.empty_like(o1)
    layer.step_fused_call(logits, x, T, o1)
    layer.step_fused_call(logits, x, T, o2)
    four = layer.step(logits, x, T)
    torch.cuda.synchronize()
    assert torch.equal(o1, o2)
    assert float((o1 - four).abs().max()) <= 2e-3
    layer.close()


def test_single_launch_decode_step_bf16_out_and_absent_expert(oracle, B):
    """bf16 output of the two-launch step, and a routed expert without a slot: the status word says
    NOT_RESIDENT and the expert contributes nothing (the other experts' terms are still merged)."""
    g = _g()
    cfg = gen.LayerConfig("t", 256, 384, 6, 2, 4, 0, "normal", seed=31)
    li = gen.layer_inputs(cfg)
    from paper_2608_21614_b200.layer import MoELayer
    layer = g.make_layer(li, FUSED, out_dtype=B.SAEM_OUT_BF16)
    out = torch.zeros((4, 256), dtype=torch.uint16, device="cuda:0")
    layer.step_fused_call(g.dev(li.logits), g.dev(li.x), 4, out)
    torch.cuda.synchronize()
    ref = oracle.moe_step(li.logits, li.x, 2, li.gate, li.up, li.down)
    g.assert_close(gen.bf16_bits_to_f32(g.host(out)), ref["out"], "bf16 out")
    layer.close()
    missing = int(ref["topk_idx"][0, 0])
    layer = MoELayer(256, 384, 6, 2, 4)
    for e in range(6):
        if e != missing:
            layer.load_expert(0, e, e, li.gate[e], li.up[e], li.down[e])
    o = torch.zeros((4, 256), dtype=torch.float32, device="cuda:0")
    layer.step_fused_call(g.dev(li.logits), g.dev(li.x), 4, o)
    torch.cuda.synchronize()
    assert layer.device_status() == B.SAEM_ERR_NOT_RESIDENT
    zero = [np.zeros_like(m) for m in (li.gate[missing], li.up[missing], li.down[missing])]
    gate, up, down = list(li.gate), list(li.up), list(li.down)
    gate[missing], up[missing], down[missing] = zero
    ref2 = oracle.moe_step(li.logits, li.x, 2, gate, up, down)
    g.assert_close(g.host(o), ref2["out"], "absent expert contributes zero")
    layer.close()


@pytest.mark.parametrize("T,E,k", [(8, 64, 4), (2, 8, 2)])
def test_single_launch_step_token_without_any_resident_expert(oracle, B, T, E, k):
    """None of token 0's experts has a slot: its output row is zero, the other tokens' rows merge what
    is resident, the status word says NOT_RESIDENT.  The first case has more than 16 active experts
    (merge by tickets), the second at most 16 (merge inside the CTA that owns the columns)."""
    g = _g()
    cfg = gen.LayerConfig("t", 256, 256, E, k, T, 0, "uniform", seed=77)
    li = gen.layer_inputs(cfg, n_distinct_experts=min(E, 6))
    ref = oracle.moe_step(li.logits, li.x, k, li.gate, li.up, li.down)
    missing = set(int(e) for e in ref["topk_idx"][0])
    from paper_2608_21614_b200.layer import MoELayer
    layer = MoELayer(256, 256, E, k, T, ffn_path=FUSED)
    for e in range(E):
        if e not in missing:
            layer.load_expert(0, e, e, li.gate[e], li.up[e], li.down[e])
    o = torch.full((T, 256), 7.0, dtype=torch.float32, device="cuda:0")
    layer.step_fused_call(g.dev(li.logits), g.dev(li.x), T, o)
    torch.cuda.synchronize()
    assert layer.device_status() == B.SAEM_ERR_NOT_RESIDENT
    gate, up, down = list(li.gate), list(li.up), list(li.down)
    for e in missing:
        gate[e], up[e], down[e] = np.zeros_like(gate[e]), np.zeros_like(up[e]), np.zeros_like(down[e])
    ref2 = oracle.moe_step(li.logits, li.x, k, gate, up, down)
    out = g.host(o)
    assert not out[0].any()
    g.assert_close(out, ref2["out"], "tokens beside the one without a resident expert")
    layer.close()


@pytest.mark.parametrize("T,E,k,d,f,fs", [
    (300, 8, 2, 256, 256, 0),        # one pair of weight blocks in gate/up, a single block in down
    (700, 12, 3, 512, 384, 384),     # odd number of f-blocks (a one-block item), in-layer shared expert, ragged tiles
    (1500, 16, 2, 256, 640, 0),      # several 256-token tiles per expert, five f-blocks
])
def test_cta_pair_tiles(oracle, T, E, k, d, f, fs):
    """The cta_group::2 form of the tiled kernels (forced: the default rule wants d_model >= 4096)."""
    g = _g()
    cfg = gen.LayerConfig("t", d, f, E, k, T, fs, "zipf", 1.1, seed=3 * T + E)
    li = gen.layer_inputs(cfg)
    layer = g.make_layer(li, PAIRS)
    g.run_stepwise_and_compare(layer, li, oracle)
    y1, o1 = layer.y_packed.clone(), layer.out.clone()
    layer.step(g.dev(li.logits), g.dev(li.x), li.cfg.tokens)
    torch.cuda.synchronize()
    assert torch.equal(y1, layer.y_packed) and torch.equal(o1, layer.out)      # run to run: bit-identical
    layer.close()
    # the pair MMA adds the same products in the same order as the one-CTA tiles: identical bits
    single = g.make_layer(li, TENSOR)
    single.step(g.dev(li.logits), g.dev(li.x), li.cfg.tokens)
    torch.cuda.synchronize()
    assert torch.equal(y1, single.y_packed) and torch.equal(o1, single.out)
    single.close()


@pytest.mark.parametrize("path", [SCALAR, TENSOR, AUTO], ids=["scalar", "tensor", "auto"])
@pytest.mark.parametrize("T,E,k,d,f,fs", [
    (1, 1, 1, 128, 128, 0),          # dense FFN, one token
    (17, 6, 2, 256, 384, 0),         # 9..64 tokens: tiled kernels under AUTO, streaming kernels under TENSOR
    (24, 40, 4, 128, 256, 256),      # 17..64 tokens with an in-layer shared expert
    (1, 60, 4, 256, 384, 256),       # decode batch 1: four one-row segments, 56 empty, shared expert
    (9, 8, 8, 128, 256, 0),          # k == E
    (33, 60, 4, 256, 128, 0),        # E not a multiple of 32, ragged T
    (70, 128, 8, 128, 128, 128),     # E = 128, k = 8
    (300, 8, 2, 256, 256, 0),        # segments beyond one 16..64-row tile; fused repack limit
    (1500, 16, 2, 128, 128, 0),      # two-kernel repack, several 256-row token tiles per expert
])
def test_small_shapes(oracle, path, T, E, k, d, f, fs):
    g = _g()
    cfg = gen.LayerConfig("t", d, f, E, k, T, fs, "zipf", 1.1, seed=T + E)
    li = gen.layer_inputs(cfg)
    layer = g.make_layer(li, path)
    g.run_stepwise_and_compare(layer, li, oracle)
    layer.close()


@pytest.mark.parametrize("path", [SCALAR, TENSOR, PAIRS, AUTO], ids=["scalar", "tensor", "cta-pairs", "auto"])
def test_segment_sizes_around_tile_edges(oracle, path):
    """One expert, k = 1: the segment is the whole batch; sizes straddle every tile boundary."""
    g = _g()
    d, f = 256, 256
    rng = np.random.default_rng(77)
    gate, up, down = gen.expert_weights(rng, d, f)
    from paper_2608_21614_b200.layer import MoELayer
    layer = MoELayer(d, f, 1, 1, 300, ffn_path=path)
    layer.load_all([gate], [up], [down])
    for T in (1, 7, 8, 9, 15, 16, 17, 31, 32, 33, 63, 64, 65, 127, 128, 129, 255, 256, 257, 300):
        x = gen.activations(rng, T, d)
        ref = oracle.expert_ffn(x, np.array([0, T], np.int32), [gate], [up], [down])
        y = torch.full((300, d), float("nan"), dtype=torch.float32, device="cuda:0")
        import paper_2608_21614_b200.binding as B
        B.saem_expert_ffn(layer.ctx.handle, 0, g.dev(x), None, T, None, y)
        torch.cuda.synchronize()
        g.assert_close(g.host(y[:T]), ref, "T=%d" % T)
        assert torch.isnan(y[T:]).all(), "rows beyond the segment were written (T=%d)" % T
    assert layer.device_status() == 0
    layer.close()


@pytest.mark.parametrize("path", [TENSOR, AUTO], ids=["tensor", "auto"])
@pytest.mark.parametrize("max_tokens,fs", [(40, 0), (48, 0), (40, 256), (48, 256), (33, 0)])
def test_token_tiles_between_32_and_64_rows(oracle, path, max_tokens, fs):
    """Contexts whose largest batch is 33..48 tokens: the streaming kernels load a token tile as
    32-row boxes, so the tile (and its shared-memory stage) must hold a whole number of boxes.  One
    routed expert with k = 1 (and optionally one in-layer shared expert) makes every segment exactly
    max_tokens rows long."""
    g = _g()
    d, f = 256, 256
    cfg = gen.LayerConfig("t", d, f, 1, 1, max_tokens, fs, "normal", seed=40 + max_tokens)
    li = gen.layer_inputs(cfg)
    layer = g.make_layer(li, path)
    assert layer.S == (1 if fs else 0)
    g.run_stepwise_and_compare(layer, li, oracle)
    y1 = layer.y_packed.clone()
    layer.step(g.dev(li.logits), g.dev(li.x), max_tokens)
    torch.cuda.synchronize()
    assert torch.equal(y1, layer.y_packed)
    layer.close()


def test_route_special_values(oracle, B):
    g = _g()
    rows = [
        [-0.0, 0.0, -np.inf, np.nan, 1.0, -1.0, 0.5, 0.5],
        [np.inf, 1.0, np.inf, 0.0, 0.0, 0.0, 0.0, 0.0],
        [-np.inf] * 8,
        [0.0] * 8,
        [300.0, 0.0, -300.0, 1.0, 2.0, 3.0, 4.0, 5.0],
        [np.nan] * 8,
    ]
    logits = np.array(rows, np.float32)
    rng = np.random.default_rng(1)
    quant = rng.integers(-2, 3, size=(64, 8)).astype(np.float32)          # many exact ties
    logits = np.concatenate([logits, quant])
    for k, renorm in ((1, 1), (3, 1), (8, 1), (3, 0)):
        cfg = B.make_config(128, 128, 8, k, len(logits), renorm=renorm)
        ctx = B.Context(cfg)
        idx = torch.empty((len(logits), k), dtype=torch.int32, device="cuda:0")
        w = torch.empty((len(logits), k), dtype=torch.float32, device="cuda:0")
        B.saem_route(ctx.handle, g.dev(logits), len(logits), idx, w)
        torch.cuda.synchronize()
        ridx, rw = oracle.route(logits, k, renorm=bool(renorm))
        assert np.array_equal(g.host(idx), ridx), (k, renorm)
        assert np.isfinite(g.host(w)).all()
        assert np.abs(g.host(w).astype(np.float64) - rw).max() <= g.W_TOL, (k, renorm)
        ctx.close()


@pytest.mark.parametrize("E,k", [(8, 2), (60, 4), (64, 6), (128, 8), (128, 128), (33, 33)])
def test_route_random(oracle, B, E, k):
    g = _g()
    rng = np.random.default_rng(E * 7 + k)
    T = 257 if k <= 8 else 40          # the repack table bounds pairs x experts
    logits = rng.standard_normal((T, E)).astype(np.float32) * 3
    ctx = B.Context(B.make_config(128, 128, E, k, T))
    idx = torch.empty((T, k), dtype=torch.int32, device="cuda:0")
    w = torch.empty((T, k), dtype=torch.float32, device="cuda:0")
    B.saem_route(ctx.handle, g.dev(logits), T, idx, w)
    ridx, rw = oracle.route(logits, k)
    assert np.array_equal(g.host(idx), ridx)
    assert np.abs(g.host(w).astype(np.float64) - rw).max() <= g.W_TOL
    ctx.close()


def test_repack_skew_and_paper_example(oracle, B):
    g = _g()
    # the paper's worked example (Sec. IV-E)
    idx = np.array([[0, 2], [1, 2], [1, 3], [0, 2]], np.int32)
    cases = [(idx, 4)]
    cases.append((np.full((50, 1), 3, np.int32), 6))                      # every token picks the same expert
    rng = np.random.default_rng(2)
    cases.append((np.stack([rng.permutation(60)[:4] for _ in range(777)]).astype(np.int32), 60))
    cases.append((np.stack([rng.permutation(64)[:6] for _ in range(2048)]).astype(np.int32), 64))   # prefill size
    # the multi-CTA index phase at its largest sizes: 128 experts top-8 at 4096 tokens (32 768 pairs), 65 535 pairs,
    # and every pair of 40 blocks on one expert
    cases.append((np.argsort(rng.random((4096, 128)), axis=1)[:, :8].astype(np.int32), 128))
    cases.append((np.argsort(rng.random((13107, 64)), axis=1)[:, :5].astype(np.int32), 64))
    cases.append((np.full((40000, 1), 5, np.int32), 9))
    for idx, E in cases:
        T, k = idx.shape
        d = 128
        x = rng.integers(0, 65535, size=(T, d)).astype(np.uint16)
        ctx = B.Context(B.make_config(d, 128, E, k, T))
        P = T * k
        counts = torch.empty(E, dtype=torch.int32, device="cuda:0")
        offsets = torch.empty(E + 1, dtype=torch.int32, device="cuda:0")
        perm = torch.empty(P, dtype=torch.int32, device="cuda:0")
        inv = torch.empty(P, dtype=torch.int32, device="cuda:0")
        xp = torch.empty((P, d), dtype=torch.uint16, device="cuda:0")
        B.saem_repack(ctx.handle, g.dev(idx), g.dev(x), T, counts, offsets, perm, inv, xp)
        rc, ro, rp, ri, rx = oracle.repack(idx, x, E)
        assert np.array_equal(g.host(counts), rc)
        assert np.array_equal(g.host(offsets), ro)
        assert np.array_equal(g.host(perm), rp)
        assert np.array_equal(g.host(inv), ri)
        assert np.array_equal(g.host(xp), rx)
        assert B.saem_last_device_status(ctx.handle) == 0
        ctx.close()


@pytest.mark.parametrize("T,S", [(700, 1), (700, 0), (100, 1)], ids=["two-kernel-shared", "two-kernel", "fused-shared"])
def test_repack_drops_invalid_expert_ids(oracle, B, T, S):
    """Expert ids outside [0, E), injected on the host: the status word says INVALID_ARG, the pair is
    dropped from every output, and the valid pairs are packed exactly as the oracle packs them (the
    oracle is given the valid pairs only, as a ragged problem: invalid pairs are routed to a spare
    expert E whose segment comes last).  With in-layer shared experts and more than 2048 pairs the
    gather runs as a second kernel over all T*k rows and must skip the rows that hold no pair."""
    g = _g()
    E, k, d = 12, 3, 128
    rng = np.random.default_rng(T + S)
    idx = np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
    bad = rng.choice(T * k, 9, replace=False)
    idx.ravel()[bad[:5]] = E + 3
    idx.ravel()[bad[5:]] = -1
    x = rng.integers(0, 65535, size=(T, d)).astype(np.uint16)
    ctx = B.Context(B.make_config(d, 128, E, k, T, n_shared=S))
    P, R = T * k, T * (k + S)
    counts = torch.empty(E + S, dtype=torch.int32, device="cuda:0")
    offsets = torch.empty(E + S + 1, dtype=torch.int32, device="cuda:0")
    perm = torch.full((P,), 12345, dtype=torch.int32, device="cuda:0")
    inv = torch.empty(P, dtype=torch.int32, device="cuda:0")
    xp = torch.full((R, d), 7, dtype=torch.uint16, device="cuda:0")
    B.saem_repack(ctx.handle, g.dev(idx), g.dev(x), T, counts, offsets, perm, inv, xp)
    assert B.saem_last_device_status(ctx.handle) == B.SAEM_ERR_INVALID_ARG
    spare = np.where((idx < 0) | (idx >= E), E, idx).astype(np.int32)
    rc, ro, rp, ri, rx = oracle.repack(spare, x, E + 1)
    valid = int(ro[E])
    assert valid == P - 9
    assert np.array_equal(g.host(counts)[:E], rc[:E])
    assert np.array_equal(g.host(offsets)[:E], ro[:E])
    assert int(g.host(offsets)[E]) == (P if S else valid)
    assert np.array_equal(g.host(perm)[:valid], rp[:valid]) and np.all(g.host(perm)[valid:] == -1)
    ri_expect = np.where(ri >= valid, -1, ri)
    assert np.array_equal(g.host(inv), ri_expect)
    assert np.array_equal(g.host(xp)[:valid], rx[:valid])
    assert np.all(g.host(xp)[valid:P] == 7)                         # rows without a pair are never written
    if S:
        assert np.array_equal(g.host(xp)[P:], np.tile(x, (S, 1)))
    ctx.close()


@pytest.mark.parametrize("fs,merge", [(256, True), (768, True), (768, False)],
                         ids=["own-context", "in-layer", "in-layer-width-forced-separate"])
def test_step_calls_agree_bit_for_bit(oracle, fs, merge):
    """saem_moe_step and saem_moe_step_host give the bits of the four separate calls, with the
    shared expert in a context of its own (width not a multiple of d_ff, or forced) and inside
    the layer's grouped launch (width 2 x d_ff)."""
    g = _g()
    cfg = gen.LayerConfig("t", 256, 384, 12, 3, 20, fs, "zipf", 1.1, seed=5)
    li = gen.layer_inputs(cfg)
    layer = g.make_layer(li, TENSOR, merge_shared=merge)
    assert (layer.S == 2) == (fs == 768 and merge)
    g.run_stepwise_and_compare(layer, li, oracle)
    logits, x = g.dev(li.logits), g.dev(li.x)
    ref_out = layer.step(logits, x, cfg.tokens).clone()
    out2 = torch.empty_like(ref_out)
    layer.step_fused_call(logits, x, cfg.tokens, out2)
    torch.cuda.synchronize()
    assert torch.equal(ref_out, out2)
    lh = torch.from_numpy(li.logits).pin_memory()
    xh = torch.from_numpy(li.x).pin_memory()
    oh = torch.empty((cfg.tokens, cfg.d_model), dtype=torch.float32).pin_memory()
    layer.step_host(lh, xh, cfg.tokens, oh)
    assert torch.equal(ref_out.cpu(), oh)
    outs = [torch.zeros_like(oh).pin_memory() for _ in range(3)]      # three steps enqueued without waiting in between
    for o in outs:
        layer.step_host_async(lh, xh, cfg.tokens, o)
    torch.cuda.synchronize()
    assert all(torch.equal(ref_out.cpu(), o) for o in outs)
    ref = oracle.moe_step(li.logits, li.x, cfg.top_k, li.gate, li.up, li.down, shared=li.shared)
    g.assert_close(oh.numpy(), ref["out"], "out via host call")
    layer.close()


def test_bf16_output_option(oracle):
    g = _g()
    from paper_2608_21614_b200 import binding as B
    cfg = gen.layer_config("c1")
    li = gen.layer_inputs(cfg)
    layer = g.make_layer(li, TENSOR, out_dtype=B.SAEM_OUT_BF16)
    out = layer.step(g.dev(li.logits), g.dev(li.x), cfg.tokens)
    torch.cuda.synchronize()
    ref = oracle.moe_step(li.logits, li.x, cfg.top_k, li.gate, li.up, li.down)
    g.assert_close(gen.bf16_bits_to_f32(g.host(out)), ref["out"], "bf16 out")
    layer.close()


def test_error_statuses(B):
    g = _g()
    cfg = B.make_config(128, 128, 4, 2, 8)
    ctx = B.Context(cfg)
    z = torch.zeros(4096, dtype=torch.float32, device="cuda:0")
    zi = torch.zeros(4096, dtype=torch.int32, device="cuda:0")
    assert B.saem_route(ctx.handle, z, 9, zi, z, check=False) == B.SAEM_ERR_SHAPE          # T = max_tokens + 1
    assert B.saem_route(ctx.handle, z, 8, zi, z, check=False) == B.SAEM_OK                 # T = max_tokens
    assert B.saem_route(ctx.handle, None, 8, zi, z, check=False) == B.SAEM_ERR_INVALID_ARG
    assert B.saem_expert_ffn(ctx.handle, 1, z, zi, 4, None, z, check=False) == B.SAEM_ERR_INVALID_ARG   # bad layer
    assert B.saem_expert_ffn(ctx.handle, 0, z, zi, 17, None, z, check=False) == B.SAEM_ERR_SHAPE
    assert B.saem_expert_ffn(ctx.handle, 0, z, zi, 4, [2], z, check=False) == B.SAEM_ERR_NOT_RESIDENT
    assert B.saem_cache_evict(ctx.handle, 0, 1, check=False) == B.SAEM_ERR_NOT_RESIDENT
    assert B.saem_cache_load(ctx.handle, 0, 1, 9, z, check=False) == B.SAEM_ERR_INVALID_ARG              # bad slot
    assert B.saem_cache_load(ctx.handle, 0, 1, B.SAEM_TEMP, z, check=False) == B.SAEM_ERR_INVALID_ARG    # no temp slots
    assert B.saem_cache_query(ctx.handle, 0, 1) == (-1, 0)
    bad = B.make_config(100, 128, 4, 2, 8)
    assert B.saem_slot_bytes(bad) == 0
    assert B.saem_create_status(bad, ctx.slot_ptr, 1 << 30, ctx.ws_ptr, 1 << 30) == B.SAEM_ERR_SHAPE
    assert B.saem_create_status(cfg, ctx.slot_ptr + 16, 1 << 30, ctx.ws_ptr, 1 << 30) == B.SAEM_ERR_ALIGNMENT
    assert B.saem_create_status(cfg, ctx.slot_ptr, 16, ctx.ws_ptr, 1 << 30) == B.SAEM_ERR_WORKSPACE
    ctx.close()


@pytest.mark.parametrize("path", [SCALAR, TENSOR], ids=["scalar", "tensor"])
def test_absent_expert_sets_device_status_and_leaves_rows(oracle, path, B):
    g = _g()
    cfg = gen.LayerConfig("t", 128, 128, 4, 2, 16, seed=3)
    li = gen.layer_inputs(cfg)
    from paper_2608_21614_b200.layer import MoELayer
    layer = MoELayer(128, 128, 4, 2, 16, ffn_path=path)
    for e in (0, 1, 3):                                   # expert 2 never loaded
        layer.load_expert(0, e, e, li.gate[e], li.up[e], li.down[e])
    layer.route(g.dev(li.logits), 16)
    layer.repack(g.dev(li.x), 16)
    layer.y_packed.fill_(float("nan"))
    layer.expert_ffn(16)
    torch.cuda.synchronize()
    ref = oracle.moe_step(li.logits, li.x, 2, li.gate, li.up, li.down)
    assert ref["counts"][2] > 0
    assert layer.device_status() == B.SAEM_ERR_NOT_RESIDENT
    assert layer.device_status() == 0                      # reading clears it
    o = ref["offsets"]
    y = g.host(layer.y_packed)
    assert np.isnan(y[o[2]:o[3]]).all()
    keep = np.r_[0:o[2], o[3]:o[4]]
    g.assert_close(y[keep], ref["y_packed"][keep], "other segments")
    layer.close()


def test_step_is_graph_capturable_and_replays_identically(oracle):
    """With every expert resident the four calls read nothing back on the host and launch
    data-independent grids, so a whole step can be captured in a CUDA graph and replayed."""
    g = _g()
    cfg = gen.LayerConfig("t", 256, 384, 12, 3, 24, 768, "zipf", 1.1, seed=7)
    li = gen.layer_inputs(cfg)
    layer = g.make_layer(li, TENSOR)
    logits, x = g.dev(li.logits), g.dev(li.x)
    eager = layer.step(logits, x, cfg.tokens).clone()
    torch.cuda.synchronize()
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        layer.step(logits, x, cfg.tokens)                  # warm-up on the capture stream
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=s):
            layer.step(logits, x, cfg.tokens)
        layer.out.zero_()
        layer.y_packed.zero_()
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
    assert torch.equal(layer.out[:cfg.tokens], eager)
    # new routing through the same graph: the device-built work lists follow the data
    li2 = gen.layer_inputs(dataclasses.replace(cfg, seed=8))
    logits.copy_(g.dev(li2.logits))
    x.copy_(g.dev(li2.x))
    torch.cuda.synchronize()
    with torch.cuda.stream(s):
        graph.replay()
        torch.cuda.synchronize()
    ref = oracle.moe_step(li2.logits, li2.x, cfg.top_k, li.gate, li.up, li.down, shared=li.shared)
    g.assert_close(g.host(layer.out[:cfg.tokens]), ref["out"], "graph replay on new inputs")
    assert layer.device_status() == 0
    layer.close()


def test_capture_step_helper_batch_1(oracle):
    """MoELayer.capture_step at batch 1 (matrix-vector kernels): replays equal the eager step and follow new inputs."""
    g = _g()
    cfg = gen.LayerConfig("t", 256, 384, 60, 4, 1, 384, "zipf", 1.1, seed=11)
    li = gen.layer_inputs(cfg)
    layer = g.make_layer(li, AUTO)
    logits, x = g.dev(li.logits), g.dev(li.x)
    eager = layer.step(logits, x, 1).clone()
    graph = layer.capture_step(logits, x, 1)
    layer.out.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(layer.out[:1], eager)
    li2 = gen.layer_inputs(dataclasses.replace(cfg, seed=12))
    logits.copy_(g.dev(li2.logits))
    x.copy_(g.dev(li2.x))
    graph.replay()
    torch.cuda.synchronize()
    ref = oracle.moe_step(li2.logits, li2.x, cfg.top_k, li.gate, li.up, li.down, shared=li.shared)
    g.assert_close(g.host(layer.out[:1]), ref["out"], "graph replay, batch 1, new inputs")
    assert layer.device_status() == 0
    layer.close()


def test_single_launch_step_in_a_graph_follows_new_inputs(oracle):
    """The one-launch decode step (a cooperative launch) recorded in a CUDA graph with other steps, as a
    decoder records its layers: replays follow new logits and activations, and the step's barrier
    counter and tickets are left ready for the next replay."""
    g = _g()
    cfg = gen.LayerConfig("t", 256, 384, 60, 4, 2, 768, "zipf", 1.1, seed=17)
    li = gen.layer_inputs(cfg)
    layer = g.make_layer(li, AUTO)
    logits, x = g.dev(li.logits), g.dev(li.x)
    out = torch.empty((2, 256), dtype=torch.float32, device="cuda:0")
    n0 = layer.launches()
    layer.step_fused_call(logits, x, 2, out)             # first call outside the capture
    assert layer.launches() - n0 in (1, 2)
    eager = out.clone()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=s):
            for _ in range(3):
                layer.step_fused_call(logits, x, 2, out)
    torch.cuda.current_stream().wait_stream(s)
    out.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, eager)
    li2 = gen.layer_inputs(dataclasses.replace(cfg, seed=18))
    logits.copy_(g.dev(li2.logits))
    x.copy_(g.dev(li2.x))
    for _ in range(2):
        graph.replay()
    torch.cuda.synchronize()
    ref = oracle.moe_step(li2.logits, li2.x, cfg.top_k, li.gate, li.up, li.down, shared=li.shared)
    g.assert_close(g.host(out), ref["out"], "graph replay of the one-launch step on new inputs")
    assert layer.device_status() == 0
    layer.close()


def test_empty_batch_and_limits(B):
    """T = 0 is a no-op everywhere (repack still zeroes counts and offsets); T = max_tokens works and
    T = max_tokens + 1 is refused before anything is enqueued."""
    g = _g()
    E, k, d, f, maxT = 6, 2, 128, 128, 5
    cfg = B.make_config(d, f, E, k, maxT)
    ctx = B.Context(cfg)
    h = ctx.handle
    n0 = B.saem_launch_count(h)
    counts = torch.full((E,), 7, dtype=torch.int32, device="cuda:0")
    offsets = torch.full((E + 1,), 7, dtype=torch.int32, device="cuda:0")
    z = torch.zeros(maxT * k * d, dtype=torch.float32, device="cuda:0")
    zi = torch.zeros(maxT * k, dtype=torch.int32, device="cuda:0")
    zx = torch.zeros((maxT * k, d), dtype=torch.uint16, device="cuda:0")
    assert B.saem_route(h, z, 0, zi, z, check=False) == B.SAEM_OK
    assert B.saem_combine(h, z, zi, z, 0, None, z, check=False) == B.SAEM_OK
    assert B.saem_expert_ffn(h, 0, zx, offsets, 0, None, z, check=False) == B.SAEM_OK
    assert B.saem_launch_count(h) == n0                       # nothing was launched
    assert B.saem_repack(h, zi, zx, 0, counts, offsets, zi, zi, zx, check=False) == B.SAEM_OK
    torch.cuda.synchronize()
    assert counts.sum().item() == 0 and offsets.sum().item() == 0
    for call in (lambda T: B.saem_route(h, z, T, zi, z, check=False),
                 lambda T: B.saem_repack(h, zi, zx, T, counts, offsets, zi, zi, zx, check=False),
                 lambda T: B.saem_combine(h, z, zi, z, T, None, z, check=False)):
        assert call(maxT) == B.SAEM_OK
        assert call(maxT + 1) == B.SAEM_ERR_SHAPE
        assert call(-1) == B.SAEM_ERR_SHAPE
    assert B.saem_expert_ffn(h, 0, zx, offsets, maxT * k + 1, None, z, check=False) == B.SAEM_ERR_SHAPE
    assert B.saem_expert_ffn(h, 0, zx.view(-1)[1:], offsets, 2, None, z, check=False) == B.SAEM_ERR_ALIGNMENT
    torch.cuda.synchronize()
    assert B.saem_last_device_status(h) == 0
    ctx.close()


@pytest.mark.parametrize("T,path", [(8, AUTO), (48, AUTO), (48, TENSOR), (700, AUTO)])
def test_ffn_counters_are_zero_between_calls(oracle, T, path):
    """Every counter through which the FFN kernels' CTAs meet (split-item arrivals of the streaming
    kernels; per-expert completion counts and the item counter of the tiled kernels, whose down launch
    starts while the gate/up launch's last items still run) is back at zero after each call, and a
    second step on other inputs is as correct as the first."""
    g = _g()
    cfg = gen.LayerConfig("t", 512, 384, 12, 3, T, 384, "zipf", 1.1, seed=5 + T)
    li = gen.layer_inputs(cfg)
    layer = g.make_layer(li, path)
    counters = layer.ctx.step_tensor(10, (656,), torch.int32)
    for seed in (5 + T, 905 + T):
        li2 = gen.layer_inputs(dataclasses.replace(cfg, seed=seed))
        li2 = dataclasses.replace(li2, gate=li.gate, up=li.up, down=li.down, shared=li.shared)
        g.run_stepwise_and_compare(layer, li2, oracle)
        torch.cuda.synchronize()
        assert int(counters.abs().sum()) == 0
    layer.close()


@pytest.mark.parametrize("T,E,k,d,f,fs", [(1500, 16, 2, 256, 640, 0), (2048, 64, 6, 256, 384, 768), (40, 8, 2, 512, 1024, 0)])
def test_tiled_kernels_many_calls_in_a_row(oracle, T, E, k, d, f, fs):
    """Several hundred steps and expert-FFN calls in a row on the tiled kernels (two-tile items whose
    epilogue runs behind the MMAs; a down launch that starts while the gate/up launch still runs and
    takes its items from a counter): no wait ever runs out, every counter is back at zero, and the
    output of every step is bit-identical to the first one's."""
    g = _g()
    cfg = gen.LayerConfig("t", d, f, E, k, T, fs, "zipf", 1.1, seed=11 * T + E)
    li = gen.layer_inputs(cfg, n_distinct_experts=min(E, 6))
    layer = g.make_layer(li, AUTO)
    g.run_stepwise_and_compare(layer, li, oracle)
    logits, x = g.dev(li.logits), g.dev(li.x)
    first = layer.step(logits, x, T).clone()
    counters = layer.ctx.step_tensor(10, (656,), torch.int32)
    for rep in range(6):
        for _ in range(50):
            out = layer.step(logits, x, T)
        for _ in range(50):
            layer.expert_ffn(T)
        layer.combine(T)
        torch.cuda.synchronize()
        assert layer.device_status() == 0
        assert int(counters.abs().sum()) == 0
        assert torch.equal(out, first)
    layer.close()


def test_bounded_device_wait_runs_out_and_context_survives(oracle, B):
    """Failure detection without a GPU fault: a wait that nothing will ever satisfy gives up after
    its limit, the kernel returns, the status word says TIMEOUT, and the same context then runs a
    correct step."""
    import time
    g = _g()
    li = gen.layer_inputs(gen.LayerConfig("t", 128, 128, 4, 2, 16, seed=1))
    layer = g.make_layer(li, TENSOR)
    # a CTA that gives up a wait skips its arrival on a split item's counter; stand in for that on the
    # host by leaving a count behind, and check that reading the TIMEOUT status clears the counters
    counters = layer.ctx.step_tensor(10, (656,), torch.int32)
    assert int(counters.abs().sum()) == 0
    counters[3] = 2
    counters[320 + 17] = 1
    counters[640] = 5
    t0 = time.perf_counter()
    B.saem_selftest_bounded_wait(layer.ctx.handle, 20000)            # 20 ms limit
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 5.0
    assert layer.device_status() == B.SAEM_ERR_TIMEOUT
    assert int(counters.abs().sum()) == 0
    assert layer.device_status() == 0
    assert B.saem_selftest_bounded_wait(layer.ctx.handle, 0, check=False) == B.SAEM_ERR_INVALID_ARG
    g.run_stepwise_and_compare(layer, li, oracle)
    layer.close()


@pytest.mark.parametrize("T,E,k,d", [(1, 60, 4, 2048), (16, 8, 2, 4096), (64, 128, 8, 2048), (33, 64, 6, 256)])
def test_route_fused_with_router_projection(oracle, B, T, E, k, d):
    """saem_route_fused: logits against the oracle's float64 router; selection and weights must be
    exactly what saem_route gives on those logits, and equal the oracle's wherever the exact logits
    are not within rounding distance of a tie."""
    g = _g()
    rng = np.random.default_rng(T * 131 + E)
    x = gen.activations(rng, T, d)
    wr = gen.router_weights(rng, E, d)
    ctx = B.Context(B.make_config(d, 128, E, k, T))
    idx = torch.empty((T, k), dtype=torch.int32, device="cuda:0")
    w = torch.empty((T, k), dtype=torch.float32, device="cuda:0")
    logits = torch.empty((T, E), dtype=torch.float32, device="cuda:0")
    B.saem_route_fused(ctx.handle, g.dev(x), g.dev(wr), T, logits, idx, w)
    idx2, w2 = torch.empty_like(idx), torch.empty_like(w)
    B.saem_route(ctx.handle, logits, T, idx2, w2)
    torch.cuda.synchronize()
    assert torch.equal(idx, idx2) and torch.equal(w, w2)                 # same gate on the same logits
    ref_logits = oracle.router_logits(x, wr)
    assert np.abs(g.host(logits).astype(np.float64) - ref_logits).max() <= 1e-4
    ridx, rw = oracle.route(ref_logits.astype(np.float32), k)
    srt = -np.sort(-ref_logits, axis=1)[:, :min(k + 1, E)]
    clear = (np.abs(np.diff(srt, axis=1)).min(axis=1) > 1e-4) if E > 1 else np.ones(T, bool)
    assert clear.mean() >= 0.9
    assert np.array_equal(g.host(idx)[clear], ridx[clear])
    assert np.abs(g.host(w).astype(np.float64) - rw)[clear].max() <= 1e-5
    # without the optional logits output
    B.saem_route_fused(ctx.handle, g.dev(x), g.dev(wr), T, None, idx2, w2)
    torch.cuda.synchronize()
    assert torch.equal(idx, idx2) and torch.equal(w, w2)
    ctx.close()


@pytest.mark.parametrize("T,E,k,d,f,fs", [(24, 12, 3, 256, 384, 768), (5, 60, 4, 256, 128, 0)])
def test_bookkeeping_comparison_mode_against_oracle(oracle, T, E, k, d, f, fs):
    """The per-expert mask / gather / dense execution / scatter-add procedure of the paper's
    Motivation 3 (the comparison mode of launch_ablation) computes the same layer output as the
    oracle, within the FFN tolerance -- so the launch-count and time contrast it reports is between
    two correct ways of doing the same step."""
    g = _g()
    from paper_2608_21614_b200.launch_ablation import BookkeepingStep
    cfg = gen.LayerConfig("t", d, f, E, k, T, fs, "zipf", 1.1, seed=21)
    li = gen.layer_inputs(cfg)
    layer = g.make_layer(li, AUTO)
    book = BookkeepingStep(cfg, li, layer)
    out = book.run(g.dev(li.logits), g.dev(li.x))
    torch.cuda.synchronize()
    ref = oracle.moe_step(li.logits, li.x, k, li.gate, li.up, li.down, shared=li.shared)
    g.assert_close(g.host(out), ref["out"], "bookkeeping step")
    assert book.ffn_calls == int((ref["counts"] > 0).sum()) + (fs // f if fs else 0)
    assert book.one.device_status() == 0 and layer.device_status() == 0
    book.close()
    layer.close()
