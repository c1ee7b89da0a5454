"""Pins of the oracle's gating: brute force, closed forms, special values, statistics."""
import numpy as np
import pytest


def _brute(logits, k):
    """Full sort per row by (value descending, index ascending), NaN as -inf."""
    v = np.where(np.isnan(logits), -np.inf, logits).astype(np.float64)
    out = np.empty((v.shape[0], k), np.int32)
    for t in range(v.shape[0]):
        order = np.lexsort((np.arange(v.shape[1]), -v[t]))
        out[t] = order[:k]
    return out


@pytest.mark.parametrize("T,E,k", [(1, 1, 1), (5, 8, 2), (64, 8, 2), (33, 60, 4), (32, 64, 6), (7, 128, 8), (9, 60, 60)])
def test_indices_match_full_sort(oracle, T, E, k):
    rng = np.random.default_rng(T * 1000 + E + k)
    logits = rng.standard_normal((T, E)).astype(np.float32)
    idx, w = oracle.route(logits, k)
    assert np.array_equal(idx, _brute(logits, k))
    assert np.allclose(w.sum(1), 1.0, atol=1e-12)
    assert np.all(np.diff(w, axis=1) <= 1e-15) and np.all(w > 0) and np.all(w <= 1)


def test_ties_and_quantised_values(oracle):
    rng = np.random.default_rng(3)
    logits = rng.integers(-2, 3, size=(200, 16)).astype(np.float32)   # many exact ties
    idx, _ = oracle.route(logits, 5)
    assert np.array_equal(idx, _brute(logits, 5))
    eq = np.zeros((3, 8), np.float32)
    idx, w = oracle.route(eq, 3)
    assert np.array_equal(idx, np.tile(np.arange(3, dtype=np.int32), (3, 1)))
    assert np.allclose(w, 1.0 / 3.0, atol=1e-15)


def test_signed_zero_inf_nan(oracle):
    row = np.array([[-0.0, 0.0, -np.inf, np.nan, 1.0, -1.0]], np.float32)
    idx, w = oracle.route(row, 6)
    assert idx.tolist() == [[4, 0, 1, 5, 2, 3]]          # +0 == -0 -> lower id; NaN ranks as -inf, after id 2
    assert np.isfinite(w).all() and abs(w.sum() - 1) < 1e-12
    assert w[0, 4] == 0.0 and w[0, 5] == 0.0
    allneg = np.full((1, 4), -np.inf, np.float32)
    idx, w = oracle.route(allneg, 2)
    assert idx.tolist() == [[0, 1]] and np.allclose(w, 0.5)
    big = np.array([[300.0, 0.0, -300.0]], np.float32)
    idx, w = oracle.route(big, 2)
    assert idx.tolist() == [[0, 1]] and w[0, 0] == pytest.approx(1.0) and w[0, 1] < 1e-100
    pinf = np.array([[np.inf, 1.0, np.inf]], np.float32)
    idx, w = oracle.route(pinf, 3)
    assert idx.tolist() == [[0, 2, 1]] and w.tolist() == [[0.5, 0.5, 0.0]]


def test_closed_forms_k1_k2(oracle):
    rng = np.random.default_rng(11)
    logits = rng.standard_normal((50, 8)).astype(np.float32)
    _, w1 = oracle.route(logits, 1)
    assert np.all(w1 == 1.0)
    idx, w2 = oracle.route(logits, 2)
    l0 = np.take_along_axis(logits, idx[:, :1].astype(np.int64), 1).astype(np.float64)
    l1 = np.take_along_axis(logits, idx[:, 1:].astype(np.int64), 1).astype(np.float64)
    from scipy.special import expit            # logistic: k = 2 softmax is sigma(l0 - l1)
    assert np.allclose(w2[:, :1], expit(l0 - l1), atol=1e-14)


def test_k_equals_E_is_full_softmax(oracle):
    from scipy.special import softmax
    rng = np.random.default_rng(12)
    logits = rng.standard_normal((10, 12)).astype(np.float32)
    idx, w = oracle.route(logits, 12)
    assert np.array_equal(np.sort(idx, 1), np.tile(np.arange(12), (10, 1)))
    full = softmax(logits.astype(np.float64), axis=1)
    assert np.allclose(w, np.take_along_axis(full, idx.astype(np.int64), 1), atol=1e-14)
    # without renormalisation the weights are the full-softmax probabilities of the chosen experts
    idx3, w3 = oracle.route(logits, 3, renorm=False)
    assert np.allclose(w3, np.take_along_axis(full, idx3.astype(np.int64), 1), atol=1e-14)
    assert np.all(w3.sum(1) < 1)


def test_uniform_routing_frequency(oracle):
    """iid logits -> every expert is selected with probability k/E (8/128 = 6.25 % in the
    paper's heat-map discussion, Motivation 1)."""
    rng = np.random.default_rng(5)
    T, E, k = 20000, 128, 8
    idx, _ = oracle.route(rng.standard_normal((T, E)).astype(np.float32), k)
    freq = np.bincount(idx.ravel(), minlength=E) / T
    assert abs(freq.mean() - k / E) < 1e-12
    assert np.all(np.abs(freq - 0.0625) < 6 * np.sqrt(0.0625 * 0.9375 / T))


def test_router_logits_equal_library_matmul(oracle):
    from paper_2608_21614_b200 import inputs as gen
    rng = np.random.default_rng(21)
    x = gen.activations(rng, 9, 192)
    w = gen.router_weights(rng, 13, 192)
    got = oracle.router_logits(x, w)
    ref = gen.bf16_bits_to_f32(x).astype(np.float64) @ gen.bf16_bits_to_f32(w).astype(np.float64).T
    assert got.shape == (9, 13) and np.allclose(got, ref, rtol=0, atol=1e-12)
    assert 0.5 < got.std() < 1.5
    onehot = gen.to_bf16_bits(np.eye(4, 192, dtype=np.float32))          # x_t = e_t picks column t of W
    assert np.array_equal(oracle.router_logits(onehot, w), gen.bf16_bits_to_f32(w)[:, :4].T.astype(np.float64))
