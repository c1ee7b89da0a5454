"""CPU-only pins of the host-side cache policy and of the temporal-coherence metric (Eq. 1)."""
import numpy as np

from paper_2608_21614_b200 import inputs as gen
from paper_2608_21614_b200.stack import plan_layer, tc_seq


def test_planner_identical_stage_means_no_transfers():
    counts = [50, 40, 30, 20, 5, 4, 3, 2]
    assert plan_layer(counts, [0, 1, 2, 3]) == []
    assert plan_layer(counts, [3, 2, 1, 0]) == []                  # slot order is irrelevant


def test_planner_disjoint_hot_sets_swap_min_c_hot():
    counts = [0, 0, 0, 0, 9, 8, 7, 0]                              # three hot experts, none resident
    moves = plan_layer(counts, [0, 1, 2, 3])
    assert [m[1] for m in moves] == [4, 5, 6]                      # hottest first
    assert sorted(m[0] for m in moves) == [1, 2, 3]                # least used residents; ties evict the higher id first
    assert [m[0] for m in moves] == [3, 2, 1]
    assert all(slot == victim for victim, _, slot in moves)       # the newcomer takes the victim's slot
    moves = plan_layer([0, 0, 0, 0, 9, 8, 7, 6], [0, 1])           # C = 2 < #hot
    assert [(m[1]) for m in moves] == [4, 5]


def test_planner_strict_improvement_and_ties():
    assert plan_layer([5, 5, 5, 5], [0, 1]) == []                  # equal counts: no gratuitous transfer
    assert plan_layer([1, 9, 9, 0], [0, 3]) == [(3, 1, 1), (0, 2, 0)]
    assert plan_layer([0, 3, 0, 0], [-1, -1]) == [(-1, 1, 0)]      # empty slots are filled first, only by used experts


def test_planner_matches_pairwise_swap_definition():
    """Second, independent formulation: repeatedly take the best non-resident and the worst
    resident and swap them while that strictly raises the resident count mass."""
    rng = np.random.default_rng(0)
    for _ in range(300):
        E, C = 8, 4
        counts = rng.integers(0, 6, size=E).tolist()
        slots = rng.permutation(E)[:C].tolist()
        got = plan_layer(counts, slots)
        res = list(slots)
        exp = []
        while True:
            non = [e for e in range(E) if e not in res]
            best = min(non, key=lambda e: (-counts[e], e))
            worst = min(res, key=lambda e: (counts[e], -e))
            if counts[best] <= counts[worst]:
                break
            exp.append((worst, best, slots.index(worst) if worst in slots else res.index(worst)))
            res[res.index(worst)] = best
        assert [(v, n) for v, n, _ in got] == [(v, n) for v, n, _ in exp]
        after = list(slots)
        for v, n, s in got:
            assert after[s] == v
            after[s] = n
        assert sorted(after) == sorted(res)


def test_tc_seq_closed_forms():
    same = np.tile(np.array([[3, 1, 0, 0], [1, 1, 1, 1]], float), (4, 1, 1))
    assert abs(tc_seq(same) - 1.0) < 1e-12                          # identical stages
    a = np.array([[1, 1, 0, 0]], float)
    b = np.array([[0, 0, 2, 5]], float)
    assert tc_seq(np.stack([a, b])) == 0.0                          # disjoint support
    c = np.array([[1, 0, 0, 0]], float)
    d = np.array([[1, 1, 0, 0]], float)
    assert abs(tc_seq(np.stack([c, d])) - 2 ** -0.5) < 1e-12        # cos 45 degrees
    assert abs(tc_seq(np.stack([c * 7, d * 3])) - 2 ** -0.5) < 1e-12   # scale-free (ratios, not counts)


def test_stage_trace_shape_and_coherence(oracle):
    tr = gen.stage_trace(4096, 4, 8, 1.2, seed=0)
    assert tr.boundaries[0] == 0 and np.all(np.diff(tr.boundaries) > 0) and tr.boundaries[-1] < 4096
    lens = np.diff(np.r_[tr.boundaries, 4096])
    assert 60 < lens.mean() < 600                                    # geometric, mean 200
    for s in range(len(tr.boundaries)):
        for l in range(4):
            assert sorted(tr.rankings[s, l]) == list(range(1, 9))
    # coherent trace: adjacent stages keep most of their routing; independent ones do not
    def coherence(trace):
        S = len(trace.boundaries)
        cnt = np.zeros((S, 4, 8))
        for s in range(S):
            step = int(trace.boundaries[s])
            for l in range(4):
                lg = np.concatenate([gen.trace_logits(trace, step + i, l, 8) for i in range(12)])
                idx, _ = oracle.route(lg, 2)
                cnt[s, l] = np.bincount(idx.ravel(), minlength=8)
        return tc_seq(cnt)
    coh = coherence(tr)
    ind = coherence(gen.stage_trace(4096, 4, 8, 1.2, seed=0, reshuffled=None))
    assert coh > ind + 0.1 and coh > 0.8
