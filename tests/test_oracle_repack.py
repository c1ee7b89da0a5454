"""Pins of the oracle's repacking: the paper's worked example, a library stable sort, invariants."""
import os

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "repack_worked_example.txt")


def _read_golden():
    rows, vals = [], {}
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, *nums = line.split()
        nums = [int(n) for n in nums]
        if key == "route":
            rows.append(nums[1:])
        else:
            vals[key] = np.array(nums, np.int32)
    return np.array(rows, np.int32), vals


def test_paper_worked_example(oracle):
    idx, g = _read_golden()
    x = (np.arange(4, dtype=np.uint16)[:, None] * 100 + np.arange(8, dtype=np.uint16)[None, :])
    counts, offsets, perm, inv, xp = oracle.repack(idx, x, 4)
    assert np.array_equal(counts, g["counts"])
    assert np.array_equal(offsets, g["offsets"])
    assert np.array_equal(perm, g["perm"])
    assert np.array_equal(inv, g["inv_perm"])
    assert np.array_equal(perm // 2, g["packed_tokens"])
    assert np.array_equal(xp[:, 0] // 100, g["packed_tokens"])      # rows really moved


@pytest.mark.parametrize("T,E,k", [(1, 1, 1), (1, 60, 4), (64, 8, 2), (37, 60, 4), (300, 64, 6), (5, 128, 8)])
def test_equals_stable_library_sort_and_invariants(oracle, T, E, k):
    rng = np.random.default_rng(T + E + k)
    idx = np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
    x = rng.integers(0, 65535, size=(T, 16)).astype(np.uint16)
    counts, offsets, perm, inv, xp = oracle.repack(idx, x, E)
    P = T * k
    assert counts.sum() == P and offsets[0] == 0 and offsets[-1] == P
    assert np.array_equal(np.diff(offsets), counts)
    assert np.array_equal(counts, np.bincount(idx.ravel(), minlength=E))
    assert np.array_equal(perm, np.argsort(idx.ravel(), kind="stable"))
    assert np.array_equal(np.sort(perm), np.arange(P))
    assert np.array_equal(inv[perm], np.arange(P))
    for e in range(E):
        seg = perm[offsets[e]:offsets[e + 1]]
        assert np.all(idx.ravel()[seg] == e) and np.all(np.diff(seg) > 0)
    assert np.array_equal(xp, x[perm // k])


def test_all_tokens_one_expert_and_empty_experts(oracle):
    idx = np.full((9, 1), 3, np.int32)
    counts, offsets, perm, inv, _ = oracle.repack(idx, None, 6)
    assert counts.tolist() == [0, 0, 0, 9, 0, 0]
    assert offsets.tolist() == [0, 0, 0, 0, 9, 9, 9]
    assert np.array_equal(perm, np.arange(9)) and np.array_equal(inv, np.arange(9))
