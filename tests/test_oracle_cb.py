"""Pins of the class-balanced oracle (oracle/cb.py): special cases that reduce to the global rule, hand-worked
values, brute force, invariances. CPU only."""
import numpy as np

import oracle
from oracle import cb


def _zhat(N, ell, seed):
    r = np.random.default_rng(seed)
    z = r.standard_normal((N, ell)) + 0.7
    z[3] = 0.0
    n = np.linalg.norm(z, axis=1, keepdims=True)
    return np.where(n > 0, z / np.where(n > 0, n, 1), 0.0)


def test_single_class_equals_global_rule():
    r = np.random.default_rng(0)
    S = r.standard_normal((4, 9))
    G = r.standard_normal((50, 9))
    ref = oracle.score(S, G)
    a, U, counts = cb.class_scores(ref["zhat"], np.zeros(50, dtype=np.int64), 1)
    assert np.allclose(a, ref["alpha"], atol=1e-13) and np.allclose(U[0], ref["u"], atol=1e-13) and counts[0] == 50
    idx, kc = cb.select(a, np.zeros(50, dtype=np.int64), 1, 0.3)
    assert np.array_equal(idx, oracle.select(ref["alpha"], 0.3)) and kc.tolist() == [15]


def test_hand_worked_two_classes():
    # class 0 lives on e1/e2, class 1 on e3: centroids are (1,1,0)/sqrt2 and (0,0,1)
    zh = np.array([[1.0, 0, 0], [0, 1.0, 0], [0, 0, 1.0], [0, 0, -1.0], [0, 0, 1.0]])
    lab = np.array([0, 0, 1, 1, 1])
    a, U, counts = cb.class_scores(zh, lab, 2)
    s = 1 / np.sqrt(2)
    assert np.allclose(U, [[s, s, 0], [0, 0, 1.0]]) and counts.tolist() == [2, 3]
    assert np.allclose(a, [s, s, 1.0, -1.0, 1.0])
    idx, kc = cb.select(a, lab, 2, 0.6)                      # k = 3 -> quotas 1.2, 1.8 -> (1, 2)
    assert kc.tolist() == [1, 2] and idx.tolist() == [0, 2, 4]


def test_allocation_rules():
    assert cb.allocate(np.array([5, 3, 2]), 5).tolist() == [3, 1, 1]      # quotas 2.5 1.5 1.0, tie -> class 0
    assert cb.allocate(np.array([1, 1, 1, 1]), 2).tolist() == [1, 1, 0, 0]
    assert cb.allocate(np.array([0, 7]), 3).tolist() == [0, 3]
    assert cb.allocate(np.array([4, 4]), 8).tolist() == [4, 4] and cb.allocate(np.array([4, 4]), 0).tolist() == [0, 0]
    r = np.random.default_rng(1)
    for _ in range(200):
        counts = r.integers(0, 40, size=r.integers(1, 9))
        N = int(counts.sum())
        k = int(r.integers(0, N + 1))
        kc = cb.allocate(counts, k)
        assert kc.sum() == k and np.all(kc <= counts) and np.all(kc >= 0)
        if N:
            assert np.all(np.abs(kc - k * counts / N) < 1.0)


def test_selection_brute_force_and_invalid_labels():
    zh = _zhat(300, 6, 2)
    r = np.random.default_rng(3)
    lab = r.integers(-1, 5, size=300)                        # -1 = no class
    a, U, counts = cb.class_scores(zh, lab, 4)               # label 4 is out of range too
    assert np.all(a[(lab < 0) | (lab >= 4)] == 0.0) and a[3] == 0.0
    assert np.all(np.abs(a) <= 1 + 1e-12)
    idx, kc = cb.select(a, lab, 4, 0.25)
    n_valid = int(np.sum((lab >= 0) & (lab < 4)))
    assert kc.sum() == int(np.floor(0.25 * n_valid + 0.5)) == len(idx) == len(set(idx.tolist()))
    pos = 0
    for c in range(4):
        mem = np.flatnonzero(lab == c)
        best = mem[np.lexsort((mem, -a[mem]))][: kc[c]]
        assert idx[pos:pos + kc[c]].tolist() == best.tolist()
        pos += kc[c]


def test_identical_rows_score_one_and_relabelling():
    zh = _zhat(120, 5, 4)
    lab = np.arange(120) % 3
    zh[lab == 1] = zh[1]                                     # class 1: all rows identical -> score 1
    a, U, _ = cb.class_scores(zh, lab, 3)
    assert np.allclose(a[lab == 1], 1.0)
    perm = np.array([2, 0, 1])
    a2, U2, _ = cb.class_scores(zh, perm[lab], 3)
    assert np.allclose(a2, a) and np.allclose(U2[perm], U)
    # each centroid maximises the mean score of its class: sum_i <zhat_i, u_c> = ||sum_i zhat_i||
    for c in range(3):
        assert np.isclose(a[lab == c].sum(), np.linalg.norm(zh[lab == c].sum(axis=0)))
