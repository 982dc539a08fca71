"""Pins for the merged form of pass 1 in the oracle (P sketches over interleaved row blocks, merged pairwise at the
freeze). Each check compares it with something it did not compute itself: the sequential oracle (P = 1), an
independent numpy replay through numpy's SVD, the Frequent-Directions guarantees (which mergeability preserves),
exactness on low-rank and short inputs, and a marked input that shows which sketch received which row. CPU only."""
import numpy as np
import pytest

import oracle
from oracle import metrics


def rng(seed):
    return np.random.default_rng(seed)


def lowrank(N, D, rank, noise, seed):
    r = rng(seed)
    Q, _ = np.linalg.qr(r.standard_normal((D, rank)))
    return r.standard_normal((N, rank)) @ Q.T * 3.0 + noise * r.standard_normal((N, D))


# ---- an independent replay: numpy SVD instead of the oracle's Jacobi, its own dealing and merge loops --------------

def np_fd(rows, ell):
    """Sequential sketch through numpy's SVD. Returns (S with ell rows, rows kept, sum of deltas)."""
    m, D = 2 * ell, rows.shape[1]
    B = np.zeros((m, D))
    fill, sd = 0, 0.0
    for g in rows:
        B[fill] = g
        fill += 1
        if fill == m:
            _, s, Vt = np.linalg.svd(B, full_matrices=False)
            d = s[ell - 1] ** 2
            B[:] = 0.0
            B[:ell - 1] = np.sqrt(np.clip(s[:ell - 1] ** 2 - d, 0, None))[:, None] * Vt[:ell - 1]
            fill, sd = ell - 1, sd + d
    S = np.zeros((ell, D))
    if fill:
        _, s, Vt = np.linalg.svd(B[:fill], full_matrices=False)
        if fill > ell:
            d = s[ell - 1] ** 2
            S[:ell - 1] = np.sqrt(np.clip(s[:ell - 1] ** 2 - d, 0, None))[:, None] * Vt[:ell - 1]
            fill, sd = ell - 1, sd + d
        else:
            S[:fill] = s[:fill, None] * Vt[:fill]
    return S, fill, sd


def np_merged(A, ell, P, block):
    parts = [[] for _ in range(P)]
    for i in range(A.shape[0]):
        parts[(i // block) % P].append(i)
    fr = [np_fd(A[ix] if ix else np.zeros((0, A.shape[1])), ell) for ix in parts]
    total = sum(f[2] for f in fr)
    s = 1
    while s < P:
        for a in range(0, P, 2 * s):
            if a + s < P:
                S, c, d = np_fd(np.concatenate([fr[a][0][:fr[a][1]], fr[a + s][0][:fr[a + s][1]]]), ell)
                fr[a] = (S, c, 0.0)
                total += d
        s *= 2
    return fr[0][0], total


# ---- pins --------------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("route", [0, 1])
def test_one_sketch_is_the_sequential_sketch_bit_for_bit(route):
    A = lowrank(300, 24, 5, 0.4, 1)
    a = oracle.run(A, 24, 5, 0.2, route=route)
    fd = oracle.OracleMergedFD(24, 5, 1, route=route)
    fd.update(A[:77])
    fd.update(A[77:])
    S, sigma = fd.finalize()
    assert np.array_equal(S, a["S"]) and np.array_equal(sigma, a["sigma"])
    assert fd.stats()["shrinks"] == a["stats"]["shrinks"]


@pytest.mark.parametrize("N,D,ell,P,block", [(200, 12, 3, 2, None), (333, 20, 4, 3, None), (500, 16, 5, 4, 7),
                                             (64, 10, 4, 8, None), (1000, 30, 6, 16, None), (90, 9, 2, 5, 1)])
def test_against_numpy_replay(N, D, ell, P, block):
    A = lowrank(N, D, min(D, 6), 0.5, N + P)
    fd = oracle.OracleMergedFD(D, ell, P, block)
    for r0 in range(0, N, 41):                        # chunking of the calls must not matter
        fd.update(A[r0:r0 + 41])
    S, _ = fd.finalize()
    S_np, sd_np = np_merged(A, ell, P, block or ell + 1)
    scale = np.linalg.norm(A) ** 2
    assert np.allclose(S.T @ S, S_np.T @ S_np, atol=1e-9 * scale)
    assert np.isclose(fd.stats()["sum_delta"], sd_np, rtol=1e-9)


def test_rows_go_to_sketches_in_blocks():
    """Row i is the unit vector e_i (N <= D): before any merge, sketch p must span exactly the rows of its blocks."""
    N = D = 40
    ell, P, block = 16, 3, 5
    fd = oracle.OracleMergedFD(D, ell, P, block)
    fd.update(np.eye(N))
    fd.finalize()
    for p, (S, kept) in enumerate(fd.frozen):
        mine = [i for i in range(N) if (i // block) % P == p]
        assert kept == len(mine) <= ell                  # no shrink: at most ell rows each
        support = np.flatnonzero(np.abs(S).sum(axis=0) > 0)
        assert support.tolist() == mine
    assert fd.stats()["rows_per_sketch"] == [15, 15, 10]


@pytest.mark.parametrize("P", [2, 4, 7, 16])
def test_guarantees_hold_for_the_merged_sketch(P):
    N, D, ell = 900, 48, 8
    A = lowrank(N, D, 5, 0.6, P)
    out = oracle.run(A, D, ell, 0.1, sketches=P)
    S, sd = out["S"], out["stats"]["sum_delta"]
    lo, hi = metrics.signed_gram_extremes(A, S)
    F2 = np.linalg.norm(A) ** 2
    assert lo >= -1e-10 * F2                              # 0 <= A^T A - S^T S
    assert hi <= sd * (1 + 1e-10)                         # every shrink, merges included, removes at most its delta
    sv = np.linalg.svd(A, compute_uv=False) ** 2
    for k in range(ell):
        assert hi <= sv[k:].sum() / (ell - k) * (1 + 1e-10)
    assert F2 - np.linalg.norm(S) ** 2 >= ell * sd * (1 - 1e-10)


@pytest.mark.parametrize("P", [2, 5])
def test_exact_below_rank_ell_and_for_short_streams(P):
    D, ell = 30, 6
    A = lowrank(400, D, 4, 0.0, 3)                        # rank 4 < ell: every delta is zero
    S = oracle.run(A, D, ell, 0.1, sketches=P)["S"]
    assert np.allclose(S.T @ S, A.T @ A, atol=1e-9 * np.linalg.norm(A) ** 2)
    A = rng(4).standard_normal((ell, D))                  # N <= ell rows in all: nothing is ever shrunk
    out = oracle.run(A, D, ell, 0.5, sketches=P, block=1)
    assert out["stats"]["shrinks"] == 0
    assert np.allclose(out["S"].T @ out["S"], A.T @ A, atol=1e-12 * np.linalg.norm(A) ** 2)


def test_merged_sketch_differs_from_the_sequential_one_but_scores_stay_close():
    """The merged sketch is a different approximation (not a reordering of the same arithmetic): it must not be
    mistaken for the sequential one, yet on a low-rank-plus-noise input both rank the examples alike."""
    N, D, ell = 1500, 64, 8
    A = lowrank(N, D, 4, 0.3, 9)
    a = oracle.run(A, D, ell, 0.1)
    b = oracle.run(A, D, ell, 0.1, sketches=4)
    F2 = np.linalg.norm(A) ** 2
    assert metrics.signed_gram_norm(a["S"], b["S"]) > 1e-6 * F2
    assert np.corrcoef(a["alpha"], b["alpha"])[0, 1] > 0.99
