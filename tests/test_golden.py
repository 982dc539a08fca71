"""The stored fixtures of tests/golden (written by make_golden.py from the oracle alone) against an independent
numpy evaluation of the same definitions, and against the oracle as it stands (a regression pin)."""
import json
import os

import numpy as np

import oracle

GOLD = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def test_scores_fixture_matches_definition_and_oracle():
    d = json.load(open(os.path.join(GOLD, "scores_small.json")))
    S, G = np.array(d["S"]), np.array(d["rows"])
    Z = G @ S.T                                              # z_i = S g_i
    nz = np.linalg.norm(Z, axis=1)
    Zh = np.where(nz[:, None] > 0, Z / np.where(nz[:, None] > 0, nz[:, None], 1.0), 0.0)
    zbar = Zh.mean(axis=0)
    u = zbar / np.linalg.norm(zbar)
    alpha = Zh @ u
    assert np.allclose(alpha, d["alpha"], atol=1e-12) and np.allclose(u, d["u"], atol=1e-12)
    assert alpha[4] == 0.0
    order = np.lexsort((np.arange(len(alpha)), -alpha))[:4]
    assert order.tolist() == d["top4"]
    out = oracle.score(S, G)
    assert np.allclose(out["alpha"], d["alpha"], atol=1e-13)


def test_fd_fixture_matches_numpy_svd_replay_and_oracle():
    d = json.load(open(os.path.join(GOLD, "fd_small.json")))
    A, ell = np.array(d["rows"]), d["ell"]
    m = 2 * ell
    B = np.zeros((m, A.shape[1]))
    fill, sum_delta, shrinks = 0, 0.0, 0
    for row in A:                                            # buffer of 2*ell rows, shrink when full
        B[fill] = row
        fill += 1
        if fill == m:
            _, s, Vt = np.linalg.svd(B, full_matrices=False)
            delta = s[ell - 1] ** 2
            B[:] = 0.0
            B[: ell - 1] = np.sqrt(np.clip(s[: ell - 1] ** 2 - delta, 0, None))[:, None] * Vt[: ell - 1]
            fill, sum_delta, shrinks = ell - 1, sum_delta + delta, shrinks + 1
    _, s, Vt = np.linalg.svd(B[:fill], full_matrices=False)
    if fill > ell:
        delta = s[ell - 1] ** 2
        s = np.sqrt(np.clip(s ** 2 - delta, 0, None))
        sum_delta, shrinks = sum_delta + delta, shrinks + 1
    sig = np.zeros(ell)
    sig[: min(ell, len(s))] = s[:ell]
    S = sig[:, None][: len(s[:ell])] * Vt[: len(s[:ell])]
    assert np.allclose(sig, d["sigma"], atol=1e-9) and np.isclose(sum_delta, d["sum_delta"], rtol=1e-10)
    assert shrinks == d["shrinks"]
    assert np.allclose(S.T @ S, np.array(d["gram"]), atol=1e-9)
    fd = oracle.OracleFD(A.shape[1], ell)
    fd.update(A)
    _, sigma = fd.finalize()
    assert np.allclose(sigma, d["sigma"], atol=1e-12)
