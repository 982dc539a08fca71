"""Pins for the CPU oracle: every check here compares the oracle with something it did not compute
itself -- a closed form, numpy's SVD/eigh on a tiny input, a guarantee the paper quotes, or an
invariance of the definitions. CPU only."""
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


# ------------------------------------------------------------------ eigen-solver

@pytest.mark.parametrize("n", [1, 2, 5, 16, 33])
def test_jacobi_eig_against_numpy(n):
    r = rng(n)
    A = r.standard_normal((n, n))
    K = A @ A.T + np.diag(r.uniform(0, 1, n))
    U, lam, _ = oracle.jacobi_eig(K)
    assert np.allclose(U.T @ U, np.eye(n), atol=1e-12)
    assert np.allclose(K @ U, U * lam, atol=1e-11 * np.linalg.norm(K))
    assert np.allclose(np.sort(lam), np.linalg.eigvalsh(K), rtol=1e-11, atol=1e-12)


def test_jacobi_eig_known_spectra():
    n = 12
    d = np.arange(1.0, n + 1)
    _, lam, sweeps = oracle.jacobi_eig(np.diag(d))
    assert sweeps == 0 and np.array_equal(lam, d)
    v = rng(0).standard_normal(n)
    K = np.eye(n) + np.outer(v, v)                        # spectrum {1 (n-1 times), 1 + |v|^2}
    _, lam, _ = oracle.jacobi_eig(K)
    lam = np.sort(lam)
    assert np.allclose(lam[:-1], 1.0, atol=1e-13) and np.isclose(lam[-1], 1.0 + v @ v, rtol=1e-13)


# ------------------------------------------------------------------ one shrink, closed form

def closed_form_case(ell, D, seed=0):
    m = 2 * ell
    r = rng(seed)
    Q, _ = np.linalg.qr(r.standard_normal((D, m)))
    sig = np.sort(r.uniform(0.5, 4.0, m))[::-1]
    rows = (sig[:, None] * Q.T)[r.permutation(m)]          # orthogonal rows in scrambled order
    return sig, Q.T, rows


@pytest.mark.parametrize("route", [0, 1])
def test_single_shrink_closed_form(route):
    """Rows sigma_j q_j^T with orthonormal q_j: the SVD is known, so the shrunk sketch is
    diag(sqrt(max(sigma_j^2 - sigma_ell^2, 0))) Q with sigma_ell the ell-th largest (1-indexed)."""
    ell, D = 6, 40
    sig, Qt, rows = closed_form_case(ell, D)
    fd = oracle.OracleFD(D, ell, route=route)
    fd.update(rows)
    B, fill = fd.buffer()
    assert fill == ell - 1 and fd.stats()["shrinks"] == 1
    delta = sig[ell - 1] ** 2
    expect = np.sqrt(np.clip(sig ** 2 - delta, 0, None))[:, None] * Qt
    assert np.allclose(B.T @ B, expect.T @ expect, atol=1e-12)
    assert np.allclose(np.linalg.norm(B, axis=1)[: ell - 1], np.sqrt(sig[: ell - 1] ** 2 - delta), atol=1e-12)
    assert np.all(B[ell - 1:] == 0.0)
    assert np.isclose(fd.stats()["sum_delta"], delta, rtol=1e-13)


def test_closed_form_pin_detects_wrong_delta_index():
    """The same closed form must reject a sketch shrunk with the (ell+1)-th singular value: shows the
    pin is sensitive to an off-by-one in the paper's delta = sigma_ell^2."""
    ell, D = 6, 40
    sig, Qt, rows = closed_form_case(ell, D)
    fd = oracle.OracleFD(D, ell, delta_rank=ell + 1)
    fd.update(rows)
    B, _ = fd.buffer()
    expect = np.sqrt(np.clip(sig ** 2 - sig[ell - 1] ** 2, 0, None))[:, None] * Qt
    assert not np.allclose(B.T @ B, expect.T @ expect, atol=1e-6)


# ------------------------------------------------------------------ exactness cases

@pytest.mark.parametrize("N", [1, 5, 8])
def test_exact_when_N_le_ell(N):
    ell, D = 8, 30
    A = rng(N).standard_normal((N, D))
    fd = oracle.OracleFD(D, ell)
    fd.update(A)
    S, sigma = fd.finalize()
    assert fd.stats()["shrinks"] == 0
    assert np.allclose(S.T @ S, A.T @ A, atol=1e-12)
    assert np.allclose(np.sort(sigma[:N])[::-1], np.linalg.svd(A, compute_uv=False), atol=1e-12)


def test_exact_when_rank_below_ell():
    """rank(A) < ell makes every delta zero, so the sketch reproduces A^T A for any N."""
    ell, D, N = 8, 25, 200
    A = lowrank(N, D, rank=5, noise=0.0, seed=3)
    fd = oracle.OracleFD(D, ell)
    fd.update(A)
    S, _ = fd.finalize()
    assert fd.stats()["shrinks"] > 10
    assert np.allclose(S.T @ S, A.T @ A, atol=1e-9 * np.linalg.norm(A) ** 2)
    assert fd.stats()["sum_delta"] <= 1e-12 * np.linalg.norm(A) ** 2


def test_partial_buffer_finalize_matches_numpy_svd():
    """ell < N < 2*ell: no shrink during the stream, one at the end; numpy's SVD gives the answer."""
    ell, D, N = 8, 30, 13
    A = rng(7).standard_normal((N, D))
    fd = oracle.OracleFD(D, ell)
    fd.update(A)
    S, sigma = fd.finalize()
    _, s, Vt = np.linalg.svd(A, full_matrices=False)
    kept = np.sqrt(np.clip(s ** 2 - s[ell - 1] ** 2, 0, None))
    expect = kept[:, None] * Vt
    assert np.allclose(S.T @ S, expect.T @ expect, atol=1e-12)
    assert np.allclose(sigma, kept[:ell], atol=1e-12)
    assert sigma[ell - 1] == 0.0


# ------------------------------------------------------------------ brute force through numpy's SVD

def fd_numpy(A, ell):
    """Third route: the same buffer schedule with numpy's SVD doing each factorisation."""
    m, D = 2 * ell, A.shape[1]
    B = np.zeros((m, D))
    fill, deltas = 0, []
    for g in A:
        B[fill] = g
        fill += 1
        if fill == m:
            _, s, Vt = np.linalg.svd(B, full_matrices=False)
            d = s[ell - 1] ** 2
            deltas.append(d)
            B = np.zeros((m, D))
            k = min(len(s), m)
            B[:k] = np.sqrt(np.clip(s ** 2 - d, 0, None))[:, None] * Vt
            B[ell - 1:] = 0
            fill = ell - 1
    _, s, Vt = np.linalg.svd(B[:fill], full_matrices=False)
    s = np.concatenate([s, np.zeros(max(0, m - len(s)))])
    Vt = np.concatenate([Vt, np.zeros((m - Vt.shape[0], D))]) if Vt.shape[0] < m else Vt
    if fill > ell:
        d = s[ell - 1] ** 2
        deltas.append(d)
        s = np.sqrt(np.clip(s ** 2 - d, 0, None))
    return (s[:, None] * Vt)[:ell], deltas


@pytest.mark.parametrize("N,D,ell,route", [(64, 32, 8, 0), (64, 32, 8, 1), (57, 19, 4, 0), (40, 6, 2, 0), (100, 24, 5, 1)])
def test_fd_against_numpy_svd_route(N, D, ell, route):
    A = lowrank(N, D, rank=3, noise=0.3, seed=N + D)
    fd = oracle.OracleFD(D, ell, route=route)
    fd.update(A[:17])
    fd.update(A[17:])                                       # chunking must not matter
    S, _ = fd.finalize()
    S_np, deltas = fd_numpy(A, ell)
    scale = np.linalg.norm(A) ** 2
    assert metrics.signed_gram_norm(S, S_np) <= 1e-11 * scale
    assert np.isclose(fd.stats()["sum_delta"], sum(deltas), rtol=1e-9)
    assert fd.stats()["shrinks"] == len(deltas)
    assert fd.stats()["rows_seen"] == N


def test_two_routes_agree_on_workload_shape():
    from paper_2510_02470_b200 import workloads as wl
    w = wl.scaled(wl.WORKLOADS["c1"], N=600, D=256, ell=16, chunk_rows=200)
    rows = wl.host_rows(w, seed=0)
    outs = []
    for route in (0, 1):
        fd = oracle.OracleFD(w.D, w.ell, route=route)
        fd.update(rows)
        outs.append(fd.finalize()[0])
    A = metrics.rows_as_f64(rows, w.D)
    assert metrics.signed_gram_norm(outs[0], outs[1]) <= 1e-10 * np.linalg.norm(A) ** 2


# ------------------------------------------------------------------ the guarantees the paper quotes

@pytest.mark.parametrize("N,D,ell,rank,noise", [(300, 40, 8, 4, 0.5), (500, 64, 16, 10, 1.0), (257, 33, 6, 20, 0.2)])
def test_fd_guarantees(N, D, ell, rank, noise):
    A = lowrank(N, D, rank, noise, seed=N)
    fd = oracle.OracleFD(D, ell)
    fd.update(A)
    S, _ = fd.finalize()
    E = A.T @ A - S.T @ S
    ev = np.linalg.eigvalsh(E)
    F2 = np.linalg.norm(A) ** 2
    assert ev.min() >= -1e-10 * F2                           # 0 <= A^T A - S^T S
    err = ev.max()
    s = np.linalg.svd(A, compute_uv=False)
    tail = np.concatenate([np.cumsum((s ** 2)[::-1])[::-1], [0.0]])   # tail[k] = ||A - A_k||_F^2
    for k in range(ell):
        assert err <= tail[k] / (ell - k) * (1 + 1e-9) + 1e-10 * F2
    for k in range(ell // 2 + 1):                            # the paper's form of the bound
        assert err <= 2.0 / ell * tail[k] * (1 + 1e-9) + 1e-10 * F2
    sd = fd.stats()["sum_delta"]
    assert err <= sd * (1 + 1e-9) + 1e-10 * F2
    assert F2 - np.linalg.norm(S) ** 2 >= ell * sd * (1 - 1e-9) - 1e-10 * F2
    # the Gram-trick metric agrees with the direct D x D computation
    lo, hi = metrics.signed_gram_extremes(A, S)
    assert np.isclose(hi, err, rtol=1e-8, atol=1e-10 * F2) and lo >= -1e-9 * F2
    assert np.isclose(metrics.signed_gram_norm(A, S), max(abs(ev.min()), err), rtol=1e-8, atol=1e-10 * F2)


# ------------------------------------------------------------------ scores

def random_case(N=50, D=20, ell=6, seed=0):
    r = rng(seed)
    S = r.standard_normal((ell, D)) * r.uniform(0.2, 3, (ell, 1))
    G = lowrank(N, D, 3, 0.4, seed + 1) + 0.7
    return S, G


def test_scores_through_M_only():
    """alpha is a function of M = S^T S: <z_i, z_j> = g_i^T M g_j. Recompute it without S."""
    S, G = random_case()
    out = oracle.score(S, G)
    M = S.T @ S
    Z2 = G @ M @ G.T
    nrm = np.sqrt(np.diag(Z2))
    Cn = Z2 / np.outer(nrm, nrm)                             # <zhat_i, zhat_j>
    alpha = Cn.sum(axis=1) / np.sqrt(Cn.sum())
    assert np.allclose(out["alpha"], alpha, atol=1e-12)
    assert np.allclose(out["znorm"], nrm, rtol=1e-12)


def test_score_range_identities_and_lemma():
    S, G = random_case(N=80, seed=5)
    out = oracle.score(S, G)
    a, zh, zn, u = out["alpha"], out["zhat"], out["znorm"], out["u"]
    assert np.all(a <= 1 + 1e-15) and np.all(a >= -1 - 1e-15)
    assert np.isclose(np.linalg.norm(u), 1.0, atol=1e-14)
    assert np.allclose(out["zbar"], zh.mean(axis=0), atol=1e-15)
    assert np.isclose(a.sum(), np.linalg.norm(zh.sum(axis=0)), rtol=1e-12)   # sum alpha = ||sum zhat||
    Z = G @ S.T
    assert np.allclose(zh * zn[:, None], Z, atol=1e-12)
    T = oracle.select(a, 0.25)
    xi = a[T].min()
    assert xi > 0
    lhs = ((Z[T] @ u) ** 2).sum()
    assert np.isclose(lhs, (zn[T] ** 2 * a[T] ** 2).sum(), rtol=1e-12)        # Lemma 1, identity
    assert lhs >= xi ** 2 * (zn[T] ** 2).sum() * (1 - 1e-12)                  # Lemma 1, bound
    assert np.linalg.norm(Z[T].mean(axis=0)) >= xi * zn[T].mean() * (1 - 1e-12)   # corollary


def test_identical_rows_score_one_and_scaling():
    S, _ = random_case()
    g = rng(1).standard_normal(S.shape[1])
    out = oracle.score(S, np.tile(g, (7, 1)))
    assert np.allclose(out["alpha"], 1.0, atol=1e-14)
    G = np.stack([g, 3.5 * g, -2.0 * g, rng(2).standard_normal(S.shape[1])])
    a = oracle.score(S, G)["alpha"]
    assert np.isclose(a[0], a[1], atol=1e-14) and np.isclose(a[0], -a[2], atol=1e-14)


def test_rotation_and_permutation_invariance():
    S, G = random_case(seed=9)
    a = oracle.score(S, G)["alpha"]
    Qr, _ = np.linalg.qr(rng(3).standard_normal((S.shape[0], S.shape[0])))
    assert np.allclose(oracle.score(Qr @ S, G)["alpha"], a, atol=1e-12)
    p = rng(4).permutation(G.shape[0])
    assert np.allclose(oracle.score(S, G[p])["alpha"], a[p], atol=1e-12)


def test_zero_conventions():
    S, G = random_case(seed=11)
    G[3] = 0.0
    Gperp = G.copy()
    # a row exactly orthogonal to every sketch row projects to z = 0
    S2 = S.copy()
    S2[:, 0] = 0.0
    Gperp[5] = 0.0
    Gperp[5, 0] = 2.0
    out = oracle.score(S2, Gperp)
    assert out["alpha"][3] == 0.0 and out["alpha"][5] == 0.0
    assert np.all(out["zhat"][3] == 0) and out["znorm"][5] == 0.0
    # opposite pairs cancel: zbar = 0 -> u = 0 -> all alpha = 0
    g = np.zeros(S.shape[1])
    g[1] = 1.0
    out = oracle.score(np.eye(4, S.shape[1]), np.stack([g, -g]))
    assert np.all(out["u"] == 0) and np.all(out["alpha"] == 0)


def test_dtype_entry_points_agree():
    import torch
    S, G = random_case(seed=13)
    Gb = torch.from_numpy(G).to(torch.bfloat16)
    G32 = Gb.to(torch.float32)
    a16 = oracle.score(S, Gb)["alpha"]
    a32 = oracle.score(S, G32)["alpha"]
    a64 = oracle.score(S, G32.to(torch.float64).numpy())["alpha"]
    assert np.array_equal(a16, a32) and np.array_equal(a32, a64)
    fds = []
    for rows in (Gb, G32, G32.to(torch.float64).numpy()):
        fd = oracle.OracleFD(S.shape[1], 4)
        fd.update(rows)
        fds.append(fd.finalize()[0])
    assert np.array_equal(fds[0], fds[1]) and np.array_equal(fds[1], fds[2])


def test_pitch_is_respected():
    S, G = random_case(seed=17)
    D = S.shape[1]
    Gp = np.full((G.shape[0], D + 5), 99.0)
    Gp[:, :D] = G
    fd1, fd2 = oracle.OracleFD(D, 4), oracle.OracleFD(D, 4)
    fd1.update(G)
    fd2.update(Gp)
    assert np.array_equal(fd1.finalize()[0], fd2.finalize()[0])
    assert np.array_equal(oracle.score(S, G)["alpha"], oracle.score(S, Gp)["alpha"])


# ------------------------------------------------------------------ selection

def test_select_k_rounding():
    assert oracle.select_k(4096, 0.1) == 410
    assert oracle.select_k(50000, 0.05) == 2500
    assert oracle.select_k(10, 0.0) == 0 and oracle.select_k(10, 1.0) == 10 and oracle.select_k(10, 2.0) == 10
    assert oracle.select_k(3, 0.5) == 2                      # 1.5 rounds half up


@pytest.mark.parametrize("kind", ["random", "ties", "constant"])
def test_select_against_lexsort(kind):
    r = rng(21)
    N = 1000
    a = {"random": r.uniform(-1, 1, N), "ties": r.integers(-3, 4, N) / 3.0, "constant": np.full(N, 0.25)}[kind]
    for rate in (0.0, 0.001, 0.1, 0.5, 1.0):
        idx = oracle.select(a, rate)
        ref = np.lexsort((np.arange(N), -a))[: oracle.select_k(N, rate)]
        assert np.array_equal(idx, ref)


# ------------------------------------------------------------------ the comparison helpers themselves

@pytest.mark.parametrize("p,q,D", [(3, 2, 4), (8, 8, 300), (64, 64, 20000)])
def test_signed_gram_norm_both_forms_against_the_dense_matrix(p, q, D):
    """|| P^T P - Q^T Q ||_2 through the QR form and through the W^(1/2) J W^(1/2) form (the one taken for operands too
    large for a QR) against numpy's eigvalsh of the D x D matrix itself where that is small, and against each other
    on a mid-size case. The square-root form is accurate to about sqrt(eps) of the operands' scale."""
    r = rng(p + q + D)
    P = r.standard_normal((p, D)) * np.linspace(2.0, 0.1, p)[:, None]
    Q = P[:q] + 1e-3 * r.standard_normal((q, D))
    a = metrics.signed_gram_norm(P, Q, method="qr")
    b = metrics.signed_gram_norm(P, Q, method="sqrt")
    scale = np.linalg.norm(P) ** 2
    assert abs(a - b) <= 1e-7 * scale
    if D <= 300:
        dense = np.abs(np.linalg.eigvalsh(P.T @ P - Q.T @ Q)).max()
        assert abs(a - dense) <= 1e-12 * scale and abs(b - dense) <= 1e-7 * scale
    lo, hi = metrics.signed_gram_extremes(P, Q)
    assert np.isclose(max(abs(lo), abs(hi)), a)
