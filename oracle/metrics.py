"""Comparison helpers for the parity tests (numpy, fp64). Test infrastructure, like the rest of oracle/.

Sketches are never compared row by row: an SVD is unique only up to signs and rotations inside
groups of equal singular values, so the comparable object is the D x D matrix S^T S (and the scores,
which are a function of S^T S alone). These helpers measure spectral norms of differences of such
matrices without forming anything D x D.
"""
from __future__ import annotations

import numpy as np


def _signed_gram_eigs(P: np.ndarray, Q: np.ndarray, method: str = "auto") -> np.ndarray:
    """Eigenvalues of P^T P - Q^T Q on its range, from a (p+q) x (p+q) symmetric problem.

    With C = [P; Q] and J = diag(I_p, -I_q), P^T P - Q^T Q = C^T J C. If C^T = Y R (thin QR, Y with
    orthonormal columns) then C^T J C = Y (R J R^T) Y^T, so the eigenvalues are those of R J R^T: accurate
    to rounding. For very large D the QR is replaced by W = C C^T and W^(1/2) J W^(1/2) (same non-zero
    eigenvalues, by similarity of XY and YX), which is accurate to about sqrt(eps) * ||W||."""
    P = np.asarray(P, dtype=np.float64)
    Q = np.asarray(Q, dtype=np.float64)
    Cm = np.concatenate([P, Q], axis=0)
    J = np.concatenate([np.ones(P.shape[0]), -np.ones(Q.shape[0])])
    assert method in ("auto", "qr", "sqrt")
    if method == "qr" or (method == "auto" and Cm.shape[0] <= Cm.shape[1] and Cm.size <= 2e8):
        R = np.linalg.qr(Cm.T, mode="r")
        M = (R * J[None, :]) @ R.T
    else:
        W = Cm @ Cm.T
        lam, V = np.linalg.eigh(W)
        Wh = (V * np.sqrt(np.clip(lam, 0.0, None))) @ V.T
        M = Wh @ (J[:, None] * Wh)
    return np.linalg.eigvalsh(0.5 * (M + M.T))


def signed_gram_norm(P: np.ndarray, Q: np.ndarray, method: str = "auto") -> float:
    """|| P^T P - Q^T Q ||_2 for P (p x D), Q (q x D) without forming a D x D matrix. method: "qr", "sqrt" (the
    W^(1/2) J W^(1/2) form) or "auto" (QR unless the stacked operand is very large)."""
    ev = _signed_gram_eigs(P, Q, method)
    return float(np.max(np.abs(ev))) if ev.size else 0.0


def signed_gram_extremes(P: np.ndarray, Q: np.ndarray):
    """(lambda_min, lambda_max) of P^T P - Q^T Q restricted to its range (0 is also an eigenvalue when
    p+q < D)."""
    ev = _signed_gram_eigs(P, Q)
    return float(ev.min()), float(ev.max())


def rows_as_f64(rows, D: int) -> np.ndarray:
    """CPU torch tensor or numpy array of rows (any supported dtype, pitch >= D) -> (n, D) float64."""
    if isinstance(rows, np.ndarray):
        return np.asarray(rows[:, :D], dtype=np.float64)
    import torch
    return rows[:, :D].to(torch.float64).numpy()


def selection_agrees(idx_test: np.ndarray, alpha_oracle: np.ndarray, keep_rate_k: int, tol: float):
    """Compares a selected index set with the oracle's, allowing differences only among examples whose
    oracle score lies within ``tol`` of the oracle's k-th score. Returns (ok, n_differences)."""
    k = keep_rate_k
    order = np.lexsort((np.arange(alpha_oracle.size), -alpha_oracle))
    ref = order[:k]
    if k == 0 or k == alpha_oracle.size:
        return set(idx_test.tolist()) == set(ref.tolist()), 0
    thr = alpha_oracle[order[k - 1]]
    diff = np.setxor1d(np.asarray(idx_test), ref)
    ok = bool(np.all(np.abs(alpha_oracle[diff] - thr) <= tol)) and len(idx_test) == k
    return ok, int(diff.size)
