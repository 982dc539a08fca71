"""CPU oracle for the class-balanced variant (CB-SAGE), plain numpy in fp64.

TEST INFRASTRUCTURE ONLY, like the rest of this package: nothing on the product path imports it.

What it follows: Algorithm 1, the class-balanced branch, and the section on agreement scoring and
selection: for each class c the mean of the normalised projections zhat_i over the class, its unit vector u_c (zero
if the mean is zero), the score <zhat_i, u_c> of every example of the class, and the top-k_c examples per class
with sum_c k_c = k.

Reading taken where the paper is silent: it only fixes sum_c k_c = k. Here k_c is proportional to the class size
n_c with largest-remainder rounding: k_c = floor(k n_c / N), and the k - sum_c floor(.) classes with the largest
fractional parts (ties: smaller class index first) get one more. Since k <= N this never exceeds n_c. Examples
whose label is outside [0, C) take no part: score 0, never selected. Within a class the order is (score
descending, index ascending); the result lists class 0's picks first, then class 1's, and so on.

Pins: tests/test_oracle_cb.py (one class equals the global rule, hand-worked allocation, brute-force selection,
identical rows score 1, invariance under relabelling).
"""
from __future__ import annotations

import numpy as np


def class_scores(zhat: np.ndarray, labels: np.ndarray, num_classes: int):
    """Returns (alpha (N,), U (C x ell) unit centroids, counts (C,))."""
    zhat = np.asarray(zhat, dtype=np.float64)
    labels = np.asarray(labels)
    N, ell = zhat.shape
    alpha = np.zeros(N)
    U = np.zeros((num_classes, ell))
    counts = np.zeros(num_classes, dtype=np.int64)
    for c in range(num_classes):
        members = np.flatnonzero(labels == c)
        counts[c] = members.size
        if members.size == 0:
            continue
        zbar = np.zeros(ell)
        for i in members:                      # ascending example order
            zbar += zhat[i]
        zbar /= members.size
        nrm = np.sqrt(np.sum(zbar * zbar))
        if nrm > 0:
            U[c] = zbar / nrm
        for i in members:
            alpha[i] = float(np.dot(zhat[i], U[c]))
    return alpha, U, counts


def allocate(counts: np.ndarray, k: int) -> np.ndarray:
    """k_c proportional to the class sizes, largest-remainder rounding, ties to the smaller class index."""
    counts = np.asarray(counts, dtype=np.int64)
    N = int(counts.sum())
    kc = np.zeros_like(counts)
    if N == 0 or k <= 0:
        return kc
    k = min(int(k), N)
    num = counts * k                            # exact integers: quota_c = num_c / N
    kc = num // N
    rem = num - kc * N                          # fractional part times N
    left = k - int(kc.sum())
    order = sorted(range(len(counts)), key=lambda c: (-int(rem[c]), c))
    for c in order[:left]:
        kc[c] += 1
    return kc


def select(alpha: np.ndarray, labels: np.ndarray, num_classes: int, keep_rate: float):
    """Returns (idx, k_c). k = floor(keep_rate * N_valid + 0.5) clamped to [0, N_valid], N_valid = examples with a
    label in [0, C)."""
    alpha = np.asarray(alpha, dtype=np.float64)
    labels = np.asarray(labels)
    counts = np.array([int(np.sum(labels == c)) for c in range(num_classes)], dtype=np.int64)
    n_valid = int(counts.sum())
    k = int(np.floor(keep_rate * n_valid + 0.5)) if np.isfinite(keep_rate) else 0
    k = max(0, min(k, n_valid))
    kc = allocate(counts, k)
    out = []
    for c in range(num_classes):
        members = [int(i) for i in np.flatnonzero(labels == c)]
        members.sort(key=lambda i: (-alpha[i], i))
        out.extend(members[: int(kc[c])])
    return np.array(out, dtype=np.int64), kc
