"""CPU oracle for structured last-layer rows, plain numpy in fp64.

TEST INFRASTRUCTURE ONLY, like the rest of this package: nothing on the product path imports it.

What it follows: the method sketches and scores per-example gradients g_i (Method section, the definition of the
per-example gradient; Limitations, on gradients of the last layer). For a softmax classifier head with weights W (C x F)
and bias b (C) on features h_i, the gradient of the cross-entropy loss of example i with respect to (W, b) is

    dL/dW = (p_i - e_{y_i}) h_i^T   (C x F),        dL/db = p_i - e_{y_i}   (C),

so with q_i = p_i - e_{y_i} the row is g_i = [vec_rowmajor(q_i h_i^T) ; q_i], of dimension D = C F + C: the outer product
q_i (x) [h_i ; 1] with the bias part moved to the end. The CUDA library accepts (q_i, h_i) instead of g_i; what it must
compute is, by definition, what the plain path computes on the materialised rows. This module materialises them in fp64
(products of the stored fp32 / bf16 values, exact in fp64) and hands them to the plain oracle: no other arithmetic.
"""
from __future__ import annotations

import numpy as np


def _as_f64(x) -> np.ndarray:
    if isinstance(x, np.ndarray):
        return np.asarray(x, dtype=np.float64)
    import torch
    return x.to(torch.float64).numpy()


def materialise(q, h) -> np.ndarray:
    """Rows g_i = [vec_rowmajor(q_i h_i^T) ; q_i] (N x (C F + C), fp64) from q (N x C) and h (N x F)."""
    q, h = _as_f64(q), _as_f64(h)
    n, C = q.shape
    F = h.shape[1]
    g = np.empty((n, C * F + C))
    g[:, : C * F] = (q[:, :, None] * h[:, None, :]).reshape(n, C * F)
    g[:, C * F:] = q
    return g


def run(q, h, ell: int, keep_rate: float, route: int = 0, sketches: int = 1) -> dict:
    """The whole path on structured rows: exactly the plain oracle on the materialised rows."""
    import oracle
    g = materialise(q, h)
    return oracle.run(g, g.shape[1], ell, keep_rate, route=route, sketches=sketches)
