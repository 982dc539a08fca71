"""Pins for the oracle's statement of structured last-layer rows: the materialised row against a hand-worked case,
against the gradient autograd computes for a softmax head (an independent route to the same vector), and the projection
through the row's structure against the projection of the materialised row. CPU only."""
import numpy as np
import torch

import oracle
from oracle import structured


def test_hand_worked_row():
    q = np.array([[0.25, -0.75]])                    # C = 2
    h = np.array([[2.0, 0.0, -4.0]])                 # F = 3
    g = structured.materialise(q, h)
    assert g.tolist() == [[0.5, 0.0, -1.0, -1.5, 0.0, 3.0, 0.25, -0.75]]


def test_row_is_the_autograd_gradient_of_a_softmax_head():
    """g_i must be the per-example gradient itself: cross-entropy of logits W h + b, differentiated by autograd with
    respect to (W, b) and flattened as [W row-major ; b]."""
    r = torch.Generator().manual_seed(0)
    C, F, N = 5, 7, 6
    W = torch.randn(C, F, generator=r, dtype=torch.float64, requires_grad=True)
    b = torch.randn(C, generator=r, dtype=torch.float64, requires_grad=True)
    h = torch.relu(torch.randn(N, F, generator=r, dtype=torch.float64))
    y = torch.randint(0, C, (N,), generator=r)
    p = torch.softmax(h @ W.T + b, dim=1).detach()
    q = p.clone()
    q[torch.arange(N), y] -= 1.0
    g = structured.materialise(q.numpy(), h.numpy())
    for i in range(N):
        loss = torch.nn.functional.cross_entropy((h[i] @ W.T + b)[None, :], y[i:i + 1])
        gW, gb = torch.autograd.grad(loss, (W, b))
        ref = torch.cat([gW.reshape(-1), gb]).numpy()
        assert np.allclose(g[i], ref, atol=1e-14)


def test_projection_through_the_structure_equals_projection_of_the_row():
    """z = S g with g = q (x) [h ; 1]: z_j = sum_c q_c (S_j[c, :] . h + S_j[bias c]) -- the identity the CUDA path uses to
    avoid forming g -- against the oracle's scores on the materialised rows."""
    r = np.random.default_rng(1)
    C, F, N, ell = 4, 6, 40, 5
    q = r.standard_normal((N, C))
    h = np.maximum(r.standard_normal((N, F)), 0)
    S = r.standard_normal((ell, C * F + C))
    ref = oracle.score(S, structured.materialise(q, h))
    Sw = S[:, : C * F].reshape(ell, C, F)
    Sb = S[:, C * F:]
    z = np.einsum("nc,jcf,nf->nj", q, Sw, h) + q @ Sb.T
    zn = np.linalg.norm(z, axis=1)
    assert np.allclose(zn, ref["znorm"], rtol=1e-12)
    zh = z / zn[:, None]
    u = zh.sum(axis=0)
    u /= np.linalg.norm(u)
    assert np.allclose(zh @ u, ref["alpha"], atol=1e-12)


def test_bf16_inputs_are_taken_exactly():
    r = np.random.default_rng(2)
    q = torch.from_numpy(r.standard_normal((3, 2)).astype(np.float32)).to(torch.bfloat16)
    h = torch.from_numpy(r.standard_normal((3, 4)).astype(np.float32)).to(torch.bfloat16)
    g = structured.materialise(q, h)
    assert np.array_equal(g[:, :8].reshape(3, 2, 4), q.double().numpy()[:, :, None] * h.double().numpy()[:, None, :])
    out = structured.run(q, h, 2, 0.5)
    assert out["S"].shape == (2, 10) and len(out["idx"]) == 2
