"""The fp64 torch replay used by the full-size GPU tests, checked against the oracle on the CPU (torch runs it on the
host here): same rows, same shrink schedule, agreement to fp64 rounding of the Gram route."""
import numpy as np
import pytest
import torch

import oracle
from oracle import metrics
import replay_f64 as rp


@pytest.mark.parametrize("N,D,ell", [(50, 40, 8), (700, 96, 12), (300, 1000, 33)])
def test_replay_matches_oracle(N, D, ell):
    r = np.random.default_rng(N)
    Q, _ = np.linalg.qr(r.standard_normal((D, 5)))
    A = (r.standard_normal((N, 5)) + 0.5) @ Q.T * 2.0 + 0.3 * r.standard_normal((N, D))
    rows = torch.from_numpy(A.astype(np.float32))
    ref = oracle.run(rows, D, ell, 0.2, route=0)
    rep = rp.ReplayFD(D, ell, torch.device("cpu"))
    for r0 in range(0, N, 37):
        rep.update(rows[r0:r0 + 37])
    S = rep.finalize()
    sc = rp.ReplayScore(S, N)
    sc.chunk(rows, sub_rows=50)
    alpha, u = sc.end()
    F2 = float(np.linalg.norm(A.astype(np.float32).astype(np.float64)) ** 2)
    assert rep.shrinks == ref["stats"]["shrinks"] and np.isclose(rep.fro_a, F2, rtol=1e-12)
    assert metrics.signed_gram_norm(S.numpy(), ref["S"]) / F2 <= 1e-10
    assert np.isclose(rep.sum_delta, ref["stats"]["sum_delta"], rtol=1e-9)
    assert np.max(np.abs(alpha - ref["alpha"])) <= 1e-8
    assert abs(rp.signed_gram_norm_device(S, torch.from_numpy(ref["S"])) - metrics.signed_gram_norm(S.numpy(), ref["S"])) <= 1e-12 * F2
    k = oracle.select_k(N, 0.2)
    assert rp.selection_agrees(ref["idx"], alpha, k, 1e-8)[0]
