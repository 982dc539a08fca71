"""GPU parity of the class-balanced variant (sage_score_classes, sage_select_classes) against oracle/cb.py."""
import numpy as np
import pytest
import torch

import oracle
from oracle import cb
import paper_2510_02470_b200 as sage

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _rows(N, D, seed, dtype=torch.float32):
    r = np.random.default_rng(seed)
    Q, _ = np.linalg.qr(r.standard_normal((D, 5)))
    A = (r.standard_normal((N, 5)) + 0.5) @ Q.T + 0.3 * r.standard_normal((N, D))
    return torch.from_numpy(A.astype(np.float32)).to(dtype)


@pytest.mark.parametrize("N,D,ell,C", [(700, 96, 8, 1), (1500, 260, 16, 7), (4000, 132, 64, 100), (300, 64, 200, 3)])
def test_class_scores_match_oracle(N, D, ell, C):
    rows = _rows(N, D, N + C)
    r = np.random.default_rng(C)
    S = (r.standard_normal((ell, D)) * np.linspace(2.0, 0.2, ell)[:, None]).astype(np.float32)
    labels = r.integers(-1, C + 1, size=N).astype(np.int32)          # -1 and C are "no class"
    ref = oracle.score(S.astype(np.float64), rows)
    a_ref, U_ref, cnt_ref = cb.class_scores(ref["zhat"], labels, C)
    fd = sage.SageFD(D, ell, torch.float32, 0)
    fd.load_sketch(torch.from_numpy(S).to(DEV))
    with pytest.raises(sage.SageError):                              # no scoring pass yet
        fd.score_classes(torch.from_numpy(labels).to(DEV), C)
    fd.score(rows.to(DEV))
    a = fd.score_classes(torch.from_numpy(labels).to(DEV), C)
    U, cnt = fd.class_centroids()
    b = fd.score_classes(torch.from_numpy(labels).to(DEV), C)        # deterministic
    torch.cuda.synchronize()
    fd.close()
    assert torch.equal(a, b)
    assert np.array_equal(cnt.cpu().numpy(), cnt_ref)
    assert np.max(np.abs(U.double().cpu().numpy() - U_ref)) <= 2e-5
    a = a.double().cpu().numpy()
    assert np.max(np.abs(a - a_ref)) <= 2e-5
    assert np.all(a[(labels < 0) | (labels >= C)] == 0.0) and np.all(np.abs(a) <= 1.0)


@pytest.mark.parametrize("N,C,rate", [(1, 1, 1.0), (257, 3, 0.3), (5000, 10, 0.1), (20000, 100, 0.05), (4097, 1000, 0.5),
                                      (999, 4, 0.0)])
def test_class_selection_is_exact(N, C, rate):
    r = np.random.default_rng(N + C)
    a = (r.integers(-20, 21, size=N) / 20.0).astype(np.float32)      # many ties
    labels = r.integers(-1, C + 1, size=N).astype(np.int32)
    idx, kc = sage.sage_select_classes(torch.from_numpy(a).to(DEV), torch.from_numpy(labels).to(DEV), C, rate)
    idx_ref, kc_ref = cb.select(a.astype(np.float64), labels, C, rate)
    assert kc == kc_ref.tolist()
    assert np.array_equal(idx.cpu().numpy(), idx_ref)


def test_full_path_with_classes_matches_oracle_within_tolerance():
    N, D, ell, C = 3000, 515, 16, 5
    rows = _rows(N, D, 77)
    labels = (np.arange(N) % C).astype(np.int32)
    ref = oracle.run(rows, D, ell, 0.2)
    a_ref, _, _ = cb.class_scores(ref["zhat"], labels, C)
    g = rows.to(DEV)
    fd = sage.SageFD(D, ell, torch.float32, 0)
    fd.update(g)
    fd.finalize()
    fd.score(g)
    lab = torch.from_numpy(labels).to(DEV)
    a = fd.score_classes(lab, C)
    idx, kc = sage.sage_select_classes(a, lab, C, 0.2)
    fd.close()
    a64 = a.double().cpu().numpy()
    assert np.max(np.abs(a64 - a_ref)) <= 1e-4
    assert kc == [120] * C
    idx_self, _ = cb.select(a64, labels, C, 0.2)                     # exact on the GPU's own scores
    assert np.array_equal(idx.cpu().numpy(), idx_self)
    idx_ref, _ = cb.select(a_ref, labels, C, 0.2)                    # vs the oracle: only near-threshold examples may differ
    diff = np.setxor1d(idx.cpu().numpy(), idx_ref)
    for i in diff:
        c = labels[i]
        thr = np.sort(a_ref[labels == c])[::-1][kc[c] - 1]
        assert abs(a_ref[i] - thr) <= 1e-4
