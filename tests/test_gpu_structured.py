"""GPU parity for structured last-layer rows: the library is given the factors (q = softmax - onehot, h = features) and
must give what the oracle gives on the materialised rows [vec(q h^T) ; q]. Through the C ABI's binding; tolerances as
in the dense tests (pass 1 forms the products exactly; the scoring pass never forms the rows: it projects the features onto
every class block of the sketch and folds the results with the other factor)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import metrics, structured
import paper_2510_02470_b200 as sage
from paper_2510_02470_b200 import workloads as wl

from helpers import TOL_SCORE, TOL_SKETCH

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def factors(N, C, F, seed, dtype, ldq=None, ldf=None):
    r = np.random.default_rng(seed)
    mu = r.standard_normal((C, F))
    cls = r.integers(0, C, N)
    h = np.maximum(mu[cls] + r.standard_normal((N, F)), 0.0)
    logits = h @ (np.maximum(mu, 0).T / np.sqrt(F))
    p = np.exp(logits - logits.max(axis=1, keepdims=True))
    p /= p.sum(axis=1, keepdims=True)
    p[np.arange(N), np.where(r.uniform(size=N) < 0.2, r.integers(0, C, N), cls)] -= 1.0
    q_t = torch.zeros((N, ldq or C), dtype=dtype)
    h_t = torch.zeros((N, ldf or F), dtype=dtype)
    q_t[:, :C] = torch.from_numpy(p.astype(np.float32)).to(dtype)
    h_t[:, :F] = torch.from_numpy(h.astype(np.float32)).to(dtype)
    return q_t, h_t


def gpu_outer(q, h, C, F, ell, keep, cuts=None, sketches=1):
    D = C * F + C
    qd, hd = q.to(DEV), h.to(DEV)
    N = q.shape[0]
    fd = sage.SageFD(D, ell, q.dtype, 0)
    if sketches > 1:
        fd.set_option(6, sketches)
    r0 = 0
    for c in (cuts or [N]):
        fd.update_outer(qd[r0:r0 + c], hd[r0:r0 + c], C, F)
        r0 += c
    fd.finalize()
    S, _ = fd.sketch()
    scores = torch.empty((N,), dtype=torch.float32, device=DEV)
    fd.score_begin(N)
    r0 = 0
    for c in (cuts or [N]):
        fd.score_chunk_outer(qd[r0:r0 + c], hd[r0:r0 + c], C, F, r0)
        r0 += c
    fd.score_end(scores)
    idx = sage.sage_select(scores, keep)
    torch.cuda.synchronize()
    st = fd.stats()
    fd.close()
    return S.double().cpu().numpy(), scores.double().cpu().numpy(), idx.cpu().numpy(), st


def check(q, h, C, F, ell, keep, S, a, idx, st, ref, tol):
    G = structured.materialise(q[:, :C], h[:, :F])
    F2 = float(np.linalg.norm(G) ** 2)
    sk = metrics.signed_gram_norm(S, ref["S"]) / F2
    da = float(np.max(np.abs(a - ref["alpha"])))
    ok, nd = metrics.selection_agrees(idx, ref["alpha"], oracle.select_k(len(a), keep), tol)
    report = {"sketch_rel": sk, "max_dalpha": da, "idx_diff": nd}
    assert sk <= TOL_SKETCH and da <= tol and ok and st["device_flags"] == 0, report
    assert st["shrinks"] == ref["stats"]["shrinks"]
    return report


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("N,C,F,ell,ldq,ldf", [(300, 3, 5, 4, None, None), (900, 10, 64, 16, 12, 64), (700, 7, 33, 8, 8, 40),
                                               (600, 16, 128, 64, 16, 128), (500, 20, 100, 128, 24, 104)])
def test_structured_rows_match_oracle(dtype, N, C, F, ell, ldq, ldf):
    q, h = factors(N, C, F, N + C, dtype, ldq, ldf)
    ref = structured.run(q[:, :C], h[:, :F], ell, 0.2, route=1)
    S, a, idx, st = gpu_outer(q, h, C, F, ell, 0.2, cuts=[N // 3, N - N // 3])
    print(check(q, h, C, F, ell, 0.2, S, a, idx, st, ref, TOL_SCORE[dtype]))


def test_structured_and_dense_calls_mix_and_agree():
    """The same rows given once as factors and once materialised (fp32): same sketch and scores up to the rounding of the
    products, and the two kinds of call may alternate on one handle."""
    N, C, F, ell = 800, 6, 40, 12
    D = C * F + C
    q, h = factors(N, C, F, 5, torch.float32)
    G = torch.from_numpy(structured.materialise(q, h).astype(np.float32))
    ref = oracle.run(G, D, ell, 0.1, route=1)
    fd = sage.SageFD(D, ell, torch.float32, 0)
    qd, hd, gd = q.to(DEV), h.to(DEV), G.to(DEV)
    fd.update_outer(qd[:300], hd[:300], C, F)
    fd.update(gd[300:500])
    fd.update_outer(qd[500:], hd[500:], C, F)
    fd.finalize()
    S, _ = fd.sketch()
    a = fd.score_outer(qd, hd, C, F).double().cpu().numpy()
    b = fd.score(gd).double().cpu().numpy()
    fd.close()
    assert metrics.signed_gram_norm(S.double().cpu().numpy(), ref["S"]) / float(np.linalg.norm(G.double().numpy()) ** 2) <= TOL_SKETCH
    assert np.max(np.abs(a - ref["alpha"])) <= 1e-4 and np.max(np.abs(a - b)) <= 1e-5


@pytest.mark.parametrize("dtype,ell,tol", [(torch.float32, 64, 2e-5), (torch.bfloat16, 128, TOL_SCORE[torch.bfloat16])])
def test_structured_scoring_over_several_sub_chunks_agrees_with_dense_rows(dtype, ell, tol):
    """c3-shaped factors (100 classes x 512 features), 45,000 rows: the per-class planes of that many rows do not fit the
    1 GiB the library allows itself, so the scoring pass takes several sub-chunks. The reference is the dense scoring
    pass of the same handle on rows materialised on the device a chunk at a time (itself checked against the oracle
    by the dense tests); fp32 products are exact, bfloat16 rows carry the rounding of each product."""
    N, C, F = 45000, 100, 512
    D = C * F + C
    g = torch.Generator(device=DEV).manual_seed(11)
    cls = torch.randint(0, C, (N,), device=DEV, generator=g)
    mu = torch.randn((C, F), device=DEV, generator=g)
    h = torch.relu(mu[cls] + torch.randn((N, F), device=DEV, generator=g))
    q = torch.softmax(h @ torch.relu(mu).T / F ** 0.5, dim=1)
    q[torch.arange(N, device=DEV), cls] -= 1.0
    q, h = q.to(dtype).contiguous(), h.to(dtype).contiguous()
    fd = sage.SageFD(D, ell, dtype, 0)
    fd.update_outer(q[:3 * ell], h[:3 * ell], C, F)
    fd.finalize()
    a = fd.score_outer(q, h, C, F).double().cpu().numpy()
    b = torch.empty((N,), dtype=torch.float32, device=DEV)
    fd.score_begin(N)
    for r0 in range(0, N, 9000):
        qs, hs = q[r0:r0 + 9000].float(), h[r0:r0 + 9000].float()
        rows = torch.cat([(qs[:, :, None] * hs[:, None, :]).reshape(qs.shape[0], C * F), qs], dim=1).to(dtype)
        fd.score_chunk(rows, r0)
        torch.cuda.synchronize()
        del rows
    fd.score_end(b)
    torch.cuda.synchronize()
    st = fd.stats()
    fd.close()
    assert st["device_flags"] == 0
    assert np.max(np.abs(a - b.double().cpu().numpy())) <= tol


def test_structured_rows_merged_sketches_and_errors():
    N, C, F, ell, P = 1200, 5, 24, 8, 3
    q, h = factors(N, C, F, 9, torch.float32)
    ref = structured.run(q, h, ell, 0.1, route=1, sketches=P)
    S, a, idx, st = gpu_outer(q, h, C, F, ell, 0.1, cuts=[500, 700], sketches=P)
    check(q, h, C, F, ell, 0.1, S, a, idx, st, ref, 1e-4)
    fd = sage.SageFD(C * F + C + 1, ell, torch.float32, 0)
    with pytest.raises(sage.SageError) as e:
        fd.update_outer(q.to(DEV), h.to(DEV), C, F)                   # C F + C != D
    assert e.value.status == 1
    fd.close()
    fd = sage.SageFD(C * F + C, ell, torch.float32, 0)
    with pytest.raises(sage.SageError) as e:
        fd.score_outer(q.to(DEV), h.to(DEV), C, F)                    # not frozen
    assert e.value.status == 2
    fd.close()


@pytest.mark.parametrize("name,rows", [("c2", 6000), ("c3", 2000)])
def test_last_layer_workloads_in_factored_form(name, rows):
    """c2 / c3 given as their factors: 10 x 512 + 10 and 100 x 512 + 100 values per row never exist on the caller's side."""
    w = wl.scaled(wl.WORKLOADS[name], N=rows)
    C = {"c2": 10, "c3": 100}[name]
    Fd = (w.D - C) // C
    q, h = wl.host_factors(w, 0, rows)
    ref = structured.run(q[:, :C], h[:, :Fd], w.ell, 0.1, route=1)
    S, a, idx, st = gpu_outer(q, h, C, Fd, w.ell, 0.1)
    print(name, check(q, h, C, Fd, w.ell, 0.1, S, a, idx, st, ref, TOL_SCORE[w.dtype]), st)
