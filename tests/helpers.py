"""Shared helpers for the GPU parity tests: run the CUDA path through the Python binding of the C ABI
and the oracle on the same bytes, and compare in the metrics the tolerances are stated in."""
import numpy as np
import torch

import oracle
from oracle import metrics
import paper_2510_02470_b200 as sage

TOL_SKETCH = 1e-4          # ||S^T S - S_o^T S_o||_2 / ||A||_F^2
TOL_SCORE = {torch.float32: 1e-4, torch.bfloat16: 2e-3}


def gpu_run(rows_cpu: torch.Tensor, D: int, ell: int, keep_rate: float, chunks=None, score_chunks=None, sketches=1, block=None):
    """rows_cpu: (N, ld) CPU tensor. Returns dict with S (ell x D fp64 numpy), sigma, alpha, idx, stats."""
    dev = torch.device("cuda", 0)
    rows = rows_cpu.to(dev)
    N = rows.shape[0]
    fd = sage.SageFD(D, ell, rows.dtype, 0)
    try:
        if sketches > 1:
            fd.set_option(6, sketches)
        if block:
            fd.set_option(7, block)
        if chunks is None:
            fd.update(rows)
        else:
            r0 = 0
            for c in chunks:
                fd.update(rows[r0:r0 + c])
                r0 += c
            assert r0 == N
        fd.finalize()
        S, sigma = fd.sketch()
        scores = torch.empty((N,), dtype=torch.float32, device=dev)
        if score_chunks is None:
            fd.score(rows, scores)
        else:
            fd.score_begin(N)
            r0 = 0
            for c in score_chunks:
                fd.score_chunk(rows[r0:r0 + c], r0)
                r0 += c
            fd.score_end(scores)
        idx = sage.sage_select(scores, keep_rate)
        zhat, znorm, u = fd.intermediates(N)
        torch.cuda.synchronize()
        return {"S": S.double().cpu().numpy(), "sigma": sigma.double().cpu().numpy(),
                "alpha": scores.double().cpu().numpy(), "idx": idx.cpu().numpy(), "stats": fd.stats(),
                "zhat": zhat.double().cpu().numpy(), "znorm": znorm.double().cpu().numpy(), "u": u.double().cpu().numpy()}
    finally:
        fd.close()


def compare(gpu: dict, ref: dict, rows_cpu: torch.Tensor, D: int, keep_rate: float, tol_score=None, label=""):
    A = metrics.rows_as_f64(rows_cpu, D)
    F2 = float(np.linalg.norm(A) ** 2)
    sk = metrics.signed_gram_norm(gpu["S"], ref["S"]) / F2 if F2 > 0 else 0.0
    tol_score = tol_score if tol_score is not None else TOL_SCORE[rows_cpu.dtype]
    da = float(np.max(np.abs(gpu["alpha"] - ref["alpha"]))) if A.shape[0] else 0.0
    k = oracle.select_k(A.shape[0], keep_rate)
    ok_sel, ndiff = metrics.selection_agrees(gpu["idx"], ref["alpha"], k, tol_score)
    report = {"label": label, "sketch_rel": sk, "max_dalpha": da, "idx_diff": ndiff, "k": k}
    assert sk <= TOL_SKETCH, report
    assert da <= tol_score, report
    assert ok_sel, report
    return report
