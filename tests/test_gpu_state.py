"""GPU tests of the two additions that follow from the method's O(ell D) state (Method, the complexity paragraph):
the checkpoint of the sketch (export / import) and the strict-memory form of the scoring pass (no N x ell store, scores
from a third pass). Both are compared with the oracle on the same rows, and with the default path."""
import numpy as np
import pytest
import torch

import oracle
import paper_2510_02470_b200 as sage

from helpers import TOL_SCORE, compare, gpu_run
from test_gpu_parity import lowrank_rows

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("dtype,N,D,ell,P", [(torch.float32, 900, 260, 16, 1), (torch.bfloat16, 700, 1032, 40, 1),
                                             (torch.float32, 1500, 132, 8, 4)])
def test_checkpoint_resumes_bit_for_bit(dtype, N, D, ell, P):
    """Sketch part of the rows, export, restore into a NEW handle, sketch the rest: the frozen sketch equals that of the
    uninterrupted run bit for bit, and matches the oracle's sketch of all rows."""
    rows = lowrank_rows(N, D, 5, 0.4, N + ell, dtype)
    whole = gpu_run(rows, D, ell, 0.1, sketches=P)
    g = rows.to(DEV)
    cut = N // 2 + 3
    a = sage.SageFD(D, ell, dtype, 0)
    if P > 1:
        a.set_option(6, P)
    a.update(g[:cut])
    blob = a.export_state()
    a.close()
    b = sage.SageFD(D, ell, dtype, 0)
    b.import_state(blob)
    assert b.stats()["rows_seen"] == cut
    b.update(g[cut:])
    b.finalize()
    S, sigma = b.sketch()
    st = b.stats()
    assert np.array_equal(S.double().cpu().numpy(), whole["S"])
    assert st["shrinks"] == whole["stats"]["shrinks"] and st["sum_delta"] == whole["stats"]["sum_delta"] and st["rows_seen"] == N
    # a frozen sketch travels too: scores from the restored copy equal the original's
    frozen = b.export_state()
    c = sage.SageFD(D, ell, dtype, 0)
    c.import_state(frozen)
    a1 = c.score(g).double().cpu().numpy()
    assert np.array_equal(a1, whole["alpha"])
    assert c.stats()["shrinks"] == st["shrinks"]
    b.close()
    c.close()
    ref = oracle.run(rows, D, ell, 0.1, route=1, sketches=P)
    compare(whole, ref, rows, D, 0.1, label="checkpoint")


def test_checkpoint_rejects_foreign_data():
    a = sage.SageFD(64, 4, torch.float32, 0)
    a.update(lowrank_rows(30, 64, 2, 0.1, 1).to(DEV))
    blob = a.export_state()
    other = sage.SageFD(65, 4, torch.float32, 0)
    with pytest.raises(sage.SageError) as e:
        other.import_state(blob)
    assert e.value.status == 1
    with pytest.raises(sage.SageError):
        a.import_state(blob[: blob.numel() // 2].contiguous())        # truncated
    bad = blob.clone()
    bad[0] = 0
    with pytest.raises(sage.SageError):
        a.import_state(bad)
    assert a.stats()["rows_seen"] == 30                               # failed imports left the handle as it was
    a.close()
    other.close()


@pytest.mark.parametrize("dtype,N,D,ell", [(torch.float32, 3000, 515, 16), (torch.bfloat16, 2500, 20008, 24), (torch.float32, 700, 1028, 128)])
def test_strict_memory_scoring_matches_default_and_oracle(dtype, N, D, ell):
    """Option 8: the scoring pass keeps nothing of size N; a third pass over the rows (here in other chunks, and in
    another order) gives the scores. Same definition, so the scores match the oracle within the tolerance and the default
    path to rounding."""
    ld = D + (-D) % 8
    rows = lowrank_rows(N, D, 5, 0.4, N + D, dtype, ld)
    ref = oracle.run(rows, D, ell, 0.1, route=1)
    base = gpu_run(rows, D, ell, 0.1)
    g = rows.to(DEV)
    fd = sage.SageFD(D, ell, dtype, 0)
    fd.update(g)
    fd.finalize()
    fd.set_option(8, 1)
    fd.score_begin(N)
    for r0 in range(0, N, 999):
        fd.score_chunk(g[r0:r0 + 999], r0)
    fd.score_end(None)
    with pytest.raises(sage.SageError):
        fd.intermediates(N)                                           # nothing of size N was kept
    scores = torch.full((N,), 7.0, dtype=torch.float32, device=DEV)
    half = N // 2
    fd.score_apply(g[half:], scores[half:])                           # second half first
    fd.score_apply(g[:half], scores[:half])
    torch.cuda.synchronize()
    a = scores.double().cpu().numpy()
    assert fd.stats()["device_flags"] == 0
    assert np.max(np.abs(a - ref["alpha"])) <= TOL_SCORE[dtype]
    assert np.max(np.abs(a - base["alpha"])) <= 2e-6
    idx = sage.sage_select(scores, 0.1).cpu().numpy()
    from oracle import metrics
    assert metrics.selection_agrees(idx, ref["alpha"], oracle.select_k(N, 0.1), TOL_SCORE[dtype])[0]
    # back to the default mode on the same handle
    fd.set_option(8, 0)
    b = fd.score(g).double().cpu().numpy()
    assert np.array_equal(b, base["alpha"])
    with pytest.raises(sage.SageError):
        fd.score_apply(g[:10], scores[:10])                           # the default mode has no third pass
    fd.close()
