"""GPU parity: the CUDA path, called through the C ABI's Python binding, against the fp64 oracle on the
same seeded bytes in the same row order. Tolerances (stated by the benchmark spec):
  sketch  ||S^T S - S_o^T S_o||_2 / ||A||_F^2 <= 1e-4
  scores  |alpha - alpha_o| <= 1e-4 for fp32 rows, <= 2e-3 for bf16 rows
  indices identical except for rows whose oracle score is within that tolerance of the k-th score."""
import numpy as np
import pytest
import torch

import oracle
from oracle import metrics
import paper_2510_02470_b200 as sage
from paper_2510_02470_b200 import workloads as wl

from helpers import TOL_SCORE, TOL_SKETCH, compare, gpu_run
import replay_f64 as rp

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def lowrank_rows(N, D, rank, noise, seed, dtype=torch.float32, ld=None):
    r = np.random.default_rng(seed)
    Q, _ = np.linalg.qr(r.standard_normal((D, rank)))
    A = (r.standard_normal((N, rank)) + 0.6) @ Q.T * 2.0 + noise * r.standard_normal((N, D))
    A *= np.exp(0.5 * r.standard_normal((N, 1)))
    ld = ld or D
    out = np.zeros((N, ld), dtype=np.float32)
    out[:, :D] = A
    return torch.from_numpy(out).to(dtype)


# ------------------------------------------------------------------ selection (bit-exact)

@pytest.mark.parametrize("kind", ["random", "ties", "constant", "signed_zero"])
@pytest.mark.parametrize("N", [1, 31, 4096, 4097, 200000])
def test_select_matches_oracle_exactly(kind, N):
    r = np.random.default_rng(N)
    a = {"random": r.uniform(-1, 1, N), "ties": r.integers(-5, 6, N) / 5.0, "constant": np.full(N, -0.5),
         "signed_zero": np.where(r.uniform(size=N) < 0.5, 0.0, -0.0) * 1.0}[kind].astype(np.float32)
    s = torch.from_numpy(a).to(DEV)
    for rate in (0.0, 1e-4, 0.1, 0.3, 1.0):
        idx = sage.sage_select(s, rate).cpu().numpy()
        ref = oracle.select(a.astype(np.float64), rate)
        assert np.array_equal(idx, ref), (kind, N, rate)


def test_select_nan_ranks_last_and_errors():
    a = torch.tensor([0.5, float("nan"), -1.0, 0.7], device=DEV)
    assert sage.sage_select(a, 0.75).cpu().tolist() == [3, 0, 2]
    with pytest.raises(sage.SageError) as e:
        sage._check(sage.lib().sage_select(a.data_ptr(), 4, float("nan"), None, None, None))
    assert e.value.status == 1


# ------------------------------------------------------------------ scoring with the oracle's sketch

@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("N,D,ell", [(300, 257, 8), (1000, 1024, 32), (130, 5130, 64), (70, 3001, 128), (50, 777, 256),
                                     (700, 16392, 256), (300, 20008, 128)])
def test_score_with_loaded_sketch(dtype, N, D, ell):
    ld = wl.padded_pitch(D, 4 if dtype == torch.float32 else 2) if D % 2 else D
    rows = lowrank_rows(N, D, 5, 0.3, N + D, dtype, ld)
    S = np.random.default_rng(1).standard_normal((ell, D)) * np.linspace(3, 0.1, ell)[:, None]
    S32 = torch.from_numpy(S.astype(np.float32))
    ref = oracle.score(S32.double().numpy(), rows)
    fd = sage.SageFD(D, ell, dtype, 0)
    fd.load_sketch(S32.to(DEV))
    g = rows.to(DEV)
    tc0 = fd.stats()["tensor_core_launches"]
    a = fd.score(g).double().cpu().numpy()
    zhat, znorm, u = fd.intermediates(N)
    tc1 = fd.stats()["tensor_core_launches"]
    fd.close()
    if D >= 16384 and dtype == torch.bfloat16:
        assert tc1 > tc0, "long bf16 rows must take the tensor-core projection (one-term bf16 sketch)"
    assert np.max(np.abs(a - ref["alpha"])) <= TOL_SCORE[dtype] * (0.1 if D < 16384 else 0.5)
    assert np.allclose(znorm.double().cpu().numpy(), ref["znorm"], rtol=2e-3 if dtype == torch.bfloat16 else 1e-4)
    # long bf16 rows are projected onto a one-term bf16 copy of the sketch: u carries its rounding (still a unit vector)
    assert np.max(np.abs(u.double().cpu().numpy() - ref["u"])) <= (TOL_SCORE[dtype] if D >= 16384 and dtype == torch.bfloat16 else 1e-4)
    assert a.min() >= -1.0 and a.max() <= 1.0


def test_score_chunked_equals_oneshot_within_rounding_and_is_deterministic():
    N, D, ell = 5000, 640, 16
    rows = lowrank_rows(N, D, 6, 0.5, 3)
    a = gpu_run(rows, D, ell, 0.1)
    b = gpu_run(rows, D, ell, 0.1)
    assert np.array_equal(a["alpha"], b["alpha"]) and np.array_equal(a["idx"], b["idx"]) and np.array_equal(a["S"], b["S"])
    c = gpu_run(rows, D, ell, 0.1, chunks=[1, 30, 33, 936, 4000], score_chunks=[777, 4223])
    assert np.array_equal(a["S"], c["S"])                    # update chunking does not change the sketch
    assert np.max(np.abs(a["alpha"] - c["alpha"])) <= 2e-6


def test_zero_rows_and_zero_consensus():
    D, ell = 96, 4
    rows = lowrank_rows(40, D, 3, 0.2, 5)
    rows[7] = 0.0
    ref = oracle.run(rows, D, ell, 0.25)
    out = gpu_run(rows, D, ell, 0.25)
    assert out["alpha"][7] == 0.0 and out["znorm"][7] == 0.0 and np.all(out["zhat"][7] == 0)
    compare(out, ref, rows, D, 0.25)
    # g and -g cancel exactly: consensus 0, all scores 0
    fd = sage.SageFD(D, ell, torch.float32, 0)
    S = torch.zeros((ell, D))
    S[0, 0] = S[1, 1] = 1.0
    fd.load_sketch(S.to(DEV))
    g = torch.zeros((2, D))
    g[0, 0], g[1, 0] = 2.0, -2.0
    a = fd.score(g.to(DEV)).cpu().numpy()
    fd.close()
    assert np.all(a == 0.0)


# ------------------------------------------------------------------ sketch + full path on small shapes

@pytest.mark.parametrize("N,D,ell", [(3, 8, 2), (4, 17, 2), (9, 33, 4), (64, 32, 8), (257, 100, 5), (1000, 300, 16),
                                     (700, 1030, 33), (600, 400, 80), (500, 260, 100)])
def test_full_path_small_shapes(N, D, ell):
    rows = lowrank_rows(N, D, min(3, D), 0.3, N * 7 + D)
    ref = oracle.run(rows, D, ell, 0.2)
    out = gpu_run(rows, D, ell, 0.2)
    compare(out, ref, rows, D, 0.2, label=f"{N}x{D} ell={ell}")
    assert out["stats"]["shrinks"] == ref["stats"]["shrinks"] and out["stats"]["rows_seen"] == N
    assert np.isclose(out["stats"]["sum_delta"], ref["stats"]["sum_delta"], rtol=1e-3, atol=1e-6 * np.linalg.norm(rows.numpy()) ** 2)


@pytest.mark.parametrize("N", [1, 5, 8])
def test_exact_when_N_le_ell(N):
    D, ell = 70, 8
    rows = lowrank_rows(N, D, 3, 0.5, N)
    out = gpu_run(rows, D, ell, 0.5)
    A = rows.double().numpy()
    assert out["stats"]["shrinks"] == 0
    assert np.allclose(out["S"].T @ out["S"], A.T @ A, atol=2e-6 * np.linalg.norm(A) ** 2)


def test_rank_deficient_input_is_reproduced():
    D, ell, N = 64, 8, 300
    rows = lowrank_rows(N, D, 4, 0.0, 11)
    out = gpu_run(rows, D, ell, 0.1)
    A = rows.double().numpy()
    assert out["stats"]["shrinks"] > 10
    assert metrics.signed_gram_norm(out["S"], A) <= 1e-4 * np.linalg.norm(A) ** 2
    compare(out, oracle.run(rows, D, ell, 0.1), rows, D, 0.1)


def test_closed_form_single_shrink():
    ell, D = 6, 40
    m = 2 * ell
    r = np.random.default_rng(0)
    Q, _ = np.linalg.qr(r.standard_normal((D, m)))
    sig = np.sort(r.uniform(0.5, 4.0, m))[::-1]
    rows = torch.from_numpy((sig[:, None] * Q.T)[r.permutation(m)].astype(np.float32))
    out = gpu_run(rows, D, ell, 0.5)
    kept = np.sqrt(np.clip(sig ** 2 - sig[ell - 1] ** 2, 0, None))
    expect = kept[:, None] * Q.T
    assert np.allclose(out["S"].T @ out["S"], expect.T @ expect, atol=1e-5 * sig[0] ** 2)
    assert np.allclose(out["sigma"], kept[:ell], atol=1e-5 * sig[0])


def test_lemma_identity_on_gpu_outputs():
    N, D, ell = 800, 200, 12
    rows = lowrank_rows(N, D, 4, 0.3, 21)
    out = gpu_run(rows, D, ell, 0.25)
    T, a, zn = out["idx"], out["alpha"], out["znorm"]
    Z = out["zhat"] * zn[:, None]
    xi = a[T].min()
    assert xi > 0
    lhs = ((Z[T] @ out["u"]) ** 2).sum()
    assert np.isclose(lhs, (zn[T] ** 2 * a[T] ** 2).sum(), rtol=1e-4)
    assert lhs >= xi ** 2 * (zn[T] ** 2).sum() * (1 - 1e-4)
    assert np.linalg.norm(Z[T].mean(axis=0)) >= xi * zn[T].mean() * (1 - 1e-4)


# ------------------------------------------------------------------ merged form of pass 1 (several sketches)

@pytest.mark.parametrize("N,D,ell,P,block", [(500, 64, 6, 2, None), (777, 130, 8, 4, 5), (40, 70, 8, 4, None), (3000, 260, 16, 16, None),
                                             (2500, 1028, 64, 4, None), (9, 33, 4, 16, 1), (1200, 516, 128, 3, None)])
def test_merged_sketches_small_shapes(N, D, ell, P, block):
    """Option 6: P sketches over interleaved row blocks, merged pairwise at the freeze, against the oracle's statement
    of the same dealing and merge order; update calls cut the stream at points unrelated to the blocks."""
    rows = lowrank_rows(N, D, min(5, D), 0.4, N + P)
    ref = oracle.run(rows, D, ell, 0.2, route=1, sketches=P, block=block)
    cuts = [N // 3, N // 2 - N // 3, N - N // 2]
    out = gpu_run(rows, D, ell, 0.2, chunks=cuts, sketches=P, block=block)
    compare(out, ref, rows, D, 0.2, label=f"{N}x{D} ell={ell} P={P}")
    assert out["stats"]["shrinks"] == ref["stats"]["shrinks"] and out["stats"]["rows_seen"] == N
    assert np.isclose(out["stats"]["sum_delta"], ref["stats"]["sum_delta"], rtol=1e-3, atol=1e-6 * np.linalg.norm(rows.numpy()) ** 2)
    again = gpu_run(rows, D, ell, 0.2, sketches=P, block=block)       # other call boundaries, same sketch
    assert np.array_equal(out["S"], again["S"]) and np.array_equal(out["idx"], again["idx"])


@pytest.mark.parametrize("P", [1, 4, 16])
def test_c1_full_merged(P):
    w = wl.WORKLOADS["c1"]
    rows = wl.host_rows(w, 0)
    ref = oracle.run(rows, w.D, w.ell, 0.1, sketches=P)
    out = gpu_run(rows, w.D, w.ell, 0.1, sketches=P)
    print(compare(out, ref, rows, w.D, 0.1, label=f"c1 P={P}"), out["stats"])
    assert out["stats"]["shrinks"] == ref["stats"]["shrinks"] and out["stats"]["device_flags"] == 0


@pytest.mark.parametrize("P", [4, 16])
def test_c2_prefix_merged(P):
    w = wl.WORKLOADS["c2"]
    rows = wl.host_rows(w, 0, 12000)
    ref = oracle.run(rows, w.D, w.ell, 0.1, route=1, sketches=P)
    out = gpu_run(rows, w.D, w.ell, 0.1, sketches=P)
    print(compare(out, ref, rows, w.D, 0.1, label=f"c2[:12000] P={P}"), out["stats"])
    assert out["stats"]["shrinks"] == ref["stats"]["shrinks"] and out["stats"]["device_flags"] == 0


def test_merged_option_rules():
    fd = sage.SageFD(64, 4, torch.float32, 0)
    rows = lowrank_rows(30, 64, 2, 0.1, 1).to(DEV)
    for bad in (0, 65, 2.5):
        with pytest.raises(sage.SageError):
            fd.set_option(6, bad)
    fd.set_option(6, 3)
    fd.update(rows)
    with pytest.raises(sage.SageError) as e:
        fd.set_option(6, 2)                                  # only before the first update
    assert e.value.status == 2
    fd.join()
    fd.finalize()
    assert fd.stats()["rows_seen"] == 30
    fd.reset()
    fd.set_option(6, 1)                                      # back to the sequential sketch after a reset
    fd.update(rows)
    fd.finalize()
    S1, _ = fd.sketch()
    fd.close()
    ref = gpu_run(rows.cpu(), 64, 4, 0.5)
    assert np.array_equal(S1.double().cpu().numpy(), ref["S"])


# ------------------------------------------------------------------ tensor-core kernels against the CUDA-core kernels

def _run_with_option(rows, D, ell, use_tc):
    dev = torch.device("cuda", 0)
    g = rows.to(dev)
    fd = sage.SageFD(D, ell, rows.dtype, 0)
    fd.set_option(4, 1.0 if use_tc else 0.0)
    fd.update(g)
    fd.finalize()
    S, _ = fd.sketch()
    a = fd.score(g)
    torch.cuda.synchronize()
    st = fd.stats()
    fd.close()
    return S.double().cpu().numpy(), a.double().cpu().numpy(), st


@pytest.mark.parametrize("dtype,N,D,ell", [(torch.float32, 900, 2052, 40), (torch.bfloat16, 700, 4104, 64),
                                           (torch.bfloat16, 600, 20008, 24), (torch.float32, 500, 1000, 128)])
def test_tensor_core_path_agrees_with_cuda_core_path(dtype, N, D, ell):
    """Same rows through option 4 = 1 (tcgen05 Gram / rebuild / projection) and option 4 = 0 (fp32 FMA kernels):
    both must match the oracle, and each other far more tightly than the tolerances."""
    rows = lowrank_rows(N, D, 6, 0.4, N + ell, dtype)
    S1, a1, st1 = _run_with_option(rows, D, ell, True)
    S0, a0, st0 = _run_with_option(rows, D, ell, False)
    assert st1["device_flags"] == 0 and st0["device_flags"] == 0 and st1["shrinks"] == st0["shrinks"]
    A = metrics.rows_as_f64(rows, D)
    F2 = float(np.linalg.norm(A) ** 2)
    assert metrics.signed_gram_norm(S1, S0) / F2 <= 2e-5
    # bf16 rows: the tensor-core path rounds the sketch to bf16 (one term for D >= 16384), the CUDA-core path does not
    assert np.max(np.abs(a1 - a0)) <= (2e-5 if dtype == torch.float32 else TOL_SCORE[dtype])
    ref = oracle.run(rows, D, ell, 0.1, route=1)
    for S, a in ((S1, a1), (S0, a0)):
        assert metrics.signed_gram_norm(S, ref["S"]) / F2 <= 1e-4
        assert np.max(np.abs(a - ref["alpha"])) <= TOL_SCORE[dtype]


@pytest.mark.parametrize("N,D,ell,ld", [(520, 1000, 16, 1100008), (515, 1000, 16, 1100008), (264, 20008, 24, 1200000),
                                        (392, 16456, 64, 1048576)])
def test_bf16_rows_a_page_or_more_apart_score_like_packed_rows(N, D, ell, ld):
    """bfloat16 rows held in a much wider matrix (row pitch of 2 MB and more): the projection then fetches two K tiles
    per row visit through 4-D TMA boxes where the shapes allow it (row counts that are multiples of 8; 515 rows take the
    2-D boxes), with the two-term sketch (D = 1000), the one-term sketch, odd numbers of K tiles and ragged last tiles.
    The scores must be those of the same rows packed tightly, far inside the tolerance, and match the oracle."""
    rows = lowrank_rows(N, D, 5, 0.4, N + D, torch.bfloat16)
    dev = torch.device("cuda", 0)
    wide = torch.zeros((N, ld), dtype=torch.bfloat16, device=dev)
    wide[:, :D] = rows.to(dev)
    wide[:, D:D + 64] = float("nan")                       # what follows a row must never be read as data
    packed = rows.to(dev)
    out = []
    for g in (wide[:, :D], packed):
        fd = sage.SageFD(D, ell, torch.bfloat16, 0)
        fd.update(g)
        fd.finalize()
        a = fd.score(g)
        torch.cuda.synchronize()
        st = fd.stats()
        S, _ = fd.sketch()
        fd.close()
        assert st["device_flags"] == 0
        out.append((S.double().cpu().numpy(), a.double().cpu().numpy()))
    assert np.array_equal(out[0][0], out[1][0])                                    # pass 1 does not depend on the pitch
    assert np.max(np.abs(out[0][1] - out[1][1])) <= 2e-5
    ref = oracle.run(rows, D, ell, 0.1, route=1)
    assert np.max(np.abs(out[0][1] - ref["alpha"])) <= TOL_SCORE[torch.bfloat16]


@pytest.mark.parametrize("N,D,ell,cuts", [(1000, 4104, 64, [300, 300, 400]), (777, 1000, 32, [97] * 8 + [1]), (900, 20008, 64, [66, 65, 64, 705]),
                                          (500, 2056, 64, [500])])
def test_rows_read_in_place_give_the_appended_result_bit_for_bit(N, D, ell, cuts):
    """bfloat16 rows, ell = 32 / 64: shrink cycles whose ell + 1 new rows lie inside one update call read them where the
    caller holds them (option 9, default) instead of appending them. The arithmetic is the same, so sketch and scores must
    equal those of the always-append form (option 9 = 0) bit for bit, whatever the calls' sizes (leftover rows, cycles that
    straddle two calls, calls shorter than a cycle); the counter of rows read in place must move, and both match the oracle."""
    assert sum(cuts) == N
    rows = lowrank_rows(N, D, 6, 0.4, N + D + ell, torch.bfloat16)
    g = rows.to(torch.device("cuda", 0))
    out = []
    for direct in (1, 0):
        fd = sage.SageFD(D, ell, torch.bfloat16, 0)
        fd.set_option(9, direct)
        r0 = 0
        for c in cuts:
            fd.update(g[r0:r0 + c])
            r0 += c
        fd.finalize()
        S, sigma = fd.sketch()
        a = fd.score(g)
        torch.cuda.synchronize()
        st = fd.stats()
        fd.close()
        assert st["device_flags"] == 0
        out.append((S.cpu().numpy().copy(), sigma.cpu().numpy().copy(), a.cpu().numpy().copy(), st))
    assert out[0][3]["rows_in_place"] > 0 and out[0][3]["rows_in_place"] % (ell + 1) == 0 and out[1][3]["rows_in_place"] == 0
    assert out[0][3]["shrinks"] == out[1][3]["shrinks"]
    assert np.array_equal(out[0][0], out[1][0]) and np.array_equal(out[0][1], out[1][1]) and np.array_equal(out[0][2], out[1][2])
    ref = oracle.run(rows, D, ell, 0.1, route=1)
    F2 = float(np.linalg.norm(metrics.rows_as_f64(rows, D)) ** 2)
    assert metrics.signed_gram_norm(out[0][0].astype(np.float64), ref["S"]) / F2 <= 1e-4
    assert np.max(np.abs(out[0][2].astype(np.float64) - ref["alpha"])) <= TOL_SCORE[torch.bfloat16]


# ------------------------------------------------------------------ the two eigen-solve kernel families

def _run_with_eig_variant(rows, D, ell, variant):
    dev = torch.device("cuda", 0)
    g = rows.to(dev)
    fd = sage.SageFD(D, ell, rows.dtype, 0)
    fd.set_option(5, float(variant))
    fd.update(g)
    fd.finalize()
    S, sigma = fd.sketch()
    a = fd.score(g)
    torch.cuda.synchronize()
    st = fd.stats()
    fd.close()
    return S.double().cpu().numpy(), sigma.double().cpu().numpy(), a.double().cpu().numpy(), st


@pytest.mark.parametrize("N,D,ell,rank", [(300, 520, 8, 3), (700, 1028, 32, 6), (900, 1028, 64, 40), (900, 772, 96, 200),
                                          (1200, 1028, 128, 12), (1500, 516, 256, 300), (150, 260, 64, 200)])
def test_cluster_eigen_solve_agrees_with_one_cta_solve(N, D, ell, rank):
    """Option 5 = 0 (cluster of 8 CTAs, Jacobi columns in distributed shared memory; buffers of 16 to 512 rows cover
    every instantiation) against option 5 = 1 (one-CTA / L2 kernels): same algorithm, so the sketches agree to
    rounding, and both match the oracle."""
    rows = lowrank_rows(N, D, rank, 0.3, 7 * N + ell)
    S0, sg0, a0, st0 = _run_with_eig_variant(rows, D, ell, 0)
    S1, sg1, a1, st1 = _run_with_eig_variant(rows, D, ell, 1)
    assert st0["device_flags"] == 0 and st1["device_flags"] == 0 and st0["shrinks"] == st1["shrinks"]
    A = metrics.rows_as_f64(rows, D)
    F2 = float(np.linalg.norm(A) ** 2)
    assert metrics.signed_gram_norm(S0, S1) / F2 <= 2e-5
    assert np.allclose(sg0, sg1, rtol=0, atol=2e-4 * max(sg1.max(), 1e-30))
    assert np.max(np.abs(a0 - a1)) <= 5e-5
    ref = oracle.run(rows, D, ell, 0.1, route=1)
    assert metrics.signed_gram_norm(S0, ref["S"]) / F2 <= 1e-4
    assert np.max(np.abs(a0 - ref["alpha"])) <= 1e-4


# ------------------------------------------------------------------ the benchmark workloads

def test_c1_full():
    w = wl.WORKLOADS["c1"]
    rows = wl.host_rows(w, 0)
    ref = oracle.run(rows, w.D, w.ell, 0.1)
    out = gpu_run(rows, w.D, w.ell, 0.1)
    rep = compare(out, ref, rows, w.D, 0.1, label="c1")
    assert out["stats"]["shrinks"] == 124 and len(out["idx"]) == 410
    print(rep, out["stats"])


def test_c2_prefix_three_keep_rates():
    w = wl.WORKLOADS["c2"]
    rows = wl.host_rows(w, 0, 4000)                          # dense pitch 5132 (16-byte multiple)
    ref = oracle.run(rows, w.D, w.ell, 0.1, route=1)
    out = gpu_run(rows, w.D, w.ell, 0.1)
    print(compare(out, ref, rows, w.D, 0.1, label="c2[:4000]"), out["stats"])
    s = torch.from_numpy(out["alpha"].astype(np.float32)).to(DEV)
    for rate in (0.05, 0.3):
        idx = sage.sage_select(s, rate).cpu().numpy()
        ok, _ = metrics.selection_agrees(idx, ref["alpha"], oracle.select_k(4000, rate), 1e-4)
        assert ok
    # unpadded pitch (ld = D, rows not 16-byte aligned) takes the generic path and must agree
    dense = rows[:, : w.D].contiguous()
    out2 = gpu_run(dense, w.D, w.ell, 0.1)
    compare(out2, ref, dense, w.D, 0.1, label="c2 dense pitch")


def test_c2_full_size():
    """The default benchmark workload at its full size (50,000 rows, 769 shrinks) against the oracle: errors of the
    tensor-core Gram / rebuild accumulate over the shrinks, so the prefix test above does not bound them."""
    w = wl.WORKLOADS["c2"]
    rows = wl.host_rows(w, 0)
    ref = oracle.run(rows, w.D, w.ell, 0.1, route=0)         # one-sided Jacobi on the rows: no Gram matrix, no rebuild
    out = gpu_run(rows, w.D, w.ell, 0.1)
    rep = compare(out, ref, rows, w.D, 0.1, label="c2 full")
    assert out["stats"]["shrinks"] == 769 and len(out["idx"]) == 5000
    print(rep, out["stats"])


def _replay_run(rows_dev, D, ell, chunk=4096):
    """fp64 replay (torch on the device) of sketch, freeze and scores for resident rows."""
    rep = rp.ReplayFD(D, ell, rows_dev.device)
    for r0 in range(0, rows_dev.shape[0], chunk):
        rep.update(rows_dev[r0:r0 + chunk])
    S = rep.finalize()
    sc = rp.ReplayScore(S, rows_dev.shape[0])
    for r0 in range(0, rows_dev.shape[0], chunk):
        sc.chunk(rows_dev[r0:r0 + chunk], sub_rows=1024)
    alpha, u = sc.end()
    return rep, S, alpha


def _replay_equals_oracle(rep, S_rep, a_rep, ref, F2):
    """The replay restates the oracle's Gram route with library routines: on the same rows they agree to fp64 rounding
    of that route (the Gram matrix squares the condition number, so about 1e-9 of ||A||_F^2, far below the tolerances)."""
    assert rep.shrinks == ref["stats"]["shrinks"]
    # (the comparison itself is good to about 1e-8 of ||A||_F^2 where the operands are too large for its QR form)
    assert metrics.signed_gram_norm(S_rep.cpu().numpy(), ref["S"]) / F2 <= 1e-7
    assert np.isclose(rep.sum_delta, ref["stats"]["sum_delta"], rtol=1e-8)
    assert np.max(np.abs(a_rep - ref["alpha"])) <= 1e-6


def _compare_with_replay(label, S_gpu, S_rep, F2, a_gpu, a_rep, idx_gpu, keep_rate, tol):
    sk = rp.signed_gram_norm_device(S_gpu.double(), S_rep) / F2
    da = float(np.max(np.abs(a_gpu - a_rep)))
    k = oracle.select_k(a_rep.size, keep_rate)
    ok, ndiff = rp.selection_agrees(idx_gpu, a_rep, k, tol)
    report = {"label": label, "sketch_rel": sk, "max_dalpha": da, "idx_diff": ndiff, "k": k}
    assert sk <= TOL_SKETCH and da <= tol and ok, report
    return report


def test_c3_prefix_bf16_against_oracle_and_replay():
    """The first 12,000 rows of c3 (92 shrinks of a 256-row buffer) against the oracle; the fp64 device replay used by
    the full-size tests is pinned to the oracle on the same rows."""
    w = wl.scaled(wl.WORKLOADS["c3"], N=12000)
    rows = wl.host_rows(w, 0)
    ref = oracle.run(rows, w.D, w.ell, 0.1, route=1)
    out = gpu_run(rows, w.D, w.ell, 0.1)
    print(compare(out, ref, rows, w.D, 0.1, label="c3[:12000]"), out["stats"])
    rep, S_rep, a_rep = _replay_run(rows.to(DEV), w.D, w.ell)
    _replay_equals_oracle(rep, S_rep, a_rep, ref, rep.fro_a)


def test_c3_full_size_properties():
    """c3 at its full size (50,000 x 51,300 bf16, 387 shrinks), where the oracle would take an hour: checks that need no
    oracle run. The Frequent-Directions bounds on A^T A - S^T S (largest eigenvalue by power iteration, at most the sum
    of the deltas; smallest not below zero), the loss of squared Frobenius norm (at least ell times that sum), scores
    of sampled rows recomputed in fp64 from the library's own S and u, the identity sum(alpha) = |sum(zhat)|, and the
    selection redone by the oracle's sort on the library's scores."""
    w = wl.WORKLOADS["c3"]
    rows = wl.host_rows(w, 0)
    g = rows.to(DEV)
    N, D, ell = w.N, w.D, w.ell
    fd = sage.SageFD(D, ell, rows.dtype, 0)
    fd.update(g)
    fd.finalize()
    S, _ = fd.sketch()
    scores = fd.score(g)
    zhat, znorm, u = fd.intermediates(N)
    idx = sage.sage_select(scores, 0.1)
    torch.cuda.synchronize()
    st = fd.stats()
    assert st["shrinks"] == 387 and st["device_flags"] == 0
    S64 = S[:, :D].double()

    def op(x):                                     # x -> A^T (A x) - S^T (S x), fp64, rows converted chunk by chunk
        y = torch.zeros_like(x)
        for r0 in range(0, N, 2500):
            a = g[r0:r0 + 2500, :D].double()
            y += a.T @ (a @ x)
        return y - S64.T @ (S64 @ x)

    gen = torch.Generator(device=DEV).manual_seed(3)
    fro_a = sum(float((g[r0:r0 + 5000, :D].double() ** 2).sum()) for r0 in range(0, N, 5000))
    x = torch.randn(D, dtype=torch.float64, device=DEV, generator=gen)
    lam_max = 0.0
    for _ in range(25):
        x = x / x.norm()
        y = op(x)
        lam_max = float(x @ y)
        x = y
    assert lam_max <= st["sum_delta"] * (1 + 1e-3), (lam_max, st["sum_delta"])
    x = torch.randn(D, dtype=torch.float64, device=DEV, generator=gen)     # smallest eigenvalue: iterate on lam_max I - M
    lam_min = 0.0
    for _ in range(25):
        x = x / x.norm()
        y = lam_max * x - op(x)
        lam_min = lam_max - float(x @ y)
        x = y
    assert lam_min >= -1e-5 * fro_a, (lam_min, fro_a)
    assert fro_a - float((S64 ** 2).sum()) >= ell * st["sum_delta"] * (1 - 1e-3)
    # scores of sampled rows from the library's own sketch and consensus, in fp64
    pick = np.random.default_rng(5).choice(N, 256, replace=False)
    z = g[torch.from_numpy(pick).to(DEV), :D].double() @ S64.T
    zn = z.norm(dim=1, keepdim=True)
    a64 = ((z / zn.clamp_min(1e-300)) @ u[:ell].double()).cpu().numpy()
    a_gpu = scores.double().cpu().numpy()
    assert np.max(np.abs(a64 - a_gpu[pick])) <= TOL_SCORE[torch.bfloat16]
    assert abs(a_gpu.sum() - float(zhat.double().sum(dim=0).norm())) <= 1e-3 * N ** 0.5
    assert np.array_equal(idx.cpu().numpy(), oracle.select(a_gpu, 0.1))
    fd.close()
    # all 50,000 rows and 387 shrinks against the fp64 replay (pinned to the oracle on the 12,000-row prefix above)
    rep, S_rep, a_rep = _replay_run(g, D, ell)
    assert rep.shrinks == 387
    print(_compare_with_replay("c3 full vs fp64 replay", S[:, :D], S_rep, rep.fro_a, a_gpu, a_rep, idx.cpu().numpy(), 0.1,
                               TOL_SCORE[torch.bfloat16]))


def test_c4_shape_small_prefix():
    """c4's generator and ell=256 on a reduced D and row count (the full D is covered by bench checks)."""
    w = wl.scaled(wl.WORKLOADS["c4"], N=1300, D=8192, chunk_rows=650)
    stream = wl.DeviceStream(w, seed=0, device=DEV)
    rows = torch.cat([stream.chunk(j) for j in range(w.num_chunks)]).cpu()
    ref = oracle.run(rows, w.D, w.ell, 0.1, route=1)
    out = gpu_run(rows, w.D, w.ell, 0.1, chunks=[650, 650], score_chunks=[650, 650])
    print(compare(out, ref, rows, w.D, 0.1, label="c4-shape"), out["stats"])


def test_c5_shape_small_prefix():
    w = wl.scaled(wl.WORKLOADS["c5"], N=600, D=111739, chunk_rows=256)
    stream = wl.DeviceStream(w, seed=0, device=DEV)
    rows = torch.cat([stream.chunk(j) for j in range(w.num_chunks)]).cpu()
    ref = oracle.run(rows, w.D, w.ell, 0.1, route=1)
    out = gpu_run(rows, w.D, w.ell, 0.1, chunks=[256, 256, 88], score_chunks=[256, 256, 88])
    print(compare(out, ref, rows, w.D, 0.1, label="c5-shape"), out["stats"])


# ------------------------------------------------------------------ streamed workloads at full row length

def _prefix_full_D(name, n_rows, chunk_rows):
    """The first n_rows rows of a streamed workload at its full D: CUDA path and fp64 replay against the oracle."""
    w = wl.scaled(wl.WORKLOADS[name], N=n_rows, chunk_rows=chunk_rows)
    stream = wl.DeviceStream(w, seed=0, device=DEV)
    chunks = [stream.rows_in_chunk(j) for j in range(w.num_chunks)]
    rows_dev = torch.cat([stream.chunk(j) for j in range(w.num_chunks)])
    rows = rows_dev.cpu()
    ref = oracle.run(rows, w.D, w.ell, 0.1, route=1)
    out = gpu_run(rows, w.D, w.ell, 0.1, chunks=chunks, score_chunks=chunks)
    print(compare(out, ref, rows, w.D, 0.1, label=f"{name}[:{n_rows}] at full D"), out["stats"])
    rep, S_rep, a_rep = _replay_run(rows_dev, w.D, w.ell, chunk=chunk_rows)
    _replay_equals_oracle(rep, S_rep, a_rep, ref, rep.fro_a)


def test_c4_prefix_at_full_D_against_oracle():
    """1,300 rows of 262,144 bf16 values, ell = 256: four shrinks of the 512-row buffer plus the freeze, the bf16
    tensor-core projection with a 256-row sketch, two chunks per pass."""
    _prefix_full_D("c4", 1300, 650)


def test_c5_prefix_at_full_D_against_oracle():
    """140 rows of 11,173,962 bf16 values, ell = 64: a shrink of the full buffer plus the shrinking freeze, at the full row length."""
    _prefix_full_D("c5", 140, 128)


def _streamed_properties(w, sample_rows=192):
    """Both passes streamed chunk by chunk, as the benchmark does for c4 and c5, with the fp64 replay fed the same chunks;
    returns what the checks need."""
    stream = wl.DeviceStream(w, seed=0, device=DEV)
    N, D, ell = w.N, w.D, w.ell
    fd = sage.SageFD(D, ell, w.dtype, 0)
    rep = rp.ReplayFD(D, ell, torch.device(DEV))
    buf = torch.zeros((w.chunk_rows, w.ld), dtype=w.dtype, device=DEV)
    for j in range(w.num_chunks):
        c = stream.chunk(j, buf)
        fd.update(c)
        rep.update(c)
        torch.cuda.synchronize()                 # the chunk buffer is refilled next
    fd.finalize()
    S, _ = fd.sketch()
    S_rep = rep.finalize()
    rsc = rp.ReplayScore(S_rep, N)
    fd.score_begin(N)
    pick = np.sort(np.random.default_rng(7).choice(N, min(sample_rows, N), replace=False))
    kept = []
    r0 = 0
    for j in range(w.num_chunks):
        c = stream.chunk(j, buf)
        fd.score_chunk(c, r0)
        rsc.chunk(c, sub_rows=64 if D > 1000000 else 1024)
        local = pick[(pick >= r0) & (pick < r0 + c.shape[0])] - r0
        if local.size:
            kept.append(c[torch.from_numpy(local).to(DEV), :D].clone())
        r0 += c.shape[0]
        torch.cuda.synchronize()
    scores = torch.empty((N,), dtype=torch.float32, device=DEV)
    fd.score_end(scores)
    a_rep, _ = rsc.end()
    zhat, znorm, u = fd.intermediates(N)
    idx = sage.sage_select(scores, 0.1)
    torch.cuda.synchronize()
    st = fd.stats()
    a_gpu = scores.double().cpu().numpy()
    # sampled rows re-scored in fp64 from the library's own S and u, a block of sketch columns at a time
    G = torch.cat(kept)
    z = torch.zeros((G.shape[0], ell), dtype=torch.float64, device=DEV)
    for c0 in range(0, D, 1 << 20):
        z += G[:, c0:c0 + (1 << 20)].double() @ S[:, c0:min(D, c0 + (1 << 20))].double().T
    a64 = ((z / z.norm(dim=1, keepdim=True).clamp_min(1e-300)) @ u[:ell].double()).cpu().numpy()
    fro_s = float((S[:, :D] ** 2).sum(dtype=torch.float64))
    fd.close()
    del buf, G, z
    sk = rp.signed_gram_norm_device(S[:, :D].double(), S_rep) / rep.fro_a
    out = {"stats": st, "fro_a": rep.fro_a, "fro_s": fro_s, "a_gpu": a_gpu, "a64": a64, "pick": pick,
           "sum_zhat_norm": float(zhat.double().sum(dim=0).norm()), "idx": idx.cpu().numpy(),
           "replay": {"sketch_rel": sk, "alpha": a_rep, "shrinks": rep.shrinks, "sum_delta": rep.sum_delta}}
    return out


def _expected_shrinks(N, ell):
    """Shrinks of a 2 ell-row buffer over N rows: one whenever the buffer fills up (ell - 1 rows survive), and one at
    the freeze if more than ell rows are in use."""
    fill = shrinks = 0
    for _ in range(N):
        fill += 1
        if fill == 2 * ell:
            shrinks += 1
            fill = ell - 1
    return shrinks + (1 if fill > ell else 0)


def _check_streamed(o, w, shrinks):
    st = o["stats"]
    assert st["shrinks"] == shrinks and st["device_flags"] == 0
    assert o["fro_a"] - o["fro_s"] >= w.ell * st["sum_delta"] * (1 - 1e-3)          # every shrink removes at least ell * delta
    assert np.max(np.abs(o["a64"] - o["a_gpu"][o["pick"]])) <= TOL_SCORE[torch.bfloat16]
    assert abs(o["a_gpu"].sum() - o["sum_zhat_norm"]) <= 1e-3 * w.N ** 0.5
    assert np.array_equal(o["idx"], oracle.select(o["a_gpu"], 0.1))
    # every row and every shrink against the fp64 replay (pinned to the oracle by the prefix tests at full D above)
    r = o["replay"]
    tol = TOL_SCORE[torch.bfloat16]
    da = float(np.max(np.abs(o["a_gpu"] - r["alpha"])))
    ok, ndiff = rp.selection_agrees(o["idx"], r["alpha"], oracle.select_k(w.N, 0.1), tol)
    report = {"workload": w.name, "sketch_rel": r["sketch_rel"], "max_dalpha": da, "idx_diff": ndiff}
    print(report)
    assert r["shrinks"] == shrinks and np.isclose(st["sum_delta"], r["sum_delta"], rtol=1e-3), report
    assert r["sketch_rel"] <= TOL_SKETCH and da <= tol and ok, report


def test_c4_full_size_against_replay():
    """c4 at its full size (200,000 x 262,144 bf16 in 25 chunks, ell = 256, 778 shrinks): property checks that need no
    reference, then sketch, scores and selection against the fp64 replay of the same chunks."""
    w = wl.WORKLOADS["c4"]
    _check_streamed(_streamed_properties(w), w, _expected_shrinks(w.N, w.ell))


def test_c5_full_size_against_replay():
    """c5 at its full size (50,000 x 11,173,962 bf16 in 98 chunks, ell = 64, 769 shrinks)."""
    w = wl.WORKLOADS["c5"]
    _check_streamed(_streamed_properties(w, sample_rows=96), w, _expected_shrinks(w.N, w.ell))


# ------------------------------------------------------------------ host pipeline and state machine

def test_select_from_host_matches_device_path():
    N, D, ell = 3000, 515, 16
    rows = lowrank_rows(N, D, 5, 0.4, 9, ld=516)
    ref = oracle.run(rows, D, ell, 0.1)
    scores, idx = sage.sage_select_from_host(rows.pin_memory(), D, ell, 0.1, chunk_rows=700)
    dev = gpu_run(rows, D, ell, 0.1, score_chunks=[700, 700, 700, 700, 200])
    assert np.array_equal(idx.numpy(), dev["idx"])
    assert np.max(np.abs(scores.double().numpy() - ref["alpha"])) <= 1e-4


def test_select_from_host_bf16_rows_read_in_place():
    """The host pipeline with bfloat16 rows and ell = 64: inside it most shrink cycles read their rows straight from the
    staging buffers the copies land in, so a copy that overwrote a buffer too early would show here. Same result as the
    device path on the same rows, and both inside the tolerance of the oracle."""
    N, D, ell = 1500, 2056, 64
    rows = lowrank_rows(N, D, 6, 0.4, 21, torch.bfloat16)
    ref = oracle.run(rows, D, ell, 0.1, route=1)
    scores, idx = sage.sage_select_from_host(rows.pin_memory(), D, ell, 0.1, chunk_rows=400)
    dev = gpu_run(rows, D, ell, 0.1, score_chunks=[400, 400, 400, 300])
    assert np.max(np.abs(scores.double().numpy() - dev["alpha"])) <= 1e-6 and np.array_equal(idx.numpy(), dev["idx"])
    assert np.max(np.abs(scores.double().numpy() - ref["alpha"])) <= TOL_SCORE[torch.bfloat16]


def test_state_machine_and_errors():
    D, ell = 64, 4
    fd = sage.SageFD(D, ell, torch.float32, 0)
    rows = lowrank_rows(20, D, 2, 0.1, 1).to(DEV)
    with pytest.raises(sage.SageError) as e:
        fd.score(rows)
    assert e.value.status == 2                               # not frozen yet
    fd.update(rows[:0])                                      # n == 0 is a no-op
    fd.update(rows)
    with pytest.raises(sage.SageError):
        sage._check(sage.lib().sage_fd_update(fd._h, rows.data_ptr(), 5, D - 1, None))   # ld < D
    fd.finalize()
    with pytest.raises(sage.SageError) as e:
        fd.update(rows)
    assert e.value.status == 2
    fd.score_begin(20)
    with pytest.raises(sage.SageError):
        fd.score_chunk(rows[:5], 3)                          # wrong offset
    fd.score_chunk(rows[:5], 0)
    with pytest.raises(sage.SageError):
        fd.score_end(torch.empty(20, device=DEV))            # rows missing
    fd.score_chunk(rows[5:], 5)
    fd.score_end(torch.empty(20, device=DEV))
    fd.reset()
    fd.update(rows)
    fd.finalize()
    assert fd.stats()["rows_seen"] == 20
    fd.close()


def test_nonfinite_rows_are_flagged_not_fatal():
    D, ell = 64, 4
    fd = sage.SageFD(D, ell, torch.float32, 0)
    S = torch.eye(ell, D)
    fd.load_sketch(S.to(DEV))
    g = lowrank_rows(10, D, 2, 0.1, 2)
    g[3, 0] = float("nan")
    g[4, 1] = float("inf")
    a = fd.score(g.to(DEV)).cpu().numpy()
    assert a[3] == 0.0 and a[4] == 0.0 and np.all(np.isfinite(a))
    assert fd.stats()["device_flags"] & 2
    fd.close()
