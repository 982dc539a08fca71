"""CPU oracle for the SAGE selection hot path (fp64, plain C++; see sage_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the benchmark's CPU
baseline leg. The CUDA package never imports this package and this package never imports it.

``build()`` compiles ``sage_oracle.cpp`` with g++ into ``liboracle_sage.so`` next to the source;
``lib()`` loads it (building on first use).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sage_oracle.cpp")
_SO = os.path.join(_HERE, "liboracle_sage.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-fopenmp", "-shared", "-fPIC", "-o", _SO, _SRC]
        subprocess.run(cmd, check=True)
    return _SO


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        i64, i32, f64, vp = C.c_int64, C.c_int, C.c_double, C.c_void_p
        L.sage_oracle_fd_create.restype = vp
        L.sage_oracle_fd_create.argtypes = [i64, i32, i32, i32]
        L.sage_oracle_fd_destroy.argtypes = [vp]
        for name in ("f64", "f32", "bf16"):
            getattr(L, f"sage_oracle_fd_update_{name}").argtypes = [vp, vp, i64, i64]
            getattr(L, f"sage_oracle_score_{name}").argtypes = [vp, i32, i64, vp, i64, i64, vp, vp, vp, vp, vp]
        L.sage_oracle_fd_finalize.argtypes = [vp]
        L.sage_oracle_fd_sketch.argtypes = [vp, vp, vp]
        L.sage_oracle_fd_buffer.argtypes = [vp, vp, vp]
        L.sage_oracle_fd_stats.argtypes = [vp, vp, vp, vp, vp]
        L.sage_oracle_select_k.restype = i64
        L.sage_oracle_select_k.argtypes = [i64, f64]
        L.sage_oracle_select.restype = i64
        L.sage_oracle_select.argtypes = [vp, i64, f64, vp]
        L.sage_oracle_jacobi_eig.restype = i32
        L.sage_oracle_jacobi_eig.argtypes = [vp, i32, vp, vp]
        _lib = L
    return _lib


def _rows_view(rows) -> Tuple[str, np.ndarray, int, int]:
    """Accepts a 2-D numpy array (float64/float32, or uint16 holding bf16 bits) or a CPU torch tensor
    (float64/float32/bfloat16) whose last dimension is contiguous. Returns (kind, array, n, ld)."""
    if not isinstance(rows, np.ndarray):
        import torch
        assert rows.device.type == "cpu"
        if rows.dtype == torch.bfloat16:
            rows = rows.view(torch.int16).numpy().view(np.uint16)
        else:
            rows = rows.numpy()
    assert rows.ndim == 2 and (rows.shape[0] == 0 or rows.strides[1] == rows.itemsize)
    kind = {np.dtype(np.float64): "f64", np.dtype(np.float32): "f32", np.dtype(np.uint16): "bf16"}[rows.dtype]
    ld = rows.strides[0] // rows.itemsize if rows.shape[0] > 1 else max(rows.shape[1], 1)
    return kind, rows, rows.shape[0], ld


class OracleFD:
    """Frequent-Directions sketch state (Method section, Algorithm 1 Phase I) in fp64."""

    def __init__(self, D: int, ell: int, delta_rank: int = 0, route: int = 0):
        self.D, self.ell = int(D), int(ell)
        self._h = lib().sage_oracle_fd_create(self.D, self.ell, delta_rank, route)
        if not self._h:
            raise ValueError("bad D/ell")

    def update(self, rows, D: Optional[int] = None) -> None:
        kind, arr, n, ld = _rows_view(rows)
        assert arr.shape[1] >= self.D
        if n:
            getattr(lib(), f"sage_oracle_fd_update_{kind}")(self._h, arr.ctypes.data, n, ld)

    def finalize(self) -> Tuple[np.ndarray, np.ndarray]:
        lib().sage_oracle_fd_finalize(self._h)
        S = np.empty((self.ell, self.D))
        sigma = np.empty(self.ell)
        lib().sage_oracle_fd_sketch(self._h, S.ctypes.data, sigma.ctypes.data)
        return S, sigma

    def buffer(self) -> Tuple[np.ndarray, int]:
        B = np.empty((2 * self.ell, self.D))
        fill = C.c_int(0)
        lib().sage_oracle_fd_buffer(self._h, B.ctypes.data, C.byref(fill))
        return B, fill.value

    def stats(self) -> dict:
        rows, shr, sd, sw = C.c_int64(0), C.c_int64(0), C.c_double(0), C.c_int(0)
        lib().sage_oracle_fd_stats(self._h, C.byref(rows), C.byref(shr), C.byref(sd), C.byref(sw))
        return {"rows_seen": rows.value, "shrinks": shr.value, "sum_delta": sd.value, "last_sweeps": sw.value}

    def __del__(self):
        if getattr(self, "_h", None):
            lib().sage_oracle_fd_destroy(self._h)
            self._h = None


def score(S: np.ndarray, rows, D: Optional[int] = None) -> dict:
    """Agreement scores (Method section, paragraph on two-pass scoring,, Algorithm 1 Phase II) for all rows at once."""
    S = np.ascontiguousarray(S, dtype=np.float64)
    ell, Ds = S.shape
    kind, arr, n, ld = _rows_view(rows)
    assert arr.shape[1] >= Ds
    zhat = np.zeros((n, ell))
    znorm = np.zeros(n)
    zbar = np.zeros(ell)
    u = np.zeros(ell)
    alpha = np.zeros(n)
    getattr(lib(), f"sage_oracle_score_{kind}")(S.ctypes.data, ell, Ds, arr.ctypes.data, n, ld, zhat.ctypes.data,
                                                znorm.ctypes.data, zbar.ctypes.data, u.ctypes.data, alpha.ctypes.data)
    return {"zhat": zhat, "znorm": znorm, "zbar": zbar, "u": u, "alpha": alpha}


def select_k(N: int, keep_rate: float) -> int:
    return int(lib().sage_oracle_select_k(int(N), float(keep_rate)))


def select(alpha: np.ndarray, keep_rate: float) -> np.ndarray:
    """Top-k indices by alpha (Algorithm 1, the top-k step), ordered (alpha desc, index asc)."""
    alpha = np.ascontiguousarray(alpha, dtype=np.float64)
    N = alpha.shape[0]
    idx = np.empty(max(select_k(N, keep_rate), 1), dtype=np.int64)
    k = lib().sage_oracle_select(alpha.ctypes.data, N, float(keep_rate), idx.ctypes.data)
    return idx[:k].copy()


def jacobi_eig(K: np.ndarray) -> Tuple[np.ndarray, np.ndarray, int]:
    K = np.ascontiguousarray(K, dtype=np.float64)
    n = K.shape[0]
    U = np.empty((n, n))
    lam = np.empty(n)
    sweeps = lib().sage_oracle_jacobi_eig(K.ctypes.data, n, U.ctypes.data, lam.ctypes.data)
    return U, lam, sweeps


class OracleMergedFD:
    """P Frequent-Directions sketches over interleaved row blocks, merged pairwise at the freeze.

    The paper's sketch is one sequential stream (Method section, first paragraph). Frequent-Directions sketches are
    mergeable (a property of the works the paper cites for it): the sketch of the stacked rows of two sketches obeys
    the same guarantee as a sketch of all the rows behind them. This class states the merged form the CUDA library
    offers as an option, in terms of the sequential sketch above and nothing else:

    * rows are dealt in blocks of ``block`` consecutive rows (default ell + 1, the number of rows between two
      shrinks of one buffer): block b of the stream, counted from 0 over everything given to ``update``, goes to
      sketch b mod P, and every sketch sees its rows in stream order;
    * at the freeze every sketch is frozen on its own (orthogonalise, shrink only if more than ell rows are in use),
      which leaves c_p <= ell non-trivial rows; then, for stride s = 1, 2, 4, ...: sketch a (a = 0, 2s, 4s, ...)
      absorbs sketch a + s, if there is one: a fresh sequential sketch is fed the c_a rows of a, then the c_{a+s} rows
      of a + s, and is frozen. Sketch 0 is the result.

    With P = 1 nothing is dealt or merged: the result is the sequential sketch, bit for bit."""

    def __init__(self, D: int, ell: int, sketches: int, block: Optional[int] = None, route: int = 0):
        assert sketches >= 1
        self.D, self.ell, self.P, self.route = int(D), int(ell), int(sketches), route
        self.block = int(block) if block else self.ell + 1
        self.subs = [OracleFD(D, ell, route=route) for _ in range(self.P)]
        self.seen = 0
        self.merge_stats = {"shrinks": 0, "sum_delta": 0.0}
        self.frozen = None          # per sketch: (S, kept rows) as frozen before any merge

    def update(self, rows) -> None:
        kind, arr, n, ld = _rows_view(rows)
        i = 0
        while i < n:
            b = self.seen // self.block
            take = min(n - i, (b + 1) * self.block - self.seen)
            self.subs[b % self.P].update(arr[i:i + take])
            i += take
            self.seen += take

    @staticmethod
    def _freeze(fd: OracleFD):
        S, sigma = fd.finalize()
        _, kept = fd.buffer()
        return S, sigma, min(kept, fd.ell)

    def finalize(self) -> Tuple[np.ndarray, np.ndarray]:
        frozen = [self._freeze(fd) for fd in self.subs]
        self.frozen = [(S.copy(), c) for S, _, c in frozen]
        s = 1
        while s < self.P:
            for a in range(0, self.P, 2 * s):
                b = a + s
                if b >= self.P:
                    continue
                (Sa, _, ca), (Sb, _, cb) = frozen[a], frozen[b]
                m = OracleFD(self.D, self.ell, route=self.route)
                m.update(Sa[:ca])
                m.update(Sb[:cb])
                frozen[a] = self._freeze(m)
                st = m.stats()
                self.merge_stats["shrinks"] += st["shrinks"]
                self.merge_stats["sum_delta"] += st["sum_delta"]
            s *= 2
        return frozen[0][0], frozen[0][1]

    def stats(self) -> dict:
        per = [fd.stats() for fd in self.subs]
        return {"rows_seen": self.seen, "shrinks": sum(p["shrinks"] for p in per) + self.merge_stats["shrinks"],
                "sum_delta": sum(p["sum_delta"] for p in per) + self.merge_stats["sum_delta"],
                "last_sweeps": per[0]["last_sweeps"], "rows_per_sketch": [p["rows_seen"] for p in per]}


def run(rows, D: int, ell: int, keep_rate: float, route: int = 0, sketches: int = 1, block: Optional[int] = None) -> dict:
    """Whole path on resident rows: sketch -> finalize -> score -> select. sketches > 1: the merged form of pass 1."""
    fd = OracleFD(D, ell, route=route) if sketches == 1 else OracleMergedFD(D, ell, sketches, block, route)
    fd.update(rows)
    S, sigma = fd.finalize()
    out = score(S, rows)
    out.update(S=S, sigma=sigma, idx=select(out["alpha"], keep_rate), stats=fd.stats())
    return out
