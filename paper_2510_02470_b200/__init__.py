"""Thin Python binding of the C ABI in ``include/sage.h`` (argument marshalling only).

Every function here has the name of the C entry point it calls; tensors are turned into raw device
pointers plus sizes, the current torch CUDA stream is passed as the ``cuda_stream`` argument, and a
non-zero status raises :class:`SageError`. All arithmetic happens in the CUDA library
(``libsage_b200.so``, built in-tree by ``python -m paper_2510_02470_b200.build``). There is no CPU
path: if the library is missing, loading it raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libsage_b200.so")
_lib: Optional[C.CDLL] = None

SAGE_F32, SAGE_BF16 = 0, 1
STATUS_NAMES = {0: "SAGE_OK", 1: "SAGE_ERR_INVALID_ARG", 2: "SAGE_ERR_BAD_STATE", 3: "SAGE_ERR_ALLOC",
                4: "SAGE_ERR_CUDA", 5: "SAGE_ERR_UNSUPPORTED", 6: "SAGE_ERR_NOT_CONVERGED", 7: "SAGE_ERR_NONFINITE"}

# name -> (restype, argtypes); the list every test of the boundary checks against include/sage.h
_i64, _i32, _f64, _vp, _u32 = C.c_int64, C.c_int32, C.c_double, C.c_void_p, C.c_uint32
SIGNATURES = {
    "sage_fd_create": (_i32, [_vp, _i64, _i32, _i32, _i32]),
    "sage_fd_destroy": (None, [_vp]),
    "sage_fd_reset": (_i32, [_vp]),
    "sage_fd_update": (_i32, [_vp, _vp, _i64, _i64, _vp]),
    "sage_fd_finalize": (_i32, [_vp, _vp]),
    "sage_fd_join": (_i32, [_vp, _vp]),
    "sage_fd_sketch": (_i32, [_vp, _vp, _vp, _vp]),
    "sage_fd_load_sketch": (_i32, [_vp, _vp, _i64, _vp]),
    "sage_score": (_i32, [_vp, _vp, _i64, _i64, _vp, _vp]),
    "sage_score_begin": (_i32, [_vp, _i64, _vp]),
    "sage_score_chunk": (_i32, [_vp, _vp, _i64, _i64, _i64, _vp]),
    "sage_score_end": (_i32, [_vp, _vp, _vp]),
    "sage_score_apply": (_i32, [_vp, _vp, _i64, _i64, _vp, _vp]),
    "sage_fd_update_outer": (_i32, [_vp, _vp, _i64, _vp, _i64, _i64, _i32, _i32, _vp]),
    "sage_score_chunk_outer": (_i32, [_vp, _vp, _i64, _vp, _i64, _i64, _i32, _i32, _i64, _vp]),
    "sage_score_outer": (_i32, [_vp, _vp, _i64, _vp, _i64, _i64, _i32, _i32, _vp, _vp]),
    "sage_score_intermediates": (_i32, [_vp, _vp, _vp, _vp]),
    "sage_fd_export_size": (_i32, [_vp, _vp]),
    "sage_fd_export": (_i32, [_vp, _vp, C.c_size_t, _vp]),
    "sage_fd_import": (_i32, [_vp, _vp, C.c_size_t, _vp]),
    "sage_select_count": (_i64, [_i64, _f64]),
    "sage_select": (_i32, [_vp, _i64, _f64, _vp, _vp, _vp]),
    "sage_score_classes": (_i32, [_vp, _vp, _i32, _vp, _vp]),
    "sage_score_class_centroids": (_i32, [_vp, _vp, _vp, _vp]),
    "sage_select_classes": (_i32, [_vp, _vp, _i64, _i32, _f64, _vp, _vp, _vp, _vp]),
    "sage_select_static": (_i32, [_vp, _i64, _f64, _vp, _vp, _vp]),
    "sage_select_from_host": (_i32, [_vp, _i64, _i64, _i64, _i32, _i32, _f64, _i64, _i32, _vp, _vp, _vp]),
    "sage_fd_stats": (_i32, [_vp, _vp]),
    "sage_fd_set_option": (_i32, [_vp, _i32, _f64]),
    "sage_fd_profile": (_i32, [_vp, _vp, _vp, _i32]),
    "sage_status_string": (C.c_char_p, [_i32]),
    "sage_last_error": (C.c_char_p, []),
    "sage_version": (C.c_char_p, []),
    "sage_launch_count": (_i64, []),
}


class SageStats(C.Structure):
    _fields_ = [("rows_seen", _i64), ("shrinks", _i64), ("sum_delta", _f64), ("last_sweeps", _i32),
                ("max_sweeps", _i32), ("last_rank", _i32), ("device_flags", _u32), ("kernel_launches", _i64),
                ("tensor_core_launches", _i64), ("rows_in_place", _i64)]


class SageError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


def lib() -> C.CDLL:
    """Loads the CUDA library; raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2510_02470_b200.build`")
        L = C.CDLL(_LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def _check(status: int, allow=()) -> int:
    if status != 0 and status not in allow:
        raise SageError(status, lib().sage_last_error().decode())
    return status


def _stream(device=None) -> int:
    return torch.cuda.current_stream(device).cuda_stream


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return SAGE_F32
    if t.dtype == torch.bfloat16:
        return SAGE_BF16
    raise TypeError(f"rows must be float32 or bfloat16, got {t.dtype}")


def _rows_args(rows: torch.Tensor, D: int) -> Tuple[int, int, int]:
    if rows.dim() != 2 or rows.shape[1] < D or (rows.shape[0] > 1 and rows.stride(1) != 1):
        raise ValueError("rows must be a 2-D tensor (n, >=D) with unit stride along D")
    ld = rows.stride(0) if rows.shape[0] > 1 else max(rows.shape[1], D)
    return rows.data_ptr(), rows.shape[0], ld


# ---- functions named after the C entry points -----------------------------------------------------

def sage_fd_create(D: int, ell: int, row_dtype: int, device: int = 0) -> int:
    h = _vp()
    _check(lib().sage_fd_create(C.byref(h), D, ell, row_dtype, device))
    return h.value


def sage_fd_destroy(h: int) -> None:
    lib().sage_fd_destroy(h)


def sage_fd_reset(h: int) -> None:
    _check(lib().sage_fd_reset(h))


def sage_fd_set_option(h: int, key: int, value: float) -> None:
    _check(lib().sage_fd_set_option(h, key, value))


def sage_fd_update(h: int, rows: torch.Tensor, D: int) -> None:
    ptr, n, ld = _rows_args(rows, D)
    _check(lib().sage_fd_update(h, ptr, n, ld, _stream(rows.device)))


def sage_fd_finalize(h: int, device=None, allow=()) -> int:
    return _check(lib().sage_fd_finalize(h, _stream(device)), allow)


def sage_fd_join(h: int, device=None) -> None:
    _check(lib().sage_fd_join(h, _stream(device)))


def sage_fd_sketch(h: int, ell: int, D: int, device) -> Tuple[torch.Tensor, torch.Tensor]:
    """Copies of the frozen sketch (ell x D) and sigma' (ell) as torch tensors on the device."""
    S, pitch, sig = _vp(), _i64(), _vp()
    _check(lib().sage_fd_sketch(h, C.byref(S), C.byref(pitch), C.byref(sig)))
    out = _borrow(S.value, (ell, D), (pitch.value * 4, 4), device).clone()
    sigma = _borrow(sig.value, (ell,), (4,), device).clone()
    return out, sigma


def sage_fd_load_sketch(h: int, S: torch.Tensor) -> None:
    assert S.dtype == torch.float32 and S.dim() == 2 and S.stride(1) == 1
    _check(lib().sage_fd_load_sketch(h, S.data_ptr(), S.stride(0), _stream(S.device)))


def sage_score(h: int, rows: torch.Tensor, D: int, scores: torch.Tensor) -> None:
    ptr, n, ld = _rows_args(rows, D)
    assert scores.dtype == torch.float32 and scores.is_contiguous() and scores.numel() >= n
    _check(lib().sage_score(h, ptr, n, ld, scores.data_ptr(), _stream(rows.device)))


def sage_score_begin(h: int, N_total: int, device=None) -> None:
    _check(lib().sage_score_begin(h, N_total, _stream(device)))


def sage_score_chunk(h: int, rows: torch.Tensor, D: int, row_offset: int) -> None:
    ptr, n, ld = _rows_args(rows, D)
    _check(lib().sage_score_chunk(h, ptr, n, ld, row_offset, _stream(rows.device)))


def sage_score_end(h: int, scores: Optional[torch.Tensor], device=None) -> None:
    """scores may be None in the strict-memory mode (option 8), where this call only forms the consensus direction."""
    if scores is None:
        _check(lib().sage_score_end(h, None, _stream(device)))
        return
    assert scores.dtype == torch.float32 and scores.is_contiguous()
    _check(lib().sage_score_end(h, scores.data_ptr(), _stream(scores.device)))


def _outer_args(q: torch.Tensor, feat: torch.Tensor, C: int, F: int):
    assert q.dim() == 2 and feat.dim() == 2 and q.shape[0] == feat.shape[0] and q.dtype == feat.dtype
    assert q.shape[1] >= C and feat.shape[1] >= F and q.stride(1) == 1 and feat.stride(1) == 1
    n = q.shape[0]
    return q.data_ptr(), (q.stride(0) if n > 1 else q.shape[1]), feat.data_ptr(), (feat.stride(0) if n > 1 else feat.shape[1]), n


def sage_fd_update_outer(h: int, q: torch.Tensor, feat: torch.Tensor, C: int, F: int) -> None:
    qp, ldq, fp, ldf, n = _outer_args(q, feat, C, F)
    _check(lib().sage_fd_update_outer(h, qp, ldq, fp, ldf, n, C, F, _stream(q.device)))


def sage_score_chunk_outer(h: int, q: torch.Tensor, feat: torch.Tensor, C: int, F: int, row_offset: int) -> None:
    qp, ldq, fp, ldf, n = _outer_args(q, feat, C, F)
    _check(lib().sage_score_chunk_outer(h, qp, ldq, fp, ldf, n, C, F, row_offset, _stream(q.device)))


def sage_score_outer(h: int, q: torch.Tensor, feat: torch.Tensor, C: int, F: int, scores: torch.Tensor) -> None:
    qp, ldq, fp, ldf, n = _outer_args(q, feat, C, F)
    assert scores.dtype == torch.float32 and scores.is_contiguous() and scores.numel() >= n
    _check(lib().sage_score_outer(h, qp, ldq, fp, ldf, n, C, F, scores.data_ptr(), _stream(q.device)))


def sage_score_apply(h: int, rows: torch.Tensor, D: int, scores: torch.Tensor) -> None:
    ptr, n, ld = _rows_args(rows, D)
    assert scores.dtype == torch.float32 and scores.is_contiguous() and scores.numel() >= n
    _check(lib().sage_score_apply(h, ptr, n, ld, scores.data_ptr(), _stream(rows.device)))


def sage_fd_export(h: int) -> torch.Tensor:
    """The checkpoint of the sketch as a CPU uint8 tensor."""
    need = C.c_size_t(0)
    _check(lib().sage_fd_export_size(h, C.byref(need)))
    buf = torch.empty((need.value,), dtype=torch.uint8)
    written = C.c_size_t(0)
    _check(lib().sage_fd_export(h, buf.data_ptr(), need.value, C.byref(written)))
    return buf[: written.value]


def sage_fd_import(h: int, blob: torch.Tensor, device=None) -> None:
    assert blob.device.type == "cpu" and blob.dtype == torch.uint8 and blob.is_contiguous()
    _check(lib().sage_fd_import(h, blob.data_ptr(), blob.numel(), _stream(device)))


def sage_score_intermediates(h: int, N: int, ell: int, device) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    zh, zn, u = _vp(), _vp(), _vp()
    _check(lib().sage_score_intermediates(h, C.byref(zh), C.byref(zn), C.byref(u)))
    zhat = _borrow(zh.value, (N, ell), (ell * 4, 4), device).clone()
    znorm = _borrow(zn.value, (N,), (4,), device).clone()
    uu = _borrow(u.value, (ell,), (4,), device).clone()
    return zhat, znorm, uu


def sage_select_count(N: int, keep_rate: float) -> int:
    return int(lib().sage_select_count(N, keep_rate))


def sage_select(scores: torch.Tensor, keep_rate: float, idx: Optional[torch.Tensor] = None) -> torch.Tensor:
    assert scores.dtype == torch.float32 and scores.is_contiguous()
    N = scores.numel()
    k = sage_select_count(N, keep_rate)
    if idx is None:
        idx = torch.empty((k,), dtype=torch.int64, device=scores.device)
    assert idx.dtype == torch.int64 and idx.numel() >= k
    k_out = _i64(0)
    _check(lib().sage_select(scores.data_ptr(), N, keep_rate, idx.data_ptr(), C.byref(k_out), _stream(scores.device)))
    return idx[: k_out.value]


def sage_score_classes(h: int, labels: torch.Tensor, num_classes: int, scores: torch.Tensor) -> None:
    assert labels.dtype == torch.int32 and labels.is_contiguous() and scores.dtype == torch.float32 and scores.is_contiguous()
    assert labels.numel() == scores.numel()
    _check(lib().sage_score_classes(h, labels.data_ptr(), num_classes, scores.data_ptr(), _stream(scores.device)))


def sage_score_class_centroids(h: int, ell: int, device) -> Tuple[torch.Tensor, torch.Tensor]:
    U, cnt, C_ = _vp(), _vp(), _i32(0)
    _check(lib().sage_score_class_centroids(h, C.byref(U), C.byref(cnt), C.byref(C_)))
    nc = C_.value
    Ut = _borrow(U.value, (nc, ell), (ell * 4, 4), device).clone()
    ct = torch.as_tensor(_DevArray(cnt.value, (nc,), (4,), "<i4"), device=device).clone()
    return Ut, ct


def sage_select_classes(scores: torch.Tensor, labels: torch.Tensor, num_classes: int, keep_rate: float):
    """Returns (idx on the device, list of k_c)."""
    assert scores.dtype == torch.float32 and scores.is_contiguous() and labels.dtype == torch.int32 and labels.is_contiguous()
    N = scores.numel()
    idx = torch.empty((max(sage_select_count(N, keep_rate), 1),), dtype=torch.int64, device=scores.device)
    kc = (C.c_int64 * num_classes)()
    k_out = _i64(0)
    _check(lib().sage_select_classes(scores.data_ptr(), labels.data_ptr(), N, num_classes, keep_rate, idx.data_ptr(), kc,
                                     C.byref(k_out), _stream(scores.device)))
    return idx[: k_out.value], [int(v) for v in kc]


def sage_select_static(scores: torch.Tensor, keep_rate: float, idx: torch.Tensor) -> torch.Tensor:
    """sage_select for callers that cannot allocate: the caller passes ``idx`` (capacity >= k) and the
    library uses its built-in scratch (N <= 262,144). Runs on the current device, current stream."""
    assert scores.dtype == torch.float32 and scores.is_contiguous()
    assert idx.dtype == torch.int64 and idx.is_contiguous()
    N = scores.numel()
    k = sage_select_count(N, keep_rate)
    assert idx.numel() >= k
    k_out = _i64(0)
    with torch.cuda.device(scores.device):
        _check(lib().sage_select_static(scores.data_ptr(), N, keep_rate, idx.data_ptr(), C.byref(k_out),
                                        _stream(scores.device)))
    return idx[: k_out.value]


def sage_select_from_host(rows: torch.Tensor, D: int, ell: int, keep_rate: float, chunk_rows: int = 0,
                          device: int = 0, want_scores: bool = True, allow=(6, 7)):
    """Whole path on HOST rows (pinned memory recommended). Returns (scores or None, idx) on the host."""
    assert rows.device.type == "cpu"
    ptr, N, ld = _rows_args(rows, D)
    k = sage_select_count(N, keep_rate)
    scores = torch.empty((N,), dtype=torch.float32).pin_memory() if want_scores else None
    idx = torch.empty((max(k, 1),), dtype=torch.int64).pin_memory()
    k_out = _i64(0)
    st = lib().sage_select_from_host(ptr, N, D, ld, ell, _dtype_code(rows), keep_rate, chunk_rows, device,
                                     scores.data_ptr() if want_scores else None, idx.data_ptr(), C.byref(k_out))
    _check(st, allow=allow)
    return scores, idx[: k_out.value]


def sage_fd_stats(h: int) -> dict:
    s = SageStats()
    _check(lib().sage_fd_stats(h, C.byref(s)))
    return {name: getattr(s, name) for name, _ in SageStats._fields_}


KERNEL_CLASSES = ("append", "gram", "gram_reduce", "eig_shrink", "rebuild", "project", "project_reduce",
                  "normalise", "score")


def sage_fd_profile(h: int) -> dict:
    ms = (C.c_double * 16)()
    n = (C.c_int64 * 16)()
    _check(lib().sage_fd_profile(h, ms, n, 16))
    return {name: {"ms": ms[i], "launches": n[i]} for i, name in enumerate(KERNEL_CLASSES)}


def sage_launch_count() -> int:
    return int(lib().sage_launch_count())


def sage_version() -> str:
    return lib().sage_version().decode()


class _DevArray:
    """Raw device memory described through __cuda_array_interface__ so that torch can view it."""

    def __init__(self, ptr: int, shape, strides_bytes, typestr: str = "<f4"):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "strides": tuple(strides_bytes), "typestr": typestr,
                                         "data": (int(ptr), False), "version": 2}


def _borrow(ptr: int, shape, strides_bytes, device) -> torch.Tensor:
    """A torch view (no copy) of library-owned device memory; callers clone what they keep."""
    return torch.as_tensor(_DevArray(ptr, shape, strides_bytes), device=device)


class SageFD:
    """Convenience owner of a handle: ``update`` rows, ``finalize``, ``score``, ``select``."""

    def __init__(self, D: int, ell: int, dtype: torch.dtype = torch.float32, device: int = 0):
        self.D, self.ell, self.dtype, self.device = D, ell, dtype, device
        self._h = sage_fd_create(D, ell, SAGE_F32 if dtype == torch.float32 else SAGE_BF16, device)

    def update(self, rows: torch.Tensor) -> None:
        assert rows.dtype == self.dtype
        sage_fd_update(self._h, rows, self.D)

    def finalize(self, allow=()) -> int:
        return sage_fd_finalize(self._h, self.device, allow)

    def join(self) -> None:
        sage_fd_join(self._h, self.device)

    def sketch(self):
        return sage_fd_sketch(self._h, self.ell, self.D, torch.device("cuda", self.device))

    def load_sketch(self, S: torch.Tensor) -> None:
        sage_fd_load_sketch(self._h, S)

    def score(self, rows: torch.Tensor, scores: Optional[torch.Tensor] = None) -> torch.Tensor:
        if scores is None:
            scores = torch.empty((rows.shape[0],), dtype=torch.float32, device=rows.device)
        sage_score(self._h, rows, self.D, scores)
        return scores

    def update_outer(self, q: torch.Tensor, feat: torch.Tensor, C: int, F: int) -> None:
        sage_fd_update_outer(self._h, q, feat, C, F)

    def score_outer(self, q: torch.Tensor, feat: torch.Tensor, C: int, F: int, scores: Optional[torch.Tensor] = None) -> torch.Tensor:
        if scores is None:
            scores = torch.empty((q.shape[0],), dtype=torch.float32, device=q.device)
        sage_score_outer(self._h, q, feat, C, F, scores)
        return scores

    def score_chunk_outer(self, q: torch.Tensor, feat: torch.Tensor, C: int, F: int, row_offset: int) -> None:
        sage_score_chunk_outer(self._h, q, feat, C, F, row_offset)

    def score_begin(self, N_total: int) -> None:
        sage_score_begin(self._h, N_total, self.device)

    def score_chunk(self, rows: torch.Tensor, row_offset: int) -> None:
        sage_score_chunk(self._h, rows, self.D, row_offset)

    def score_end(self, scores: Optional[torch.Tensor] = None) -> None:
        sage_score_end(self._h, scores)

    def score_apply(self, rows: torch.Tensor, scores: torch.Tensor) -> None:
        sage_score_apply(self._h, rows, self.D, scores)

    def export_state(self) -> torch.Tensor:
        return sage_fd_export(self._h)

    def import_state(self, blob: torch.Tensor) -> None:
        sage_fd_import(self._h, blob, self.device)

    def score_classes(self, labels: torch.Tensor, num_classes: int, scores: Optional[torch.Tensor] = None) -> torch.Tensor:
        if scores is None:
            scores = torch.empty((labels.numel(),), dtype=torch.float32, device=labels.device)
        sage_score_classes(self._h, labels, num_classes, scores)
        return scores

    def class_centroids(self):
        return sage_score_class_centroids(self._h, self.ell, torch.device("cuda", self.device))

    def intermediates(self, N: int):
        return sage_score_intermediates(self._h, N, self.ell, torch.device("cuda", self.device))

    def stats(self) -> dict:
        return sage_fd_stats(self._h)

    def profile(self) -> dict:
        return sage_fd_profile(self._h)

    def reset(self) -> None:
        sage_fd_reset(self._h)

    def set_option(self, key: int, value: float) -> None:
        sage_fd_set_option(self._h, key, value)

    def close(self) -> None:
        if self._h:
            sage_fd_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
