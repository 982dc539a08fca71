"""Seeded synthetic gradient-row workloads.

This module only *produces inputs*: matrices of per-example "gradient" rows with the shapes, dtypes
and value structure of the five benchmark workloads (low-rank signal plus noise with log-normal row
norms; last-layer outer-product gradients of a softmax head; block-structured full-model rows).
It holds none of the selection method's arithmetic (no sketching, projection, scoring or selection),
so the CUDA path and the CPU oracle can both be fed from it without sharing any code of the method.

The paper measured on image-classification datasets with a ResNet-18; none of those datasets or
gradients are available offline, so these generators stand in for them by shape and structure:

* ``c1``  N=4,096   D=1,024       ell=32   fp32  rank-16 signal + noise, 10 % pure-noise rows
* ``c2``  N=50,000  D=5,130       ell=64   fp32  (softmax(logits) - onehot(y)) outer [h; 1], 10 classes
* ``c3``  N=50,000  D=51,300      ell=128  bf16  same generator with 100 classes
* ``c4``  N=200,000 D=262,144     ell=256  bf16  rank-64 signal + noise, generated on device in chunks
* ``c5``  N=50,000  D=11,173,962  ell=64   bf16  per-layer blocks, block-wise rank-8 + noise, chunked

Every generator is chunk-deterministic: the rows of chunk ``j`` depend only on ``(seed, workload, j)``,
so a row prefix of a workload is byte-identical to the same rows of the full workload, and the second
pass over a streamed workload regenerates exactly the bytes of the first.

Rows are returned as a 2-D torch tensor of shape ``(n, ld)`` with ``ld >= D`` the row pitch in elements
(the smallest pitch whose byte size is a multiple of 16, zero padded), dtype float32 or bfloat16.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Iterator, Optional, Tuple

import numpy as np
import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    N: int
    D: int
    ell: int
    dtype: torch.dtype
    keep_rates: Tuple[float, ...]
    chunk_rows: int          # rows per generated chunk (also the streaming granularity)
    on_device: bool          # True: chunks are generated on the GPU and never stored as N x D
    description: str

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == torch.float32 else 2

    @property
    def ld(self) -> int:
        return padded_pitch(self.D, self.elem_bytes)

    @property
    def num_chunks(self) -> int:
        return (self.N + self.chunk_rows - 1) // self.chunk_rows


def padded_pitch(D: int, elem_bytes: int) -> int:
    """Smallest pitch (in elements) >= D whose size in bytes is a multiple of 16."""
    per16 = 16 // elem_bytes
    return ((D + per16 - 1) // per16) * per16


WORKLOADS = {
    "c1": Workload("c1", 4096, 1024, 32, torch.float32, (0.1,), 1024, False,
                   "rank-16 signal + N(0,0.1^2) noise, lognormal(0,0.5) row norms, 10% pure-noise rows"),
    "c2": Workload("c2", 50000, 5130, 64, torch.float32, (0.05, 0.1, 0.3), 1000, False,
                   "last-layer rows (softmax-onehot) x [h;1], 10-class Gaussian mixture in R^512, 20% flipped labels"),
    "c3": Workload("c3", 50000, 51300, 128, torch.bfloat16, (0.1,), 500, False,
                   "last-layer rows, 100 classes, 10% label noise, rounded to bf16"),
    "c4": Workload("c4", 200000, 262144, 256, torch.bfloat16, (0.1,), 8192, True,
                   "rank-64 signal + noise, lognormal row norms, device-generated 8,192-row chunks"),
    "c5": Workload("c5", 50000, 11173962, 64, torch.bfloat16, (0.1,), 512, True,
                   "ResNet-18-sized rows: 21 per-layer blocks, rank-8 per block + noise, 512-row chunks"),
}


def scaled(w: Workload, N: Optional[int] = None, D: Optional[int] = None, ell: Optional[int] = None,
           chunk_rows: Optional[int] = None) -> Workload:
    """A smaller (or larger) instance of the same generator, for tests."""
    return dataclasses.replace(w, N=N or w.N, D=D or w.D, ell=ell or w.ell,
                               chunk_rows=chunk_rows or w.chunk_rows)


# ----------------------------------------------------------------------------------------------
# host generators (numpy, Philox counter-based streams keyed by (seed, tag, chunk))
# ----------------------------------------------------------------------------------------------

def _rng(seed: int, tag: int, chunk: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[(seed << 20) ^ (tag << 8), chunk]))


def _pad_to(rows: np.ndarray, ld: int) -> np.ndarray:
    n, D = rows.shape
    if ld == D:
        return np.ascontiguousarray(rows)
    out = np.zeros((n, ld), dtype=rows.dtype)
    out[:, :D] = rows
    return out


def _lowrank_chunk(w: Workload, seed: int, chunk: int, rank: int, noise_frac: float) -> np.ndarray:
    """Rows s_i (c_i Q + n_i); a seeded subset of rows keeps only the noise term."""
    n0 = chunk * w.chunk_rows
    n = min(w.chunk_rows, w.N - n0)
    qr = _rng(seed, 1)
    Q, _ = np.linalg.qr(qr.standard_normal((w.D, rank)))          # D x rank, orthonormal columns
    r = _rng(seed, 2, chunk)
    coef = r.standard_normal((n, rank))
    noise = 0.1 * r.standard_normal((n, w.D))
    scale = np.exp(0.5 * r.standard_normal(n))
    signal = coef @ Q.T
    if noise_frac > 0:
        perm = _rng(seed, 3).permutation(w.N)
        is_noise = np.zeros(w.N, dtype=bool)
        is_noise[perm[: int(round(noise_frac * w.N))]] = True
        signal[is_noise[n0:n0 + n]] = 0.0
    return (scale[:, None] * (signal + noise)).astype(np.float32)


def _lastlayer_chunk(w: Workload, seed: int, chunk: int, classes: int, flip_frac: float, factors: bool = False):
    """Rows [vec((p - e_y) h^T) ; (p - e_y)] for a nearest-mean softmax head over a Gaussian mixture; with
    ``factors`` the pair (p - e_y, h) the rows are outer products of, instead of the rows."""
    feat = (w.D - classes) // classes
    assert classes * feat + classes == w.D, "D must equal classes*features + classes"
    n0 = chunk * w.chunk_rows
    n = min(w.chunk_rows, w.N - n0)
    mu = _rng(seed, 11).standard_normal((classes, feat))
    W0 = np.maximum(mu, 0.0) / math.sqrt(feat)
    cls_all = np.arange(w.N) % classes
    cls_all = cls_all[_rng(seed, 12).permutation(w.N)]
    flip = np.zeros(w.N, dtype=bool)
    flip[_rng(seed, 13).permutation(w.N)[: int(round(flip_frac * w.N))]] = True
    shift = _rng(seed, 14).integers(1, classes, size=w.N)          # uniformly random *other* class
    y_all = np.where(flip, (cls_all + shift) % classes, cls_all)
    c = cls_all[n0:n0 + n]
    y = y_all[n0:n0 + n]
    r = _rng(seed, 15, chunk)
    h = np.maximum(mu[c] + r.standard_normal((n, feat)), 0.0)
    logits = h @ W0.T
    logits -= logits.max(axis=1, keepdims=True)
    p = np.exp(logits)
    p /= p.sum(axis=1, keepdims=True)
    p[np.arange(n), y] -= 1.0                                       # p - onehot(y)
    if factors:
        return p.astype(np.float32), h.astype(np.float32)
    rows = np.empty((n, w.D), dtype=np.float32)
    rows[:, : classes * feat] = (p[:, :, None] * h[:, None, :]).reshape(n, classes * feat)
    rows[:, classes * feat:] = p
    return rows


def host_chunk(w: Workload, seed: int, chunk: int) -> torch.Tensor:
    """Chunk ``chunk`` of a host-generated workload as a CPU tensor of shape (n, ld)."""
    if w.name == "c1":
        rows = _lowrank_chunk(w, seed, chunk, rank=16, noise_frac=0.1)
    elif w.name == "c2":
        rows = _lastlayer_chunk(w, seed, chunk, classes=10, flip_frac=0.2)
    elif w.name == "c3":
        rows = _lastlayer_chunk(w, seed, chunk, classes=100, flip_frac=0.1)
    else:
        raise ValueError(f"{w.name} is generated on the device; use device_chunk")
    t = torch.from_numpy(_pad_to(rows, padded_pitch(w.D, 4 if w.dtype == torch.float32 else 2)))
    return t if w.dtype == torch.float32 else t.to(torch.bfloat16)


def host_factors(w: Workload, seed: int = 0, n_rows: Optional[int] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """The last-layer workloads (c2, c3) in factored form: q = softmax - onehot (n x C) and the features h (n x F), in the
    workload's dtype and with padded pitches, such that row i of the workload's structured variant is
    [vec_rowmajor(q_i h_i^T) ; q_i] with the products taken exactly from the stored values. (For fp32 this is the
    workload's own row up to the rounding of the product; for bf16 the factors are rounded, not the products.)"""
    classes = {"c2": 10, "c3": 100}[w.name]
    flip = {"c2": 0.2, "c3": 0.1}[w.name]
    n_rows = w.N if n_rows is None else min(n_rows, w.N)
    feat = (w.D - classes) // classes
    eb = w.elem_bytes
    q = torch.zeros((n_rows, padded_pitch(classes, eb)), dtype=w.dtype)
    h = torch.zeros((n_rows, padded_pitch(feat, eb)), dtype=w.dtype)
    done = chunk = 0
    while done < n_rows:
        qc, hc = _lastlayer_chunk(w, seed, chunk, classes, flip, factors=True)
        take = min(qc.shape[0], n_rows - done)
        q[done:done + take, :classes] = torch.from_numpy(qc[:take]).to(w.dtype)
        h[done:done + take, :feat] = torch.from_numpy(hc[:take]).to(w.dtype)
        done += take
        chunk += 1
    return q, h


def host_rows(w: Workload, seed: int = 0, n_rows: Optional[int] = None) -> torch.Tensor:
    """The first ``n_rows`` rows (default: all N) of a host-generated workload, shape (n_rows, ld)."""
    n_rows = w.N if n_rows is None else min(n_rows, w.N)
    out = torch.empty((n_rows, w.ld), dtype=w.dtype)
    done = 0
    chunk = 0
    while done < n_rows:
        t = host_chunk(w, seed, chunk)
        take = min(t.shape[0], n_rows - done)
        out[done:done + take] = t[:take]
        done += take
        chunk += 1
    return out


# ----------------------------------------------------------------------------------------------
# device generators (torch ops on the given device; chunk-deterministic via a per-chunk seed)
# ----------------------------------------------------------------------------------------------

def resnet18_blocks(D: int = 11173962) -> Tuple[int, ...]:
    """Per-layer block sizes of a CIFAR-style ResNet-18 with a 10-way head: each conv together with
    its BatchNorm scale and shift, then the fully connected layer. They sum to 11,173,962; for other
    D (tests) the same proportions are used."""
    def conv(cin, cout, k):
        return cin * cout * k * k + 2 * cout
    blocks = [conv(3, 64, 3)]
    blocks += [conv(64, 64, 3)] * 4
    blocks += [conv(64, 128, 3), conv(128, 128, 3), conv(64, 128, 1), conv(128, 128, 3), conv(128, 128, 3)]
    blocks += [conv(128, 256, 3), conv(256, 256, 3), conv(128, 256, 1), conv(256, 256, 3), conv(256, 256, 3)]
    blocks += [conv(256, 512, 3), conv(512, 512, 3), conv(256, 512, 1), conv(512, 512, 3), conv(512, 512, 3)]
    blocks += [512 * 10 + 10]
    total = sum(blocks)
    assert total == 11173962
    if D == total:
        return tuple(blocks)
    sizes = [max(8, int(b * D / total)) for b in blocks]
    sizes[-2] += D - sum(sizes)
    assert sizes[-2] > 0 and sum(sizes) == D
    return tuple(sizes)


def _dev_gen(device, seed: int, tag: int, chunk: int = 0) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(((seed * 1000003 + tag) * 1000003 + chunk) & 0x7FFFFFFFFFFFFFFF)
    return g


class DeviceStream:
    """Chunked device-side generator for the streamed workloads (c4, c5).

    ``chunk(j)`` returns rows ``[j*chunk_rows, ...)`` as a (n, ld) tensor on ``device``; it depends only on
    (seed, j), so both passes of the method see the same bytes. The basis matrices are built once."""

    def __init__(self, w: Workload, seed: int = 0, device="cuda", sub_rows: int = 64):
        self.w, self.seed, self.device = w, seed, torch.device(device)
        self.sub_rows = sub_rows
        if w.name == "c4":
            g = _dev_gen(self.device, seed, 41)
            self.Q = torch.randn((64, w.D), generator=g, device=self.device) / math.sqrt(w.D)
        elif w.name == "c5":
            self.blocks = resnet18_blocks(w.D)
            g = _dev_gen(self.device, seed, 51)
            self.Qb = [torch.randn((8, d), generator=g, device=self.device) / math.sqrt(d) for d in self.blocks]
        else:
            raise ValueError("DeviceStream serves c4 and c5")

    def rows_in_chunk(self, j: int) -> int:
        return min(self.w.chunk_rows, self.w.N - j * self.w.chunk_rows)

    def chunk(self, j: int, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        w = self.w
        n = self.rows_in_chunk(j)
        if out is None:
            out = torch.zeros((n, w.ld), dtype=w.dtype, device=self.device)
        g = _dev_gen(self.device, self.seed, 42 if w.name == "c4" else 52, j)
        # Three passes over a sub-block: the noise is drawn, the low-rank signal is added to it in place
        # (x = sigma * noise + coef Q), and the row scale is applied while the result is rounded into the output.
        for r0 in range(0, n, self.sub_rows):
            r = min(self.sub_rows, n - r0)
            scale = torch.exp(0.5 * torch.randn((r, 1), generator=g, device=self.device))
            if w.name == "c4":
                coef = torch.randn((r, 64), generator=g, device=self.device)
                x = torch.randn((r, w.D), generator=g, device=self.device)
                x.addmm_(coef, self.Q, beta=0.1)
                torch.mul(x, scale, out=out[r0:r0 + r, : w.D])
            else:
                c0 = 0
                for d, Q in zip(self.blocks, self.Qb):
                    coef = torch.randn((r, 8), generator=g, device=self.device)
                    x = torch.randn((r, d), generator=g, device=self.device)
                    x.addmm_(coef, Q, beta=math.sqrt(2.0 / d))
                    torch.mul(x, scale, out=out[r0:r0 + r, c0:c0 + d])
                    c0 += d
        return out[:n]

    def __iter__(self) -> Iterator[torch.Tensor]:
        for j in range(self.w.num_chunks):
            yield self.chunk(j)
