"""An fp64 replay of the selection path with torch on the device, for comparisons at sizes the CPU oracle cannot
reach in a test run.

Test infrastructure only. It restates the oracle's Gram route (Gram matrix -> symmetric eigen-decomposition ->
delta = the ell-th largest eigenvalue -> rows rebuilt with the factors sqrt(max(1 - delta/lambda, 0))) with library
routines in double precision (torch.matmul, torch.linalg.eigh), shares nothing with the CUDA library, and is itself
checked against the CPU oracle on row prefixes by the tests that use it. The chain is: oracle == replay on a prefix
(to fp64 rounding), replay versus the CUDA path at full size (within the benchmark's tolerances)."""
import numpy as np
import torch


class ReplayFD:
    def __init__(self, D: int, ell: int, device):
        self.D, self.ell, self.m = D, ell, 2 * ell
        self.dev = device
        self.B = torch.zeros((self.m, D), dtype=torch.float64, device=device)
        self.fill = 0
        self.shrinks = 0
        self.sum_delta = 0.0
        self.fro_a = 0.0

    def _factor(self, r: int, shrink: bool) -> None:
        ell = self.ell
        Bc = self.B[:r]
        K = Bc @ Bc.T
        lam, U = torch.linalg.eigh(K)
        lam = lam.flip(0)
        U = U.flip(1)
        if shrink:
            delta = float(lam[ell - 1]) if r >= ell else 0.0
            keep = min(ell - 1, r)
            self.sum_delta += max(delta, 0.0)
            self.shrinks += 1
        else:
            delta = 0.0
            keep = min(r, ell)
        lk = lam[:keep]
        f = torch.where(lk > 0, torch.sqrt(torch.clamp(1.0 - delta / lk.clamp_min(1e-300), min=0.0)), torch.zeros_like(lk))
        new = (U[:, :keep] * f).T @ Bc
        self.B.zero_()
        self.B[:keep] = new
        self.fill = keep

    def update(self, rows: torch.Tensor) -> None:
        """rows: (n, >= D) tensor on the device, any floating dtype; converted exactly to fp64 a buffer-load at a time."""
        n = rows.shape[0]
        i = 0
        while i < n:
            take = min(n - i, self.m - self.fill)
            blk = rows[i:i + take, : self.D].double()
            self.fro_a += float((blk * blk).sum())
            self.B[self.fill:self.fill + take] = blk
            del blk
            self.fill += take
            i += take
            if self.fill == self.m:
                self._factor(self.m, True)

    def finalize(self) -> torch.Tensor:
        if self.fill:
            self._factor(self.fill, self.fill > self.ell)
        self.S = self.B[: self.ell].clone()
        return self.S


class ReplayScore:
    """z = S g, zhat, sum of zhat, u, alpha in fp64; rows are fed in chunks, zhat (N x ell) is kept."""

    def __init__(self, S: torch.Tensor, N: int):
        self.S = S
        self.zhat = torch.zeros((N, S.shape[0]), dtype=torch.float64, device=S.device)
        self.next = 0

    def chunk(self, rows: torch.Tensor, sub_rows: int = 64) -> None:
        D = self.S.shape[1]
        for r0 in range(0, rows.shape[0], sub_rows):
            g = rows[r0:r0 + sub_rows, :D].double()
            z = g @ self.S.T
            nrm = z.norm(dim=1, keepdim=True)
            zh = torch.where(nrm > 0, z / nrm.clamp_min(1e-300), torch.zeros_like(z))
            self.zhat[self.next:self.next + zh.shape[0]] = zh
            self.next += zh.shape[0]

    def end(self):
        s = self.zhat.sum(dim=0)
        n = s.norm()
        u = s / n if float(n) > 0 else torch.zeros_like(s)
        return (self.zhat @ u).cpu().numpy(), u.cpu().numpy()


def signed_gram_norm_device(P: torch.Tensor, Q: torch.Tensor) -> float:
    """|| P^T P - Q^T Q ||_2 for fp64 device tensors P (p x D), Q (q x D) without a D x D matrix. With C = [P; Q] and
    J = diag(I_p, -I_q) the non-zero eigenvalues of C^T J C are those of R J R^T (C^T = Y R, thin QR; used while C is
    small) and also those of W^(1/2) J W^(1/2), W = C C^T (used for large C; accurate to about 1e-8 of ||W||)."""
    C = torch.cat([P, Q], dim=0)
    J = torch.cat([torch.ones(P.shape[0]), -torch.ones(Q.shape[0])]).to(C)
    if C.numel() <= 2e8:
        R = torch.linalg.qr(C.T, mode="r").R
        M = (R * J[None, :]) @ R.T
    else:
        W = C @ C.T
        lam, V = torch.linalg.eigh(W)
        Wh = (V * lam.clamp_min(0).sqrt()) @ V.T
        M = Wh @ (J[:, None] * Wh)
    del C
    ev = torch.linalg.eigvalsh(0.5 * (M + M.T))
    return float(ev.abs().max())


def selection_agrees(idx_test: np.ndarray, alpha_ref: np.ndarray, k: int, tol: float):
    """Index sets may differ only among examples whose reference score lies within tol of the reference's k-th score."""
    order = np.lexsort((np.arange(alpha_ref.size), -alpha_ref))
    ref = order[:k]
    if k == 0 or k == alpha_ref.size:
        return set(idx_test.tolist()) == set(ref.tolist()), 0
    thr = alpha_ref[order[k - 1]]
    diff = np.setxor1d(np.asarray(idx_test), ref)
    return bool(np.all(np.abs(alpha_ref[diff] - thr) <= tol)) and len(idx_test) == k, int(diff.size)
