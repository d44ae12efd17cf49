"""Direct transition of a weight matrix to the TSVD form, W ~ U diag(S) V (Algorithm 2 of the
paper, Section "Direct Transition Algorithm to TSVD form"), on the current CUDA device.

This is the one-time conversion that produces the operands of the forward; it is not the hot path.
Per iteration: the top-q singular pairs of the residual (torch.linalg.svd, a library routine),
their ternarisation by Algorithm 1 (the library's own kernel, `tsvd_ternarize`), all scales refitted
by Eq. 4, S* = [(U^T U) o (V V^T)]^+ diag(U^T W V^T) (plain library GEMMs and a pseudo-inverse, in
float64 because the Gram entries are integer counts up to M*N), and the new residual (one GEMM).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

from . import binding

THETA_DEFAULT = 0.576   # Section "Optimal theta in Practice": about 33 degrees, nonzero rate about 0.29


def ternarize(x, theta: float = THETA_DEFAULT):
    """Algorithm 1 on the rows of a CUDA float32 tensor [n_vec, len]; returns (int8 [n_vec, len],
    int32 [n_vec] nonzero counts, -1 where no ternary vector lies within theta)."""
    import torch
    if not x.is_cuda or x.dtype != torch.float32 or x.dim() != 2 or x.stride(1) != 1:
        raise binding.TSVDError(binding.TSVD_E_SHAPE, "ternarize")
    n_vec, length = x.shape
    t = torch.empty((n_vec, length), dtype=torch.int8, device=x.device)
    nnz = torch.empty(n_vec, dtype=torch.int32, device=x.device)
    stream = torch.cuda.current_stream(x.device).cuda_stream
    binding.tsvd_ternarize(x.data_ptr(), n_vec, length, x.stride(0), theta, t.data_ptr(), t.stride(0),
                           nnz.data_ptr(), stream)
    return t, nnz


def lsq_scales(U, V, W):
    """Eq. 4 for int8 U [M,K], V [K,N] and W [M,N] on the device; returns float64 S [K]."""
    import torch
    Ud, Vd, Wd = U.double(), V.double(), W.double()
    gram = (Ud.T @ Ud) * (Vd @ Vd.T)
    rhs = ((Ud.T @ Wd) * Vd).sum(dim=1)
    return torch.linalg.pinv(gram, hermitian=True) @ rhs


@dataclass
class Transition:
    U: "object"               # torch int8 [M, K]
    S: "object"               # torch float32 [K]
    V: "object"               # torch int8 [K, N]
    residual_fro: List[float]

    @property
    def nonzero_rate(self) -> float:
        M, K = self.U.shape
        N = self.V.shape[1]
        nz = int((self.U != 0).sum().item()) + int((self.V != 0).sum().item())
        return nz / (K * (M + N)) if K else 0.0


def direct_transition(W, theta: float = THETA_DEFAULT, q: int = 1, max_rank: Optional[int] = None,
                      rel_fro_tol: Optional[float] = None) -> Transition:
    """Algorithm 2.  W: CUDA float32 [M, N].  Stops at max_rank components or when the residual
    falls to rel_fro_tol * ||W||_F.  Raises if a singular vector has no ternary vector within theta."""
    import torch
    if not W.is_cuda or W.dtype != torch.float32 or W.dim() != 2:
        raise binding.TSVDError(binding.TSVD_E_SHAPE, "direct_transition")
    if max_rank is None and rel_fro_tol is None:
        raise ValueError("give an exit condition")
    M, N = W.shape
    U = torch.zeros((M, 0), dtype=torch.int8, device=W.device)
    V = torch.zeros((0, N), dtype=torch.int8, device=W.device)
    S = torch.zeros(0, dtype=torch.float64, device=W.device)
    Wd = W.double()
    R = W.clone()
    w_fro = float(torch.linalg.norm(Wd))
    res = [w_fro]
    while True:
        if max_rank is not None and U.shape[1] >= max_rank:
            break
        if rel_fro_tol is not None and res[-1] <= rel_fro_tol * w_fro:
            break
        u, _, v = torch.linalg.svd(R, full_matrices=False)
        take = q if max_rank is None else min(q, max_rank - U.shape[1])
        T_u, nu = ternarize(u[:, :take].T.contiguous(), theta)      # [take, M]
        T_v, nv = ternarize(v[:take, :].contiguous(), theta)        # [take, N]
        if int(nu.min().item()) < 0 or int(nv.min().item()) < 0:
            raise ValueError("no ternary vector within theta of a singular vector (Theorem 1 bounds when this can happen)")
        U = torch.cat([U, T_u.T.contiguous()], dim=1)
        V = torch.cat([V, T_v], dim=0)
        S = lsq_scales(U, V, W)
        Rd = Wd - (U.double() * S[None, :]) @ V.double()
        res.append(float(torch.linalg.norm(Rd)))
        R = Rd.float()
    return Transition(U=U, S=S.float(), V=V, residual_fro=res)
