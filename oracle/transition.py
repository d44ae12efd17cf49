"""CPU checker for the direct transition W -> (U, S, V) (test infrastructure only).

Plain numpy in float64, in the paper's order and notation (Section "Direct Transition Algorithm
to TSVD form"): the ternarisation T(x, theta) of Algorithm 1, the existence bound gamma_N of
Theorem 1, the least-squares scales S* of Eq. 4 and the greedy loop of Algorithm 2.  The SVD and
the pseudo-inverse are numpy's library routines, used as the steps the paper names.

Nothing in the GPU library imports this module, and this module imports nothing of it.

Readings of the paper taken here:
  * Algorithm 1 is stated for a unit vector; here the cumulative sums are divided by ||x||_2, which
    is the same thing for a unit vector and makes the angle test scale-free for any other.
  * Ties: Algorithm 1 keeps every entry whose magnitude is at least the magnitude of the entry that
    reaches the threshold, so equal magnitudes at the cut are all kept (the result may then hold
    more nonzeros than the index found).  An entry equal to zero that is kept gets +1 (x >= 0).
  * Theorem 2 is printed with the assumption theta > pi/4; its bound sin^2(2 theta) sigma_0^2 only
    says something for 2 theta < pi/2, and the paper's own theta = 0.576 is below pi/4, so the
    assumption is read as theta < pi/4.
  * Exit condition of Algorithm 2: the paper leaves it open; here a rank limit and/or a relative
    Frobenius residual.

Pins: tests/test_transition_pins.py (brute force over all ternary vectors, hand-worked 4-vectors,
Theorem 1's bound and the N <= 55 remark, a generic least-squares solve for Eq. 4, the first
inequality of Theorem 2, the nonzero rate of about 0.29 at theta = 0.576 on a [512, 256] Laplace
matrix).
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import List, Optional

import numpy as np


class NoTernarisation(ValueError):
    """No ternary vector lies within the angle theta of x (Algorithm 1's error exit)."""


def ternarize(x: np.ndarray, theta: float) -> np.ndarray:
    """Algorithm 1: the sparsest ternary vector whose angle to x is at most theta.

    x: one vector (any real dtype; evaluated in float64).  Returns int8 of the same length.
    """
    x = np.asarray(x, dtype=np.float64).ravel()
    if x.size == 0:
        raise NoTernarisation("empty vector")
    norm = float(np.sqrt(np.sum(x * x)))
    if norm == 0.0:
        raise NoTernarisation("zero vector")
    o_x = np.sort(np.abs(x))[::-1]                       # magnitudes, descending
    s_x = np.cumsum(o_x)                                 # sum of the k largest
    n_x = np.sqrt(np.arange(1, x.size + 1, dtype=np.float64))
    c_x = s_x / n_x / norm                               # cosine between x and its top-k sign vector
    reach = c_x >= math.cos(theta)
    i_x = int(np.argmax(reach))
    if not reach[i_x]:
        raise NoTernarisation("no ternary vector within theta")
    t_x = np.where(x >= 0, 1, -1)
    t_x = np.where(np.abs(x) < o_x[i_x], 0, t_x)
    return t_x.astype(np.int8)


def gamma(N: int) -> float:
    """Theorem 1: every unit vector of dimension N has a ternary vector within arccos(gamma_N)."""
    k = np.arange(1, N + 1, dtype=np.float64)
    return float(1.0 / np.sqrt(np.sum((np.sqrt(k) - np.sqrt(k - 1.0)) ** 2)))


def lsq_scales(U: np.ndarray, V: np.ndarray, W: np.ndarray) -> np.ndarray:
    """Eq. 4: S* = [(U^T U) o (V V^T)]^+ diag(U^T W V^T), the minimiser of ||W - U diag(S) V||_F."""
    U = np.asarray(U, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    gram = (U.T @ U) * (V @ V.T)
    rhs = np.einsum("mk,mn,kn->k", U, W, V)              # diag(U^T W V^T)
    return np.linalg.pinv(gram) @ rhs


@dataclass
class Transition:
    U: np.ndarray             # int8 [M, K]
    S: np.ndarray             # float64 [K]
    V: np.ndarray             # int8 [K, N]
    residual_fro: List[float]  # ||W - U diag(S) V||_F after every iteration (index 0: ||W||_F)
    sigma: List[np.ndarray]    # singular values of the residual each iteration started from

    @property
    def nonzero_rate(self) -> float:
        """r of Table S1: nonzeros of U and V over K (M + N)."""
        M, K = self.U.shape
        N = self.V.shape[1]
        return float((np.count_nonzero(self.U) + np.count_nonzero(self.V)) / (K * (M + N))) if K else 0.0


def direct_transition(W: np.ndarray, theta: float = 0.576, q: int = 1, max_rank: Optional[int] = None,
                      rel_fro_tol: Optional[float] = None) -> Transition:
    """Algorithm 2: greedy transition of W [M, N] to the TSVD form U diag(S) V.

    Every iteration takes the top-q singular pairs of the residual, ternarises them (Algorithm 1),
    appends them to U and V, refits all of S by Eq. 4 and recomputes the residual.  Stops when the
    rank reaches max_rank or the residual falls to rel_fro_tol * ||W||_F.
    """
    W = np.asarray(W, dtype=np.float64)
    M, N = W.shape
    if max_rank is None and rel_fro_tol is None:
        raise ValueError("give an exit condition")
    U = np.zeros((M, 0), dtype=np.int8)
    V = np.zeros((0, N), dtype=np.int8)
    S = np.zeros(0)
    R = W.copy()
    w_fro = float(np.linalg.norm(W))
    res = [w_fro]
    sig = []
    while True:
        if max_rank is not None and U.shape[1] >= max_rank:
            break
        if rel_fro_tol is not None and res[-1] <= rel_fro_tol * w_fro:
            break
        u, s, v = np.linalg.svd(R, full_matrices=False)
        sig.append(s)
        take = q if max_rank is None else min(q, max_rank - U.shape[1])
        T_u = np.stack([ternarize(u[:, j], theta) for j in range(take)], axis=1)
        T_v = np.stack([ternarize(v[j, :], theta) for j in range(take)], axis=0)
        U = np.concatenate([U, T_u], axis=1)
        V = np.concatenate([V, T_v], axis=0)
        S = lsq_scales(U, V, W)
        R = W - (U.astype(np.float64) * S[None, :]) @ V.astype(np.float64)
        res.append(float(np.linalg.norm(R)))
    return Transition(U=U, S=S, V=V, residual_fro=res, sigma=sig)
