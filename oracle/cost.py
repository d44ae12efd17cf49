"""The paper's analytic cost model (test infrastructure; reporting check only).

Section "Hardware Cost of Basic Instruction": one d-bit multiplication is
counted as (d-2) additions.  Table S1 gives the per-column operation counts of
the TSVD map; Table S2 the acceleration rate; Eq. 3 the critical rank.
"""
from __future__ import annotations


def tsvd_counts(M: int, N: int, K: int, r: float):
    """(multiplications, additions) per input column of U diag(S) V (.) -- Table S1, last row."""
    return K, r * K * (M + N)


def equivalent_adds(muls: float, adds: float, d: int) -> float:
    """Cost in additions with 1 Mul = (d-2) Add."""
    return muls * (d - 2) + adds


def acceleration_from_counts(mul_orig: float, add_orig: float, mul_tsvd: float,
                             add_tsvd: float, d: int) -> float:
    """Ratio of equivalent-addition costs, as used for the acc(d) columns of Tables 1-3."""
    return equivalent_adds(mul_orig, add_orig, d) / equivalent_adds(mul_tsvd, add_tsvd, d)


def acceleration_rate(M: int, N: int, K: int, r: float, d: int) -> float:
    """Table S2, TSVD row: M N (d-1) / (K (d-2) + r K (M+N))."""
    return M * N * (d - 1) / (K * (d - 2) + r * K * (M + N))


def critical_rank(M: int, N: int, r: float, d: int) -> float:
    """Eq. 3: the rank at which TSVD costs as much as the dense map."""
    return (d - 1) * M * N / (d + r * (M + N) - 2)
