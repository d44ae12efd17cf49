"""The five synthetic TSVD workloads and a builder for arbitrary (ragged) cases.

Shapes, densities and value distributions stand in for the layers the paper
converts (BERT-base FFN at sequence length 128, OPT-6.7B projections at
sequence length 2048); only shapes, ternary density and value scale are taken
from there.  U and V are i.i.d. Bernoulli(density) x Rademacher, which is the
nonzero-rate model the paper's cost table uses (Table S1: r*K*(M+N) additions).
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, Tuple

import numpy as np

from . import rng

# tensor ids inside one seed
_TID_U, _TID_V, _TID_S, _TID_X = 1, 2, 3, 4


@dataclass(frozen=True)
class CaseSpec:
    name: str
    M: int
    N: int
    K: int
    B: int
    density: float
    x_dtype: str            # "f32" | "bf16" | "i8"
    s_dist: str             # "uniform" (0.01,1) | "lognormal" (mu 0, sigma 0.5)
    s_sorted: bool
    seed: int
    density_u: float = -1.0  # < 0: same as density
    row_density_spread: float = 0.0  # > 0: per-row density varies by this relative amount


@dataclass
class Case:
    spec: CaseSpec
    U: np.ndarray            # int8 [M,K]
    V: np.ndarray            # int8 [K,N]
    S: np.ndarray            # float32 [K]
    x: np.ndarray            # [B,N] token-major: float32, uint16 (bf16 bits) or int8
    meta: Dict[str, float] = field(default_factory=dict)

    def x_as_f64(self) -> np.ndarray:
        """Exact widening of the stored activations to float64."""
        if self.spec.x_dtype == "bf16":
            return rng.bf16_bits_to_f32(self.x).astype(np.float64)
        return self.x.astype(np.float64)


CONFIGS: Dict[str, CaseSpec] = {
    "cfg1": CaseSpec("cfg1", M=256, N=256, K=256, B=8, density=0.3, x_dtype="f32",
                     s_dist="uniform", s_sorted=True, seed=0),
    "cfg2": CaseSpec("cfg2", M=3072, N=768, K=768, B=4096, density=0.25, x_dtype="bf16",
                     s_dist="lognormal", s_sorted=False, seed=2),
    "cfg3_b1": CaseSpec("cfg3_b1", M=4096, N=4096, K=4096, B=1, density=0.2, x_dtype="bf16",
                        s_dist="lognormal", s_sorted=True, seed=3),
    "cfg3_b4": CaseSpec("cfg3_b4", M=4096, N=4096, K=4096, B=4, density=0.2, x_dtype="bf16",
                        s_dist="lognormal", s_sorted=True, seed=3),
    "cfg3_b16": CaseSpec("cfg3_b16", M=4096, N=4096, K=4096, B=16, density=0.2, x_dtype="bf16",
                         s_dist="lognormal", s_sorted=True, seed=3),
    "cfg4": CaseSpec("cfg4", M=16384, N=4096, K=4096, B=2048, density=0.1, x_dtype="bf16",
                     s_dist="lognormal", s_sorted=False, seed=4),
    "cfg5_d05": CaseSpec("cfg5_d05", M=4096, N=4096, K=8192, B=256, density=0.05, x_dtype="i8",
                         s_dist="uniform", s_sorted=False, seed=50),
    "cfg5_d20": CaseSpec("cfg5_d20", M=4096, N=4096, K=8192, B=256, density=0.2, x_dtype="i8",
                         s_dist="uniform", s_sorted=False, seed=51),
    "cfg5_d50": CaseSpec("cfg5_d50", M=4096, N=4096, K=8192, B=256, density=0.5, x_dtype="i8",
                         s_dist="uniform", s_sorted=False, seed=52),
}


def scaled(spec: CaseSpec, **kw) -> CaseSpec:
    """A copy of `spec` with some fields replaced (smaller or ragged variants for tests)."""
    return replace(spec, **kw)


def _ternary_matrix(seed: int, tid: int, rows: int, cols: int, density: float,
                    spread: float) -> np.ndarray:
    if spread <= 0.0:
        return rng.ternary(seed, tid, rows * cols, density).reshape(rows, cols)
    # per-row density: density * (1 + spread*(2u-1)), clipped to [0,1]; rows stay i.i.d. inside
    u = rng.uniform01(seed, tid + 100, 0, 0, rows)
    dens = np.clip(density * (1.0 + spread * (2.0 * u - 1.0)), 0.0, 1.0)
    out = np.empty((rows, cols), dtype=np.int8)
    for r in range(rows):
        nz = rng.uniform01(seed, tid, 0, r * cols, cols) < dens[r]
        neg = (rng.raw_u64(seed, tid, 1, r * cols, cols) >> np.uint64(63)).astype(bool)
        out[r] = np.where(nz, np.where(neg, -1, 1), 0).astype(np.int8)
    return out


def make_weights(spec: CaseSpec) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    du = spec.density if spec.density_u < 0 else spec.density_u
    U = _ternary_matrix(spec.seed, _TID_U, spec.M, spec.K, du, spec.row_density_spread)
    V = _ternary_matrix(spec.seed, _TID_V, spec.K, spec.N, spec.density, spec.row_density_spread)
    if spec.s_dist == "uniform":
        S = rng.uniform(spec.seed, _TID_S, spec.K, 0.01, 1.0)
    elif spec.s_dist == "lognormal":
        S = np.exp(0.5 * rng.normal(spec.seed, _TID_S, spec.K))
    else:
        raise ValueError(spec.s_dist)
    if spec.s_sorted:
        S = np.sort(S)[::-1]
    return U, V, np.ascontiguousarray(S, dtype=np.float32)


def make_x(spec: CaseSpec, b_start: int = 0, b_count: int | None = None) -> np.ndarray:
    """Activations for tokens b_start..b_start+b_count, token-major [b_count, N]."""
    if b_count is None:
        b_count = spec.B - b_start
    n = b_count * spec.N
    off = b_start * spec.N
    if spec.x_dtype == "i8":
        span = 255
        v = np.floor(rng.uniform01(spec.seed, _TID_X, 0, off, n) * span).astype(np.int64)
        return (np.minimum(v, span - 1) - 127).astype(np.int8).reshape(b_count, spec.N)
    u1 = rng.uniform01(spec.seed, _TID_X, 0, off, n)
    u2 = rng.uniform01(spec.seed, _TID_X, 1, off, n)
    g = (np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)).astype(np.float32)
    if spec.x_dtype == "f32":
        return g.reshape(b_count, spec.N)
    if spec.x_dtype == "bf16":
        return rng.f32_to_bf16_bits(g).reshape(b_count, spec.N)
    raise ValueError(spec.x_dtype)


def widen_x(x: np.ndarray, x_dtype: str) -> np.ndarray:
    """The stored activations as the array a double-precision consumer takes: bf16 bit patterns
    and fp32 widened exactly to float64, int8 left as it is."""
    if x_dtype == "bf16":
        return rng.bf16_bits_to_f32(x).astype(np.float64)
    if x_dtype == "i8":
        return x
    return x.astype(np.float64)


def set_entries(x: np.ndarray, x_dtype: str, tokens, cols, value: float) -> np.ndarray:
    """A copy of the stored activations x [B,N] with x[tokens, cols] = value (outliers, zeros,
    extreme int8 codes); `value` must be representable in the storage type."""
    out = x.copy()
    tokens = np.atleast_1d(np.asarray(tokens))
    cols = np.atleast_1d(np.asarray(cols))
    if x_dtype == "bf16":
        bits = rng.f32_to_bf16_bits(np.array([value], dtype=np.float32))[0]
        if float(rng.bf16_bits_to_f32(np.array([bits], dtype=np.uint16))[0]) != float(value):
            raise ValueError("value is not a bf16 number")
        out[np.ix_(tokens, cols)] = bits
    else:
        out[np.ix_(tokens, cols)] = np.asarray(value).astype(out.dtype)
    return out


def laplace_matrix(seed: int, M: int, N: int) -> np.ndarray:
    """A float32 [M, N] matrix of i.i.d. Laplace entries: the random matrix the paper profiles its
    decomposition on (shape [512, 256] in its Figures 1a and 2a)."""
    return rng.laplace(seed, 7, M * N).astype(np.float32).reshape(M, N)


def make_case(spec: CaseSpec) -> Case:
    U, V, S = make_weights(spec)
    return Case(spec=spec, U=U, V=V, S=S, x=make_x(spec))
