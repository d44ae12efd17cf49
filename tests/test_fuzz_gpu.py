"""Seeded random cases through the default dispatch (whatever path the library picks for the shape and
batch), against the CPU checker element by element: ragged shapes from 1 to a few thousand, every
activation type, one to 300 tokens, random nonzero rates, signed S with zeros, bias on and off."""
import numpy as np
import pytest

import gen
from tests import _util

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2308_07641_b200 import build
    build.build()


def _case(i):
    g = np.random.default_rng(7000 + i)
    big = i % 4 == 0                                            # every fourth case: contractions of 1024+ columns
    M = int(g.integers(1, 700))
    N = int(g.integers(1024, 2600)) if big else int(g.integers(1, 900))
    K = int(g.integers(1024, 2200)) if (big and i % 8 == 0) else int(g.integers(1, 900))
    B = int(g.choice([1, 2, 3, 4, 5, 7, 8, 9, 13, 16, 17, 33, 64, 65, 130, 300]))
    x_dtype = ("bf16", "f32", "i8")[i % 3]
    base = {"bf16": "cfg2", "f32": "cfg1", "i8": "cfg5_d20"}[x_dtype]
    density = float(g.choice([0.02, 0.1, 0.28, 0.5, 0.9]))
    spec = gen.scaled(gen.CONFIGS[base], name=f"fuzz{i}_{x_dtype}_{M}x{N}x{K}_B{B}", M=M, N=N, K=K, B=B,
                      density=density, seed=7000 + i, row_density_spread=0.5 if i % 5 == 0 else 0.0)
    U, V, S = gen.make_weights(spec)
    S = (S * g.choice([-1.0, 1.0], K)).astype(np.float32)
    S[g.random(K) < 0.1] = 0.0
    # a bias comparable to |y|: a few times sqrt(r K) * sqrt(r N) * scale of x
    scale = {"bf16": 1.0, "f32": 1.0, "i8": 74.0}[x_dtype] * max(1.0, density * np.sqrt(float(K) * float(N)))
    bias = (scale * g.standard_normal(M)).astype(np.float32) if i % 2 else None
    return spec, (U, V, S), bias


@pytest.mark.parametrize("i", range(72))
def test_random_case_default_path(i):
    spec, weights, bias = _case(i)
    _util.run_and_check(spec, weights=weights, bias=bias, expect_status=(0, 10))


def _stream_case(i):
    """Aligned rows of 1024 to 4096 values and batches around and beyond 4 x 148 token slots: the regime
    of the digit conversion that keeps its blocks resident and walks them over the tokens."""
    g = np.random.default_rng(9100 + i)
    M = int(g.integers(1, 400))
    N = 16 * int(g.integers(64, 257))
    K = 16 * int(g.integers(64, 257)) if i % 2 == 0 else int(g.integers(1030, 4096))
    B = (591, 592, 593, 640, 1183, 1185, 1300, 1777, 2049)[i % 9]
    x_dtype = ("bf16", "f32", "i8")[i % 3]
    base = {"bf16": "cfg2", "f32": "cfg1", "i8": "cfg5_d20"}[x_dtype]
    spec = gen.scaled(gen.CONFIGS[base], name=f"stream{i}_{x_dtype}_{M}x{N}x{K}_B{B}", M=M, N=N, K=K, B=B,
                      density=float(g.choice([0.05, 0.28, 0.6])), seed=9100 + i)
    U, V, S = gen.make_weights(spec)
    S = (S * g.choice([-1.0, 1.0], K)).astype(np.float32)
    return spec, (U, V, S), (0x200 if x_dtype == "bf16" and i % 2 == 0 else 0)


@pytest.mark.parametrize("i", range(12))
def test_random_case_resident_digit_conversion(i):
    spec, weights, flags = _stream_case(i)
    _util.run_and_check(spec, weights=weights, flags=flags, expect_status=(0, 10))


def _cluster_case(i):
    """Five to 32 tokens on contractions of up to 4096 columns: the cluster kernels of the tensor-core path
    (slabs of zero to eight blocks per CTA, ragged rows and columns, every activation type, bias)."""
    g = np.random.default_rng(9500 + i)
    M = int(g.integers(1, 900))
    N = int(g.choice([1, 100, 128, 129, 500, 512, 513, 1024, 2000, 3000, 4096]))
    K = int(g.choice([1, 127, 128, 300, 640, 1030, 2500, 4096]))
    B = int(g.choice([5, 8, 9, 15, 16, 17, 24, 31, 32]))
    x_dtype = ("bf16", "f32", "i8")[i % 3]
    base = {"bf16": "cfg2", "f32": "cfg1", "i8": "cfg5_d20"}[x_dtype]
    density = float(g.choice([0.05, 0.28, 0.7]))
    spec = gen.scaled(gen.CONFIGS[base], name=f"cluster{i}_{x_dtype}_{M}x{N}x{K}_B{B}", M=M, N=N, K=K, B=B,
                      density=density, seed=9500 + i)
    U, V, S = gen.make_weights(spec)
    S = (S * g.choice([-1.0, 1.0], K)).astype(np.float32)
    scale = {"bf16": 1.0, "f32": 1.0, "i8": 74.0}[x_dtype] * max(1.0, density * np.sqrt(float(K) * float(N)))
    bias = (scale * g.standard_normal(M)).astype(np.float32) if i % 2 else None
    flags = 0x40 | (0x200 if x_dtype == "bf16" and i % 4 == 0 else 0)
    return spec, (U, V, S), bias, flags


@pytest.mark.parametrize("i", range(30))
def test_random_case_cluster_kernels(i):
    spec, weights, bias, flags = _cluster_case(i)
    _util.run_and_check(spec, weights=weights, bias=bias, flags=flags, expect_status=(0, 10))
