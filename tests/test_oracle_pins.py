"""Pins for the CPU checker: what the paper and the mathematics fix, independent of it.

Each test names the passage it rests on.  None of them re-types the checker's
loop: they use a dense reconstruction through numpy's matmul, exact Python
integers/fractions, hand-worked numbers stored under tests/golden/, the
Winograd closed forms, and algebraic invariants.
"""
import itertools
import json
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from gen import rng

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_case(seed, M, K, N, B, density=0.4):
    U = rng.ternary(seed, 1, M * K, density).reshape(M, K)
    V = rng.ternary(seed, 2, K * N, density).reshape(K, N)
    S = rng.uniform(seed, 3, K, -2.0, 2.0).astype(np.float32)
    x = rng.normal(seed, 4, B * N).reshape(B, N)
    return U, S, V, x


def _dense(U, S, V, x):
    """W' = U diag(S) V built densely, then W' x (definition, Eq. 1-2)."""
    W = U.astype(np.float64) @ np.diag(S.astype(np.float64)) @ V.astype(np.float64)
    return x @ W.T


# P1 -- brute-force dense reconstruction on tiny shapes (Eq. 2 and the display after it)
@pytest.mark.parametrize("seed", range(40))
def test_dense_reconstruction_random_tiny(seed):
    g = np.random.default_rng(seed)
    M, K, N = (int(g.integers(1, 9)) for _ in range(3))
    B = int(g.integers(1, 4))
    U, S, V, x = _rand_case(1000 + seed, M, K, N, B)
    res = oracle.forward(U, S, V, x)
    ref = _dense(U, S, V, x)
    scale = max(1.0, np.abs(ref).max())
    assert res.y.shape == (B, M)
    assert np.abs(res.y - ref).max() <= 1e-12 * scale
    assert np.abs(res.zraw - x @ V.T.astype(np.float64)).max() <= 1e-12 * max(1.0, np.abs(x).max() * N)


def test_dense_reconstruction_exhaustive_2x2():
    """All 3^4 x 3^4 ternary pairs (U,V) of shape 2x2 with fixed S, x."""
    S = np.array([1.5, -0.25], dtype=np.float32)
    x = np.array([[0.75, -2.0], [3.0, 0.125]], dtype=np.float64)
    vals = (-1, 0, 1)
    mats = [np.array(t, dtype=np.int8).reshape(2, 2) for t in itertools.product(vals, repeat=4)]
    for U in mats:
        Ud = U.astype(np.float64) * S.astype(np.float64)[None, :]
        for V in mats:
            got = oracle.forward(U, S, V, x).y
            ref = x @ (Ud @ V.astype(np.float64)).T
            assert np.array_equal(got, ref), (U, V)   # everything here is dyadic: exact


# P2 -- exact arithmetic: integer x and dyadic S must agree with rational evaluation exactly
@pytest.mark.parametrize("seed", range(5))
def test_exact_rational(seed):
    g = np.random.default_rng(seed)
    M, K, N, B = 5, 7, 6, 2
    U = g.integers(-1, 2, size=(M, K)).astype(np.int8)
    V = g.integers(-1, 2, size=(K, N)).astype(np.int8)
    S_frac = [Fraction(int(g.integers(-64, 65)), 32) for _ in range(K)]
    S = np.array([float(f) for f in S_frac], dtype=np.float32)
    xi = g.integers(-1000, 1001, size=(B, N))
    res = oracle.forward(U, S, V, xi.astype(np.float64))
    for b in range(B):
        z = [sum(int(V[k, n]) * int(xi[b, n]) for n in range(N)) for k in range(K)]
        for k in range(K):
            assert res.zraw[b, k] == z[k]
        for m in range(M):
            yv = sum(int(U[m, k]) * S_frac[k] * z[k] for k in range(K))
            assert Fraction(res.y[b, m]) == yv
    # the int8 entry point must agree with the float one on int8-range inputs
    x8 = g.integers(-127, 128, size=(B, N)).astype(np.int8)
    r8 = oracle.forward(U, S, V, x8)
    rf = oracle.forward(U, S, V, x8.astype(np.float64))
    assert r8.zraw.dtype == np.int64
    assert np.array_equal(r8.zraw.astype(np.float64), rf.zraw)
    assert np.array_equal(r8.y, rf.y)


# P3 -- hand-worked cases (tests/golden/handworked_forward.json)
def test_handworked_golden():
    with open(os.path.join(GOLDEN, "handworked_forward.json")) as f:
        data = json.load(f)
    assert len(data["cases"]) >= 4
    for c in data["cases"]:
        U = np.array(c["U"], dtype=np.int8)
        V = np.array(c["V"], dtype=np.int8)
        S = np.array(c["S"], dtype=np.float32)
        x = np.array(c["x"], dtype=np.float64)
        bias = np.array(c["bias"], dtype=np.float32) if "bias" in c else None
        res = oracle.forward(U, S, V, x, bias)
        assert np.array_equal(res.zraw, np.array(c["zraw"])), c["name"]
        assert np.array_equal(res.y, np.array(c["y"])), c["name"]


# bias (the supplement's architecture listing keeps bias=True on every converted layer): one
# addition per output after the U-stage, pinned by the dense form W' x + b, exact rationals, the
# hand-worked case above, the int8 entry point and the operation count
@pytest.mark.parametrize("seed", range(6))
def test_bias_dense_and_exact(seed):
    g = np.random.default_rng(50 + seed)
    M, K, N, B = (int(g.integers(1, 9)) for _ in range(4))
    U, S, V, x = _rand_case(2000 + seed, M, K, N, B)
    bias = g.integers(-40, 41, size=M).astype(np.float32) / 8.0
    res = oracle.forward(U, S, V, x, bias)
    ref = _dense(U, S, V, x) + bias.astype(np.float64)[None, :]
    assert np.abs(res.y - ref).max() <= 1e-12 * max(1.0, np.abs(ref).max())
    # the bias enters after everything else: exactly the no-bias result plus b, and nowhere else
    plain = oracle.forward(U, S, V, x)
    assert np.array_equal(res.y, plain.y + bias.astype(np.float64)[None, :])
    assert np.array_equal(res.zraw, plain.zraw)
    assert res.adds == plain.adds + B * M and res.muls == plain.muls
    # integer activations, dyadic S and bias: exact rational evaluation
    xi = g.integers(-100, 101, size=(B, N)).astype(np.int8)
    Sf = [Fraction(int(g.integers(-64, 65)), 32) for _ in range(K)]
    S2 = np.array([float(f) for f in Sf], dtype=np.float32)
    r8 = oracle.forward(U, S2, V, xi, bias)
    for b in range(B):
        for m in range(M):
            yv = sum(int(U[m, k]) * Sf[k] * sum(int(V[k, n]) * int(xi[b, n]) for n in range(N))
                     for k in range(K)) + Fraction(float(bias[m]))
            assert Fraction(r8.y[b, m]) == yv
    with pytest.raises(ValueError):
        oracle.forward(U, S, V, x, np.zeros(M + 1, np.float32))


# P4 -- Winograd minimal filtering is a lossless TSVD (Section "Connection with Winograd",
# and the unfolded F(2,3) matrix of Section "TSVD in Convolution Layer")
_BT = np.array([[1, 0, -1, 0], [0, 1, 1, 0], [0, -1, 1, 0], [0, 1, 0, -1]], dtype=np.int8)
_G = np.array([[1, 0, 0], [0.5, 0.5, 0.5], [0.5, -0.5, 0.5], [0, 0, 1]], dtype=np.float64)
_AT = np.array([[1, 1, 1, 0], [0, 1, -1, -1]], dtype=np.int8)


@pytest.mark.parametrize("seed", range(6))
def test_winograd_f23(seed):
    g = np.random.default_rng(seed)
    w = g.integers(-16, 17, size=3) / 8.0           # dyadic taps: G w exact in float32
    d = g.integers(-50, 51, size=(3, 4)) / 4.0      # three tiles
    S = (_G @ w).astype(np.float32)
    assert np.array_equal(S.astype(np.float64), _G @ w)
    res = oracle.forward(_AT, S, _BT, d)
    direct = np.stack([d[:, 0] * w[0] + d[:, 1] * w[1] + d[:, 2] * w[2],
                       d[:, 1] * w[0] + d[:, 2] * w[1] + d[:, 3] * w[2]], axis=1)
    assert np.array_equal(res.y, direct)
    # the same numbers through the paper's unfolded 2x4 matrix
    Wc = np.array([[w[0], w[1], w[2], 0.0], [0.0, w[0], w[1], w[2]]])
    assert np.array_equal(res.y, d @ Wc.T)


@pytest.mark.parametrize("seed", range(4))
def test_winograd_f2x2_3x3(seed):
    g = np.random.default_rng(100 + seed)
    ker = g.integers(-8, 9, size=(3, 3)) / 4.0
    tile = g.integers(-20, 21, size=(2, 4, 4)) / 2.0
    U = np.kron(_AT, _AT).astype(np.int8)            # [4,16]
    V = np.kron(_BT, _BT).astype(np.int8)            # [16,16]
    assert set(np.unique(U)) <= {-1, 0, 1} and set(np.unique(V)) <= {-1, 0, 1}
    Sd = (_G @ ker @ _G.T).reshape(16)
    S = Sd.astype(np.float32)
    assert np.array_equal(S.astype(np.float64), Sd)
    res = oracle.forward(U, S, V, tile.reshape(2, 16))
    for t in range(2):
        direct = np.zeros((2, 2))
        for i in range(2):
            for j in range(2):
                direct[i, j] = sum(ker[p, q] * tile[t, i + p, j + q]
                                   for p in range(3) for q in range(3))
        assert np.array_equal(res.y[t].reshape(2, 2), direct)


# P5 -- invariants of the definition
def test_linearity_sign_permutation_scaling():
    U, S, V, x1 = _rand_case(7, 9, 13, 11, 3)
    x2 = rng.normal(8, 4, 3 * 11).reshape(3, 11)
    f = lambda U_, S_, V_, x_: oracle.forward(U_, S_, V_, x_).y
    y1, y2 = f(U, S, V, x1), f(U, S, V, x2)
    a, b = 0.75, -2.5
    scale = np.abs(y1).max() + np.abs(y2).max()
    assert np.abs(f(U, S, V, a * x1 + b * x2) - (a * y1 + b * y2)).max() <= 1e-13 * scale
    assert np.array_equal(f(U, S, -V, x1), -y1)
    assert np.array_equal(f(-U, S, V, x1), -y1)
    assert np.array_equal(f(-U, S, -V, x1), y1)
    assert np.array_equal(f(U, -S, V, x1), -y1)
    assert np.array_equal(f(U, 4.0 * S, V, x1), 4.0 * y1)          # power of two: exact
    perm = np.random.default_rng(3).permutation(13)
    yp = f(U[:, perm], S[perm], V[perm, :], x1)
    assert np.abs(yp - y1).max() <= 1e-13 * scale
    # a zero row of V removes S[k] from the map; a zero row of U zeroes that output
    V0 = V.copy(); V0[5, :] = 0
    S_big = S.copy(); S_big[5] = 1e6
    assert np.array_equal(f(U, S, V0, x1), f(U, S_big, V0, x1))
    U0 = U.copy(); U0[2, :] = 0
    assert np.all(f(U0, S, V, x1)[:, 2] == 0.0)


# P6 -- operation counts of Table S1: nnz(V) + nnz(U) additions and K multiplications per column
def test_operation_counts():
    M, K, N, B = 17, 23, 19, 4
    U, S, V, x = _rand_case(11, M, K, N, B, density=0.3)
    res = oracle.forward(U, S, V, x)
    assert res.adds == B * (np.count_nonzero(U) + np.count_nonzero(V))
    assert res.muls == B * K
    from oracle import cost
    r = (np.count_nonzero(U) + np.count_nonzero(V)) / (K * (M + N))
    muls, adds = cost.tsvd_counts(M, N, K, r)
    assert muls * B == res.muls and abs(adds * B - res.adds) < 1e-6


# P7 -- plus/minus split (Section "Connection with BNN"): U = U+ - U-, V = V+ - V-
def test_plus_minus_split():
    U, S, V, x = _rand_case(21, 6, 10, 8, 2)
    Up, Um = (U == 1).astype(np.int8), (U == -1).astype(np.int8)
    Vp, Vm = (V == 1).astype(np.int8), (V == -1).astype(np.int8)
    assert not np.any(Up & Um) and not np.any(Vp & Vm)
    f = lambda U_, V_: oracle.forward(U_, S, V_, x)
    full = f(U, V)
    parts = [f(Up, Vp), f(Up, Vm), f(Um, Vp), f(Um, Vm)]
    y = parts[0].y - parts[1].y - parts[2].y + parts[3].y
    assert np.abs(y - full.y).max() <= 1e-13 * max(1.0, np.abs(full.y).max())
    assert sum(p.adds for p in parts) == 2 * full.adds       # same FLOPS per split product


# P8 -- special case that is a library routine: S = 1 and U a 0/1 selection gives V x
def test_reduces_to_matvec():
    K, N, B = 64, 96, 5
    V = rng.ternary(31, 2, K * N, 0.3).reshape(K, N)
    U = np.eye(K, dtype=np.int8)
    S = np.ones(K, dtype=np.float32)
    x8 = rng.int8_uniform(31, 4, B * N).reshape(B, N)
    res = oracle.forward(U, S, V, x8)
    ref = x8.astype(np.int64) @ V.T.astype(np.int64)
    assert np.array_equal(res.zraw, ref)
    assert np.array_equal(res.y, ref.astype(np.float64))


def test_rejects_non_ternary():
    U = np.array([[2]], dtype=np.int8)
    with pytest.raises(ValueError):
        oracle.forward(U, np.ones(1, np.float32), np.ones((1, 1), np.int8), np.ones((1, 1)))


# cost model against the paper's printed acceleration rates (Tables 1-3)
def test_cost_model_golden():
    from oracle import cost
    with open(os.path.join(GOLDEN, "acceleration_rates.json")) as f:
        data = json.load(f)
    for r in data["rows"]:
        acc = cost.acceleration_from_counts(r["mul_orig"], r["add_orig"], r["mul_tsvd"],
                                            r["add_tsvd"], r["d"])
        assert abs(acc - r["acc"]) <= r["tol"], r["name"]
    # Table S2 formula equals the ratio of Table S1 counts; Eq. 3 is where it equals 1
    M, N, r_, d = 512, 256, 0.29, 32
    Kc = cost.critical_rank(M, N, r_, d)
    assert abs(cost.acceleration_rate(M, N, Kc, r_, d) - 1.0) < 1e-12
    muls, adds = cost.tsvd_counts(M, N, 100, r_)
    assert abs(cost.acceleration_rate(M, N, 100, r_, d)
               - cost.equivalent_adds(M * N, M * N, d) / cost.equivalent_adds(muls, adds, d)) < 1e-9
