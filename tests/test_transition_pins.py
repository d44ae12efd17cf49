"""Pins for the CPU checker of the direct transition W -> (U, S, V) (oracle/transition.py): what the
paper and the mathematics fix, independent of the checker's own code."""
import itertools
import json
import math
import os

import numpy as np
import pytest

import gen
from oracle import transition as tr

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
THETA = 0.576


def _cos(x, t):
    return float(np.dot(x, t) / (np.linalg.norm(x) * math.sqrt(np.count_nonzero(t))))


# Algorithm 1 against its definition: the sparsest ternary vector within the angle, by brute force
# over all 3^n ternary vectors (Section "Direct Transition Algorithm", the policy stated before Eq. 5
# of that section and the structure of the optimum).
@pytest.mark.parametrize("seed", range(12))
def test_ternarize_is_the_sparsest_vector_within_the_angle(seed):
    g = np.random.default_rng(seed)
    n = int(g.integers(2, 8))
    x = g.standard_normal(n)
    x /= np.linalg.norm(x)
    theta = float(g.uniform(0.3, 0.9))
    best_nnz, best_cos = None, {}
    for cand in itertools.product((-1, 0, 1), repeat=n):
        t = np.array(cand, dtype=np.float64)
        k = int(np.count_nonzero(t))
        if k == 0:
            continue
        c = _cos(x, t)
        best_cos[k] = max(best_cos.get(k, -2.0), c)
        if c >= math.cos(theta) - 1e-15 and (best_nnz is None or k < best_nnz):
            best_nnz = k
    if best_nnz is None:
        with pytest.raises(tr.NoTernarisation):
            tr.ternarize(x, theta)
        return
    t = tr.ternarize(x, theta)
    assert set(np.unique(t)) <= {-1, 0, 1}
    assert np.count_nonzero(t) == best_nnz                      # the sparsest
    assert _cos(x, t) >= math.cos(theta) - 1e-15                # within the angle
    assert abs(_cos(x, t) - best_cos[best_nnz]) <= 1e-12        # and the closest among the equally sparse
    nz = t != 0
    assert np.all(t[nz] == np.sign(x[nz]))                      # signs of x on its largest magnitudes
    assert np.abs(x[nz]).min() >= np.abs(x[~nz]).max() if (~nz).any() else True


def test_ternarize_handworked():
    with open(os.path.join(GOLDEN, "handworked_ternarize.json")) as f:
        data = json.load(f)
    assert len(data["cases"]) >= 4
    for c in data["cases"]:
        x = np.array(c["x"], dtype=np.float64)
        if c["t"] is None:
            with pytest.raises(tr.NoTernarisation):
                tr.ternarize(x, c["theta"])
        else:
            assert tr.ternarize(x, c["theta"]).tolist() == c["t"], c["name"]


def test_ternarize_scale_and_sign_invariance():
    x = gen.rng.normal(5, 1, 300)
    t = tr.ternarize(x, THETA)
    assert np.array_equal(tr.ternarize(8.0 * x, THETA), t)      # the angle does not see the length
    assert np.array_equal(tr.ternarize(-x, THETA), -t)
    p = np.random.default_rng(0).permutation(x.size)
    assert np.array_equal(tr.ternarize(x[p], THETA), t[p])
    # a larger angle never needs more nonzeros
    assert np.count_nonzero(tr.ternarize(x, 0.8)) <= np.count_nonzero(t) <= np.count_nonzero(tr.ternarize(x, 0.5))


# Theorem 1: gamma_N bounds the best cosine from below for every unit vector, it is attained, and the
# remark after it: gamma_N >= cos(pi/4) exactly up to N = 55.
def test_theorem_1_bound():
    assert tr.gamma(1) == 1.0
    assert tr.gamma(55) >= math.cos(math.pi / 4) > tr.gamma(56)
    for N in (2, 5, 17, 64, 300):
        gN = tr.gamma(N)
        g = np.random.default_rng(N)
        for _ in range(20):
            x = g.standard_normal(N)
            x /= np.linalg.norm(x)
            t = tr.ternarize(x, math.acos(gN) + 1e-12)          # must exist by the theorem
            assert _cos(x, t) >= gN - 1e-12
        # the minimiser of the proof, a[k] proportional to sqrt(k) - sqrt(k-1): every prefix gives gamma_N
        k = np.arange(1, N + 1, dtype=np.float64)
        a = gN * (np.sqrt(k) - np.sqrt(k - 1))
        assert abs(np.linalg.norm(a) - 1.0) < 1e-12
        c = np.cumsum(a) / np.sqrt(k)
        assert np.abs(c - gN).max() < 1e-12
        with pytest.raises(tr.NoTernarisation):
            tr.ternarize(a, math.acos(gN) - 1e-6)


# Eq. 4 against a generic least-squares solve of the same problem (a library routine on the
# vectorised rank-one terms), including a rank-deficient case (duplicate components)
@pytest.mark.parametrize("seed", range(6))
def test_lsq_scales_is_the_least_squares_solution(seed):
    g = np.random.default_rng(seed)
    M, N, K = (int(g.integers(3, 12)) for _ in range(3))
    U = g.integers(-1, 2, (M, K)).astype(np.int8)
    V = g.integers(-1, 2, (K, N)).astype(np.int8)
    if seed % 2 and K > 1:
        U[:, -1] = U[:, 0]; V[-1, :] = V[0, :]                   # singular Gram matrix: the pseudo-inverse matters
    W = g.standard_normal((M, N))
    S = tr.lsq_scales(U, V, W)
    A = np.stack([np.outer(U[:, k], V[k, :]).ravel() for k in range(K)], axis=1).astype(np.float64)
    ref, *_ = np.linalg.lstsq(A, W.ravel(), rcond=None)
    fit = lambda s: np.linalg.norm(W - (U * s[None, :]) @ V.astype(np.float64))
    assert abs(fit(S) - fit(ref)) <= 1e-10 * max(1.0, fit(ref))  # the same minimum
    assert np.abs(S - ref).max() <= 1e-8 * max(1.0, np.abs(ref).max())   # and the same (minimum-norm) minimiser
    # first-order condition: the residual is orthogonal to every rank-one term
    R = W - (U * S[None, :]) @ V.astype(np.float64)
    assert np.abs(A.T @ R.ravel()).max() <= 1e-9 * max(1.0, np.abs(W).max() * M * N)


# Algorithm 2: exact reconstruction when W already is a TSVD of orthogonal ternary components, the
# residual never grows, Theorem 2's first inequality per iteration, and the paper's nonzero rate
def test_transition_recovers_a_ternary_rank_one_matrix():
    u = np.array([1, 0, -1, 1, 0, 0], dtype=np.float64)
    v = np.array([0, 1, 1, -1, 0], dtype=np.float64)
    W = 2.5 * np.outer(u, v)
    out = tr.direct_transition(W, THETA, max_rank=1)
    assert out.residual_fro[-1] <= 1e-12 * out.residual_fro[0]
    # the singular pair is determined up to a common sign
    assert (np.array_equal(out.U[:, 0], u) and np.array_equal(out.V[0], v)) or \
           (np.array_equal(out.U[:, 0], -u) and np.array_equal(out.V[0], -v))
    assert abs(out.S[0] - 2.5) < 1e-12


def test_transition_residual_and_theorem_2():
    W = gen.laplace_matrix(11, 96, 64).astype(np.float64)
    out = tr.direct_transition(W, THETA, q=1, max_rank=40)
    res = np.array(out.residual_fro)
    assert np.all(np.diff(res) <= 1e-12 * res[0])               # refitting all of S cannot lose ground
    for i, sigma in enumerate(out.sigma):
        # Theorem 2 (read with theta < pi/4): fitting only the new component already reaches
        # sin^2(2 theta) sigma_0^2 + ||sigma[1:]||^2; Eq. 4 over all components is at least as good
        bound = math.sin(2 * THETA) ** 2 * sigma[0] ** 2 + float(np.sum(sigma[1:] ** 2))
        assert res[i + 1] ** 2 <= bound * (1 + 1e-12)
        assert bound <= (1 - math.cos(2 * THETA) ** 2 / min(W.shape)) * res[i] ** 2 * (1 + 1e-12)
    assert out.U.shape == (96, 40) and out.V.shape == (40, 64) and out.S.shape == (40,)
    assert set(np.unique(out.U)) <= {-1, 0, 1} and set(np.unique(out.V)) <= {-1, 0, 1}


def test_nonzero_rate_on_the_laplace_matrix_of_the_paper():
    """Section "Optimal theta in Practice": on a [512, 256] Laplace matrix, theta = 0.576 gives a
    nonzero rate r of about 0.29."""
    W = gen.laplace_matrix(1, 512, 256)
    out = tr.direct_transition(W, THETA, q=8, max_rank=64)
    assert abs(out.nonzero_rate - 0.29) <= 0.02, out.nonzero_rate
