"""GPU parity of the direct transition W -> (U, S, V): the library's Algorithm 1 kernel, called
through the C ABI, against the CPU checker entry by entry; Eq. 4 and Algorithm 2 of the device-side
driver against the checker on what is unique (the scales for given U, V; the residuals and the
nonzero rate), because singular vectors computed in float32 and in float64 may ternarise a few
entries at the cut differently; and the forward on operands produced this way."""
import math

import numpy as np
import pytest

import gen
from oracle import transition as otr
from tests import _util

pytestmark = pytest.mark.gpu
THETA = 0.576


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2308_07641_b200 import build
    build.build()


def _ternarize_gpu(x32, theta, ld_extra=0):
    import torch
    from paper_2308_07641_b200 import binding
    n_vec, length = x32.shape
    xs = torch.zeros((n_vec, length + ld_extra), dtype=torch.float32, device="cuda")
    xs[:, :length] = torch.from_numpy(x32).cuda()
    t = torch.full((n_vec, length + ld_extra), 7, dtype=torch.int8, device="cuda")
    nnz = torch.full((n_vec,), -5, dtype=torch.int32, device="cuda")
    binding.tsvd_ternarize(xs.data_ptr(), n_vec, length, xs.stride(0), theta, t.data_ptr(), t.stride(0), nnz.data_ptr())
    torch.cuda.synchronize()
    tt = t.cpu().numpy()
    assert np.all(tt[:, length:] == 7)                      # padding untouched
    return tt[:, :length], nnz.cpu().numpy()


def _check_against_checker(x32, theta, **kw):
    t, nnz = _ternarize_gpu(x32, theta, **kw)
    for v in range(x32.shape[0]):
        try:
            ref = otr.ternarize(x32[v].astype(np.float64), theta)
        except otr.NoTernarisation:
            assert nnz[v] == -1 and not t[v].any(), v
            continue
        assert np.array_equal(t[v], ref), (v, int(np.count_nonzero(t[v])), int(np.count_nonzero(ref)))
        assert nnz[v] == np.count_nonzero(ref)


@pytest.mark.parametrize("length", [1, 2, 7, 63, 64, 1000, 2048, 2049, 4096, 5000, 16384, 32768])
def test_ternarize_matches_the_checker(length):
    n_vec = 5
    x = gen.rng.normal(100 + length, 1, n_vec * length).reshape(n_vec, length)
    x /= np.linalg.norm(x, axis=1, keepdims=True)
    _check_against_checker(x.astype(np.float32), THETA, ld_extra=3)


@pytest.mark.parametrize("theta", [0.2, 0.45, 0.8, 1.2, math.pi / 2])
def test_ternarize_angles_including_unreachable_ones(theta):
    x = gen.rng.normal(7, 2, 6 * 777).reshape(6, 777).astype(np.float32)      # not normalised: the test is scale-free
    x[3] *= 1e-20
    x[4] *= 1e18
    _check_against_checker(x, theta)


def test_ternarize_ties_zeros_and_degenerate_vectors():
    g = np.random.default_rng(3)
    rows = [np.round(g.standard_normal(900) * 3) / 3,                 # many equal magnitudes, many exact zeros
            np.ones(900), -np.ones(900),
            np.concatenate([[5.0], np.zeros(899)]),
            np.zeros(900),                                            # zero vector: no ternarisation
            np.where(g.random(900) < 0.9, 0.0, g.standard_normal(900)),
            np.repeat(g.standard_normal(9), 100)]
    x = np.stack(rows).astype(np.float32)
    for theta in (0.3, THETA, 0.9):
        _check_against_checker(x, theta)


def test_ternarize_rejects_too_long_vectors():
    import torch
    from paper_2308_07641_b200 import binding
    n = binding.TSVD_TERNARIZE_MAX_LEN + 1
    x = torch.zeros(n, device="cuda"); t = torch.zeros(n, dtype=torch.int8, device="cuda")
    with pytest.raises(binding.TSVDError) as e:
        binding.tsvd_ternarize(x.data_ptr(), 1, n, n, THETA, t.data_ptr(), n)
    assert e.value.status == binding.TSVD_E_TOOBIG


def test_scales_of_eq_4_match_the_checker():
    import torch
    from paper_2308_07641_b200 import transition
    g = np.random.default_rng(8)
    M, N, K = 70, 50, 33
    U = g.integers(-1, 2, (M, K)).astype(np.int8); V = g.integers(-1, 2, (K, N)).astype(np.int8)
    U[:, 5] = U[:, 2]; V[5] = V[2]                                    # a duplicated component: singular Gram matrix
    W = gen.laplace_matrix(8, M, N)
    S = transition.lsq_scales(torch.from_numpy(U).cuda(), torch.from_numpy(V).cuda(), torch.from_numpy(W).cuda()).cpu().numpy()
    ref = otr.lsq_scales(U, V, W)
    assert np.abs(S - ref).max() <= 1e-9 * max(1.0, np.abs(ref).max())


def test_direct_transition_on_the_laplace_matrix_of_the_paper():
    """[512, 256] Laplace matrix, theta = 0.576 (Section "Optimal theta in Practice"): nonzero rate about
    0.29; residuals as the checker's within the effect of float32 singular vectors."""
    import torch
    from paper_2308_07641_b200 import transition
    W = gen.laplace_matrix(1, 512, 256)
    out = transition.direct_transition(torch.from_numpy(W).cuda(), THETA, q=8, max_rank=64)
    ref = otr.direct_transition(W, THETA, q=8, max_rank=64)
    U, V, S = out.U.cpu().numpy(), out.V.cpu().numpy(), out.S.cpu().numpy()
    assert U.shape == (512, 64) and V.shape == (64, 256)
    assert set(np.unique(U)) <= {-1, 0, 1} and set(np.unique(V)) <= {-1, 0, 1}
    assert abs(out.nonzero_rate - 0.29) <= 0.02
    assert abs(out.nonzero_rate - ref.nonzero_rate) <= 0.01
    res, rres = np.array(out.residual_fro), np.array(ref.residual_fro)
    assert np.all(np.diff(res) <= 1e-6 * res[0])
    assert np.abs(res - rres).max() <= 2e-3 * rres[0]
    # the scales returned are the least-squares scales of the returned U, V (Eq. 4), by the checker
    S_ref = otr.lsq_scales(U, V, W)
    assert np.abs(S - S_ref).max() <= 1e-5 * np.abs(S_ref).max()
    # and the reported residual is the residual of the returned factors
    R = W.astype(np.float64) - (U * S.astype(np.float64)[None, :]) @ V.astype(np.float64)
    assert abs(np.linalg.norm(R) - res[-1]) <= 1e-5 * res[0]


def test_forward_on_operands_from_the_transition():
    """Operands with the structure the paper's layers have (rows of V and columns of U are ternarised
    singular vectors, K beyond min(M, N), S from a pseudo-inverse: signed, unsorted): the forward against
    the checker on every path, and against W x within the decomposition's own residual."""
    import torch
    from paper_2308_07641_b200 import TSVDLinear, transition
    M, N = 384, 200
    W = gen.laplace_matrix(5, M, N)
    out = transition.direct_transition(torch.from_numpy(W).cuda(), THETA, q=16, max_rank=320)
    U, V, S = out.U.cpu().numpy(), out.V.cpu().numpy(), out.S.cpu().numpy()
    for B, flags in ((3, 0x20), (7, 0x20), (40, 0x40), (150, 0x40), (9, 0x10)):
        spec = gen.scaled(gen.CONFIGS["cfg2"], name=f"transition_B{B}", M=M, N=N, K=U.shape[1], B=B, seed=77)
        _util.run_and_check(spec, flags=flags, weights=(U, V, S), expect_status=(0, 10))
    # the map approximates W x as well as the factors approximate W
    x = gen.make_x(gen.scaled(gen.CONFIGS["cfg1"], M=M, N=N, K=U.shape[1], B=5, seed=78))
    layer = TSVDLinear(U, S, V)
    try:
        y = layer.forward(torch.from_numpy(x).cuda()).double().cpu().numpy()
    finally:
        layer.close()
    exact = x.astype(np.float64) @ W.astype(np.float64).T
    rel = np.linalg.norm(y - exact) / np.linalg.norm(exact)
    assert rel <= 1.5 * out.residual_fro[-1] / out.residual_fro[0] + 1e-3
