"""Pins for the CPU checker of the convolution forms (oracle/conv.py): the four matrices of Eq. 5,
and the staged evaluation V(.) -> diag(s)(.) -> U(.) against the plain correlation with the kernel
that U diag(S) V reshapes to, which in turn is pinned to a library routine and to nested loops."""
import itertools

import numpy as np
import pytest
from scipy import signal

from oracle import conv as oc


def test_dense_correlation_is_the_textbook_one():
    g = np.random.default_rng(0)
    x = g.standard_normal((2, 7, 9, 3)); W = g.standard_normal((4, 3, 3, 2))
    y = oc.conv2d_dense(x, W)
    assert y.shape == (2, 5, 8, 4)
    for n, o in itertools.product(range(2), range(4)):
        ref = sum(signal.correlate2d(x[n, :, :, c], W[o, c], mode="valid") for c in range(3))
        assert np.abs(y[n, :, :, o] - ref).max() < 1e-12
    # stride, padding, dilation by nested loops on a tiny case
    x = g.standard_normal((1, 5, 6, 2)); W = g.standard_normal((3, 2, 2, 3))
    s, p, d = (2, 1), (1, 2), (2, 1)
    y = oc.conv2d_dense(x, W, s, p, d)
    Ho, Wo = (5 + 2 - 2 * 1 - 1) // 2 + 1, (6 + 4 - 1 * 2 - 1) // 1 + 1
    assert y.shape == (1, Ho, Wo, 3)
    for ho, wo, o in itertools.product(range(Ho), range(Wo), range(3)):
        acc = 0.0
        for c, a, b in itertools.product(range(2), range(2), range(3)):
            h, w = ho * 2 + a * 2 - 1, wo * 1 + b * 1 - 2
            if 0 <= h < 5 and 0 <= w < 6:
                acc += W[o, c, a, b] * x[0, h, w, c]
        assert abs(y[0, ho, wo, o] - acc) < 1e-12
    # the paper's unfolded F(2,3) example: two outputs of a 3-tap kernel on four inputs
    w3 = np.array([0.5, -1.25, 2.0]); x4 = np.array([1.0, 2.0, -3.0, 4.0])
    y = oc.conv2d_dense(x4.reshape(1, 1, 4, 1), w3.reshape(1, 1, 1, 3))
    Wc = np.array([[w3[0], w3[1], w3[2], 0.0], [0.0, w3[0], w3[1], w3[2]]])
    assert np.array_equal(y.ravel(), Wc @ x4)


@pytest.mark.parametrize("form", [0, 1, 2, 3])
def test_the_four_matrices_of_eq_5(form):
    C_out, C_in, K1, K2 = 5, 3, 2, 4
    W = np.arange(C_out * C_in * K1 * K2, dtype=np.float64).reshape(C_out, C_in, K1, K2)
    Wm = oc.kernel_to_matrix(W, form)
    assert Wm.shape == oc.matrix_shape(form, C_out, C_in, K1, K2)
    assert Wm.shape == [(5, 24), (40, 3), (10, 12), (20, 6)][form]
    assert np.array_equal(oc.matrix_to_kernel(Wm, form, C_out, C_in, K1, K2), W)
    (v1, v2), (u1, u2) = oc.form_kernels(form, K1, K2)
    assert (v1 * u1, v2 * u2) == (K1, K2)            # the two stage kernels compose to the layer's
    # entry (row (o, a_u, b_u), column (c, a_v, b_v)) is W[o, c, a_u + a_v, b_u + b_v] (one of each pair is 0)
    for o, c, a, b in itertools.product(range(C_out), range(C_in), range(K1), range(K2)):
        au, av = (a, 0) if u1 > 1 else (0, a)
        bu, bv = (b, 0) if u2 > 1 else (0, b)
        assert Wm[(o * u1 + au) * u2 + bu, (c * v1 + av) * v2 + bv] == W[o, c, a, b]


@pytest.mark.parametrize("form", [0, 1, 2, 3])
@pytest.mark.parametrize("geom", [((1, 1), (0, 0), (1, 1)), ((2, 1), (1, 2), (1, 1)), ((1, 2), (2, 1), (2, 1)),
                                  ((2, 2), (1, 1), (1, 2))])
def test_staged_evaluation_equals_the_convolution_with_the_reconstructed_kernel(form, geom):
    stride, pad, dil = geom
    g = np.random.default_rng(10 * form + stride[0])
    C_out, C_in, K1, K2, K = 4, 3, 3, 2, 7
    M, N = oc.matrix_shape(form, C_out, C_in, K1, K2)
    U = g.integers(-1, 2, (M, K)).astype(np.int8)
    V = g.integers(-1, 2, (K, N)).astype(np.int8)
    S = (g.integers(-16, 17, K) / 8.0).astype(np.float32)
    x = g.integers(-20, 21, (2, 8, 9, C_in)) / 4.0
    Wk = oc.matrix_to_kernel((U * S.astype(np.float64)[None, :]) @ V.astype(np.float64), form, C_out, C_in, K1, K2)
    ref = oc.conv2d_dense(x, Wk, stride, pad, dil)
    got = oc.conv2d_tsvd(x, U, S, V, form, C_out, C_in, K1, K2, stride, pad, dil)
    assert got.shape == ref.shape
    assert np.array_equal(got, ref)                  # dyadic values: exact in any order
    # int8 activations take the integer V-stage and give the same numbers
    x8 = g.integers(-128, 128, (1, 6, 7, C_in)).astype(np.int8)
    assert np.array_equal(oc.conv2d_tsvd(x8, U, S, V, form, C_out, C_in, K1, K2, stride, pad, dil),
                          oc.conv2d_dense(x8.astype(np.float64), Wk, stride, pad, dil))


def test_pointwise_kernel_is_the_linear_layer():
    import oracle
    g = np.random.default_rng(5)
    U = g.integers(-1, 2, (6, 5)).astype(np.int8); V = g.integers(-1, 2, (5, 4)).astype(np.int8)
    S = g.standard_normal(5).astype(np.float32)
    x = g.standard_normal((3, 2, 2, 4))
    y = oc.conv2d_tsvd(x, U, S, V, 0, 6, 4, 1, 1)
    assert np.abs(y.reshape(12, 6) - oracle.forward(U, S, V, x.reshape(12, 4)).y).max() < 1e-13


def test_grouped_and_depthwise_layers():
    """Groups are independent layers on their own channels: against nested loops over the grouped
    kernel that the per-group U diag(S) V reshape to (a depth-wise 7x7 layer of rank 5 among them)."""
    g = np.random.default_rng(21)
    for (G, co, ci, K1, K2, K, form, geom) in [(6, 1, 1, 7, 7, 5, 0, ((1, 1), (3, 3), (1, 1))),
                                               (3, 2, 4, 3, 3, 6, 2, ((2, 1), (1, 1), (1, 1))),
                                               (2, 3, 2, 2, 3, 4, 1, ((1, 2), (0, 1), (1, 1)))]:
        stride, pad, dil = geom
        M, N = oc.matrix_shape(form, co, ci, K1, K2)
        Us = [g.integers(-1, 2, (M, K)).astype(np.int8) for _ in range(G)]
        Vs = [g.integers(-1, 2, (K, N)).astype(np.int8) for _ in range(G)]
        Ss = [(g.integers(-16, 17, K) / 8.0).astype(np.float32) for _ in range(G)]
        x = g.integers(-20, 21, (2, 9, 8, G * ci)) / 4.0
        Wk = np.concatenate([oc.matrix_to_kernel((Us[i] * Ss[i].astype(np.float64)[None, :]) @ Vs[i].astype(np.float64),
                                                 form, co, ci, K1, K2) for i in range(G)], axis=0)
        got = oc.conv2d_tsvd_grouped(x, Us, Ss, Vs, form, G * co, G * ci, K1, K2, stride, pad, dil)
        assert np.array_equal(got, oc.conv2d_dense_grouped(x, Wk, G, stride, pad, dil))
        # the grouped correlation itself, by nested loops on one output position per channel
        n, Ho, Wo, Co = got.shape
        for o in range(Co):
            grp = o // co
            ho, wo = Ho // 2, Wo // 3
            acc = 0.0
            for c, a, b in itertools.product(range(ci), range(K1), range(K2)):
                h, w = ho * stride[0] + a * dil[0] - pad[0], wo * stride[1] + b * dil[1] - pad[1]
                if 0 <= h < 9 and 0 <= w < 8:
                    acc += Wk[o, c, a, b] * x[1, h, w, grp * ci + c]
            assert abs(got[1, ho, wo, o] - acc) < 1e-12
