"""CPU checker for the convolution forms of a TSVD layer (test infrastructure only).

Section "TSVD in Convolution Layer": the kernel W [C_out, C_in, K1, K2] is reshaped to one of the
four matrices of Eq. 5,

    form 0   [C_out,        C_in * K1 * K2]      kernel_U = [1, 1],    kernel_V = [K1, K2]
    form 1   [C_out*K1*K2,  C_in]                kernel_U = [K1, K2],  kernel_V = [1, 1]
    form 2   [C_out*K1,     C_in * K2]           kernel_U = [K1, 1],   kernel_V = [1, K2]
    form 3   [C_out*K2,     C_in * K1]           kernel_U = [1, K2],   kernel_V = [K1, 1]

decomposed as U diag(S) V, and applied as the convolution V(.), the channel-wise scale diag(s)(.)
and the convolution U(.).  `conv2d_tsvd` evaluates exactly that, in the paper's order, in float64,
with additions and subtractions at the nonzeros of V and U only (through the forward checker,
applied to the patches of each stage's input).  Index order inside the products of Eq. 5: as
written there, the left factor slowest (row (c_out, k1, k2), column (c_in, k1, k2)).

Readings where the paper is silent:
  * correlation, not flipped convolution (the frameworks the paper's listing comes from);
  * stride, padding and dilation of the layer go, per direction, to the stage whose kernel spans
    that direction (to V(.) where neither does); the other stage has stride 1 and no padding there.
    Zero padding of the intermediate is exact because the stages have no bias;
  * groups: a grouped layer (the depth-wise layers of the listing: groups = channels, rank 5) is one
    independent TSVD per group on that group's channels, each with its own U, S, V of equal shapes
    (`conv2d_tsvd_grouped`); the listing's "rank" is read as the rank of each group.

Nothing in the GPU library imports this module, and this module imports nothing of it.
Pins: tests/test_conv_pins.py.
"""
from __future__ import annotations

from typing import Tuple

import numpy as np

from . import forward as _forward

Pair = Tuple[int, int]

# per form: (kernel_V, kernel_U) as functions of (K1, K2)
_KERNELS = {0: (lambda k1, k2: (k1, k2), lambda k1, k2: (1, 1)),
            1: (lambda k1, k2: (1, 1), lambda k1, k2: (k1, k2)),
            2: (lambda k1, k2: (1, k2), lambda k1, k2: (k1, 1)),
            3: (lambda k1, k2: (k1, 1), lambda k1, k2: (1, k2))}


def form_kernels(form: int, K1: int, K2: int) -> Tuple[Pair, Pair]:
    """(kernel_V, kernel_U) of a form."""
    kv, ku = _KERNELS[form]
    return kv(K1, K2), ku(K1, K2)


def matrix_shape(form: int, C_out: int, C_in: int, K1: int, K2: int) -> Pair:
    """Shape [M, N] of the matrix of Eq. 5 that the form decomposes."""
    (v1, v2), (u1, u2) = form_kernels(form, K1, K2)
    return C_out * u1 * u2, C_in * v1 * v2


def kernel_to_matrix(W: np.ndarray, form: int) -> np.ndarray:
    """W [C_out, C_in, K1, K2] as the matrix of its form: row (c_out, a_u, b_u), column (c_in, a_v, b_v)."""
    C_out, C_in, K1, K2 = W.shape
    if form == 0:
        return W.reshape(C_out, C_in * K1 * K2)
    if form == 1:
        return W.transpose(0, 2, 3, 1).reshape(C_out * K1 * K2, C_in)
    if form == 2:
        return W.transpose(0, 2, 1, 3).reshape(C_out * K1, C_in * K2)
    if form == 3:
        return W.transpose(0, 3, 1, 2).reshape(C_out * K2, C_in * K1)
    raise ValueError(form)


def matrix_to_kernel(Wm: np.ndarray, form: int, C_out: int, C_in: int, K1: int, K2: int) -> np.ndarray:
    """Inverse of kernel_to_matrix."""
    if form == 0:
        return Wm.reshape(C_out, C_in, K1, K2)
    if form == 1:
        return Wm.reshape(C_out, K1, K2, C_in).transpose(0, 3, 1, 2)
    if form == 2:
        return Wm.reshape(C_out, K1, C_in, K2).transpose(0, 2, 1, 3)
    if form == 3:
        return Wm.reshape(C_out, K2, C_in, K1).transpose(0, 2, 3, 1)
    raise ValueError(form)


def _out_size(L: int, k: int, s: int, p: int, d: int) -> int:
    return (L + 2 * p - d * (k - 1) - 1) // s + 1


def _patches(x: np.ndarray, kernel: Pair, stride: Pair, pad: Pair, dil: Pair) -> np.ndarray:
    """x [n, H, W, C] -> [n, Ho, Wo, C, a, b]: the values under each kernel position (zero outside)."""
    n, H, W, C = x.shape
    (k1, k2), (sh, sw), (ph, pw), (dh, dw) = kernel, stride, pad, dil
    Ho, Wo = _out_size(H, k1, sh, ph, dh), _out_size(W, k2, sw, pw, dw)
    out = np.zeros((n, Ho, Wo, C, k1, k2), dtype=x.dtype)
    for ho in range(Ho):
        for wo in range(Wo):
            for a in range(k1):
                for b in range(k2):
                    h, w = ho * sh + a * dh - ph, wo * sw + b * dw - pw
                    if 0 <= h < H and 0 <= w < W:
                        out[:, ho, wo, :, a, b] = x[:, h, w, :]
    return out


def conv2d_tsvd(x: np.ndarray, U: np.ndarray, S: np.ndarray, V: np.ndarray, form: int, C_out: int, C_in: int,
                K1: int, K2: int, stride: Pair = (1, 1), padding: Pair = (0, 0), dilation: Pair = (1, 1)) -> np.ndarray:
    """x [n, H, W, C_in] (float64, or int8 for the integer V-stage) -> y [n, Ho, Wo, C_out] float64.

    U int8 [M, K], S float32 [K], V int8 [K, N] with [M, N] = matrix_shape(form, ...)."""
    (v1, v2), (u1, u2) = form_kernels(form, K1, K2)
    M, N = matrix_shape(form, C_out, C_in, K1, K2)
    K = S.shape[0]
    assert U.shape == (M, K) and V.shape == (K, N)
    # the stage whose kernel spans a direction takes the layer's stride, padding and dilation there
    sv = (stride[0] if v1 > 1 or u1 == 1 else 1, stride[1] if v2 > 1 or u2 == 1 else 1)
    pv = (padding[0] if v1 > 1 or u1 == 1 else 0, padding[1] if v2 > 1 or u2 == 1 else 0)
    dv = (dilation[0] if v1 > 1 else 1, dilation[1] if v2 > 1 else 1)
    su = (stride[0] if sv[0] == 1 else 1, stride[1] if sv[1] == 1 else 1)
    pu = (padding[0] if u1 > 1 else 0, padding[1] if u2 > 1 else 0)
    du = (dilation[0] if u1 > 1 else 1, dilation[1] if u2 > 1 else 1)
    # V(.) as a convolution, then diag(s)(.) channel-wise: t [n, Hv, Wv, K]
    pa = _patches(x, (v1, v2), sv, pv, dv)
    n, Hv, Wv = pa.shape[:3]
    cols = np.ascontiguousarray(pa.reshape(n * Hv * Wv, C_in * v1 * v2))
    ident = np.eye(K, dtype=np.int8)                       # "U" of a V-only product: passes t through
    t = _forward(ident, S, V, cols).y.reshape(n, Hv, Wv, K)
    # U(.) as a convolution over t: y[c_out] = sum_{k,a,b} U[(c_out,a,b), k] t_patch[k,a,b]
    pb = _patches(t, (u1, u2), su, pu, du)
    Ho, Wo = pb.shape[1:3]
    cols_u = np.ascontiguousarray(pb.reshape(n * Ho * Wo, K * u1 * u2))
    Uc = np.ascontiguousarray(U.reshape(C_out, u1, u2, K).transpose(0, 3, 1, 2).reshape(C_out, K * u1 * u2))
    ones = np.ones(K * u1 * u2, dtype=np.float32)
    y = _forward(Uc, ones, np.eye(K * u1 * u2, dtype=np.int8), cols_u).y
    return y.reshape(n, Ho, Wo, C_out)


def conv2d_dense(x: np.ndarray, W: np.ndarray, stride: Pair = (1, 1), padding: Pair = (0, 0),
                 dilation: Pair = (1, 1)) -> np.ndarray:
    """Plain correlation of x [n, H, W, C_in] with W [C_out, C_in, K1, K2] in float64 (the definition a
    converted layer approximates); used by the pins and to compare a decomposition with its source."""
    C_out, C_in, K1, K2 = W.shape
    pa = _patches(np.asarray(x, dtype=np.float64), (K1, K2), stride, padding, dilation)
    return np.einsum("nhwcab,ocab->nhwo", pa, np.asarray(W, dtype=np.float64))


def conv2d_tsvd_grouped(x: np.ndarray, Us, Ss, Vs, form: int, C_out: int, C_in: int, K1: int, K2: int,
                        stride: Pair = (1, 1), padding: Pair = (0, 0), dilation: Pair = (1, 1)) -> np.ndarray:
    """A grouped layer: group g maps input channels [g*C_in/G, (g+1)*C_in/G) to output channels
    [g*C_out/G, (g+1)*C_out/G) by its own TSVD (Us[g], Ss[g], Vs[g]); G = len(Us)."""
    G = len(Us)
    ci, co = C_in // G, C_out // G
    assert ci * G == C_in and co * G == C_out
    outs = [conv2d_tsvd(np.ascontiguousarray(x[..., g * ci:(g + 1) * ci]), Us[g], Ss[g], Vs[g], form, co, ci, K1, K2,
                        stride, padding, dilation) for g in range(G)]
    return np.concatenate(outs, axis=-1)


def conv2d_dense_grouped(x: np.ndarray, W: np.ndarray, groups: int, stride: Pair = (1, 1), padding: Pair = (0, 0),
                         dilation: Pair = (1, 1)) -> np.ndarray:
    """Plain grouped correlation; W [C_out, C_in / groups, K1, K2]."""
    C_out = W.shape[0]
    ci, co = W.shape[1], C_out // groups
    outs = [conv2d_dense(x[..., g * ci:(g + 1) * ci], W[g * co:(g + 1) * co], stride, padding, dilation)
            for g in range(groups)]
    return np.concatenate(outs, axis=-1)
