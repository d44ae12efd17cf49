"""The convolution forms of a TSVD layer (Section "TSVD in Convolution Layer" of the paper) on the
current CUDA device, composed from the library's calls: `tsvd_forward_v` applies a stage's ternary
matrix (and, for V(.), the channel-wise scale diag(s)(.)) to the patches of the stage's input, which
`tsvd_forward_v_patches` reads in place (channels a multiple of 16, tensor-core kernels) and
`tsvd_im2col` gathers into a patch matrix otherwise.  Marshalling and index bookkeeping only; the
arithmetic runs in the library.

The kernel W [C_out, C_in, K1, K2] is decomposed as one of the four matrices of Eq. 5:

    form 0  [C_out, C_in*K1*K2]      V(.) a [K1,K2] convolution, U(.) a [1,1] one
    form 1  [C_out*K1*K2, C_in]      V(.) [1,1],   U(.) [K1,K2]
    form 2  [C_out*K1, C_in*K2]      V(.) [1,K2],  U(.) [K1,1]
    form 3  [C_out*K2, C_in*K1]      V(.) [K1,1],  U(.) [1,K2]

with rows ordered (c_out, a, b) and columns (c_in, a, b) as the products are written there.  Per
direction, the layer's stride, padding and dilation go to the stage whose kernel spans that direction
(to V(.) where neither does).  Images are NHWC; no bias inside the stages.  A grouped layer (the
depth-wise layers of the paper's listing: one TSVD of rank 5 per channel) is passed as lists of
per-group U, S, V and runs as one layer whose matrices are block-diagonal: group g's ternary entries
sit at its own channels and its own rank components, zeros elsewhere, so both stages stay the same two
ternary products.
"""
from __future__ import annotations

from typing import Tuple

import numpy as np

from . import binding

Pair = Tuple[int, int]


def _stage_kernels(form: int, K1: int, K2: int) -> Tuple[Pair, Pair]:
    return {0: ((K1, K2), (1, 1)), 1: ((1, 1), (K1, K2)), 2: ((1, K2), (K1, 1)), 3: ((K1, 1), (1, K2))}[form]


def _out(L: int, k: int, s: int, p: int, d: int) -> int:
    return (L + 2 * p - d * (k - 1) - 1) // s + 1


class TSVDConv2d:
    """A convolution layer in TSVD form.  U int8 [M, K], S float32 [K], V int8 [K, N] with [M, N] the
    shape of the chosen matrix of Eq. 5; or, for a grouped layer, lists of G such triples of equal
    shapes, each for C_out/G output and C_in/G input channels."""

    def __init__(self, U, S, V, form: int, C_out: int, C_in: int, K1: int, K2: int, stride: Pair = (1, 1),
                 padding: Pair = (0, 0), dilation: Pair = (1, 1)):
        (v1, v2), (u1, u2) = _stage_kernels(form, K1, K2)
        if isinstance(U, (list, tuple)):
            U, S, V = self._block_diagonal(U, S, V, C_out, C_in, (v1, v2), (u1, u2))
        U = np.ascontiguousarray(U, dtype=np.int8)
        V = np.ascontiguousarray(V, dtype=np.int8)
        S = np.ascontiguousarray(S, dtype=np.float32)
        K = S.shape[0]
        if U.shape != (C_out * u1 * u2, K) or V.shape != (K, C_in * v1 * v2):
            raise binding.TSVDError(binding.TSVD_E_SHAPE, "TSVDConv2d")
        self.form, self.C_out, self.C_in, self.K = form, C_out, C_in, K
        self.kv, self.ku = (v1, v2), (u1, u2)
        v_first = [v1 > 1 or u1 == 1, v2 > 1 or u2 == 1]      # per direction: does V(.) take stride and padding?
        self.sv = tuple(stride[i] if v_first[i] else 1 for i in range(2))
        self.pv = tuple(padding[i] if v_first[i] else 0 for i in range(2))
        self.dv = tuple(dilation[i] if (v1, v2)[i] > 1 else 1 for i in range(2))
        self.su = tuple(1 if v_first[i] else stride[i] for i in range(2))
        self.pu = tuple(0 if v_first[i] else padding[i] for i in range(2))
        self.du = tuple(dilation[i] if (u1, u2)[i] > 1 else 1 for i in range(2))
        # the patch gather lists a patch as (a, b, channel); the matrices list (channel, a, b): reorder once
        Vp = V.reshape(K, C_in, v1, v2).transpose(0, 2, 3, 1).reshape(K, v1 * v2 * C_in)
        Up = U.reshape(C_out, u1, u2, K).reshape(C_out, u1 * u2 * K)
        # stage 1: t = diag(S)(V patches); stage 2: y = U patches-of-t (scale 1).  The unused second
        # matrix of each handle is a single row of zeros.
        self.h_v = binding.tsvd_pack(np.zeros((1, K), np.int8), S, np.ascontiguousarray(Vp))
        self.h_u = binding.tsvd_pack(np.zeros((1, C_out), np.int8), np.ones(C_out, np.float32), np.ascontiguousarray(Up))

    @staticmethod
    def _block_diagonal(Us, Ss, Vs, C_out, C_in, kv, ku):
        """G per-group layers as one: rank components concatenated, group g's entries at its channels."""
        G = len(Us)
        co, ci = C_out // G, C_in // G
        Kg = np.asarray(Ss[0]).shape[0]
        if co * G != C_out or ci * G != C_in or len(Ss) != G or len(Vs) != G:
            raise binding.TSVDError(binding.TSVD_E_SHAPE, "TSVDConv2d")
        (v1, v2), (u1, u2) = kv, ku
        U = np.zeros((C_out, u1, u2, G * Kg), np.int8)
        V = np.zeros((G * Kg, C_in, v1, v2), np.int8)
        S = np.zeros(G * Kg, np.float32)
        for g in range(G):
            Ug, Vg = np.asarray(Us[g], dtype=np.int8), np.asarray(Vs[g], dtype=np.int8)
            if Ug.shape != (co * u1 * u2, Kg) or Vg.shape != (Kg, ci * v1 * v2):
                raise binding.TSVDError(binding.TSVD_E_SHAPE, "TSVDConv2d")
            U[g * co:(g + 1) * co, :, :, g * Kg:(g + 1) * Kg] = Ug.reshape(co, u1, u2, Kg)
            V[g * Kg:(g + 1) * Kg, g * ci:(g + 1) * ci] = Vg.reshape(Kg, ci, v1, v2)
            S[g * Kg:(g + 1) * Kg] = np.asarray(Ss[g], dtype=np.float32)
        return U.reshape(C_out * u1 * u2, G * Kg), S, V.reshape(G * Kg, C_in * v1 * v2)

    def forward(self, x, flags: int = 0):
        """x: CUDA tensor [n, H, W, C_in] (float32, bfloat16 or int8), contiguous.  Returns float32
        [n, Ho, Wo, C_out]."""
        import torch
        if not x.is_cuda or x.dim() != 4 or not x.is_contiguous() or x.shape[3] != self.C_in:
            raise binding.TSVDError(binding.TSVD_E_SHAPE, "TSVDConv2d.forward")
        dt = {torch.float32: binding.TSVD_F32, torch.bfloat16: binding.TSVD_BF16, torch.int8: binding.TSVD_I8}[x.dtype]
        n, H, W, _ = x.shape
        stream = torch.cuda.current_stream(x.device).cuda_stream
        (v1, v2), (u1, u2) = self.kv, self.ku
        Hv, Wv = _out(H, v1, self.sv[0], self.pv[0], self.dv[0]), _out(W, v2, self.sv[1], self.pv[1], self.dv[1])
        t = torch.empty((n * Hv * Wv, self.K), dtype=torch.float32, device=x.device)
        self._stage(self.h_v, x, dt, n, H, W, self.C_in, (v1, v2), self.sv, self.pv, self.dv, t, flags, stream)
        Ho, Wo = _out(Hv, u1, self.su[0], self.pu[0], self.du[0]), _out(Wv, u2, self.su[1], self.pu[1], self.du[1])
        y = torch.empty((n * Ho * Wo, self.C_out), dtype=torch.float32, device=x.device)
        self._stage(self.h_u, t, binding.TSVD_F32, n, Hv, Wv, self.K, (u1, u2), self.su, self.pu, self.du, y, flags, stream)
        return y.view(n, Ho, Wo, self.C_out)

    @staticmethod
    def _stage(handle, img, dt, n, H, W, C, kernel, stride, pad, dil, out, flags, stream):
        """One ternary stage as a convolution over `img` (NHWC, C channels) into `out` [pixels, rank].  A
        [1,1] stage without stride or padding reads the pixels as they are; otherwise the patches are read in
        place when the library can do that (tensor-core kernels, channels a multiple of 16), else gathered
        into a patch matrix first."""
        import torch
        k1, k2 = kernel
        B = out.shape[0]
        if kernel == (1, 1) and stride == (1, 1) and pad == (0, 0):
            binding.tsvd_forward_v(handle, img.data_ptr(), C, out.data_ptr(), out.stride(0), B, dt, flags, stream)
            return
        forced = flags & (binding.TSVD_FLAG_PATH_SIMPLE | binding.TSVD_FLAG_PATH_DECODE)
        if C % 16 == 0 and not forced and (B > binding.TSVD_DECODE_MAX_B or flags & binding.TSVD_FLAG_PATH_TENSOR):
            try:
                binding.tsvd_forward_v_patches(handle, img.data_ptr(), dt, n, H, W, C, k1, k2, stride, pad, dil,
                                               out.data_ptr(), out.stride(0), flags, stream)
                return
            except binding.TSVDError as e:
                if e.status != binding.TSVD_E_SHAPE:      # "not in place for this call": gather first
                    raise
        cols = torch.empty((B, k1 * k2 * C), dtype=img.dtype, device=img.device)
        binding.tsvd_im2col(img.data_ptr(), dt, n, H, W, C, k1, k2, stride, pad, dil, cols.data_ptr(), cols.stride(0), stream)
        binding.tsvd_forward_v(handle, cols.data_ptr(), cols.stride(0), out.data_ptr(), out.stride(0), B, dt, flags, stream)

    __call__ = forward

    def status(self) -> int:
        """The worse of the two stages' device status words (see tsvd_last_status)."""
        a, b = binding.tsvd_last_status(self.h_v), binding.tsvd_last_status(self.h_u)
        return a if a == binding.TSVD_E_TIMEOUT or b == binding.TSVD_OK else b

    def close(self):
        for name in ("h_v", "h_u"):
            h = getattr(self, name, None)
            if h:
                binding.tsvd_destroy(h)
                setattr(self, name, None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
