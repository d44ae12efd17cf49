"""Ternary-SVD linear map y = U(diag(S)(V x)) on one B200, behind the C ABI of include/tsvd.h.

`binding` mirrors the C entry points one to one; `TSVDLinear` is a small
convenience over them for torch tensors (it owns a handle and passes data
pointers and the current stream; it computes nothing itself).
"""
from __future__ import annotations

from . import binding
from .binding import (DTYPES, TSVD_BF16, TSVD_F32, TSVD_I8, TSVD_FLAG_OUT_F32,  # noqa: F401
                      TSVD_FLAG_PATH_DECODE, TSVD_FLAG_PATH_SIMPLE, TSVD_FLAG_PATH_TENSOR,
                      TSVD_FLAG_WIDE_X, TSVDError)


def device_activations(x_np, x_dtype: str):
    """A host array of stored activations ([B,N] float32, int8, or uint16 holding bf16 bit
    patterns) as a CUDA tensor of the matching torch dtype.  Marshalling only."""
    import numpy as np
    import torch
    if x_dtype == "bf16":
        return torch.from_numpy(np.ascontiguousarray(x_np).view(np.int16).copy()).cuda().view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(x_np)).cuda()


class TSVDLinear:
    """A packed TSVD layer living on the current CUDA device."""

    def __init__(self, U, S, V, pack_flags: int = 0):
        self.handle = binding.tsvd_pack(U, S, V, pack_flags)
        self.info = binding.tsvd_info(self.handle)

    def set_bias(self, bias) -> None:
        binding.tsvd_set_bias(self.handle, bias)

    def reserve(self, B_max: int, x_dtype: str) -> None:
        binding.tsvd_reserve(self.handle, B_max, DTYPES[x_dtype])

    @staticmethod
    def _dtype_of(x) -> int:
        import torch
        if x.dtype == torch.float32:
            return TSVD_F32
        if x.dtype == torch.bfloat16:
            return TSVD_BF16
        if x.dtype == torch.int8:
            return TSVD_I8
        raise TSVDError(binding.TSVD_E_DTYPE, "TSVDLinear.forward")

    def forward(self, x, out=None, flags: int = 0, z_out=None):
        """x: CUDA tensor [B,N] (float32, bfloat16 or int8), row stride >= N. Returns y [B,M]."""
        import torch
        if not x.is_cuda or x.dim() != 2 or x.stride(1) != 1:
            raise TSVDError(binding.TSVD_E_SHAPE, "TSVDLinear.forward")
        B = x.shape[0]
        dt = self._dtype_of(x)
        out_dtype = torch.bfloat16 if (dt == TSVD_BF16 and not flags & TSVD_FLAG_OUT_F32) else torch.float32
        if out is None:
            out = torch.empty((B, self.info["M"]), dtype=out_dtype, device=x.device)
        stream = torch.cuda.current_stream(x.device).cuda_stream
        binding.tsvd_forward_ex(self.handle, x.data_ptr(), x.stride(0), out.data_ptr(), out.stride(0),
                                B, dt, flags, z_out.data_ptr() if z_out is not None else 0, stream)
        return out

    __call__ = forward

    def close(self):
        if getattr(self, "handle", None):
            binding.tsvd_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
