"""Helpers for the GPU parity tests: run a case through the C ABI and compare with the CPU checker."""
from __future__ import annotations

import numpy as np

import gen
import oracle

# Tolerances (stated for this map's outputs):
#   int8 activations: z = V x bit-exact int32
#   fp32 outputs:     max|y - y_ref| <= 1e-5 * max|y_ref|
#   bf16 outputs:     |y - y_ref| <= 1e-2 * |y_ref| + 1e-3 per element
F32_REL_MAX = 1e-5
BF16_RTOL, BF16_ATOL = 1e-2, 1e-3


def torch_x(case_x: np.ndarray, x_dtype: str):
    from paper_2308_07641_b200 import device_activations
    return device_activations(case_x, x_dtype)


def run_gpu(layer, x_np: np.ndarray, x_dtype: str, flags: int = 0, want_z: bool = True):
    """Forward through TSVDLinear; returns (y as float64 numpy [B,M], z numpy or None, y_is_bf16)."""
    import torch
    x = torch_x(x_np, x_dtype)
    B = x.shape[0]
    K = layer.info["K"]
    z = None
    if want_z:
        z = torch.full((B, K), -12345, dtype=torch.int32 if x_dtype == "i8" else torch.float32,
                       device="cuda")
    y = layer.forward(x, flags=flags, z_out=z)
    torch.cuda.synchronize()
    y_bf16 = y.dtype == torch.bfloat16
    y64 = y.float().double().cpu().numpy()
    return y64, (z.cpu().numpy() if z is not None else None), y_bf16


def oracle_x(x_np: np.ndarray, x_dtype: str) -> np.ndarray:
    return gen.widen_x(x_np, x_dtype)


def check_outputs(y64: np.ndarray, z, ref: "oracle.OracleResult", x_dtype: str, y_bf16: bool, what=""):
    """Apply the stated tolerances; returns a dict of error figures."""
    err = np.abs(y64 - ref.y)
    out = {}
    if y_bf16:
        tol = BF16_RTOL * np.abs(ref.y) + BF16_ATOL
        bad = err > tol
        out["violations"] = int(bad.sum())
        out["worst_ratio"] = float((err / tol).max())
        assert not bad.any(), (f"{what}: {bad.sum()} of {bad.size} bf16 outputs outside tolerance; "
                               f"worst err/tol = {out['worst_ratio']:.3g}")
    else:
        scale = np.abs(ref.y).max()
        out["max_err_over_max"] = float(err.max() / scale) if scale > 0 else float(err.max())
        assert err.max() <= F32_REL_MAX * scale + (0.0 if scale > 0 else 0.0), \
            f"{what}: max|y-y_ref| = {err.max():.3g} > 1e-5 * max|y_ref| = {F32_REL_MAX * scale:.3g}"
    if z is not None:
        if x_dtype == "i8":
            assert z.dtype == np.int32
            assert np.array_equal(z.astype(np.int64), ref.zraw), f"{what}: int32 z is not bit-exact"
        else:
            zs = max(1.0, np.abs(ref.zraw).max())
            assert np.abs(z.astype(np.float64) - ref.zraw).max() <= 1e-6 * zs, f"{what}: z_out off"
    return out


def run_and_check(spec: "gen.CaseSpec", flags: int = 0, sample_tokens=None, pack_flags: int = 0,
                  weights=None, x=None, bias=None, expect_status=0):
    """Build the case (or take the given weights (U, V, S) / activations / bias), run it on the GPU at
    full batch, compare with the checker (all tokens, or a sample), and check the device status word
    (expect_status: a status, a collection of allowed statuses, or None for no check)."""
    from paper_2308_07641_b200 import TSVDLinear, binding
    U, V, S = weights if weights is not None else gen.make_weights(spec)
    if x is None:
        x = gen.make_x(spec)
    layer = TSVDLinear(U, S, V, pack_flags)
    try:
        if bias is not None:
            layer.set_bias(bias)
        y64, z, y_bf16 = run_gpu(layer, x, spec.x_dtype, flags)
        status = binding.tsvd_last_status(layer.handle)
    finally:
        layer.close()
    if expect_status is not None:
        allowed = (expect_status,) if isinstance(expect_status, int) else tuple(expect_status)
        assert status in allowed, f"{spec.name}: device status {status}, expected one of {allowed}"
    if sample_tokens is None:
        idx = np.arange(x.shape[0])
    else:
        idx = np.asarray(sample_tokens)
    ref = oracle.forward(U, S, V, oracle_x(x[idx], spec.x_dtype), bias)
    out = check_outputs(y64[idx], None if z is None else z[idx], ref, spec.x_dtype, y_bf16, spec.name)
    out["status"] = status
    return out
