"""ctypes binding of libtsvd: the same names as include/tsvd.h, argument marshalling only.

Every step of the map runs in the CUDA library.  There is no Python or CPU
implementation behind these calls: if libtsvd.so is missing the import of the
symbols fails loudly.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtsvd.so")

TSVD_F32, TSVD_BF16, TSVD_I8 = 0, 1, 2
TSVD_OK = 0
(TSVD_E_NULL, TSVD_E_SHAPE, TSVD_E_VALUE, TSVD_E_DTYPE, TSVD_E_ALIGN, TSVD_E_CUDA,
 TSVD_E_TIMEOUT, TSVD_E_NOMEM, TSVD_E_TOOBIG, TSVD_E_RANGE, TSVD_E_INTERNAL) = range(1, 12)
TSVD_MAX_CONTRACTION = 65280
TSVD_STATIC_SCRATCH_BYTES = 4 << 20
TSVD_FLAG_OUT_F32 = 0x1
TSVD_FLAG_PATH_SIMPLE = 0x10
TSVD_FLAG_PATH_DECODE = 0x20
TSVD_DECODE_MAX_B = 16       # largest batch the decode kernels serve (tsvd.h)
TSVD_INDEX_MAX_B = 4         # largest batch the index-list kernels serve
TSVD_FLAG_PATH_TENSOR = 0x40
TSVD_FLAG_PATH_INDEX = 0x80      # index-list kernels, for handles packed with TSVD_PACK_INDEX_LISTS
TSVD_PACK_INDEX_LISTS = 0x1      # tsvd_pack flag
TSVD_INDEX_MAX_COLUMNS = 32768
TSVD_FLAG_TEST_STALL = 0x100
TSVD_FLAG_WIDE_X = 0x200         # bf16 activations as four digits (outliers up to 2^16 of the bulk)

DTYPES = {"f32": TSVD_F32, "bf16": TSVD_BF16, "i8": TSVD_I8}

# every symbol include/tsvd.h declares
EXPORTS = ("tsvd_pack", "tsvd_forward", "tsvd_forward_ex", "tsvd_forward_host", "tsvd_forward_static",
           "tsvd_reserve", "tsvd_set_bias", "tsvd_ternarize", "tsvd_forward_v", "tsvd_forward_v_patches", "tsvd_im2col", "tsvd_last_status", "tsvd_plan", "tsvd_info", "tsvd_index_bytes", "tsvd_unpack", "tsvd_profile_enable", "tsvd_profile_read",
           "tsvd_launch_count", "tsvd_destroy", "tsvd_strerror")

_lib: Optional[ctypes.CDLL] = None


class TSVDError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {tsvd_strerror(status)} (status {status})")


def use_library(path: Optional[str]) -> None:
    """Make the binding call the library at `path` (e.g. a checked build, see build.build_checked)
    from now on; None goes back to the regular libtsvd.so.  Handles do not carry over."""
    global _lib, LIB_PATH
    LIB_PATH = path or os.path.join(_HERE, "libtsvd.so")
    _lib = None


def lib() -> ctypes.CDLL:
    """Load libtsvd.so (built by paper_2308_07641_b200.build); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2308_07641_b200.build` "
                              "(needs nvcc); there is no fallback implementation")
        L = ctypes.CDLL(LIB_PATH)
        vp, ci, cu = ctypes.c_void_p, ctypes.c_int, ctypes.c_uint
        L.tsvd_pack.argtypes = [vp, vp, vp, ci, ci, ci, cu, ctypes.POINTER(vp)]
        L.tsvd_pack.restype = ci
        L.tsvd_forward.argtypes = [vp, vp, vp, ci, ci, vp]
        L.tsvd_forward.restype = ci
        L.tsvd_forward_ex.argtypes = [vp, vp, ci, vp, ci, ci, ci, cu, vp, vp]
        L.tsvd_forward_ex.restype = ci
        L.tsvd_forward_host.argtypes = [vp, vp, vp, ci, ci, cu, vp]
        L.tsvd_forward_host.restype = ci
        L.tsvd_forward_static.argtypes = [vp, vp, vp, ci, ci, vp]
        L.tsvd_forward_static.restype = ci
        L.tsvd_reserve.argtypes = [vp, ci, ci]
        L.tsvd_reserve.restype = ci
        L.tsvd_set_bias.argtypes = [vp, vp]
        L.tsvd_set_bias.restype = ci
        L.tsvd_ternarize.argtypes = [vp, ci, ci, ci, ctypes.c_double, vp, ci, vp, vp]
        L.tsvd_ternarize.restype = ci
        L.tsvd_forward_v.argtypes = [vp, vp, ci, vp, ci, ci, ci, cu, vp]
        L.tsvd_forward_v.restype = ci
        L.tsvd_forward_v_patches.argtypes = [vp, vp, ci] + [ci] * 12 + [vp, ci, cu, vp]
        L.tsvd_forward_v_patches.restype = ci
        L.tsvd_im2col.argtypes = [vp, ci] + [ci] * 12 + [vp, ctypes.c_longlong, vp]
        L.tsvd_im2col.restype = ci
        L.tsvd_last_status.argtypes = [vp]
        L.tsvd_last_status.restype = ci
        L.tsvd_info.argtypes = [vp, ctypes.POINTER(ci), ctypes.POINTER(ci), ctypes.POINTER(ci),
                                ctypes.POINTER(ctypes.c_size_t), ctypes.POINTER(ctypes.c_double),
                                ctypes.POINTER(ctypes.c_double)]
        L.tsvd_info.restype = ci
        L.tsvd_index_bytes.argtypes = [vp, ctypes.POINTER(ctypes.c_size_t), ctypes.POINTER(ctypes.c_size_t)]
        L.tsvd_index_bytes.restype = ci
        L.tsvd_unpack.argtypes = [vp, vp, vp, vp]
        L.tsvd_unpack.restype = ci
        L.tsvd_plan.argtypes = [vp, ci, ci, cu, ctypes.POINTER(cu), ctypes.POINTER(ci), ctypes.POINTER(ci)]
        L.tsvd_plan.restype = ci
        L.tsvd_profile_enable.argtypes = [vp, ci]
        L.tsvd_profile_enable.restype = ci
        L.tsvd_profile_read.argtypes = [vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(cu)]
        L.tsvd_profile_read.restype = ci
        L.tsvd_launch_count.argtypes = []
        L.tsvd_launch_count.restype = ctypes.c_ulonglong
        L.tsvd_destroy.argtypes = [vp]
        L.tsvd_destroy.restype = None
        L.tsvd_strerror.argtypes = [ci]
        L.tsvd_strerror.restype = ctypes.c_char_p
        _lib = L
    return _lib


def tsvd_strerror(status: int) -> str:
    return lib().tsvd_strerror(int(status)).decode()


def _check(status: int, what: str) -> None:
    if status != TSVD_OK:
        raise TSVDError(status, what)


def _np_ptr(a: Optional[np.ndarray]) -> Optional[int]:
    return None if a is None else a.ctypes.data


def tsvd_pack(U: np.ndarray, S: np.ndarray, V: np.ndarray, flags: int = 0) -> int:
    """Pack host arrays U int8 [M,K], S float32 [K], V int8 [K,N]; returns the handle."""
    U = np.ascontiguousarray(U, dtype=np.int8)
    V = np.ascontiguousarray(V, dtype=np.int8)
    S = np.ascontiguousarray(S, dtype=np.float32)
    M, K = U.shape
    K2, N = V.shape
    if K2 != K or S.shape != (K,):
        raise TSVDError(TSVD_E_SHAPE, "tsvd_pack")
    h = ctypes.c_void_p()
    _check(lib().tsvd_pack(U.ctypes.data, S.ctypes.data, V.ctypes.data, M, K, N, flags,
                           ctypes.byref(h)), "tsvd_pack")
    return h.value


def tsvd_forward(h: int, x_ptr: int, y_ptr: int, B: int, dtype: int, stream: int = 0) -> None:
    """Raw device pointers (e.g. torch.Tensor.data_ptr()) and a cudaStream_t value."""
    _check(lib().tsvd_forward(h, x_ptr, y_ptr, B, dtype, stream or None), "tsvd_forward")


def tsvd_forward_ex(h: int, x_ptr: int, ldx: int, y_ptr: int, ldy: int, B: int, dtype: int,
                    flags: int = 0, z_out_ptr: int = 0, stream: int = 0) -> None:
    _check(lib().tsvd_forward_ex(h, x_ptr, ldx, y_ptr, ldy, B, dtype, flags, z_out_ptr or None,
                                 stream or None), "tsvd_forward_ex")


def tsvd_forward_host(h: int, x_ptr: int, y_ptr: int, B: int, dtype: int, flags: int = 0,
                      z_out_ptr: int = 0) -> None:
    """Host pointers (numpy .ctypes.data or pinned torch tensors' data_ptr())."""
    _check(lib().tsvd_forward_host(h, x_ptr, y_ptr, B, dtype, flags, z_out_ptr or None),
           "tsvd_forward_host")


def tsvd_forward_static(h: int, x_ptr: int, y_ptr: int, B: int, dtype: int, stream: int = 0) -> None:
    """tsvd_forward without any allocation: the intermediate lives in a fixed array inside the
    library (TSVD_STATIC_SCRATCH_BYTES); larger requests raise with status TSVD_E_TOOBIG."""
    _check(lib().tsvd_forward_static(h, x_ptr, y_ptr, B, dtype, stream or None), "tsvd_forward_static")


def tsvd_reserve(h: int, B_max: int, dtype: int) -> None:
    """Size the handle's scratch for forwards of up to B_max tokens (no allocation afterwards)."""
    _check(lib().tsvd_reserve(h, B_max, dtype), "tsvd_reserve")


def tsvd_set_bias(h: int, bias: Optional[np.ndarray]) -> None:
    """Attach (or with None remove) a float32 bias [M], added after the U-stage."""
    if bias is not None:
        bias = np.ascontiguousarray(bias, dtype=np.float32)
        if bias.shape != (tsvd_info(h)["M"],):
            raise TSVDError(TSVD_E_SHAPE, "tsvd_set_bias")
    _check(lib().tsvd_set_bias(h, _np_ptr(bias)), "tsvd_set_bias")


TSVD_TERNARIZE_MAX_LEN = 32768


def tsvd_forward_v(h: int, x_ptr: int, ldx: int, t_ptr: int, ldt: int, B: int, dtype: int, flags: int = 0,
                   stream: int = 0) -> None:
    """t = diag(S)(V x) only (fp32 [B][K]); raw device pointers."""
    _check(lib().tsvd_forward_v(h, x_ptr, ldx, t_ptr, ldt, B, dtype, flags, stream or None), "tsvd_forward_v")


def tsvd_forward_v_patches(h: int, x_ptr: int, dtype: int, n_img: int, H: int, W: int, C: int, k1: int, k2: int, stride,
                           pad, dil, t_ptr: int, ldt: int, flags: int = 0, stream: int = 0) -> None:
    """t = diag(S)(V patches) with the patches of an NHWC image batch read in place; raw device pointers."""
    _check(lib().tsvd_forward_v_patches(h, x_ptr, dtype, n_img, H, W, C, k1, k2, stride[0], stride[1], pad[0], pad[1],
                                        dil[0], dil[1], t_ptr, ldt, flags, stream or None), "tsvd_forward_v_patches")


def tsvd_im2col(x_ptr: int, dtype: int, n_img: int, H: int, W: int, C: int, k1: int, k2: int, stride, pad, dil,
                out_ptr: int, ld_out: int, stream: int = 0) -> None:
    """Patches of an NHWC image batch, feature order (a, b, c); stride, pad, dil are (h, w) pairs."""
    _check(lib().tsvd_im2col(x_ptr, dtype, n_img, H, W, C, k1, k2, stride[0], stride[1], pad[0], pad[1], dil[0], dil[1],
                             out_ptr, ld_out, stream or None), "tsvd_im2col")


def tsvd_ternarize(x_ptr: int, n_vec: int, length: int, ldx: int, theta: float, t_ptr: int, ldt: int,
                   nnz_ptr: int = 0, stream: int = 0) -> None:
    """Algorithm 1 on n_vec device vectors (float32 in, int8 out); raw device pointers."""
    _check(lib().tsvd_ternarize(x_ptr, n_vec, length, ldx, float(theta), t_ptr, ldt, nnz_ptr or None,
                                stream or None), "tsvd_ternarize")


def tsvd_last_status(h: int) -> int:
    return int(lib().tsvd_last_status(h))


def tsvd_info(h: int) -> dict:
    M, K, N = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
    pb = ctypes.c_size_t()
    du, dv = ctypes.c_double(), ctypes.c_double()
    _check(lib().tsvd_info(h, ctypes.byref(M), ctypes.byref(K), ctypes.byref(N), ctypes.byref(pb),
                           ctypes.byref(du), ctypes.byref(dv)), "tsvd_info")
    return {"M": M.value, "K": K.value, "N": N.value, "packed_bytes": pb.value,
            "density_u": du.value, "density_v": dv.value}


def tsvd_unpack(h: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    info = tsvd_info(h)
    U = np.empty((info["M"], info["K"]), dtype=np.int8)
    V = np.empty((info["K"], info["N"]), dtype=np.int8)
    S = np.empty(info["K"], dtype=np.float32)
    _check(lib().tsvd_unpack(h, U.ctypes.data, S.ctypes.data, V.ctypes.data), "tsvd_unpack")
    return U, S, V


def tsvd_index_bytes(h: int):
    """(bytes of V's index lists, bytes of U's); zeros when the handle has none."""
    v, u = ctypes.c_size_t(), ctypes.c_size_t()
    _check(lib().tsvd_index_bytes(h, ctypes.byref(v), ctypes.byref(u)), "tsvd_index_bytes")
    return v.value, u.value


def tsvd_plan(h: int, B: int, dtype: int, flags: int = 0) -> dict:
    """The dispatch decision for a forward with these arguments (nothing is launched)."""
    path, dx, dt = ctypes.c_uint(), ctypes.c_int(), ctypes.c_int()
    _check(lib().tsvd_plan(h, B, dtype, flags, ctypes.byref(path), ctypes.byref(dx), ctypes.byref(dt)),
           "tsvd_plan")
    name = {TSVD_FLAG_PATH_SIMPLE: "simple", TSVD_FLAG_PATH_DECODE: "decode",
            TSVD_FLAG_PATH_TENSOR: "tensor", TSVD_FLAG_PATH_INDEX: "index"}[path.value]
    return {"path": name, "digits_x": dx.value, "digits_t": dt.value}


N_STAGES = 4
STAGE_NAMES = ("x_digits", "v_stage", "t_digits", "u_stage")


def tsvd_profile_enable(h: int, mode) -> None:
    """mode 0/False: off; 1/True: CUDA-event pairs around every kernel; 2: time stamps written by
    the kernels themselves (works inside a captured graph)."""
    _check(lib().tsvd_profile_enable(h, int(mode)), "tsvd_profile_enable")


def tsvd_profile_read(h: int):
    """Returns ([ms summed per stage], [launches per stage]) since the last read."""
    ms = (ctypes.c_float * N_STAGES)()
    n = (ctypes.c_uint * N_STAGES)()
    _check(lib().tsvd_profile_read(h, ms, n), "tsvd_profile_read")
    return list(ms), list(n)


def tsvd_launch_count() -> int:
    return int(lib().tsvd_launch_count())


def tsvd_destroy(h: int) -> None:
    if h:
        lib().tsvd_destroy(h)
