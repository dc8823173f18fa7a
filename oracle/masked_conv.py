"""ctypes wrapper around the plain-C oracle (oracle/masked_conv_oracle.c).

The C file is the oracle; this module only compiles it with gcc (-O2, OpenMP over output
rows) and marshals numpy arrays.  See the C file's header for what is computed and which
passages of the paper it follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "masked_conv_oracle.c")
_SRC_ALG2 = os.path.join(_HERE, "alg2_fp32.c")      # the paper's three CPU stages in fp32 (a second baseline)
_LIB = os.path.join(_HERE, "libasx_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or stale."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= max(os.path.getmtime(_SRC), os.path.getmtime(_SRC_ALG2))):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC",
                           "-o", tmp, _SRC, _SRC_ALG2, "-lm"])
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, i32p = ctypes.c_int64, ctypes.POINTER(ctypes.c_int32)
        fp, dp, u8p = (ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_double),
                       ctypes.POINTER(ctypes.c_uint8))
        i64p = ctypes.POINTER(ctypes.c_int64)
        ci = ctypes.c_int
        lib.asxo_bf16_round.argtypes = [fp, fp, i64]
        lib.asxo_bf16_round.restype = None
        lib.asxo_kept_list.argtypes = [u8p, i64, i32p]
        lib.asxo_kept_list.restype = i64
        conv_args = [fp, ci, ci, ci, ci, fp, ci, ci, ci, ci, ci, fp, u8p, i64, ci]
        lib.asxo_masked_conv.argtypes = conv_args + [dp]
        lib.asxo_masked_conv.restype = ci
        lib.asxo_masked_conv_rows.argtypes = conv_args + [i64p, i64, dp]
        lib.asxo_masked_conv_rows.restype = ci
        lib.asxo_alg2_fp32.argtypes = [fp, ci, ci, ci, ci, fp, ci, ci, ci, ci, ci, fp, u8p, ci, fp]
        lib.asxo_alg2_fp32.restype = ci
        _lib = lib
    return _lib


def n_threads() -> int:
    """Threads the OpenMP loops will use (OMP_NUM_THREADS, else all cores)."""
    env = os.environ.get("OMP_NUM_THREADS")
    return int(env) if env else (os.cpu_count() or 1)


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _ptr(a: np.ndarray, ctype):
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def bf16_round(a) -> np.ndarray:
    """Round fp32 values to bfloat16 (nearest, ties to even); returned as fp32."""
    a = _f32(a)
    out = np.empty_like(a)
    _load().asxo_bf16_round(_ptr(a, ctypes.c_float), _ptr(out, ctypes.c_float), a.size)
    return out


def tf32_operand(a) -> np.ndarray:
    """The value a TF32 tensor-core contraction uses for an fp32 operand: sign, exponent and the
    upper 10 mantissa bits; the lower 13 mantissa bits are dropped (towards zero).  Returned as fp32.
    For the fp32-storage path (Appendix A stores fp32): oracle result = masked_conv(tf32_operand(x),
    tf32_operand(w), ..., storage="fp32")."""
    a = _f32(a)
    return (a.view(np.uint32) & np.uint32(0xFFFFE000)).view(np.float32)


def kept_list(mask) -> np.ndarray:
    """Ascending positions with mask == 1, int32."""
    mask = np.ascontiguousarray(mask, dtype=np.uint8).ravel()
    kept = np.empty(mask.size, dtype=np.int32)
    c = _load().asxo_kept_list(_ptr(mask, ctypes.c_uint8), mask.size, _ptr(kept, ctypes.c_int32))
    return kept[:c].copy()


def _geometry(x, w, stride, pad):
    Nb, H, W, C_in = x.shape
    C_out, kh, kw, C_in2 = w.shape
    if C_in != C_in2:
        raise ValueError("channel mismatch")
    Ho = (H + 2 * pad - kh) // stride + 1
    Wo = (W + 2 * pad - kw) // stride + 1
    return Nb, H, W, C_in, C_out, kh, kw, Ho, Wo


def _act_code(relu, storage: str = "bf16") -> int:
    """Activation code of the C oracle: False/None/"none" -> 0, True/"relu" -> 1, "silu" -> 2;
    plus 16 for fp32 storage (x and w taken as given instead of being rounded to bf16)."""
    code = {"none": 0, "relu": 1, "silu": 2}[relu] if isinstance(relu, str) else int(bool(relu))
    return code + {"bf16": 0, "fp32": 16}[storage]


def masked_conv(x, w, bias: Optional[np.ndarray], mask, stride: int, pad: int,
                relu, storage: str = "bf16") -> np.ndarray:
    """y[Nb][Ho][Wo][C_out] in fp64.  x is NHWC fp32, w is [C_out][kh][kw][C_in] fp32 (both are
    rounded to bf16 inside), bias fp32 or None, mask uint8 of Ho*Wo or Nb*Ho*Wo entries.
    `relu` is a bool (ReLU or identity) or one of "none", "relu", "silu"; storage="fp32" keeps x and w
    as given (the paper's fp32 storage) instead of rounding them to bf16."""
    x, w = _f32(x), _f32(w)
    Nb, H, W, C_in, C_out, kh, kw, Ho, Wo = _geometry(x, w, stride, pad)
    mask = np.ascontiguousarray(mask, dtype=np.uint8).ravel()
    b = None if bias is None else _f32(bias)
    y = np.empty((Nb, Ho, Wo, C_out), dtype=np.float64)
    rc = _load().asxo_masked_conv(
        _ptr(x, ctypes.c_float), Nb, H, W, C_in, _ptr(w, ctypes.c_float), C_out, kh, kw,
        stride, pad, None if b is None else _ptr(b, ctypes.c_float),
        _ptr(mask, ctypes.c_uint8), mask.size, _act_code(relu, storage), _ptr(y, ctypes.c_double))
    if rc:
        raise ValueError(f"oracle rejected the arguments (code {rc})")
    return y


def masked_conv_rows(x, w, bias, mask, stride: int, pad: int, relu, sel, storage: str = "bf16") -> np.ndarray:
    """The same definition at selected lowered rows only: returns [len(sel)][C_out] fp64."""
    x, w = _f32(x), _f32(w)
    Nb, H, W, C_in, C_out, kh, kw, Ho, Wo = _geometry(x, w, stride, pad)
    mask = np.ascontiguousarray(mask, dtype=np.uint8).ravel()
    b = None if bias is None else _f32(bias)
    sel = np.ascontiguousarray(sel, dtype=np.int64).ravel()
    y = np.empty((sel.size, C_out), dtype=np.float64)
    rc = _load().asxo_masked_conv_rows(
        _ptr(x, ctypes.c_float), Nb, H, W, C_in, _ptr(w, ctypes.c_float), C_out, kh, kw,
        stride, pad, None if b is None else _ptr(b, ctypes.c_float),
        _ptr(mask, ctypes.c_uint8), mask.size, _act_code(relu, storage),
        _ptr(sel, ctypes.c_int64), sel.size, _ptr(y, ctypes.c_double))
    if rc:
        raise ValueError(f"oracle rejected the arguments (code {rc})")
    return y


def alg2_fp32(x, w, bias: Optional[np.ndarray], mask, stride: int, pad: int, relu: bool) -> np.ndarray:
    """Appendix A, Algorithm 2 as the paper runs it on a CPU, in fp32: indirection buffer over the
    kept positions, dense product on the reduced range, reverse in-place expansion.  x [Nb][H][W][C_in],
    w [C_out][kh][kw][C_in], mask of Ho*Wo entries (shared by the batch).  Returns fp32
    [Nb][Ho][Wo][C_out].  Inputs are used as given (no bfloat16 rounding)."""
    lib = _load()
    x, w = _f32(x), _f32(w)
    Nb, H, W, C_in = x.shape
    C_out, kh, kw, _ = w.shape
    Ho, Wo = (H + 2 * pad - kh) // stride + 1, (W + 2 * pad - kw) // stride + 1
    m = np.ascontiguousarray(mask, dtype=np.uint8)
    if m.size != Ho * Wo:
        raise ValueError("the mask must have Ho*Wo entries")
    b = None if bias is None else _f32(bias)
    y = np.empty((Nb, Ho, Wo, C_out), dtype=np.float32)
    rc = lib.asxo_alg2_fp32(_ptr(x, ctypes.c_float), Nb, H, W, C_in, _ptr(w, ctypes.c_float), C_out, kh, kw,
                            stride, pad, None if b is None else _ptr(b, ctypes.c_float),
                            _ptr(m, ctypes.c_uint8), int(bool(relu)), _ptr(y, ctypes.c_float))
    if rc != 0:
        raise ValueError("bad geometry")
    return y
