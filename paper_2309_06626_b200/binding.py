"""ctypes binding of include/asx.h: same names, argument marshalling only."""
from __future__ import annotations

import ctypes
import os
from typing import Tuple

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libasx.so")
_lib = None

ACT_RELU, RECOMPACT, IMPL_NAIVE, OUT_COMPACT, IN_COMPACT, ACT_SILU, F32, IMPL_ROW_GATHER, IMPL_WINDOW_PATCH = 1, 2, 4, 8, 16, 32, 64, 128, 256

# every symbol include/asx.h declares
EXPORTS = (
    "asx_status_string", "asx_create_layer", "asx_set_mask", "asx_set_mask_random", "asx_recompact", "asx_run",
    "asx_get_kept", "asx_get_kept_host", "asx_get_mask", "asx_last_device_status", "asx_destroy",
    "asx_compact_scratch_bytes", "asx_compact", "asx_compact_status", "asx_compact_static",
    "asx_mask_from_scores", "asx_set_mask_from_scores", "asx_mask_from_activation", "asx_set_input_mask", "asx_set_residual",
    "asx_last_run_form", "asx_set_wait_limit", "asx_debug_set_split_counter",
)
COMPACT_STATIC_MAX_ROWS = 1 << 24
FORM_NONE, FORM_NAIVE, FORM_ROW_GATHER_COPY, FORM_ROW_GATHER_TMA, FORM_WINDOW_PATCH = 0, 1, 2, 3, 4


class AsxError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {lib().asx_status_string(code).decode()} (status {code})")
        self.code = code


def lib_path() -> str:
    return _LIB_PATH


def lib():
    """Load libasx.so (once).  There is no fallback: a missing library is an error."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2309_06626_b200.build` "
                "(needs nvcc); this package has no CPU or PyTorch fallback")
        L = ctypes.CDLL(_LIB_PATH)
        vp, i64, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
        L.asx_status_string.argtypes = [ci]
        L.asx_status_string.restype = ctypes.c_char_p
        L.asx_create_layer.argtypes = [ci] * 6 + [ctypes.POINTER(vp)]
        L.asx_set_mask.argtypes = [vp, vp, i64, vp]
        L.asx_set_mask_random.argtypes = [vp, i64, ctypes.c_double, ci, ctypes.c_uint64, vp]
        L.asx_recompact.argtypes = [vp, vp]
        L.asx_run.argtypes = [vp, vp, ci, ci, ci, vp, vp, vp, ci, vp]
        L.asx_get_kept.argtypes = [vp, ctypes.POINTER(i64), ctypes.POINTER(vp)]
        L.asx_get_kept_host.argtypes = [vp, vp, i64, ctypes.POINTER(i64)]
        L.asx_get_mask.argtypes = [vp, vp, i64]
        L.asx_last_device_status.argtypes = [vp]
        L.asx_destroy.argtypes = [vp]
        L.asx_compact_scratch_bytes.argtypes = [i64]
        L.asx_compact_scratch_bytes.restype = i64
        L.asx_compact.argtypes = [vp, i64, vp, vp, vp, i64, vp]
        L.asx_compact_status.argtypes = [vp, vp]
        L.asx_compact_static.argtypes = [vp, i64, vp, vp, vp]
        L.asx_set_input_mask.argtypes = [vp, vp, i64, vp]
        L.asx_set_residual.argtypes = [vp, vp]
        L.asx_last_run_form.argtypes = [vp, ctypes.POINTER(ci)]
        L.asx_set_wait_limit.argtypes = [vp, i64]
        L.asx_debug_set_split_counter.argtypes = [vp, i64, ctypes.c_int32, vp]
        L.asx_mask_from_activation.argtypes = [vp, i64, ci, vp, vp]
        L.asx_mask_from_scores.argtypes = [vp, ci, ci, ci, ci, ctypes.c_double, vp]
        L.asx_set_mask_from_scores.argtypes = [vp, vp, ci, ci, ci, ci, ctypes.c_double, vp]
        for name in EXPORTS:
            if name not in ("asx_status_string", "asx_compact_scratch_bytes"):
                getattr(L, name).restype = ci
        _lib = L
    return _lib


def _check(code: int, what: str) -> None:
    if code != 0:
        raise AsxError(code, what)


def _stream_ptr(stream=None) -> int:
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


class MaskedConvLayer:
    """One convolution layer with a row mask: create_layer / set_mask / run."""

    def __init__(self, C_in: int, C_out: int, kh: int, kw: int, stride: int, pad: int):
        self._h = ctypes.c_void_p()
        _check(lib().asx_create_layer(C_in, C_out, kh, kw, stride, pad, ctypes.byref(self._h)),
               "asx_create_layer")
        self.C_in, self.C_out, self.kh, self.kw, self.stride, self.pad = C_in, C_out, kh, kw, stride, pad

    def out_hw(self, H: int, W: int) -> Tuple[int, int]:
        return ((H + 2 * self.pad - self.kh) // self.stride + 1,
                (W + 2 * self.pad - self.kw) // self.stride + 1)

    def set_mask(self, mask, stream=None) -> None:
        """mask: uint8 torch tensor (CPU or CUDA) or numpy array, 1 = keep, 0 = drop."""
        import numpy as np
        import torch
        if isinstance(mask, torch.Tensor):
            m = mask.contiguous()
            if m.dtype != torch.uint8:
                raise TypeError("mask must be uint8")
            ptr, rows = m.data_ptr(), m.numel()
        else:
            m = np.ascontiguousarray(mask, dtype=np.uint8)
            ptr, rows = m.ctypes.data, m.size
        _check(lib().asx_set_mask(self._h, ptr, rows, _stream_ptr(stream)), "asx_set_mask")

    def set_input_mask(self, mask, stream=None) -> None:
        """The mask of the layer that produced this layer's (compact) input; see ASX_IN_COMPACT."""
        import numpy as np
        import torch
        if isinstance(mask, torch.Tensor):
            m = mask.contiguous()
            if m.dtype != torch.uint8:
                raise TypeError("mask must be uint8")
            ptr, rows = m.data_ptr(), m.numel()
        else:
            m = np.ascontiguousarray(mask, dtype=np.uint8)
            ptr, rows = m.ctypes.data, m.size
        _check(lib().asx_set_input_mask(self._h, ptr, rows, _stream_ptr(stream)), "asx_set_input_mask")

    def set_residual(self, residual=None) -> None:
        """CUDA bf16 tensor laid out like the output, added before the activation; None switches it off.
        The caller keeps the tensor alive while the layer runs."""
        _check(lib().asx_set_residual(self._h, 0 if residual is None else residual.data_ptr()), "asx_set_residual")

    def set_mask_random(self, rows: int, sparsity: float, block: int, seed: int, stream=None) -> None:
        _check(lib().asx_set_mask_random(self._h, rows, float(sparsity), block, seed, _stream_ptr(stream)),
               "asx_set_mask_random")

    def set_mask_from_scores(self, score, Ho: int, Wo: int, sparsity: float, stream=None) -> None:
        """Mask of Algorithm 1's getMask for this layer from a host fp32 score map [H0][W0]."""
        import numpy as np
        sc = np.ascontiguousarray(score, dtype=np.float32)
        _check(lib().asx_set_mask_from_scores(self._h, sc.ctypes.data, sc.shape[0], sc.shape[1], Ho, Wo,
                                              float(sparsity), _stream_ptr(stream)), "asx_set_mask_from_scores")

    def last_run_form(self) -> int:
        """Producer form of the last run (the FORM_* constants)."""
        f = ctypes.c_int(0)
        _check(lib().asx_last_run_form(self._h, ctypes.byref(f)), "asx_last_run_form")
        return f.value

    def set_wait_limit(self, cycles: int) -> None:
        _check(lib().asx_set_wait_limit(self._h, int(cycles)), "asx_set_wait_limit")

    def recompact(self, stream=None) -> None:
        _check(lib().asx_recompact(self._h, _stream_ptr(stream)), "asx_recompact")

    def recompact_raw(self, stream_ptr: int) -> int:
        return lib().asx_recompact(self._h, stream_ptr)

    def run(self, x, w, bias=None, out=None, flags: int = ACT_RELU, stream=None):
        """x: CUDA bf16 [Nb][H][W][C_in]; w: CUDA bf16 [C_out][kh][kw][C_in]; bias: CUDA fp32 or
        None.  Returns the CUDA bf16 output [Nb][Ho][Wo][C_out] (allocated by torch unless
        `out` is given).  With the F32 flag x, w and the output are float32 instead."""
        import torch
        dt = torch.float32 if flags & F32 else torch.bfloat16
        if x.dtype != dt or w.dtype != dt:
            raise TypeError("x and w must be float32 with the F32 flag, else bfloat16")
        if not (x.is_cuda and w.is_cuda and x.is_contiguous() and w.is_contiguous()):
            raise ValueError("x and w must be contiguous CUDA tensors")
        Nb, H, W, C = x.shape
        if C != self.C_in or tuple(w.shape) != (self.C_out, self.kh, self.kw, self.C_in):
            raise ValueError("tensor shapes do not match the layer")
        Ho, Wo = self.out_hw(H, W)
        if out is None:
            out = torch.empty((Nb, Ho, Wo, self.C_out), dtype=dt, device=x.device)
        elif tuple(out.shape) != (Nb, Ho, Wo, self.C_out) or out.dtype != dt or not out.is_contiguous():
            raise ValueError("bad output tensor")
        bptr = 0
        if bias is not None:
            if bias.dtype != torch.float32 or not bias.is_cuda or bias.numel() != self.C_out:
                raise ValueError("bias must be a CUDA fp32 vector of C_out entries")
            bptr = bias.data_ptr()
        _check(lib().asx_run(self._h, x.data_ptr(), Nb, H, W, w.data_ptr(), bptr, out.data_ptr(),
                             flags, _stream_ptr(stream)), "asx_run")
        return out

    def run_raw(self, x_ptr: int, Nb: int, H: int, W: int, w_ptr: int, b_ptr: int, y_ptr: int,
                flags: int, stream_ptr: int) -> int:
        """asx_run with raw pointers; returns the status code."""
        return lib().asx_run(self._h, x_ptr, Nb, H, W, w_ptr, b_ptr, y_ptr, flags, stream_ptr)

    def kept(self):
        """The kept-row list as a numpy int32 array (copied to the host)."""
        import numpy as np
        cnt = ctypes.c_int64()
        _check(lib().asx_get_kept_host(self._h, None, 0, ctypes.byref(cnt)), "asx_get_kept_host")
        out = np.empty(cnt.value, dtype=np.int32)
        _check(lib().asx_get_kept_host(self._h, out.ctypes.data, out.size, ctypes.byref(cnt)),
               "asx_get_kept_host")
        return out

    def mask(self, rows: int):
        import numpy as np
        m = np.empty(rows, dtype=np.uint8)
        _check(lib().asx_get_mask(self._h, m.ctypes.data, rows), "asx_get_mask")
        return m

    def device_status(self) -> int:
        return lib().asx_last_device_status(self._h)

    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h:
            lib().asx_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def mask_from_scores(score, Ho: int, Wo: int, sparsity: float):
    """Algorithm 1's getMask for one layer on the host: numpy uint8 [Ho*Wo] from a fp32 score map."""
    import numpy as np
    sc = np.ascontiguousarray(score, dtype=np.float32)
    out = np.empty(Ho * Wo, dtype=np.uint8)
    _check(lib().asx_mask_from_scores(sc.ctypes.data, sc.shape[0], sc.shape[1], Ho, Wo, float(sparsity),
                                      out.ctypes.data), "asx_mask_from_scores")
    return out


def mask_from_activation(x_dev, stream=None):
    """mask[r] = 1 iff a channel of row r of the CUDA bf16 tensor x_dev [..., C] is positive; returns a
    CUDA uint8 tensor with one entry per row (allocated by torch)."""
    import torch
    if x_dev.dtype != torch.bfloat16 or not x_dev.is_cuda or not x_dev.is_contiguous():
        raise ValueError("x must be a contiguous CUDA bfloat16 tensor")
    C = x_dev.shape[-1]
    rows = x_dev.numel() // C
    out = torch.empty(rows, dtype=torch.uint8, device=x_dev.device)
    _check(lib().asx_mask_from_activation(x_dev.data_ptr(), rows, C, out.data_ptr(), _stream_ptr(stream)),
           "asx_mask_from_activation")
    return out


def compact_mask(mask_dev, stream=None):
    """Stand-alone S1 on a CUDA uint8 tensor: returns (kept int32 tensor of mask.numel()
    entries, count int32 tensor of one entry, scratch tensor).  Only the first `count`
    entries of `kept` are defined."""
    import torch
    rows = mask_dev.numel()
    kept = torch.empty(max(rows, 1), dtype=torch.int32, device=mask_dev.device)
    count = torch.empty(1, dtype=torch.int32, device=mask_dev.device)
    nbytes = lib().asx_compact_scratch_bytes(rows)
    scratch = torch.empty((nbytes + 7) // 8, dtype=torch.int64, device=mask_dev.device)
    _check(lib().asx_compact(mask_dev.data_ptr(), rows, kept.data_ptr(), count.data_ptr(),
                             scratch.data_ptr(), scratch.numel() * 8, _stream_ptr(stream)), "asx_compact")
    return kept, count, scratch
