"""Masked convolution as a compacted GEMM on B200: Python binding of the C-ABI library.

The binding only marshals arguments (device pointers of torch tensors, sizes, the current
CUDA stream); every step of the path runs in the library's CUDA kernels.  Importing the
package does not load the library; the first call does, and fails loudly if the library
has not been built.
"""
from .binding import (AsxError, MaskedConvLayer, compact_mask, mask_from_scores, mask_from_activation, lib, lib_path, EXPORTS,
                      ACT_RELU, RECOMPACT, IMPL_NAIVE, OUT_COMPACT, IN_COMPACT, ACT_SILU, F32, IMPL_ROW_GATHER, IMPL_WINDOW_PATCH,
                      FORM_NONE, FORM_NAIVE, FORM_ROW_GATHER_COPY, FORM_ROW_GATHER_TMA, FORM_WINDOW_PATCH)

__all__ = ["AsxError", "MaskedConvLayer", "compact_mask", "mask_from_scores", "mask_from_activation", "lib", "lib_path", "EXPORTS",
           "ACT_RELU", "RECOMPACT", "IMPL_NAIVE", "OUT_COMPACT", "IN_COMPACT", "ACT_SILU", "F32", "IMPL_ROW_GATHER", "IMPL_WINDOW_PATCH",
           "FORM_NONE", "FORM_NAIVE", "FORM_ROW_GATHER_COPY", "FORM_ROW_GATHER_TMA", "FORM_WINDOW_PATCH"]
