"""CPU oracle for the masked convolution: test infrastructure, not part of the product.

Only the tests, the smoke check and the benchmark's CPU-baseline leg import this package.
It shares no code with the CUDA path and never imports it.
"""
from .masked_conv import (alg2_fp32, build, bf16_round, kept_list, masked_conv, masked_conv_rows,
                          n_threads, tf32_operand)
from .get_mask import get_mask, mask_from_activation, pooled_score

__all__ = ["alg2_fp32", "build", "bf16_round", "kept_list", "masked_conv", "masked_conv_rows", "n_threads", "tf32_operand",
           "get_mask", "mask_from_activation", "pooled_score"]
