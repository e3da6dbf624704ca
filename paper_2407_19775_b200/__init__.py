"""B200-native dynamic blockwise 8-bit quantization of shard-boundary hidden states.

``workloads`` (seeded input generators) imports without the CUDA library; the binding
loads ``libbq.so`` on first use and raises if it has not been built.
"""
from . import bq4, mmd, mtpp, transport, tune, workloads
from .binding import (BF16, DYNAMIC_TREE, F16, F32, USER, BqError, Codebook, bq_dequantize, bq_quantize, bq_roundtrip,
                      debug_build, kernel_status, n_blocks, set_staging)

from .tune import autotune_block
from .bq4 import Codebook4, bq4_dequantize, bq4_dequantize_s16, bq4_quantize, bq4_quantize_s16
from .mmd import DecomposedLinear, mmd_rowquant, mmd_select_features, mmd_side_columns
from .pipeline import HostBoundary

__all__ = ["workloads", "transport", "mtpp", "tune", "autotune_block", "HostBoundary", "Codebook4", "bq4_quantize", "bq4_dequantize", "bq4_quantize_s16", "bq4_dequantize_s16", "DecomposedLinear", "mmd_rowquant", "mmd_select_features", "mmd_side_columns", "Codebook", "BqError", "bq_quantize", "bq_dequantize", "bq_roundtrip", "n_blocks", "set_staging", "kernel_status", "debug_build",
           "F32", "F16", "BF16", "DYNAMIC_TREE", "USER"]
