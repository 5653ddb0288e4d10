"""B200 (sm_100a) library for block-wise 4-bit optimal-float quantisation (BOF4 / BOF4-S / OPQ).

The product is the C-ABI shared library ``libbof4.so`` (declared in ``include/bof4.h``); this
package holds its CUDA sources (``csrc/``), the build step (``build.py``) and a thin ctypes
binding with the same function names (``binding.py``).
"""
from .binding import (BF16, F32, METRIC_MAE, METRIC_MAE_NORMALIZED, METRIC_MSE, METRIC_MSE_NORMALIZED, NORM_ABS, NORM_SIGNED, OP_EM, OP_OPQ,
                      Bof4Error, bof4_default_init, bof4_dequantize, bof4_em_step,
                      bof4_fit_codebook, bof4_fit_codebook_joint, bof4_m_step, bof4_gemm_tc, bof4_gemv, bof4_last_error, bof4_opq_threshold, bof4_outlier_count, bof4_quantize,
                      bof4_quantize_batch, bof4_dequantize_batch, bof4_quantize_opq, bof4_scales_compress, bof4_scales_expand, bof4_theoretical_codebook, bof4_theoretical_codebook_batch, bof4_theoretical_codebook_general,
                      bof4_workspace_bytes, opq_split)

__all__ = ["BF16", "F32", "METRIC_MAE", "METRIC_MAE_NORMALIZED", "METRIC_MSE", "METRIC_MSE_NORMALIZED", "NORM_ABS", "NORM_SIGNED", "OP_EM", "OP_OPQ",
           "Bof4Error", "bof4_default_init", "bof4_dequantize", "bof4_em_step", "bof4_fit_codebook", "bof4_fit_codebook_joint", "bof4_m_step", "bof4_gemm_tc",
           "bof4_gemv", "bof4_last_error", "bof4_opq_threshold", "bof4_outlier_count", "bof4_quantize", "bof4_quantize_opq",
           "bof4_quantize_batch", "bof4_dequantize_batch", "bof4_scales_compress", "bof4_scales_expand", "bof4_theoretical_codebook", "bof4_theoretical_codebook_batch", "bof4_theoretical_codebook_general", "bof4_workspace_bytes", "opq_split"]
