"""Dithered backprop on NVIDIA B200: NSD quantization of the preactivation gradient and the
two sparse backward products, as hand-written CUDA kernels behind a C ABI (`include/dbp.h`).

This package is a thin binding: argument marshalling only. Every step runs in the CUDA
library `libdbp.so`; importing the binding fails loudly if the library has not been built.
"""
from .binding import (Context, SparseGradient, DbpError, lib_path, load_library,
                      nsd_quantize, nsd_decode_dense, dithered_linear_backward,
                      dithered_conv_backward, dithered_linear_backward_host,
                      dithered_conv_backward_host, relu_backward, maxpool2x2_backward,
                      network_backward, average_weight_gradients, nsd_step_size_noalloc, kernel_launches, layer_seed, DBP_FORCE_SPARSE, DBP_FORCE_DENSE, DBP_DX_F32, DBP_DW_ASYNC,
                      EXPORTED_SYMBOLS)

__all__ = [
    "Context", "SparseGradient", "DbpError", "lib_path", "load_library", "nsd_quantize",
    "nsd_decode_dense", "dithered_linear_backward", "dithered_conv_backward",
    "dithered_linear_backward_host", "dithered_conv_backward_host", "relu_backward",
    "maxpool2x2_backward", "network_backward", "average_weight_gradients", "nsd_step_size_noalloc", "kernel_launches", "layer_seed", "DBP_FORCE_SPARSE", "DBP_FORCE_DENSE",
    "DBP_DX_F32", "DBP_DW_ASYNC", "EXPORTED_SYMBOLS",
]
