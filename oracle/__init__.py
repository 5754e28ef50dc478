"""CPU oracle for dithered backprop -- TEST INFRASTRUCTURE, not part of the product.

Plain, slow, obviously-correct implementations of what the CUDA path computes:
NSD quantization (Section 3.1 Eq. (nsd), Algorithm 1) and the two dithered backward
products (Eqs. (qda), (qdw)) for linear and convolution layers, in fp64.
Nothing here is imported by, or shares code with, the CUDA library or its binding.
"""
from .nsd import (splitmix64_at, dither_u, mean_std, step_size, nsd_codes,
                  nsd_codes_literal_f64, nsd_codes_exact_python, derive_layer_seed)
from .products import (linear_backward, conv_backward, conv_forward,
                       linear_backward_bruteforce, conv_backward_bruteforce,
                       conv_dW_entry, conv_dX_entry, strided_out_size, conv_forward_strided,
                       conv_backward_strided, conv_backward_strided_bruteforce)

from .distributed import node_weight_gradient, parameter_server_average, distributed_weight_gradient
from .chain import relu_backward, maxpool2x2_backward, layer_backward, chain_backward

__all__ = [
    "node_weight_gradient", "parameter_server_average", "distributed_weight_gradient",
    "relu_backward", "maxpool2x2_backward", "layer_backward", "chain_backward",
    "splitmix64_at", "dither_u", "mean_std", "step_size", "nsd_codes",
    "nsd_codes_literal_f64", "nsd_codes_exact_python", "derive_layer_seed",
    "linear_backward", "conv_backward", "conv_forward",
    "linear_backward_bruteforce", "conv_backward_bruteforce", "conv_dW_entry", "conv_dX_entry",
    "strided_out_size", "conv_forward_strided", "conv_backward_strided", "conv_backward_strided_bruteforce",
]
