"""Data-parallel dithered backward pass (Section 3.6), test infrastructure.

N nodes hold one shard of the batch each. Every node quantizes ITS preactivation gradient with its own step
size Delta_n = s * std(delta_n) and its own dither sequence, forms its weight gradient from the quantized
gradient (Eq. (qdw)), and the parameter server averages the N weight gradients. The dither noises of the nodes
are independent, so the variance of the averaged quantization error falls like 1/N.
"""
import numpy as np

from .nsd import nsd_codes, step_size
from .products import linear_backward


def node_weight_gradient(delta, X, scale, seed):
    """One node: NSD of its delta [B,N] (Algorithm 1), then dW = delta~^T X in fp64."""
    D = step_size(delta, scale)
    codes, _, _ = nsd_codes(delta, seed, D)
    return linear_backward(codes, D, X, np.zeros((delta.shape[1], X.shape[1])))["dW"]


def parameter_server_average(grads):
    """Element-wise mean of the nodes' gradients, added in node order."""
    acc = np.zeros_like(np.asarray(grads[0], dtype=np.float64))
    for g in grads:
        acc = acc + np.asarray(g, dtype=np.float64)
    return acc / len(grads)


def distributed_weight_gradient(deltas, Xs, scale, seeds):
    """deltas[n] [B_n,N], Xs[n] [B_n,K], one seed per node -> averaged dithered dW [N,K]."""
    return parameter_server_average([node_weight_gradient(d, X, scale, s) for d, X, s in zip(deltas, Xs, seeds)])
