"""Whole-network dithered backward pass (test infrastructure).

Section 3 of the paper, backward equations with Eqs. (qdz), (qda), (qdw): for
l = L ... 1

    delta_z^l     = delta_a^l (.) f'(z^l)                    (ReLU derivative mask)
    delta~_z^l    = NSD(delta_z^l, s)                        (Algorithm 1)
    delta_W^l     = delta~_z^l a^{l-1 T}
    delta_a^{l-1} = W^{l T} delta~_z^l                       (from the QUANTIZED gradient)

A 2x2 max-pool between layers routes each pooled gradient to the window element that was
the (first) maximum in the forward pass. Each layer draws its own dither: its seed is
output l of the SplitMix64 sequence started at the network seed.
"""
import numpy as np

from .nsd import derive_layer_seed, nsd_codes, step_size
from .products import conv_backward, linear_backward


def relu_backward(delta_a, mask):
    """delta_z = delta_a (.) f'(z), fp32 like the stored gradient."""
    d = np.asarray(delta_a, dtype=np.float32)
    return d if mask is None else (d * np.asarray(mask, dtype=np.float32)).astype(np.float32)


def maxpool2x2_backward(g, argmax):
    """g [B,C,H/2,W/2], argmax in {0,1,2,3} (row-major position inside the 2x2 window)
    -> gradient [B,C,H,W] with g at the argmax element of each window, zero elsewhere."""
    g = np.asarray(g)
    B, C, h, w = g.shape
    out = np.zeros((B, C, h, 2, w, 2), dtype=g.dtype)
    for r in range(2):
        for c in range(2):
            sel = (np.asarray(argmax) == (2 * r + c))
            out[:, :, :, r, :, c] = np.where(sel, g, 0)
    return out.reshape(B, C, 2 * h, 2 * w)


def layer_backward(kind, delta_z, X, W, scale, seed, Delta=None, with_abs=False):
    """One layer: NSD then both products. `Delta` overrides s*std (used when a test feeds
    the step size found by another implementation)."""
    D = step_size(delta_z, scale) if Delta is None else np.float32(Delta)
    codes, nnz, nsat = nsd_codes(delta_z, seed, D)
    fn = linear_backward if kind == "linear" else conv_backward
    out = fn(codes, D, X, W, with_abs=with_abs)
    out.update(codes=codes, Delta=D, nnz=nnz, nsat=nsat)
    return out


def chain_backward(kinds, Xs, Ws, relu_masks, pool_argmax, delta_out, scale, seed,
                   delta_z_feed=None):
    """Free-running backward pass; returns one dict per layer (forward order) with
    delta_z, codes, Delta, nnz, dW, dX. With `delta_z_feed` (list, forward order) every
    layer reads the given delta_z instead of the one propagated from above
    (layer-by-layer comparison against another implementation)."""
    L = len(kinds)
    res = [None] * L
    delta_a = np.asarray(delta_out, dtype=np.float32)
    for l in range(L - 1, -1, -1):
        if delta_z_feed is not None and delta_z_feed[l] is not None:
            dz = np.asarray(delta_z_feed[l], dtype=np.float32)
        else:
            dz = relu_backward(delta_a, relu_masks[l])
        r = layer_backward(kinds[l], dz, Xs[l], Ws[l], scale, derive_layer_seed(seed, l))
        r["delta_z"] = dz
        res[l] = r
        if l > 0:
            g = r["dX"].astype(np.float32)              # stored as fp32 between layers
            if kinds[l] == "linear" and kinds[l - 1] == "conv":
                B, C = relu_masks[l - 1].shape[:2]
                g = g.reshape(B, C, pool_argmax[l - 1].shape[2], pool_argmax[l - 1].shape[3]) \
                    if pool_argmax[l - 1] is not None else g.reshape(relu_masks[l - 1].shape)
            if pool_argmax[l - 1] is not None:
                g = maxpool2x2_backward(g, pool_argmax[l - 1])
            delta_a = g
    return res
