"""Pins for the fp64 product oracle (Eqs. (qda), (qdw) and their convolutional analogues):
brute-force loops, adjoint identities, the 1x1-conv == linear special case, an independent
library's autograd, unbiasedness of the weight gradient (Eq. (dw_unbiased))."""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl


def _tiny_linear(B=4, N=3, K=5, seed=0):
    r = np.random.default_rng(seed)
    codes = r.integers(-3, 4, size=(B, N)).astype(np.int8)
    codes[r.random((B, N)) < 0.4] = 0
    return codes, np.float32(0.125), r.normal(size=(B, K)).astype(np.float32), \
        r.normal(size=(N, K)).astype(np.float32)


def _tiny_conv(B=2, Co=3, Ci=2, H=4, W=5, k=3, seed=0):
    r = np.random.default_rng(seed)
    codes = r.integers(-3, 4, size=(B, Co, H, W)).astype(np.int8)
    codes[r.random(codes.shape) < 0.5] = 0
    return codes, np.float32(0.25), r.normal(size=(B, Ci, H, W)).astype(np.float32), \
        r.normal(size=(Co, Ci, k, k)).astype(np.float32)


def test_linear_matches_bruteforce():
    c, D, X, W = _tiny_linear()
    a, b = oracle.linear_backward(c, D, X, W), oracle.linear_backward_bruteforce(c, D, X, W)
    for key in ("dW", "dX", "db"):
        np.testing.assert_allclose(a[key], b[key], rtol=0, atol=1e-13)
    assert a["dW"].shape == W.shape and a["dX"].shape == X.shape


@pytest.mark.parametrize("k,H,W", [(3, 4, 5), (1, 3, 4), (3, 1, 1), (3, 2, 7), (5, 6, 5), (5, 2, 3)])
def test_conv_matches_bruteforce(k, H, W):
    c, D, X, Wt = _tiny_conv(k=k, H=H, W=W, seed=k + H)
    a, b = oracle.conv_backward(c, D, X, Wt), oracle.conv_backward_bruteforce(c, D, X, Wt)
    for key in ("dW", "dX", "db"):
        np.testing.assert_allclose(a[key], b[key], rtol=0, atol=1e-13)


@pytest.mark.parametrize("k", [1, 3, 5])
def test_conv_matches_library_autograd(k):
    c, D, X, Wt = _tiny_conv(B=3, Co=4, Ci=5, H=6, W=7, k=k, seed=5)
    Xt = torch.tensor(X, dtype=torch.float64, requires_grad=True)
    Wtt = torch.tensor(Wt, dtype=torch.float64, requires_grad=True)
    z = torch.nn.functional.conv2d(Xt, Wtt, padding=(k - 1) // 2)
    np.testing.assert_allclose(oracle.conv_forward(X, Wt), z.detach().numpy(), atol=1e-12)
    g = torch.tensor(c.astype(np.float64) * float(D))
    z.backward(g)
    o = oracle.conv_backward(c, D, X, Wt)
    np.testing.assert_allclose(o["dW"], Wtt.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(o["dX"], Xt.grad.numpy(), atol=1e-12)


def test_adjoint_identities():
    """<delta~, conv(X,W)> = <dX, X> = <dW, W> (the products are the adjoints of z)."""
    c, D, X, Wt = _tiny_conv(B=2, Co=5, Ci=4, H=6, W=6, k=3, seed=9)
    o = oracle.conv_backward(c, D, X, Wt)
    lhs = (c.astype(np.float64) * float(D) * oracle.conv_forward(X, Wt)).sum()
    assert abs(lhs - (o["dX"] * X).sum()) < 1e-12 * max(1, abs(lhs))
    assert abs(lhs - (o["dW"] * Wt).sum()) < 1e-12 * max(1, abs(lhs))
    c, D, X, W = _tiny_linear(6, 5, 7, seed=2)
    o = oracle.linear_backward(c, D, X, W)
    lhs = (c.astype(np.float64) * float(D) * (X.astype(np.float64) @ W.astype(np.float64).T)).sum()
    assert abs(lhs - (o["dX"] * X).sum()) < 1e-12 and abs(lhs - (o["dW"] * W).sum()) < 1e-12


def test_1x1_conv_is_linear_on_positions():
    c, D, X, Wt = _tiny_conv(B=2, Co=3, Ci=4, H=3, W=5, k=1, seed=4)
    o = oracle.conv_backward(c, D, X, Wt)
    cm = c.transpose(0, 2, 3, 1).reshape(-1, 3)
    Xm = X.transpose(0, 2, 3, 1).reshape(-1, 4)
    l = oracle.linear_backward(cm, D, Xm, Wt.reshape(3, 4))
    np.testing.assert_allclose(o["dW"].reshape(3, 4), l["dW"], atol=1e-13)
    np.testing.assert_allclose(o["dX"].transpose(0, 2, 3, 1).reshape(-1, 4), l["dX"], atol=1e-13)
    np.testing.assert_allclose(o["db"], l["db"], atol=1e-13)


def test_abs_sums_bound_the_terms():
    c, D, X, Wt = _tiny_conv(seed=8)
    o = oracle.conv_backward(c, D, X, Wt, with_abs=True)
    assert np.all(o["S_dW"] >= np.abs(o["dW"]) - 1e-15) and np.all(o["S_dX"] >= np.abs(o["dX"]) - 1e-15)
    pos = oracle.conv_backward(np.abs(c), D, np.abs(X), np.abs(Wt))
    np.testing.assert_allclose(o["S_dW"], pos["dW"], atol=1e-13)
    c, D, X, W = _tiny_linear(seed=3)
    o = oracle.linear_backward(c, D, X, W, with_abs=True)
    np.testing.assert_allclose(o["S_dX"], np.abs(c * float(D)) @ np.abs(W).astype(np.float64), atol=1e-13)


def test_weight_gradient_is_unbiased():
    """Eq. (dw_unbiased): the mean over dither draws of delta~^T X is delta^T X."""
    r = np.random.default_rng(1)
    d = (r.laplace(0, 1e-3, size=(4, 3)) * (r.random((4, 3)) < 0.7)).astype(np.float32)
    X = r.random((4, 5)).astype(np.float32)
    W = r.normal(size=(3, 5)).astype(np.float32)
    D = oracle.step_size(d, 2.0)
    M = 6000
    acc_w = np.zeros((3, 5))
    acc_x = np.zeros((4, 5))
    for s in range(M):
        o = oracle.linear_backward(oracle.nsd_codes(d, s, D)[0], D, X, W)
        acc_w += o["dW"]
        acc_x += o["dX"]
    dense_w = d.astype(np.float64).T @ X.astype(np.float64)
    dense_x = d.astype(np.float64) @ W.astype(np.float64)
    # per-term error variance <= Delta^2/4 (Eq. (bounded variance)); sum of B (or N) terms
    bw = 5 * float(D) / 2 * np.sqrt((X.astype(np.float64) ** 2).sum(axis=0) / M)
    bx = 5 * float(D) / 2 * np.sqrt((W.astype(np.float64) ** 2).sum(axis=0) / M)
    assert np.all(np.abs(acc_w / M - dense_w) <= bw[None, :])
    assert np.all(np.abs(acc_x / M - dense_x) <= bx[None, :])


def test_small_step_limit_recovers_dense_products():
    L = wl.linear_layer(8, 6, 10, data_seed=77)
    D = np.float32(1e-7)                              # codes up to ~1e4 would saturate, so
    d = np.clip(L.delta, -100 * D, 100 * D)           # keep |x|/Delta <= 100
    c, _, nsat = oracle.nsd_codes(d, 0, D)
    assert nsat == 0
    o = oracle.linear_backward(c, D, L.X, L.W)
    dense = d.astype(np.float64).T @ L.X.astype(np.float64)
    assert np.abs(o["dW"] - dense).max() <= 8 * float(D) * np.abs(L.X).max()


@pytest.mark.parametrize("k", [1, 3])
def test_single_entry_routines_match_the_full_products(k):
    c, D, X, Wt = _tiny_conv(B=3, Co=4, Ci=5, H=5, W=6, k=k, seed=21)
    full = oracle.conv_backward(c, D, X, Wt, with_abs=True)
    r = np.random.default_rng(0)
    for _ in range(25):
        co, ci, ky, kx = r.integers(4), r.integers(5), r.integers(k), r.integers(k)
        v, s = oracle.conv_dW_entry(c, D, X, co, ci, ky, kx, k)
        assert abs(v - full["dW"][co, ci, ky, kx]) < 1e-12 and abs(s - full["S_dW"][co, ci, ky, kx]) < 1e-12
        b, y, x = r.integers(3), r.integers(5), r.integers(6)
        v, s = oracle.conv_dX_entry(c, D, Wt, b, ci, y, x)
        assert abs(v - full["dX"][b, ci, y, x]) < 1e-12 and abs(s - full["S_dX"][b, ci, y, x]) < 1e-12
