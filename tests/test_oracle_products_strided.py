"""Pins for the strided-convolution definitions of the fp64 product oracle: brute-force loops,
an independent library's autograd, the stride-1 special case, the adjoint identities, and the
phase picture (a stride-2 1x1 layer is the 1x1 layer on every other row and column)."""
import numpy as np
import pytest
import torch

import oracle


def _case(B, Co, Ci, H, W, k, s, seed):
    r = np.random.default_rng(seed)
    Ho, Wo = oracle.strided_out_size(H, k, s), oracle.strided_out_size(W, k, s)
    codes = r.integers(-3, 4, size=(B, Co, Ho, Wo)).astype(np.int8)
    codes[r.random(codes.shape) < 0.5] = 0
    return codes, np.float32(0.25), r.normal(size=(B, Ci, H, W)).astype(np.float32), \
        r.normal(size=(Co, Ci, k, k)).astype(np.float32)


def test_out_size_matches_the_library():
    for H in range(1, 12):
        for k in (1, 3, 5):
            for s in (1, 2, 3):
                z = torch.nn.functional.conv2d(torch.zeros(1, 1, H, H), torch.zeros(1, 1, k, k), stride=s,
                                               padding=(k - 1) // 2)
                assert z.shape[2] == oracle.strided_out_size(H, k, s)


@pytest.mark.parametrize("k,s,H,W", [(3, 2, 6, 8), (1, 2, 4, 6), (3, 2, 5, 7), (1, 2, 5, 3), (3, 3, 7, 7), (5, 2, 8, 6)])
def test_strided_matches_bruteforce(k, s, H, W):
    c, D, X, Wt = _case(2, 3, 2, H, W, k, s, seed=10 * k + s + H)
    a = oracle.conv_backward_strided(c, D, X, Wt, s)
    b = oracle.conv_backward_strided_bruteforce(c, D, X, Wt, s)
    for key in ("dW", "dX", "db"):
        np.testing.assert_allclose(a[key], b[key], rtol=0, atol=1e-13)
    assert a["dX"].shape == X.shape and a["dW"].shape == Wt.shape


@pytest.mark.parametrize("k,s", [(1, 2), (3, 2), (3, 3), (5, 2)])
def test_strided_matches_library_autograd(k, s):
    c, D, X, Wt = _case(3, 4, 5, 8, 10, k, s, seed=k + s)
    Xt = torch.tensor(X, dtype=torch.float64, requires_grad=True)
    Wtt = torch.tensor(Wt, dtype=torch.float64, requires_grad=True)
    z = torch.nn.functional.conv2d(Xt, Wtt, stride=s, padding=(k - 1) // 2)
    np.testing.assert_allclose(oracle.conv_forward_strided(X, Wt, s), z.detach().numpy(), atol=1e-12)
    z.backward(torch.tensor(c.astype(np.float64) * float(D)))
    o = oracle.conv_backward_strided(c, D, X, Wt, s)
    np.testing.assert_allclose(o["dW"], Wtt.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(o["dX"], Xt.grad.numpy(), atol=1e-12)


@pytest.mark.parametrize("k", [1, 3])
def test_stride_one_is_the_plain_convolution(k):
    c, D, X, Wt = _case(2, 3, 4, 5, 6, k, 1, seed=3)
    a, b = oracle.conv_backward_strided(c, D, X, Wt, 1, with_abs=True), oracle.conv_backward(c, D, X, Wt, with_abs=True)
    for key in ("dW", "dX", "db", "S_dW", "S_dX"):
        np.testing.assert_allclose(a[key], b[key], rtol=0, atol=1e-13)


def test_strided_adjoint_identities():
    c, D, X, Wt = _case(2, 5, 4, 8, 6, 3, 2, seed=9)
    o = oracle.conv_backward_strided(c, D, X, Wt, 2)
    lhs = (c.astype(np.float64) * float(D) * oracle.conv_forward_strided(X, Wt, 2)).sum()
    assert abs(lhs - (o["dX"] * X).sum()) < 1e-12 * max(1, abs(lhs))
    assert abs(lhs - (o["dW"] * Wt).sum()) < 1e-12 * max(1, abs(lhs))


def test_stride_two_pointwise_layer_lives_on_the_even_positions():
    c, D, X, Wt = _case(2, 3, 4, 6, 8, 1, 2, seed=11)
    o = oracle.conv_backward_strided(c, D, X, Wt, 2)
    sub = oracle.conv_backward(c, D, X[:, :, ::2, ::2], Wt)
    np.testing.assert_allclose(o["dW"], sub["dW"], atol=1e-13)
    np.testing.assert_allclose(o["dX"][:, :, ::2, ::2], sub["dX"], atol=1e-13)
    assert not o["dX"][:, :, 1::2, :].any() and not o["dX"][:, :, :, 1::2].any()


def test_abs_sums_bound_the_strided_terms():
    c, D, X, Wt = _case(2, 3, 4, 6, 6, 3, 2, seed=12)
    o = oracle.conv_backward_strided(c, D, X, Wt, 2, with_abs=True)
    assert (np.abs(o["dW"]) <= o["S_dW"] + 1e-12).all() and (np.abs(o["dX"]) <= o["S_dX"] + 1e-12).all()
