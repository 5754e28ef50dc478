"""Pins for the data-parallel form (Section 3.6): the server's average of the nodes' dithered weight gradients
is unbiased for the average of the exact ones, and the variance of its quantization error falls like 1/N (the
nodes' dithers are independent)."""
import numpy as np

import oracle
import workloads as wl


def _nodes(N, B=4, n=12, k=10, seed=0):
    ds, Xs = [], []
    for i in range(N):
        L = wl.linear_layer(B, n, k, data_seed=seed + 31 * i, scale=3.0)
        ds.append(L.delta), Xs.append(L.X)
    return ds, Xs


def _exact(ds, Xs):
    return oracle.parameter_server_average([d.astype(np.float64).T @ X.astype(np.float64) for d, X in zip(ds, Xs)])


def test_average_is_the_plain_mean():
    r = np.random.default_rng(1)
    g = [r.normal(size=(3, 4)) for _ in range(5)]
    np.testing.assert_allclose(oracle.parameter_server_average(g), np.mean(g, axis=0), atol=1e-15)
    np.testing.assert_array_equal(oracle.parameter_server_average(g[:1]), g[0])


def test_one_node_is_the_single_machine_gradient():
    ds, Xs = _nodes(1)
    D = oracle.step_size(ds[0], 3.0)
    codes, _, _ = oracle.nsd_codes(ds[0], 7, D)
    ref = oracle.linear_backward(codes, D, Xs[0], np.zeros((12, 10)))["dW"]
    np.testing.assert_array_equal(oracle.distributed_weight_gradient(ds, Xs, 3.0, [7]), ref)


def _error_power(ds, Xs, trials, seed0):
    N = len(ds)
    exact = _exact(ds, Xs)
    errs = np.stack([oracle.distributed_weight_gradient(ds, Xs, 3.0, [seed0 + 1000 * t + i for i in range(N)]) - exact
                     for t in range(trials)])
    return errs.mean(axis=0), (errs ** 2).mean(axis=0).sum()


def test_unbiased_and_variance_falls_like_one_over_n():
    """Independent dithers: the error power of the average is the sum of the nodes' own error powers over N^2,
    i.e. 1/N of their mean. Every power is a Monte-Carlo estimate over 300 dither draws."""
    for N in (4, 16):
        ds, Xs = _nodes(N)
        bias, p = _error_power(ds, Xs, 300, seed0=17 * N)
        # the mean error over the trials is noise of total size sqrt(p / trials)
        assert np.linalg.norm(bias) <= 4.0 * np.sqrt(p / 300)
        own = [_error_power(ds[i:i + 1], Xs[i:i + 1], 300, seed0=5000 + 7 * i)[1] for i in range(N)]
        predicted = sum(own) / N ** 2
        assert 0.8 <= p / predicted <= 1.25, (N, p, predicted)
        assert p < np.mean(own) / (0.7 * N)
