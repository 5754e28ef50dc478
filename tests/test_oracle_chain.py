"""Pins for the whole-network backward oracle and for the input generators."""
import numpy as np
import torch

import oracle
import workloads as wl


def test_maxpool_backward_matches_library():
    r = np.random.default_rng(0)
    a = torch.tensor(r.normal(size=(2, 3, 4, 6)), requires_grad=True)   # no ties
    y = torch.nn.functional.max_pool2d(a, 2)
    g = torch.tensor(r.normal(size=tuple(y.shape)))
    y.backward(g)
    win = a.detach().reshape(2, 3, 2, 2, 3, 2).permute(0, 1, 2, 4, 3, 5).reshape(2, 3, 2, 3, 4)
    am = win.argmax(-1).numpy()
    np.testing.assert_array_equal(oracle.maxpool2x2_backward(g.numpy(), am), a.grad.numpy())


def test_relu_backward_is_mask_product():
    d = np.array([1.5, -2.0, 3.0], dtype=np.float32)
    np.testing.assert_array_equal(oracle.relu_backward(d, np.array([True, False, True])),
                                  np.array([1.5, 0.0, 3.0], dtype=np.float32))
    assert oracle.relu_backward(d, None) is not None


def test_chain_composes_layers_by_hand():
    """Two linear layers: the chain equals NSD + products applied by hand, and the lower
    layer's gradient comes from the QUANTIZED upper gradient (Eq. (qda))."""
    c = wl.mlp_chain(batch=16, dims=(12, 9, 5), data_seed=5)
    res = oracle.chain_backward(c.kinds, c.X, c.W, c.relu_mask, c.pool_argmax, c.delta_out, 2.0, 3)
    s1, s0 = oracle.derive_layer_seed(3, 1), oracle.derive_layer_seed(3, 0)
    D1 = oracle.step_size(c.delta_out, 2.0)
    q1, _, _ = oracle.nsd_codes(c.delta_out, s1, D1)
    top = oracle.linear_backward(q1, D1, c.X[1], c.W[1])
    np.testing.assert_array_equal(res[1]["codes"], q1)
    np.testing.assert_allclose(res[1]["dW"], top["dW"], atol=0)
    dz0 = (top["dX"].astype(np.float32) * c.relu_mask[0]).astype(np.float32)
    np.testing.assert_array_equal(res[0]["delta_z"], dz0)
    D0 = oracle.step_size(dz0, 2.0)
    q0, _, _ = oracle.nsd_codes(dz0, s0, D0)
    np.testing.assert_array_equal(res[0]["codes"], q0)
    np.testing.assert_allclose(res[0]["dW"], oracle.linear_backward(q0, D0, c.X[0], c.W[0])["dW"], atol=0)
    # dense (unquantized) gradient differs: the chain is not using delta_z for dX
    dense_dx = c.delta_out.astype(np.float64) @ c.W[1].astype(np.float64)
    assert np.abs(dense_dx - top["dX"]).max() > 0


def test_chain_feed_and_conv_pool_shapes():
    c = wl.vgg_chain(batch=2, cfg=[4, "M", 6, 6, "M"], hw=8, data_seed=9)
    res = oracle.chain_backward(c.kinds, c.X, c.W, c.relu_mask, c.pool_argmax, c.delta_out, 2.0, 0)
    assert [r["dW"].shape for r in res] == [w.shape for w in c.W]
    assert [r["delta_z"].shape for r in res[:-1]] == [m.shape for m in c.relu_mask[:-1]]
    feed = [r["delta_z"] for r in res]
    again = oracle.chain_backward(c.kinds, c.X, c.W, c.relu_mask, c.pool_argmax, c.delta_out,
                                  2.0, 0, delta_z_feed=feed)
    for a, b in zip(res, again):
        np.testing.assert_array_equal(a["codes"], b["codes"])
    # masked positions carry no gradient and therefore no code
    assert not res[1]["codes"][~c.relu_mask[1]].any()


def test_generators_are_seeded_and_distributed_as_stated():
    a, b = wl.config3(batch=2), wl.config3(batch=2)
    assert np.array_equal(a.delta, b.delta) and np.array_equal(a.X, b.X) and np.array_equal(a.W, b.W)
    assert abs((a.X == 0).mean() - 0.5) < 0.01 and a.X.min() >= 0
    assert abs(a.W.std() - (2 / 576) ** 0.5) / (2 / 576) ** 0.5 < 0.02
    assert abs((a.delta == 0).mean() - 0.5) < 0.01
    assert abs(a.delta.std() - 1e-4) / 1e-4 < 0.02          # b sqrt(2p) with p = 1/2
    n = wl.normal(1, 1, 200000)
    assert abs(n.mean()) < 0.01 and abs(n.std() - 1) < 0.01
    l = wl.laplace(1, 2, 200000, 2.0)
    assert abs(np.abs(l).mean() - 2.0) < 0.03                # E|x| = b
    assert len(wl.RESNET50_SET) == 16
    L5 = wl.config5_layer(15, batch=1)
    assert L5.delta.shape == (1, 2048, 7, 7) and L5.dtype == "bf16"


def test_bf16_helpers_match_library_rounding():
    x = np.random.default_rng(0).normal(size=4096).astype(np.float32)
    bits = wl.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16)
    assert np.array_equal(bits.view(np.int16), ref.view(torch.int16).numpy())
    assert np.array_equal(wl.bf16_bits_to_f32(bits), ref.float().numpy())
