"""The two-launch backward pass of small fp32 linear layers (no caller's sparse structure) against the CPU
oracle: step size to 1e-6, the number of non-zero codes exactly (the oracle quantizes with the CUDA path's
step size), dW, dX, db to 1e-5 (relative Frobenius and |err| <= 1e-5 sum|terms|). The codes themselves never
leave the kernel; a wrong code shows in nnz and in the products."""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl

pytestmark = pytest.mark.gpu
TOL = 1e-5


@pytest.fixture(scope="module")
def ctx():
    import paper_2004_04729_b200 as dbp
    c = dbp.Context(0)
    yield c
    c.close()


def _cu(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def _check_products(out, ref, keys):
    for key in keys:
        got = out[key].double().cpu().numpy()
        fro = np.linalg.norm(got - ref[key]) / max(np.linalg.norm(ref[key]), 1e-300)
        assert fro <= TOL, (key, fro)
        bound = TOL * ref["S_" + key] + 1e-30
        assert np.all(np.abs(got - ref[key]) <= bound), (key, float((np.abs(got - ref[key]) / bound).max()))


def _fused_was_used(ctx, fn):
    ctx.profile_enable(True)
    ctx.profile_select(None)
    ctx.profile_read()
    out = fn()
    torch.cuda.synchronize()
    pr = ctx.profile_read()
    ctx.profile_enable(False)
    assert pr["fused"][1] == 1 and pr["statistics"][1] == 0 and pr["dx"][1] == 0 and pr["dw"][1] == 0, pr
    return out


@pytest.mark.parametrize("B,N,K", [
    (128, 300, 784),     # config 1
    (256, 100, 300),     # LeNet-300-100, second layer
    (256, 10, 100),      # rows of 10 codes: nothing is 16-byte aligned along N
    (128, 10, 512),      # the VGG classifier
    (33, 7, 50),         # ragged everywhere, K % 4 != 0: element-wise accesses along K
    (1, 1, 1),
    (70, 129, 65),       # one past a tile in every direction
])
def test_small_linear_matches_the_oracle(ctx, B, N, K):
    import paper_2004_04729_b200 as dbp
    L = wl.linear_layer(B, N, K, data_seed=500 + B + N + K, scale=2.0, seed=7)
    d, X, W = _cu(L.delta), _cu(L.X), _cu(L.W)
    out = _fused_was_used(ctx, lambda: dbp.dithered_linear_backward(ctx, d, X, W, L.seed, L.scale, need_db=True))
    assert ctx.last_device_status() == (0, 0)
    D, nnz = ctx.last_step()
    D = np.float32(D)
    want = oracle.step_size(L.delta, L.scale)
    assert abs(float(D) - float(want)) <= 1e-6 * float(want) + 1e-45
    codes, onnz, _ = oracle.nsd_codes(L.delta, L.seed, D)
    assert nnz == onnz
    _check_products(out, oracle.linear_backward(codes, D, L.X, L.W, with_abs=True), ("dW", "dX", "db"))


def test_small_linear_one_product_and_given_step(ctx):
    """dW alone (its tiles count the codes), dX alone, and a step size passed in instead of computed."""
    import paper_2004_04729_b200 as dbp
    L = wl.linear_layer(96, 40, 72, data_seed=611, scale=3.0, seed=11)
    d, X, W = _cu(L.delta), _cu(L.X), _cu(L.W)
    D = oracle.step_size(L.delta, L.scale)
    codes, onnz, _ = oracle.nsd_codes(L.delta, L.seed, D)
    ref = oracle.linear_backward(codes, D, L.X, L.W, with_abs=True)
    din = torch.tensor([float(D)], dtype=torch.float32, device="cuda")
    for kw, keys in ((dict(need_dX=False, need_db=True), ("dW", "db")), (dict(need_dW=False), ("dX",)), ({}, ("dW", "dX"))):
        out = _fused_was_used(ctx, lambda: dbp.dithered_linear_backward(ctx, d, X, W, L.seed, 0.0, delta_in=din, **kw))
        got_D, nnz = ctx.last_step()
        assert np.float32(got_D) == D and nnz == onnz
        _check_products(out, ref, keys)


def test_small_linear_degenerate_inputs(ctx):
    """sigma = 0: step size 0, no non-zero code, zero gradients, no error. NaN in delta_z: reported, gradients zero.
    Values far outside +-127 steps: clipped and counted."""
    import paper_2004_04729_b200 as dbp
    X, W = _cu(np.random.default_rng(1).random((16, 24))), _cu(np.random.default_rng(2).standard_normal((12, 24)))
    d = torch.full((16, 12), 0.1, dtype=torch.float32, device="cuda")
    out = dbp.dithered_linear_backward(ctx, d, X, W, 0, 2.0, need_db=True)
    assert ctx.last_step() == (0.0, 0) and ctx.last_device_status() == (0, 0)
    assert all(float(out[k].abs().max()) == 0.0 for k in ("dW", "dX", "db"))
    d2 = d.clone()
    d2[3, 4] = float("nan")
    out = dbp.dithered_linear_backward(ctx, d2, X, W, 0, 2.0)
    st, _ = ctx.last_device_status()
    assert st == -5 and float(out["dW"].abs().max()) == 0.0 and float(out["dX"].abs().max()) == 0.0
    rng = np.random.default_rng(3)
    x = rng.standard_normal((16, 12)).astype(np.float32)
    x[5, 5] = 1e4
    din = torch.tensor([1.0], dtype=torch.float32, device="cuda")
    out = dbp.dithered_linear_backward(ctx, _cu(x), X, W, 9, 0.0, delta_in=din)
    st, nsat = ctx.last_device_status()
    assert st == -6 and nsat == 1
    codes, _, osat = oracle.nsd_codes(x, 9, np.float32(1.0))
    assert osat == 1 and codes[5, 5] == 127
    _check_products(out, oracle.linear_backward(codes, np.float32(1.0), X.cpu().numpy(), W.cpu().numpy(), with_abs=True), ("dW", "dX"))


def test_larger_layers_and_a_callers_structure_take_the_general_path(ctx):
    import paper_2004_04729_b200 as dbp
    L = wl.linear_layer(64, 32, 48, data_seed=77, scale=2.0)
    d, X, W = _cu(L.delta), _cu(L.X), _cu(L.W)
    ctx.profile_enable(True)
    ctx.profile_select(None)
    ctx.profile_read()
    dbp.dithered_linear_backward(ctx, d, X, W, L.seed, L.scale, q_out=dbp.SparseGradient(d.numel()))
    dbp.dithered_linear_backward(ctx, d, X, W, L.seed, L.scale, flags=dbp.DBP_FORCE_SPARSE)
    torch.cuda.synchronize()
    pr = ctx.profile_read()
    ctx.profile_enable(False)
    assert pr["fused"][1] == 0 and pr["statistics"][1] == 2


def test_relu_mask_folded_into_the_call(ctx):
    """dbp_set_relu_mask: the next call quantizes delta_a (.) mask. A small linear layer applies the mask while it
    reads delta_a; a convolution runs the ReLU-derivative kernel first. Either way the results are those of the
    call on delta_z = delta_a (.) mask, and the setting lasts for one call."""
    import paper_2004_04729_b200 as dbp
    rng = np.random.default_rng(12)
    L = wl.linear_layer(96, 52, 136, data_seed=901, scale=2.0, seed=3)
    mask = (rng.random(L.delta.shape) < 0.6).astype(np.uint8)
    dz = (L.delta * mask).astype(np.float32)
    d, X, W, m = _cu(L.delta), _cu(L.X), _cu(L.W), torch.from_numpy(mask).cuda()
    ctx.set_relu_mask(m)
    out = _fused_was_used(ctx, lambda: dbp.dithered_linear_backward(ctx, d, X, W, L.seed, L.scale, need_db=True))
    D, nnz = ctx.last_step()
    D = np.float32(D)
    want = oracle.step_size(dz, L.scale)
    assert abs(float(D) - float(want)) <= 1e-6 * float(want)
    codes, onnz, _ = oracle.nsd_codes(dz, L.seed, D)
    assert nnz == onnz
    _check_products(out, oracle.linear_backward(codes, D, L.X, L.W, with_abs=True), ("dW", "dX", "db"))
    # consumed: the same call again quantizes delta itself
    dbp.dithered_linear_backward(ctx, d, X, W, L.seed, L.scale)
    _, nnz2 = ctx.last_step()
    assert nnz2 == oracle.nsd_codes(L.delta, L.seed, np.float32(ctx.last_step()[0]))[1] and nnz2 != nnz
    # convolutions: bit-identical to the two-step form. fp32 3x3 layers on the tensor-core kernels apply the mask
    # in the statistics kernel and in the quantizer (planes of 64 positions and more, tiny planes with stacked
    # images, odd plane sizes); a 1x1 layer runs the ReLU-derivative kernel first.
    for (B, Ci, Co, H, W, k) in ((4, 16, 24, 8, 8, 3), (32, 16, 16, 4, 4, 3), (3, 8, 8, 5, 7, 3), (2, 8, 16, 9, 9, 3), (4, 16, 8, 6, 6, 1)):
        C = wl.conv_layer(B, Ci, Co, H, W, k, data_seed=902 + H, scale=2.0)
        cm = (rng.random(C.delta.shape) < 0.5).astype(np.uint8)
        cd, cX, cW, cmask = _cu(C.delta), _cu(C.X), _cu(C.W), torch.from_numpy(cm).cuda()
        ref = dbp.dithered_conv_backward(ctx, dbp.relu_backward(ctx, cd, cmask), cX, cW, C.seed, C.scale, need_db=True)
        ref_step = ctx.last_step()
        ctx.set_relu_mask(cmask)
        got = dbp.dithered_conv_backward(ctx, cd, cX, cW, C.seed, C.scale, need_db=True)
        assert ctx.last_step() == ref_step, (B, Ci, Co, H, W, k)
        assert torch.equal(got["dX"], ref["dX"]) and torch.equal(got["db"], ref["db"])
        assert (got["dW"] - ref["dW"]).abs().max().item() <= 1e-5 * ref["dW"].abs().max().item()
    # the oracle on delta_z for one of them
    dz = (C.delta * cm).astype(np.float32)
    D = np.float32(ref_step[0])
    codes, onnz, _ = oracle.nsd_codes(dz, C.seed, D)
    assert onnz == ref_step[1]


@pytest.mark.parametrize("net", ["mlp", "vgg"])
def test_network_backward_without_delta_z_matches_the_step_by_step_form(ctx, net):
    """LeNet-300-100 and VGG-16 chains: with nobody asking for delta_z or the sparse structure the masks are folded
    into the calls; the gradients are those of the step-by-step form (dW to the tolerance: other kernels add in
    another order; everything else is bit for bit the same)."""
    import paper_2004_04729_b200 as dbp
    c = wl.mlp_chain(batch=64) if net == "mlp" else wl.vgg_chain(batch=8, device="cuda")
    cu = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).cuda()
    Xs, Ws = [cu(a) for a in c.X], [cu(a) for a in c.W]
    masks = [None if mk is None else cu(mk.astype(np.uint8)) for mk in c.relu_mask]
    pools = [cu(a) for a in c.pool_argmax]
    dout = cu(c.delta_out)
    ref = dbp.network_backward(ctx, c.kinds, Xs, Ws, masks, pools, dout, c.scale, 0, keep_delta_z=True)
    got = dbp.network_backward(ctx, c.kinds, Xs, Ws, masks, pools, dout, c.scale, 0, with_sparse=False)
    torch.cuda.synchronize()
    for a, b in zip(ref, got):
        num = (a["dW"] - b["dW"]).norm().item()
        assert num <= 2e-5 * a["dW"].norm().item(), (net, num / a["dW"].norm().item())


def test_relu_mask_corner_cases(ctx):
    """A mask that does not start on a 4-byte boundary takes the form with a separate ReLU-derivative pass (same
    results); bf16 tensors refuse a mask, and the refused call still consumes it."""
    import paper_2004_04729_b200 as dbp
    rng = np.random.default_rng(5)
    L = wl.linear_layer(40, 24, 56, data_seed=950, scale=2.0, seed=1)
    mask = (rng.random(L.delta.shape) < 0.5).astype(np.uint8)
    d, X, W = _cu(L.delta), _cu(L.X), _cu(L.W)
    store = torch.zeros(mask.size + 1, dtype=torch.uint8, device="cuda")
    store[1:] = torch.from_numpy(mask.ravel()).cuda()
    odd = store[1:].view(mask.shape)                     # one byte past an aligned address
    assert odd.data_ptr() % 4 == 1 and odd.is_contiguous()
    ctx.set_relu_mask(torch.from_numpy(mask).cuda())
    ref = dbp.dithered_linear_backward(ctx, d, X, W, L.seed, L.scale)
    ref_step = ctx.last_step()
    ctx.set_relu_mask(odd)
    got = dbp.dithered_linear_backward(ctx, d, X, W, L.seed, L.scale)
    assert ctx.last_step() == ref_step
    assert torch.equal(got["dX"], ref["dX"]) and torch.equal(got["dW"], ref["dW"])
    db16, X16, W16 = (t.to(torch.bfloat16) for t in (d, X, W))
    ctx.set_relu_mask(odd)
    with pytest.raises(dbp.DbpError):
        dbp.dithered_linear_backward(ctx, db16, X16, W16, L.seed, L.scale)
    out = dbp.dithered_linear_backward(ctx, db16, X16, W16, L.seed, L.scale)     # the mask is gone
    torch.cuda.synchronize()
    assert out["dW"].isfinite().all()
