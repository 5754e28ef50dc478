"""Stride-2 convolution layers (3x3 and 1x1, the down-sampling layers of residual networks) against the CPU
oracle's strided definitions: codes bit-exact, dW / dX / db within the same bars as the stride-1 layers
(relative Frobenius error <= 1e-5 and |err| <= 1e-5 * sum|terms| per element)."""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    import paper_2004_04729_b200 as dbp
    c = dbp.Context(0)
    yield c
    c.close()


def _dev(a, dtype):
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()
    return t.to(torch.bfloat16) if dtype == "bf16" else t


def _check(out, ref, tol, keys=("dW", "dX", "db")):
    for key in keys:
        got = out[key].double().cpu().numpy()
        assert got.shape == ref[key].shape
        fro = np.linalg.norm(got - ref[key]) / max(np.linalg.norm(ref[key]), 1e-300)
        assert fro <= tol, (key, fro)
        bound = tol * ref["S_" + key] + 1e-30
        assert np.all(np.abs(got - ref[key]) <= bound), (key, float((np.abs(got - ref[key]) / bound).max()))


def _run(ctx, L, tol, flags=0):
    import paper_2004_04729_b200 as dbp
    d, X, W = (_dev(a, L.dtype) for a in (L.delta, L.X, L.W))
    q = dbp.SparseGradient(d.numel())
    out = dbp.dithered_conv_backward(ctx, d, X, W, L.seed, L.scale, q_out=q, need_db=True, stride=2,
                                     flags=flags | dbp.DBP_DX_F32)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == (0, 0)
    D = np.float32(q.delta.item())
    assert abs(float(D) - L.scale * oracle.mean_std(L.delta)[1]) <= 1e-6 * float(D)
    codes, nnz, _ = oracle.nsd_codes(L.delta, L.seed, D)
    assert np.array_equal(dbp.nsd_decode_dense(ctx, q).cpu().numpy().reshape(codes.shape), codes)
    assert int(q.nnz.item()) == nnz
    ref = oracle.conv_backward_strided(codes, D, L.X, L.W, 2, with_abs=True)
    _check(out, ref, tol)
    return out, codes, D


@pytest.mark.parametrize("B,Ci,Co,H,W,k", [
    (2, 16, 24, 8, 8, 3),        # the smallest planes: 4x4 outputs
    (2, 64, 64, 16, 16, 3),
    (3, 32, 40, 12, 20, 3),      # rectangular, channel counts that fill no tile
    (1, 128, 128, 56, 56, 3),    # ResNet stage-2 down-sampling 3x3
    (2, 256, 256, 28, 28, 3),
    (2, 512, 512, 14, 14, 3),    # 7x7 outputs
    (2, 128, 64, 20, 20, 3),     # whole channel tiles per phase, one 64-channel code panel
    (3, 384, 192, 8, 12, 3),     # three channel tiles per phase, ragged output-channel tile
    (2, 3, 8, 10, 6, 3),         # 12 phase channels: off the tensor-core kernels
    (2, 64, 128, 16, 16, 1),
    (1, 256, 512, 56, 56, 1),    # ResNet stage-2 shortcut projection
    (3, 512, 1024, 28, 28, 1),
    (2, 1024, 2048, 14, 14, 1),
    (2, 24, 40, 6, 10, 1),
])
def test_stride2_bf16(ctx, B, Ci, Co, H, W, k):
    L = wl.conv_layer(B, Ci, Co, H, W, k, data_seed=7 * B + Ci + Co + H, scale=5.0, dtype="bf16", stride=2)
    _run(ctx, L, 1e-5)


@pytest.mark.parametrize("B,Ci,Co,H,W,k", [
    (2, 16, 16, 8, 8, 3),
    (2, 64, 64, 32, 32, 3),
    (3, 24, 40, 12, 20, 3),
    (2, 128, 64, 16, 16, 3),     # whole channel tiles per phase (the kernels skip the taps that are zero by construction)
    (1, 128, 128, 24, 24, 3),
    (4, 128, 128, 8, 8, 3),      # 4x4 outputs: images stacked for the weight gradient
    (2, 3, 8, 10, 6, 3),
    (2, 64, 128, 16, 16, 1),
    (2, 20, 12, 6, 10, 1),
])
def test_stride2_fp32(ctx, B, Ci, Co, H, W, k):
    L = wl.conv_layer(B, Ci, Co, H, W, k, data_seed=11 * B + Ci + Co + H, scale=2.0, dtype="f32", stride=2)
    _run(ctx, L, 1e-5)


def test_stride2_bf16_outputs_and_single_products(ctx):
    """bf16 dX (the default) rounds the fp32 result once; each product alone equals the pair."""
    import paper_2004_04729_b200 as dbp
    L = wl.conv_layer(2, 64, 64, 16, 16, 3, data_seed=99, scale=5.0, dtype="bf16", stride=2)
    d, X, W = (_dev(a, "bf16") for a in (L.delta, L.X, L.W))
    both = dbp.dithered_conv_backward(ctx, d, X, W, 3, 5.0, stride=2, flags=dbp.DBP_DX_F32)
    lo = dbp.dithered_conv_backward(ctx, d, X, W, 3, 5.0, stride=2)
    assert lo["dX"].dtype == torch.bfloat16 and lo["dX"].shape == X.shape
    assert torch.equal(lo["dX"], both["dX"].to(torch.bfloat16))
    only_w = dbp.dithered_conv_backward(ctx, d, X, W, 3, 5.0, stride=2, need_dX=False)
    only_x = dbp.dithered_conv_backward(ctx, d, X, W, 3, 5.0, stride=2, need_dW=False, flags=dbp.DBP_DX_F32)
    assert only_w["dX"] is None and only_x["dW"] is None
    fro = lambda a, b: float((a.double() - b.double()).norm() / b.double().norm())
    assert fro(only_w["dW"], both["dW"]) <= 1e-5 and fro(only_x["dX"], both["dX"]) <= 1e-5
    # the asynchronous-dW flag is accepted and changes nothing
    again = dbp.dithered_conv_backward(ctx, d, X, W, 3, 5.0, stride=2, flags=dbp.DBP_DX_F32 | dbp.DBP_DW_ASYNC)
    ctx.join()
    assert torch.equal(again["dX"], both["dX"]) and fro(again["dW"], both["dW"]) <= 1e-5


def test_stride2_pointwise_layer_is_zero_off_the_even_positions(ctx):
    import paper_2004_04729_b200 as dbp
    L = wl.conv_layer(2, 32, 48, 12, 12, 1, data_seed=5, scale=5.0, dtype="bf16", stride=2)
    d, X, W = (_dev(a, "bf16") for a in (L.delta, L.X, L.W))
    out = dbp.dithered_conv_backward(ctx, d, X, W, 0, 5.0, stride=2)
    dX = out["dX"].float()
    assert not dX[:, :, 1::2, :].any() and not dX[:, :, :, 1::2].any() and dX[:, :, ::2, ::2].any()


def test_stride2_host_entry_point(ctx):
    import paper_2004_04729_b200 as dbp
    L = wl.conv_layer(2, 32, 32, 16, 16, 3, data_seed=21, scale=2.0, dtype="f32", stride=2)
    d, X, W = (torch.from_numpy(a).pin_memory() for a in (L.delta, L.X, L.W))
    dW = torch.empty(L.W.shape, dtype=torch.float32).pin_memory()
    dX = torch.empty(L.X.shape, dtype=torch.float32).pin_memory()
    db = torch.empty(32, dtype=torch.float32).pin_memory()
    D, nnz = dbp.dithered_conv_backward_host(ctx, d, X, W, 4, 2.0, dW, dX, db, stride=2)
    codes, nnz_ref, _ = oracle.nsd_codes(L.delta, 4, np.float32(D))
    assert nnz == nnz_ref
    ref = oracle.conv_backward_strided(codes, np.float32(D), L.X, L.W, 2, with_abs=True)
    _check({"dW": dW, "dX": dX, "db": db}, ref, 1e-5)


def test_stride2_with_relu_mask(ctx):
    """The ReLU derivative set for the call applies to delta (the layer's own output positions)."""
    import paper_2004_04729_b200 as dbp
    L = wl.conv_layer(2, 32, 32, 16, 16, 3, data_seed=31, scale=2.0, dtype="f32", stride=2)
    r = np.random.default_rng(3)
    mask = (r.random(L.delta.shape) < 0.6).astype(np.uint8)
    d, X, W = (_dev(a, "f32") for a in (L.delta, L.X, L.W))
    ctx.set_relu_mask(torch.from_numpy(mask).cuda())
    got = dbp.dithered_conv_backward(ctx, d, X, W, 9, 2.0, stride=2)
    want = dbp.dithered_conv_backward(ctx, _dev(L.delta * mask, "f32"), X, W, 9, 2.0, stride=2)
    assert torch.equal(got["dX"], want["dX"])
    assert float((got["dW"].double() - want["dW"].double()).norm() / want["dW"].double().norm()) <= 1e-5


def test_stride2_rejects_what_it_cannot_do(ctx):
    import paper_2004_04729_b200 as dbp
    d = torch.zeros(1, 8, 3, 4, device="cuda")
    X = torch.zeros(1, 8, 7, 8, device="cuda")       # odd height
    W = torch.zeros(8, 8, 3, 3, device="cuda")
    with pytest.raises(ValueError):
        dbp.dithered_conv_backward(ctx, d, X, W, 0, 2.0, stride=2)
    lib = dbp.binding.load_library()
    rc = lib.dithered_conv_backward(ctx._h, d.data_ptr(), X.data_ptr(), W.data_ptr(), dbp.binding._dtype_code(d),
                                    1, 8, 8, 7, 8, 3, 2, 1, 0, 2.0, None, None, None, None, None, 0)
    assert rc == -2
    rc = lib.dithered_conv_backward(ctx._h, d.data_ptr(), X.data_ptr(), W.data_ptr(), dbp.binding._dtype_code(d),
                                    1, 8, 8, 6, 8, 3, 3, 1, 0, 2.0, None, None, None, None, None, 0)
    assert rc == -2


def test_stride2_leaves_the_weight_gradient_scratch_clean(ctx):
    """A strided 3x3 layer and a plain one share the weight-gradient scratch: whatever one leaves there would show
    up in the other's dW. Alternate them (both widths of the code operand) and compare with each layer run alone."""
    import paper_2004_04729_b200 as dbp
    fro = lambda a, b: float((a.double() - b.double()).norm() / b.double().norm())
    for co in (64, 128):
        S = wl.conv_layer(2, 128, co, 16, 16, 3, data_seed=41 + co, scale=5.0, dtype="bf16", stride=2)
        P = wl.conv_layer(2, 512, co, 8, 8, 3, data_seed=43 + co, scale=5.0, dtype="bf16")
        s_in = [_dev(a, "bf16") for a in (S.delta, S.X, S.W)]
        p_in = [_dev(a, "bf16") for a in (P.delta, P.X, P.W)]
        plain_alone = dbp.dithered_conv_backward(ctx, *p_in, 1, 5.0)["dW"].clone()
        strided_alone = dbp.dithered_conv_backward(ctx, *s_in, 1, 5.0, stride=2)["dW"].clone()
        for _ in range(2):
            a = dbp.dithered_conv_backward(ctx, *s_in, 1, 5.0, stride=2)["dW"]
            b = dbp.dithered_conv_backward(ctx, *p_in, 1, 5.0)["dW"]
            assert fro(a, strided_alone) <= 1e-5 and fro(b, plain_alone) <= 1e-5


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_stride2_with_a_given_step_size(ctx, dtype):
    """scale <= 0 and a device step size: no statistics kernel runs, so the weights take the other route."""
    import paper_2004_04729_b200 as dbp
    L = wl.conv_layer(2, 128, 64, 16, 16, 3, data_seed=51, scale=2.0, dtype=dtype, stride=2)
    d, X, W = (_dev(a, dtype) for a in (L.delta, L.X, L.W))
    D = np.float32(2.0 * oracle.mean_std(L.delta)[1])
    step = torch.tensor([float(D)], dtype=torch.float32, device="cuda")
    out = dbp.dithered_conv_backward(ctx, d, X, W, 6, 0.0, delta_in=step, need_db=True, stride=2, flags=dbp.DBP_DX_F32)
    torch.cuda.synchronize()
    codes, _, _ = oracle.nsd_codes(L.delta, 6, D)
    _check(out, oracle.conv_backward_strided(codes, D, L.X, L.W, 2, with_abs=True), 1e-5)


@pytest.mark.parametrize("B,Ci,Co,H,W,dtype", [
    (4, 1, 6, 32, 32, "f32"),        # LeNet-5 C1 (same padding)
    (4, 6, 16, 14, 14, "f32"),       # LeNet-5 C3
    (2, 3, 64, 32, 32, "f32"),       # an AlexNet-for-CIFAR first layer
    (2, 64, 192, 8, 8, "f32"),
    (3, 10, 7, 5, 9, "f32"),         # planes smaller than the kernel's reach in one direction
    (2, 16, 24, 12, 12, "bf16"),
    (1, 128, 40, 7, 7, "bf16"),
])
def test_5x5_layers(ctx, B, Ci, Co, H, W, dtype):
    """5x5 kernels (stride 1, padding 2) against the oracle's definition: codes bit-exact, products within 1e-5."""
    import paper_2004_04729_b200 as dbp
    L = wl.conv_layer(B, Ci, Co, H, W, 5, data_seed=3 * B + Ci + Co, scale=2.0, dtype=dtype)
    d, X, W_ = (_dev(a, dtype) for a in (L.delta, L.X, L.W))
    q = dbp.SparseGradient(d.numel())
    out = dbp.dithered_conv_backward(ctx, d, X, W_, 8, 2.0, q_out=q, need_db=True, flags=dbp.DBP_DX_F32)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == (0, 0)
    D = np.float32(q.delta.item())
    codes, nnz, _ = oracle.nsd_codes(L.delta, 8, D)
    assert np.array_equal(dbp.nsd_decode_dense(ctx, q).cpu().numpy().reshape(codes.shape), codes)
    _check(out, oracle.conv_backward(codes, D, L.X, L.W, with_abs=True), 1e-5)
    with pytest.raises(dbp.DbpError):
        dbp.dithered_conv_backward(ctx, d, X, W_, 8, 2.0, flags=dbp.DBP_FORCE_DENSE)
