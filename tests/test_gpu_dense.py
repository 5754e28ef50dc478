"""The dense tensor-core path (bf16 linear / 1x1 layers) against the CPU oracle, and the
density crossover that chooses between it and the sparse kernels. Same bars as the sparse
path: codes bit-exact, dW and dX within 1e-5 (relative Frobenius and |err| <= 1e-5 sum|terms|);
products of bf16 values are exact in fp32, only the accumulation order differs."""
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


def _t(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda().to(torch.bfloat16)


def _f32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def _run(ctx, L, flags):
    import paper_2004_04729_b200 as dbp
    cast = _t if L.dtype == "bf16" else _f32
    d, X, W = cast(L.delta), cast(L.X), cast(L.W)
    q = dbp.SparseGradient(d.numel())
    fn = dbp.dithered_linear_backward if L.kind == "linear" else dbp.dithered_conv_backward
    out = fn(ctx, d, X, W, L.seed, L.scale, q_out=q, need_db=True, flags=flags | dbp.DBP_DX_F32)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == (0, 0)
    D = np.float32(q.delta.item())
    codes, nnz, _ = oracle.nsd_codes(L.delta, L.seed, D)
    assert np.array_equal(dbp.nsd_decode_dense(ctx, q).cpu().numpy().reshape(codes.shape), codes)
    ofn = oracle.linear_backward if L.kind == "linear" else oracle.conv_backward
    ref = ofn(codes, D, L.X, L.W, with_abs=True)
    for key in ("dW", "dX", "db"):
        got = out[key].double().cpu().numpy()
        fro = np.linalg.norm(got - ref[key]) / max(np.linalg.norm(ref[key]), 1e-300)
        assert fro <= TOL, (key, fro)
        bound = TOL * ref["S_" + key] + 1e-30
        assert np.all(np.abs(got - ref[key]) <= bound), (key, float((np.abs(got - ref[key]) / bound).max()))
    return out


@pytest.mark.parametrize("B,Ci,Co,H,W", [
    (2, 64, 64, 16, 16),      # one k-stage, narrow N tile
    (1, 256, 64, 56, 56),     # ResNet stage-1 reduce, positions % 8 == 0
    (2, 64, 256, 28, 28),     # expand: K = 256 output channels over four stages for dX
    (3, 512, 128, 14, 14),    # 196 positions per image: 4-element groups
    (5, 128, 512, 7, 7),      # 49 positions per image: element-wise loads, ragged row tiles
    (2, 72, 40, 5, 9),        # channel counts that fill neither tile
    (1, 1024, 256, 14, 14),
    (3, 64, 64, 3, 3),        # slab staging, smallest plane (9 positions): 15 images per row tile
    (2, 136, 128, 8, 7),      # slab staging, 56 positions, ragged channel tile
    (4, 64, 192, 9, 7),       # slab staging, 63 positions
    (7, 2048, 512, 7, 7),     # ResNet stage-4 reduce at a small batch, rows end inside a tile
    (4, 72, 320, 8, 8),       # two accumulators with a ragged second one, input channels fill no 16-group
    (3, 264, 136, 12, 12),    # two input-channel tiles, the second nearly empty; 144 positions = 2.25 chunks
    (2, 512, 256, 16, 8),     # two full accumulators, two full input-channel tiles
])
def test_dense_path_conv1x1(ctx, B, Ci, Co, H, W):
    import paper_2004_04729_b200 as dbp
    L = wl.conv_layer(B, Ci, Co, H, W, 1, data_seed=B + Ci + Co, scale=5.0, dtype="bf16")
    _run(ctx, L, dbp.DBP_FORCE_DENSE)


@pytest.mark.parametrize("B,Ci,Co,H,W", [
    (2, 64, 64, 32, 32),      # config-3 shape at batch 2 (bf16)
    (1, 64, 64, 56, 56),      # ResNet stage 1: 25 position tiles per image, last one half full
    (2, 128, 128, 28, 28),
    (2, 256, 256, 14, 14),    # two accumulators per CTA for dX; 196 positions: unaligned rows
    (3, 512, 512, 7, 7),      # four accumulators; one ragged tile per image
    (1, 72, 40, 9, 11),       # channel counts that fill no tile, odd width
    (2, 16, 24, 3, 62),       # widest supported row
    (2, 8, 8, 1, 1),          # a single position: every tap but the centre is masked
    (2, 64, 192, 12, 12),     # row-shift dX kernel, 16-aligned planes, three stages
    (3, 200, 128, 6, 6),      # row-shift dX kernel, slabs of 36 positions, ragged channel tile
    (5, 64, 64, 5, 7),        # row-shift dX kernel, odd plane size: byte-aligned slabs
    (240, 512, 64, 8, 8),     # row-shift dX kernel, four accumulators per CTA
    (2, 64, 32, 6, 4),        # row-shift dW kernel: 24 positions, 16-byte activation copies with slab-staged codes
    (3, 136, 96, 20, 16),     # row-shift kernels: 320 positions = two segments per image, ragged channel tile
])
def test_dense_path_conv3x3(ctx, B, Ci, Co, H, W):
    import paper_2004_04729_b200 as dbp
    L = wl.conv_layer(B, Ci, Co, H, W, 3, data_seed=B + Ci + Co + H, scale=5.0 if Ci > 64 else 2.0, dtype="bf16")
    _run(ctx, L, dbp.DBP_FORCE_DENSE)


@pytest.mark.parametrize("B,Ci,Co,H,W", [
    (4, 64, 64, 32, 32),      # config-3 shape at batch 4: weights resident in shared memory (one ci block, 18 taps)
    (2, 128, 128, 16, 16),    # config-4 stage 2
    (2, 256, 256, 8, 8),      # two ci blocks: weights streamed
    (3, 512, 512, 4, 4),      # several images per patch
    (5, 512, 512, 2, 2),      # config-4 last stage: 4 positions per image
    (2, 72, 40, 9, 11),       # channel counts that fill no tile, odd width (element-wise staging)
    (2, 8, 16, 1, 1),         # a single position
    (32, 64, 64, 4, 4),       # tiny planes, dW on images stacked 16 to a tall image (two tall images)
    (128, 16, 24, 2, 2),      # 53 images of 6 rows each would be 318 rows: the largest divisor below is 32
    (12, 8, 8, 3, 5),         # odd plane sizes stacked (12 images of 20 positions)
    (7, 16, 16, 6, 6),        # a prime batch: 7 images in one tall image
    (9, 8, 16, 7, 8),         # 56 + 8 = 64 positions with the extra row: the largest plane that is stacked
])
def test_dense_path_conv3x3_fp32_operands(ctx, B, Ci, Co, H, W):
    """fp32 layers on the tensor cores: weights and activations enter as two bf16 pieces each (the sum of the
    pieces is within 2^-18 of the fp32 value, a code times a piece is exact), same bars as everywhere."""
    import paper_2004_04729_b200 as dbp
    L = wl.conv_layer(B, Ci, Co, H, W, 3, data_seed=B + Ci + Co + H, scale=2.0, dtype="f32")
    _run(ctx, L, dbp.DBP_FORCE_DENSE)


@pytest.mark.parametrize("B,Ci,Co,H,W", [(4, 3, 64, 32, 32), (2, 5, 16, 7, 9), (3, 12, 8, 4, 4)])
def test_dense_path_first_layer_dw_fp32(ctx, B, Ci, Co, H, W):
    """A network's first layer (few input channels, no dX wanted): the fp32 weight gradient alone runs on the
    tensor cores, the activations being padded to eight channels while they are split into bf16 pieces."""
    import paper_2004_04729_b200 as dbp
    L = wl.conv_layer(B, Ci, Co, H, W, 3, data_seed=5 + Ci, scale=2.0, dtype="f32")
    d, X, Wt = _f32(L.delta), _f32(L.X), _f32(L.W)
    q = dbp.SparseGradient(d.numel())
    out = dbp.dithered_conv_backward(ctx, d, X, Wt, L.seed, L.scale, q_out=q, need_dX=False, flags=dbp.DBP_FORCE_DENSE)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == (0, 0)
    D = np.float32(q.delta.item())
    codes, nnz, _ = oracle.nsd_codes(L.delta, L.seed, D)
    ref = oracle.conv_backward(codes, D, L.X, L.W, with_abs=True)
    got = out["dW"].double().cpu().numpy()
    assert np.linalg.norm(got - ref["dW"]) / np.linalg.norm(ref["dW"]) <= TOL
    assert np.all(np.abs(got - ref["dW"]) <= TOL * ref["S_dW"] + 1e-30)


@pytest.mark.parametrize("B,N,K", [(128, 300, 784), (256, 512, 2048), (70, 10, 512), (33, 100, 304)])
def test_dense_path_linear(ctx, B, N, K):
    import paper_2004_04729_b200 as dbp
    L = wl.linear_layer(B, N, K, data_seed=N + K, scale=2.0, dtype="bf16")
    if K % 8:
        pytest.skip("dense path needs Cin % 8 == 0")
    _run(ctx, L, dbp.DBP_FORCE_DENSE)


@pytest.mark.parametrize("B,Ci,Co,H,W,k", [
    (2, 64, 64, 16, 16, 3), (2, 128, 128, 14, 14, 3), (3, 64, 128, 7, 7, 3), (2, 64, 128, 28, 28, 1),
    (1, 256, 64, 56, 56, 1), (3, 512, 128, 14, 14, 1), (5, 128, 512, 7, 7, 1), (2, 72, 40, 5, 9, 1),
    (2, 64, 64, 9, 9, 1), (2, 136, 128, 8, 8, 1), (3, 40, 64, 10, 10, 1),
    (2, 64, 64, 28, 28, 3), (1, 64, 64, 56, 56, 3), (2, 72, 40, 9, 11, 3), (2, 16, 24, 3, 62, 3), (3, 136, 96, 20, 16, 3),
])
def test_dense_bf16_dx_is_the_rounded_f32_dx(ctx, B, Ci, Co, H, W, k):
    """The bf16 store path of dX rounds the same accumulators the fp32 store path writes."""
    import paper_2004_04729_b200 as dbp
    L = wl.conv_layer(B, Ci, Co, H, W, k, data_seed=7 + H, scale=5.0, dtype="bf16")
    d, X, W_ = _t(L.delta), _t(L.X), _t(L.W)
    a = dbp.dithered_conv_backward(ctx, d, X, W_, L.seed, L.scale, flags=dbp.DBP_FORCE_DENSE | dbp.DBP_DX_F32)
    b = dbp.dithered_conv_backward(ctx, d, X, W_, L.seed, L.scale, flags=dbp.DBP_FORCE_DENSE)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == (0, 0)
    assert b["dX"].dtype == torch.bfloat16 and a["dX"].dtype == torch.float32
    assert torch.equal(a["dX"].to(torch.bfloat16), b["dX"])


def test_dense_and_sparse_paths_agree_and_unsupported_is_refused(ctx):
    import paper_2004_04729_b200 as dbp
    L = wl.conv_layer(2, 128, 128, 14, 14, 1, data_seed=3, scale=5.0, dtype="bf16")
    a = _run(ctx, L, dbp.DBP_FORCE_DENSE)
    b = _run(ctx, L, dbp.DBP_FORCE_SPARSE)
    for key in ("dW", "dX"):
        ref = b[key].double()
        assert (a[key].double() - ref).norm() <= 2e-5 * ref.norm()
    L3 = wl.conv_layer(1, 12, 16, 6, 6, 3, data_seed=4, dtype="bf16")
    with pytest.raises(dbp.DbpError) as e:          # channel count not a multiple of 8
        dbp.dithered_conv_backward(ctx, _t(L3.delta), _t(L3.X), _t(L3.W), 0, 2.0, flags=dbp.DBP_FORCE_DENSE)
    assert e.value.status == -2
    Lf = wl.conv_layer(1, 16, 16, 6, 6, 1, data_seed=4)
    with pytest.raises(dbp.DbpError) as e:          # fp32 operands have no dense path
        dbp.dithered_conv_backward(ctx, torch.from_numpy(Lf.delta).cuda(), torch.from_numpy(Lf.X).cuda(),
                                   torch.from_numpy(Lf.W).cuda(), 0, 2.0, flags=dbp.DBP_FORCE_DENSE)
    assert e.value.status == -2


def test_crossover_uses_the_measured_density(ctx):
    """With crossover 0.5 a layer at ~10 % density switches to the sparse kernels once the
    first call's density has been read back; with crossover 0 it stays dense. Both paths give
    the same gradients, so only the kernel mix (profile counters) tells them apart."""
    import paper_2004_04729_b200 as dbp
    c2 = dbp.Context(0)
    L = wl.conv_layer(2, 64, 64, 16, 16, 1, data_seed=9, scale=5.0, dtype="bf16")
    d, X, W = _t(L.delta), _t(L.X), _t(L.W)
    c2.set_crossover(0.5)
    c2.profile_enable(True)
    dbp.dithered_conv_backward(c2, d, X, W, 0, 5.0)          # estimate starts at 1.0 -> dense
    torch.cuda.synchronize()
    first = c2.profile_read()
    assert first["weight_taps"][1] == 0
    dbp.dithered_conv_backward(c2, d, X, W, 0, 5.0)          # now ~0.1 < 0.5 -> sparse
    torch.cuda.synchronize()
    second = c2.profile_read()
    assert second["weight_taps"][1] == 1
    c2.set_crossover(0.0)
    dbp.dithered_conv_backward(c2, d, X, W, 0, 5.0)
    torch.cuda.synchronize()
    assert c2.profile_read()["weight_taps"][1] == 0
    c2.close()


def test_back_to_back_calls_are_ordered(ctx):
    """Two layers enqueued without a synchronisation in between, the second quantizing the dX of
    the first (Eq. (qda) feeds the layer below): the second call's kernels may become resident
    while the first call's are draining, but must not read dX before it is complete. Checked
    layer by layer against the oracle, the oracle reading the CUDA path's own dX."""
    import paper_2004_04729_b200 as dbp
    L2 = wl.conv_layer(4, 128, 256, 14, 14, 1, data_seed=21, scale=5.0, dtype="bf16")   # upper layer: 128 -> 256
    L1 = wl.conv_layer(4, 64, 128, 14, 14, 1, data_seed=22, scale=5.0, dtype="bf16")    # lower layer: 64 -> 128
    d2, X2, W2 = _t(L2.delta), _t(L2.X), _t(L2.W)
    X1, W1 = _t(L1.X), _t(L1.W)
    for rep in range(3):                                  # repeated: the workspaces are reused every time
        q2, q1 = dbp.SparseGradient(d2.numel()), dbp.SparseGradient(L1.delta.size)
        o2 = dbp.dithered_conv_backward(ctx, d2, X2, W2, 7, 5.0, q_out=q2, flags=dbp.DBP_FORCE_DENSE)
        o1 = dbp.dithered_conv_backward(ctx, o2["dX"], X1, W1, 8, 5.0, q_out=q1, flags=dbp.DBP_FORCE_DENSE | dbp.DBP_DX_F32)
        torch.cuda.synchronize()
        assert ctx.last_device_status() == (0, 0)
        for (q, o, delta_np, X, W, seed, f32) in ((q2, o2, L2.delta, L2.X, L2.W, 7, False),
                                                  (q1, o1, o2["dX"].float().cpu().numpy(), L1.X, L1.W, 8, True)):
            D = np.float32(q.delta.item())
            codes, nnz, _ = oracle.nsd_codes(delta_np, seed, D)
            assert np.array_equal(dbp.nsd_decode_dense(ctx, q).cpu().numpy().reshape(codes.shape), codes)
            ref = oracle.conv_backward(codes, D, X, W, with_abs=True)
            got = o["dW"].double().cpu().numpy()
            assert np.all(np.abs(got - ref["dW"]) <= TOL * ref["S_dW"] + 1e-30)
            gx = o["dX"].double().cpu().numpy()
            slack = 0.0 if f32 else 2.0 ** -8
            assert np.all(np.abs(gx - ref["dX"]) <= slack * np.abs(ref["dX"]) + TOL * ref["S_dX"] + 1e-30)


def test_async_dw_matches_the_synchronous_call(ctx):
    """DBP_DW_ASYNC: dW of a layer is still being computed on the context's second stream while the
    next layers are quantized (their codes go to the other set of buffers). After dbp_join the
    results are those of the synchronous calls: dX bit for bit, dW up to the order of the additions."""
    import paper_2004_04729_b200 as dbp
    shapes = [(2, 256, 64, 28, 28, 1), (2, 64, 64, 28, 28, 3), (3, 512, 128, 14, 14, 1), (3, 128, 128, 7, 7, 3),
              (2, 64, 256, 28, 28, 1)]
    layers = [wl.conv_layer(B, Ci, Co, H, W, k, data_seed=31 + i, scale=5.0, dtype="bf16")
              for i, (B, Ci, Co, H, W, k) in enumerate(shapes)]
    dev = [(_t(L.delta), _t(L.X), _t(L.W)) for L in layers]
    ref = [dbp.dithered_conv_backward(ctx, d, X, W, L.seed, L.scale) for L, (d, X, W) in zip(layers, dev)]
    torch.cuda.synchronize()
    for _ in range(2):                                   # twice: both buffer sets get reused
        out = [dbp.dithered_conv_backward(ctx, d, X, W, L.seed, L.scale, flags=dbp.DBP_DW_ASYNC)
               for L, (d, X, W) in zip(layers, dev)]
        ctx.join()
        torch.cuda.synchronize()
        assert ctx.last_device_status() == (0, 0)
        for a, b in zip(ref, out):
            assert torch.equal(a["dX"], b["dX"])
            scale = a["dW"].abs().max().item()
            assert (a["dW"] - b["dW"]).abs().max().item() <= 1e-5 * scale


@pytest.mark.parametrize("B,Ci,Co,H,W,k,dtype", [
    (2, 256, 64, 28, 28, 1, "bf16"), (3, 128, 128, 14, 14, 3, "bf16"), (2, 64, 64, 16, 16, 3, "f32"),
    (4, 24, 40, 9, 9, 3, "f32"),                       # gather kernels (Cin % 8 == 0 but fp32 1x1 / odd widths)
])
def test_repeated_calls_are_bit_identical(ctx, B, Ci, Co, H, W, k, dtype):
    """Identical calls give identical codes, nnz, step size and dX (bit for bit): the path is chosen from the
    layer's shape and the caller's threshold, not from the timing of a read-back. dW of the TMA-fed kernels is
    added up at the L2 in the order the CTAs arrive, so it is compared to within the tolerance."""
    import paper_2004_04729_b200 as dbp
    L = wl.conv_layer(B, Ci, Co, H, W, k, data_seed=91, scale=2.0, dtype=dtype)
    cast = _t if dtype == "bf16" else _f32
    d, X, Wt = cast(L.delta), cast(L.X), cast(L.W)
    outs = []
    for _ in range(3):
        q = dbp.SparseGradient(d.numel())
        out = dbp.dithered_conv_backward(ctx, d, X, Wt, L.seed, L.scale, q_out=q)
        torch.cuda.synchronize()
        outs.append((dbp.nsd_decode_dense(ctx, q).clone(), q.delta.item(), q.nnz.item(), out["dX"].clone(), out["dW"].clone()))
    for codes, delta, nnz, dX, dW in outs[1:]:
        assert torch.equal(codes, outs[0][0]) and delta == outs[0][1] and nnz == outs[0][2]
        assert torch.equal(dX, outs[0][3])
        scale = outs[0][4].abs().max().item()
        assert (dW - outs[0][4]).abs().max().item() <= 1e-5 * scale
