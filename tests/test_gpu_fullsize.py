"""Parity at the configurations' full sizes, in the launch configuration `bench.py` times.

The fp64 product oracle would take minutes on these tensors, so the codes are compared in
full (bit-exact, the oracle's quantizer is fast) and the gradients on sampled outputs, each
computed by the oracle from the defining sum."""
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


def _full_size_case(ctx, L, nsamples=48):
    import paper_2004_04729_b200 as dbp
    tdt = torch.bfloat16 if L.dtype == "bf16" else torch.float32
    d, X, W = (torch.from_numpy(a).to(tdt).cuda() for a in (L.delta, L.X, L.W))
    q = dbp.SparseGradient(d.numel())
    out = dbp.dithered_conv_backward(ctx, d, X, W, L.seed, L.scale, q_out=q,
                                     flags=dbp.DBP_DX_F32 if L.dtype == "bf16" else 0)   # default path choice
    torch.cuda.synchronize()
    assert ctx.last_device_status() == (0, 0)
    D = np.float32(q.delta.item())
    D_ref = oracle.step_size(L.delta, L.scale)
    assert abs(float(D) - float(D_ref)) <= 1e-6 * float(D_ref)
    codes, nnz, _ = oracle.nsd_codes(L.delta, L.seed, D)
    got = dbp.nsd_decode_dense(ctx, q).cpu().numpy().reshape(codes.shape)
    assert np.array_equal(got, codes) and q.nnz.item() == nnz
    dW, dX = out["dW"].cpu().numpy(), out["dX"].cpu().numpy()
    r = np.random.default_rng(123)
    B, Co, H, Wd = codes.shape
    Ci = L.X.shape[1]
    for _ in range(nsamples):
        co, ci, ky, kx = r.integers(Co), r.integers(Ci), r.integers(L.k), r.integers(L.k)
        v, s = oracle.conv_dW_entry(codes, D, L.X, co, ci, ky, kx, L.k)
        assert abs(float(dW[co, ci, ky, kx]) - v) <= TOL * s + 1e-30, ("dW", co, ci, ky, kx)
        b, y, x = r.integers(B), r.integers(H), r.integers(Wd)
        v, s = oracle.conv_dX_entry(codes, D, L.W, b, ci, y, x)
        assert abs(float(dX[b, ci, y, x]) - v) <= TOL * s + 1e-30, ("dX", b, ci, y, x)
    # corners and edges of the image, where border handling lives
    for (b, y, x) in ((0, 0, 0), (B - 1, H - 1, Wd - 1), (B // 2, 0, Wd - 1), (1 % B, H - 1, 0)):
        v, s = oracle.conv_dX_entry(codes, D, L.W, b, Ci - 1, y, x)
        assert abs(float(dX[b, Ci - 1, y, x]) - v) <= TOL * s + 1e-30


def test_config3_full_size(ctx):
    _full_size_case(ctx, wl.config3())           # B128, fp32: the sparse kernels


@pytest.mark.parametrize("idx", range(16))
def test_config5_full_size_layers(ctx, idx):
    _full_size_case(ctx, wl.config5_layer(idx))  # B64, bf16: every shape of the set bench.py times


@pytest.mark.parametrize("idx", range(16))
def test_config5_full_size_as_bench_calls_it(ctx, idx, nsamples=32):
    """The call `bench.py` times: no sparse structure asked for (the product-path quantizer
    runs instead of the compacting one), default flags, dX stored as bf16. Delta and nnz come
    back through dbp_last_step; the codes never leave the library, so the oracle's codes (given
    the CUDA path's Delta) stand behind every sampled gradient entry.
    Bars: nnz exact; dW within 1e-5 sum|terms|; dX = one bf16 rounding (2^-8 relative) on top."""
    import paper_2004_04729_b200 as dbp
    L = wl.config5_layer(idx)
    d, X, W = (torch.from_numpy(a).to(torch.bfloat16).cuda() for a in (L.delta, L.X, L.W))
    out = dbp.dithered_conv_backward(ctx, d, X, W, L.seed, L.scale)
    D, nnz_gpu = ctx.last_step()
    assert ctx.last_device_status() == (0, 0)
    D = np.float32(D)
    D_ref = oracle.step_size(L.delta, L.scale)
    assert abs(float(D) - float(D_ref)) <= 1e-6 * float(D_ref)
    codes, nnz, _ = oracle.nsd_codes(L.delta, L.seed, D)
    assert nnz_gpu == nnz
    assert out["dX"].dtype == torch.bfloat16
    dW, dX = out["dW"].cpu().numpy(), out["dX"].float().cpu().numpy()
    r = np.random.default_rng(321 + idx)
    B, Co, H, Wd = codes.shape
    Ci = L.X.shape[1]
    pos = [(r.integers(B), r.integers(H), r.integers(Wd)) for _ in range(nsamples)]
    pos += [(0, 0, 0), (B - 1, H - 1, Wd - 1), (B // 2, 0, Wd - 1), (1, H - 1, 0)]
    for (b, y, x) in pos:
        co, ci, ky, kx = r.integers(Co), r.integers(Ci), r.integers(L.k), r.integers(L.k)
        v, sa = oracle.conv_dW_entry(codes, D, L.X, co, ci, ky, kx, L.k)
        assert abs(float(dW[co, ci, ky, kx]) - v) <= TOL * sa + 1e-30, ("dW", co, ci, ky, kx)
        v, sa = oracle.conv_dX_entry(codes, D, L.W, b, ci, y, x)
        assert abs(float(dX[b, ci, y, x]) - v) <= 2.0 ** -8 * abs(v) + TOL * sa + 1e-30, ("dX", b, ci, y, x)


@pytest.mark.parametrize("idx", [3, 9, 13, 15])
def test_config5_full_size_bf16_dx_is_the_rounded_f32_dx(ctx, idx):
    """bench.py stores dX as bf16: at full size (persistent CTAs over many tiles, one or two
    accumulators per tile, padded small planes) those stores must be the fp32 results rounded."""
    import paper_2004_04729_b200 as dbp
    L = wl.config5_layer(idx)
    d, X, W = (torch.from_numpy(a).to(torch.bfloat16).cuda() for a in (L.delta, L.X, L.W))
    a = dbp.dithered_conv_backward(ctx, d, X, W, L.seed, L.scale, need_dW=False, flags=dbp.DBP_DX_F32)
    b = dbp.dithered_conv_backward(ctx, d, X, W, L.seed, L.scale, need_dW=False)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == (0, 0)
    assert b["dX"].dtype == torch.bfloat16
    assert torch.equal(a["dX"].to(torch.bfloat16), b["dX"])
