"""Parity of the CUDA path (through the C ABI) with the CPU oracle.

Bars: Delta within 1e-6 relative; codes and nnz bit-exact when the oracle is given the GPU's
Delta; dW and dX within relative Frobenius error 1e-5 and |err| <= 1e-5 * sum|terms|
elementwise (fp32 accumulation of exact int8 x fp32 products)."""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl

pytestmark = pytest.mark.gpu

REL_DELTA = 1e-6
TOL = 1e-5


@pytest.fixture(scope="module")
def ctx():
    import paper_2004_04729_b200 as dbp
    c = dbp.Context(0)
    yield c
    c.close()


def _t(a, dtype="f32"):
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t.to(torch.bfloat16) if dtype == "bf16" else t


def _check_sparse_structure(q, codes_np):
    """bitmap/offsets/values describe exactly the dense codes."""
    n = codes_np.size
    flat = codes_np.ravel()
    bm = q.bitmap.cpu().numpy().view(np.uint32)
    off = q.offsets.cpu().numpy().view(np.uint16)
    val = q.values.cpu().numpy()
    nseg = (n + 1023) // 1024
    padded = np.zeros(nseg * 1024, dtype=np.int8)
    padded[:n] = flat
    bits = (padded != 0).reshape(-1, 32)
    words = (bits.astype(np.uint64) << np.arange(32, dtype=np.uint64)).sum(axis=1).astype(np.uint32)
    assert np.array_equal(bm, words)
    cnt = bits.sum(axis=1).reshape(nseg, 32)
    excl = np.cumsum(cnt, axis=1) - cnt
    assert np.array_equal(off.reshape(nseg, 32), excl.astype(np.uint16))
    for g in range(min(nseg, 64)):
        seg = padded[g * 1024:(g + 1) * 1024]
        nz = seg[seg != 0]
        assert np.array_equal(val[g * 1024:g * 1024 + nz.size], nz)


def _nsd_case(ctx, d_np, scale, seed, dtype="f32", check_structure=True):
    import paper_2004_04729_b200 as dbp
    d = _t(d_np, dtype)
    q = dbp.nsd_quantize(ctx, d, seed, scale)
    codes = dbp.nsd_decode_dense(ctx, q).cpu().numpy().reshape(d_np.shape)
    D_gpu = np.float32(q.delta.item())
    D_ref = oracle.step_size(d_np, scale)
    if D_ref > 0:
        assert abs(float(D_gpu) - float(D_ref)) <= REL_DELTA * float(D_ref)
    else:
        assert D_gpu == 0
    ref, nnz, nsat = oracle.nsd_codes(d_np, seed, D_gpu)
    assert np.array_equal(codes, ref)
    assert q.nnz.item() == nnz
    if check_structure:
        _check_sparse_structure(q, ref)
    return q, codes, D_gpu


@pytest.mark.parametrize("n", [1, 5, 31, 1023, 1024, 1025, 4099, 70001])
def test_nsd_codes_ragged_sizes(ctx, n):
    d = (wl.laplace(7, n, n, 1e-3) * wl.bernoulli(7, n + 1, n, 0.5)).astype(np.float32)
    _nsd_case(ctx, d, 2.0, seed=n)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("scale", [2.0, 5.0])
def test_nsd_codes_layer_shapes(ctx, dtype, scale):
    L = wl.config1()
    d = wl.round_to_bf16(L.delta) if dtype == "bf16" else L.delta
    _, codes, _ = _nsd_case(ctx, d, scale, 0, dtype)
    C = wl.config3(batch=4)
    d = wl.round_to_bf16(C.delta) if dtype == "bf16" else C.delta
    _, codes, _ = _nsd_case(ctx, d, scale, 0, dtype)
    p0 = {2.0: 0.78383, 5.0: 0.90067}[scale]        # closed form for this input recipe
    assert abs((codes == 0).mean() - p0) < 0.01
    assert np.abs(codes).max() <= 127


def test_nsd_seed_and_override_and_determinism(ctx):
    import paper_2004_04729_b200 as dbp
    L = wl.config1()
    d = _t(L.delta)
    a = dbp.nsd_decode_dense(ctx, dbp.nsd_quantize(ctx, d, 3, 2.0)).cpu().numpy()
    b = dbp.nsd_decode_dense(ctx, dbp.nsd_quantize(ctx, d, 3, 2.0)).cpu().numpy()
    c = dbp.nsd_decode_dense(ctx, dbp.nsd_quantize(ctx, d, 4, 2.0)).cpu().numpy()
    assert np.array_equal(a, b) and not np.array_equal(a, c)
    step = torch.tensor([1.5e-3], dtype=torch.float32, device="cuda")
    q = dbp.nsd_quantize(ctx, d, 3, 0.0, delta_in=step)
    assert q.delta.item() == np.float32(1.5e-3)
    ref, nnz, _ = oracle.nsd_codes(L.delta, 3, np.float32(1.5e-3))
    assert np.array_equal(dbp.nsd_decode_dense(ctx, q).cpu().numpy().reshape(ref.shape), ref)
    assert q.nnz.item() == nnz


def test_nsd_degenerate_inputs(ctx):
    import paper_2004_04729_b200 as dbp
    z = torch.zeros(5000, device="cuda")
    q = dbp.nsd_quantize(ctx, z, 0, 2.0)
    assert q.delta.item() == 0 and q.nnz.item() == 0
    assert not dbp.nsd_decode_dense(ctx, q).any()
    assert ctx.last_device_status() == (0, 0)
    # constant non-zero tensor: sigma = 0 as well
    q = dbp.nsd_quantize(ctx, torch.full((3000,), 0.25, device="cuda"), 0, 2.0)
    assert q.delta.item() == 0 and q.nnz.item() == 0
    bad = torch.randn(4096, device="cuda")
    bad[17] = float("nan")
    q = dbp.nsd_quantize(ctx, bad, 0, 2.0)
    assert q.nnz.item() == 0 and not dbp.nsd_decode_dense(ctx, q).any()
    st, _ = ctx.last_device_status()
    assert st == -5
    assert ctx.last_device_status() == (0, 0)          # the record is cleared by the read
    # saturation: values beyond 127 steps are clipped and counted
    x = np.array([1000.0, -1000.0, 0.4, 0.0] * 300, dtype=np.float32)
    step = torch.tensor([1.0], dtype=torch.float32, device="cuda")
    q = dbp.nsd_quantize(ctx, _t(x), 1, 0.0, delta_in=step)
    got = dbp.nsd_decode_dense(ctx, q).cpu().numpy()
    ref, nnz, nsat = oracle.nsd_codes(x, 1, 1.0)
    assert np.array_equal(got, ref) and got.max() == 127 and got.min() == -127
    assert ctx.last_device_status() == (-6, nsat)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_step_size_is_shift_invariant(ctx, dtype):
    """Algorithm 1's std is about the mean: a constant tensor whose value is not a binary
    fraction has sigma = 0 exactly (Delta = 0, every code 0), and a mean of 100 sigma must not
    cost accuracy (raw moments sum(x^2)/n - mean^2 would cancel on both)."""
    import paper_2004_04729_b200 as dbp
    for n in (3000, 70001, 1 << 20):
        c = torch.full((n,), 0.1, device="cuda")
        c = c.to(torch.bfloat16) if dtype == "bf16" else c
        q = dbp.nsd_quantize(ctx, c, 0, 2.0)
        assert q.delta.item() == 0 and q.nnz.item() == 0
        assert not dbp.nsd_decode_dense(ctx, q).any()
    assert ctx.last_device_status() == (0, 0)
    if dtype == "f32":
        # a bf16 tensor with this offset would hold almost no information about sigma
        for n, seed in ((70001, 5), (1 << 20, 6)):
            lap = wl.laplace(seed, 1, n, 1e-3)
            d = (lap + 100.0 * lap.std()).astype(np.float32)
            _nsd_case(ctx, d, 2.0, seed=seed, check_structure=False)
            out = torch.zeros(1, device="cuda")
            dbp.nsd_step_size_noalloc(_t(d), 2.0, out)
            ref = float(oracle.step_size(d, 2.0))
            assert abs(out.item() - ref) <= REL_DELTA * ref


def test_bounded_wait_runs_out_and_is_reported(ctx):
    """A device-side wait that nothing satisfies gives up after its clock budget: the kernel
    returns, the status word says DBP_ETIMEOUT once, and the context keeps working."""
    import paper_2004_04729_b200 as dbp
    assert ctx.last_device_status() == (0, 0)
    ctx.selftest_bounded_wait(100000)
    assert ctx.last_device_status()[0] == -8
    assert ctx.last_device_status() == (0, 0)            # cleared by the read
    L = wl.config1()
    _nsd_case(ctx, L.delta, 2.0, 0)                      # the context is still usable


def _compare(name, got, ref, S):
    got = got.double().cpu().numpy()
    err = np.abs(got - ref)
    fro = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300)
    assert fro <= TOL, (name, fro)
    bound = TOL * S + 1e-30
    assert np.all(err <= bound), (name, float((err / bound).max()))


def _layer_case(ctx, L, need_db=True, dx_f32=True):
    import paper_2004_04729_b200 as dbp
    d, X, W = _t(L.delta, L.dtype), _t(L.X, L.dtype), _t(L.W, L.dtype)
    q = dbp.SparseGradient(d.numel())
    # the sparse kernels are the subject here (the dense path has its own test file)
    flags = dbp.DBP_FORCE_SPARSE | (dbp.DBP_DX_F32 if (L.dtype == "bf16" and dx_f32) else 0)
    fn = dbp.dithered_linear_backward if L.kind == "linear" else dbp.dithered_conv_backward
    out = fn(ctx, d, X, W, L.seed, L.scale, q_out=q, need_db=need_db, flags=flags)
    D = np.float32(q.delta.item())
    D_ref = oracle.step_size(L.delta, L.scale)
    assert abs(float(D) - float(D_ref)) <= REL_DELTA * float(D_ref)
    ref_codes, nnz, _ = oracle.nsd_codes(L.delta, L.seed, D)
    codes = dbp.nsd_decode_dense(ctx, q).cpu().numpy().reshape(L.delta.shape)
    assert np.array_equal(codes, ref_codes) and q.nnz.item() == nnz
    ofn = oracle.linear_backward if L.kind == "linear" else oracle.conv_backward
    ref = ofn(ref_codes, D, L.X, L.W, with_abs=True)
    _compare("dW", out["dW"], ref["dW"], ref["S_dW"])
    if dx_f32 or L.dtype == "f32":
        _compare("dX", out["dX"], ref["dX"], ref["S_dX"])
    else:   # bf16 output: one rounding to 8 significant bits on top of the fp32 bound
        got = out["dX"].double().cpu().numpy()
        assert np.all(np.abs(got - ref["dX"]) <= 2.0 ** -8 * np.abs(ref["dX"]) + TOL * ref["S_dX"] + 1e-30)
    if need_db:
        _compare("db", out["db"], ref["db"], ref["S_db"])
    return out, ref


def test_config1_linear_layer(ctx):
    _layer_case(ctx, wl.config1())


@pytest.mark.parametrize("B,N,K", [(1, 1, 1), (3, 10, 100), (5, 33, 7), (16, 100, 300), (2, 65, 130)])
def test_linear_ragged_shapes(ctx, B, N, K):
    _layer_case(ctx, wl.linear_layer(B, N, K, data_seed=B * 1000 + N))


def test_config3_conv3x3_reduced_batch(ctx):
    _layer_case(ctx, wl.config3(batch=4))


@pytest.mark.parametrize("B,Ci,Co,H,W,k", [
    (2, 3, 8, 6, 6, 3), (1, 64, 64, 7, 7, 3), (2, 16, 40, 5, 9, 3), (1, 128, 32, 14, 14, 3),
    (2, 8, 8, 1, 1, 3), (1, 4, 4, 2, 2, 3), (1, 32, 32, 3, 70, 3), (1, 130, 20, 4, 4, 3),
    (2, 64, 64, 8, 8, 1), (1, 256, 64, 7, 7, 1), (2, 64, 256, 5, 5, 1), (1, 3, 5, 4, 6, 1),
    (1, 72, 33, 9, 3, 1)])
def test_conv_shapes(ctx, B, Ci, Co, H, W, k):
    _layer_case(ctx, wl.conv_layer(B, Ci, Co, H, W, k, data_seed=Ci * 7 + Co + H))


@pytest.mark.parametrize("idx", [0, 2, 6, 10, 14, 15])
def test_config5_bf16_layers_reduced_batch(ctx, idx):
    L = wl.config5_layer(idx, batch=2)
    out, _ = _layer_case(ctx, L, dx_f32=True)
    _layer_case(ctx, L, dx_f32=False, need_db=False)
    nnz_frac = 1.0 - (out["dW"] == 0).float().mean().item()
    assert nnz_frac > 0.5


def test_all_zero_gradient_gives_zero_products(ctx):
    import paper_2004_04729_b200 as dbp
    L = wl.config3(batch=1)
    d = torch.zeros_like(_t(L.delta))
    out = dbp.dithered_conv_backward(ctx, d, _t(L.X), _t(L.W), 0, 2.0, need_db=True)
    assert not out["dW"].any() and not out["dX"].any() and not out["db"].any()


def test_argument_errors_are_reported_not_run(ctx):
    import paper_2004_04729_b200 as dbp
    L = wl.conv_layer(1, 4, 4, 4, 4, 3, data_seed=1)
    d, X, W = _t(L.delta), _t(L.X), _t(L.W)
    with pytest.raises(dbp.DbpError) as e:
        dbp.dithered_conv_backward(ctx, d, X, W, 0, 2.0, pad=0)
    assert e.value.status == -2
    with pytest.raises(dbp.DbpError) as e:
        dbp.dithered_conv_backward(ctx, d, X, W, 0, 2.0, flags=dbp.DBP_FORCE_SPARSE | dbp.DBP_FORCE_DENSE)
    assert e.value.status == -1
    with pytest.raises(dbp.DbpError) as e:      # misaligned base pointer
        dbp.dithered_conv_backward(ctx, d.flatten()[1:17].view(1, 1, 4, 4), X[:, :1], W[:1, :1], 0, 2.0)
    assert e.value.status == -1
    with pytest.raises(dbp.DbpError) as e:      # scale <= 0 without a step to read
        dbp.nsd_quantize(ctx, d, 0, 0.0)
    assert e.value.status == -1


def test_host_entry_points_match_device_ones(ctx):
    import paper_2004_04729_b200 as dbp
    L = wl.config3(batch=2)
    dev = dbp.dithered_conv_backward(ctx, _t(L.delta), _t(L.X), _t(L.W), 0, 2.0, need_db=True)
    hd, hX, hW = (torch.from_numpy(a).pin_memory() for a in (L.delta, L.X, L.W))
    dW = torch.empty(L.W.shape, dtype=torch.float32).pin_memory()
    dX = torch.empty(L.X.shape, dtype=torch.float32).pin_memory()
    db = torch.empty(L.W.shape[0], dtype=torch.float32).pin_memory()
    D, nnz = dbp.dithered_conv_backward_host(ctx, hd, hX, hW, 0, 2.0, dW, dX, db)
    ref_codes, ref_nnz, _ = oracle.nsd_codes(L.delta, 0, np.float32(D))
    assert nnz == ref_nnz
    assert torch.equal(dX, dev["dX"].cpu()) and torch.equal(db, dev["db"].cpu())
    ref = oracle.conv_backward(ref_codes, np.float32(D), L.X, L.W, with_abs=True)
    _compare("dW", dW, ref["dW"], ref["S_dW"])
    L1 = wl.config1()
    hd, hX, hW = (torch.from_numpy(a).pin_memory() for a in (L1.delta, L1.X, L1.W))
    dW = torch.empty(L1.W.shape, dtype=torch.float32).pin_memory()
    dX = torch.empty(L1.X.shape, dtype=torch.float32).pin_memory()
    D, nnz = dbp.dithered_linear_backward_host(ctx, hd, hX, hW, 0, 2.0, dW, dX)
    rc, rn, _ = oracle.nsd_codes(L1.delta, 0, np.float32(D))
    ref = oracle.linear_backward(rc, np.float32(D), L1.X, L1.W, with_abs=True)
    assert nnz == rn
    _compare("dW", dW, ref["dW"], ref["S_dW"])
    _compare("dX", dX, ref["dX"], ref["S_dX"])


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,N", [(1, 1), (3, 5), (7, 33), (64, 300), (129, 257)])
def test_codes_of_the_internal_quantization(ctx, dtype, B, N):
    """Without q_out the library quantizes into its own dense code array only. An identity
    weight matrix makes dX = Delta * codes, so the codes (clipped ones and a NaN included) can
    be compared with the oracle's bit for bit, and nnz / the clip count through the status."""
    import paper_2004_04729_b200 as dbp
    x = (wl.laplace(11, B, B * N, 3.0) * wl.bernoulli(11, N, B * N, 0.5)).astype(np.float32).reshape(B, N)
    if B * N >= 15:
        x.flat[3], x.flat[8], x.flat[14] = 500.0, -700.0, 127.5
    if dtype == "bf16":
        x = _t(x, "bf16").float().cpu().numpy()
    eye = np.eye(N, dtype=np.float32)
    step = torch.tensor([1.0], dtype=torch.float32, device="cuda")
    ctx.last_device_status()
    out = dbp.dithered_linear_backward(ctx, _t(x, dtype), _t(np.zeros((B, N), np.float32), dtype), _t(eye, dtype),
                                       5, 0.0, delta_in=step, need_dW=False, flags=dbp.DBP_DX_F32 | dbp.DBP_FORCE_SPARSE)
    ref, nnz, nsat = oracle.nsd_codes(x, 5, np.float32(1.0))
    assert np.array_equal(out["dX"].cpu().numpy(), ref.astype(np.float32))
    assert ctx.last_device_status() == ((-6, nsat) if nsat else (0, 0))
    if B * N >= 15:
        assert nsat == 2
        x.flat[5] = np.nan                               # NaN with a given step size: code 0, others unchanged
        out = dbp.dithered_linear_backward(ctx, _t(x, dtype), _t(np.zeros((B, N), np.float32), dtype), _t(eye, dtype),
                                           5, 0.0, delta_in=step, need_dW=False, flags=dbp.DBP_DX_F32 | dbp.DBP_FORCE_SPARSE)
        ref2 = ref.copy()
        ref2.flat[5] = 0
        assert np.array_equal(out["dX"].cpu().numpy(), ref2.astype(np.float32))
        ctx.last_device_status()
