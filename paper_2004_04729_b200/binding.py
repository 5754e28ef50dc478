"""ctypes binding of `libdbp.so` (same names as the C ABI in `include/dbp.h`).

PyTorch is used only for device memory (`torch.empty(..., device="cuda")`, `data_ptr()`),
pinned host buffers and the CUDA stream handle. No arithmetic of the method happens here.
"""
import ctypes
import os
from typing import Optional

import torch

HERE = os.path.dirname(os.path.abspath(__file__))

DBP_F32, DBP_BF16 = 0, 1
DBP_FORCE_SPARSE, DBP_FORCE_DENSE, DBP_DX_F32, DBP_DW_ASYNC = 1, 2, 4, 8
DBP_SEGMENT = 1024

EXPORTED_SYMBOLS = [
    "dbp_create", "dbp_destroy", "dbp_set_stream", "dbp_status_string",
    "dbp_last_device_status", "dbp_sparse_bytes", "nsd_quantize", "nsd_decode_dense",
    "dithered_linear_backward", "dithered_conv_backward", "dithered_linear_backward_host",
    "dithered_conv_backward_host", "dbp_relu_backward", "dbp_maxpool2x2_backward",
    "dbp_profile_enable", "dbp_profile_select", "dbp_profile_read", "dbp_set_crossover", "nsd_step_size_noalloc",
    "dbp_last_step", "dbp_layer_seed", "dbp_selftest_bounded_wait", "dbp_last_error", "dbp_wait_stats", "dbp_join", "dbp_kernel_launches", "dbp_measure_fma_peak", "dbp_set_relu_mask",
]

KERNEL_KINDS = ["statistics", "quantize", "weight_taps", "dx", "dw", "db", "decode", "glue",
                "dx_dense", "dw_dense", "fused"]


class DbpError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        detail = load_library().dbp_last_error().decode() if status == -3 else ""
        super().__init__(f"{where}: {_status_string(status)} ({status})" + (f" [{detail}]" if detail else ""))


class _Sparse(ctypes.Structure):
    _fields_ = [("bitmap", ctypes.c_void_p), ("offsets", ctypes.c_void_p),
                ("values", ctypes.c_void_p), ("delta", ctypes.c_void_p),
                ("nnz", ctypes.c_void_p), ("numel", ctypes.c_longlong)]


_lib = None


def lib_path() -> str:
    return os.path.join(HERE, "libdbp.so")


def load_library():
    """Loads the CUDA library; raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    path = lib_path()
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: build it with `python -m paper_2004_04729_b200.build`")
    lib = ctypes.CDLL(path)
    vp, ll, ull, i32, u32, f32 = (ctypes.c_void_p, ctypes.c_longlong, ctypes.c_ulonglong,
                                  ctypes.c_int, ctypes.c_uint, ctypes.c_float)
    lib.dbp_create.argtypes = [ctypes.POINTER(vp), i32, vp]
    lib.dbp_destroy.argtypes = [vp]
    lib.dbp_set_stream.argtypes = [vp, vp]
    lib.dbp_set_relu_mask.argtypes = [vp, vp]
    lib.dbp_status_string.argtypes = [i32]
    lib.dbp_status_string.restype = ctypes.c_char_p
    lib.dbp_last_device_status.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(ll)]
    lib.dbp_sparse_bytes.argtypes = [ll] + [ctypes.POINTER(ctypes.c_size_t)] * 3
    lib.nsd_quantize.argtypes = [vp, vp, i32, ll, ull, f32, vp, ctypes.POINTER(_Sparse)]
    lib.nsd_decode_dense.argtypes = [vp, ctypes.POINTER(_Sparse), vp]
    lib.dithered_linear_backward.argtypes = [vp, vp, vp, vp, i32, ll, ll, ll, ull, f32, vp,
                                             ctypes.POINTER(_Sparse), vp, vp, vp, u32]
    lib.dithered_conv_backward.argtypes = [vp, vp, vp, vp, i32, ll, ll, ll, ll, ll, i32, i32, i32,
                                           ull, f32, vp, ctypes.POINTER(_Sparse), vp, vp, vp, u32]
    lib.dithered_linear_backward_host.argtypes = [vp, vp, vp, vp, i32, ll, ll, ll, ull, f32,
                                                  vp, vp, vp, u32, ctypes.POINTER(f32),
                                                  ctypes.POINTER(ll)]
    lib.dithered_conv_backward_host.argtypes = [vp, vp, vp, vp, i32, ll, ll, ll, ll, ll, i32, i32,
                                                i32, ull, f32, vp, vp, vp, u32,
                                                ctypes.POINTER(f32), ctypes.POINTER(ll)]
    lib.dbp_set_crossover.argtypes = [vp, f32]
    lib.nsd_step_size_noalloc.argtypes = [vp, i32, ll, f32, vp, vp]
    lib.dbp_profile_enable.argtypes = [vp, i32]
    lib.dbp_profile_select.argtypes = [vp, u32]
    lib.dbp_profile_read.argtypes = [vp, i32, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ll)]
    lib.dbp_selftest_bounded_wait.argtypes = [vp, ll]
    lib.dbp_join.argtypes = [vp]
    lib.dbp_kernel_launches.argtypes = []
    lib.dbp_kernel_launches.restype = ll
    lib.dbp_measure_fma_peak.argtypes = [vp, ctypes.POINTER(ctypes.c_double)]
    lib.dbp_wait_stats.argtypes = [vp, ctypes.POINTER(ull), i32]
    lib.dbp_last_step.argtypes = [vp, ctypes.POINTER(f32), ctypes.POINTER(ll)]
    lib.dbp_layer_seed.argtypes = [ull, i32]
    lib.dbp_relu_backward.argtypes = [vp, vp, vp, vp, ll]
    lib.dbp_maxpool2x2_backward.argtypes = [vp, vp, vp, vp, ll, ll, ll]
    for name in EXPORTED_SYMBOLS:
        if name not in ("dbp_status_string", "dbp_layer_seed", "dbp_last_error", "dbp_kernel_launches"):
            getattr(lib, name).restype = i32
    lib.dbp_layer_seed.restype = ull
    lib.dbp_last_error.argtypes = []
    lib.dbp_last_error.restype = ctypes.c_char_p
    _lib = lib
    return lib


def _status_string(status: int) -> str:
    return load_library().dbp_status_string(int(status)).decode()


def _check(status, where):
    if status != 0:
        raise DbpError(status, where)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return DBP_F32
    if t.dtype == torch.bfloat16:
        return DBP_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _dev(t: torch.Tensor, name: str):
    if not (t.is_cuda and t.is_contiguous()):
        raise ValueError(f"{name} must be a contiguous CUDA tensor")
    return t


class Context:
    """One library context (workspace + stream). Uses torch's current stream by default."""

    def __init__(self, device: int = 0, stream: Optional[torch.cuda.Stream] = None):
        lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("dithered backprop needs a CUDA device; there is no CPU path")
        self.device = int(device)
        with torch.cuda.device(self.device):
            s = stream if stream is not None else torch.cuda.current_stream()
            h = ctypes.c_void_p()
            _check(lib.dbp_create(ctypes.byref(h), self.device, ctypes.c_void_p(s.cuda_stream)),
                   "dbp_create")
        self._h = h
        self._stream = s

    def set_stream(self, stream: torch.cuda.Stream):
        _check(load_library().dbp_set_stream(self._h, ctypes.c_void_p(stream.cuda_stream)),
               "dbp_set_stream")
        self._stream = stream

    def last_device_status(self):
        st, sat = ctypes.c_int(), ctypes.c_longlong()
        _check(load_library().dbp_last_device_status(self._h, ctypes.byref(st), ctypes.byref(sat)),
               "dbp_last_device_status")
        return st.value, sat.value

    def set_relu_mask(self, mask: Optional[torch.Tensor]):
        """The next backward call on this context quantizes delta (.) mask (uint8, one byte per element, non-zero
        where the forward pre-activation was positive); fp32 only. Consumed by that call."""
        if mask is not None and not (mask.is_cuda and mask.is_contiguous() and mask.dtype == torch.uint8):
            raise ValueError("mask must be a contiguous CUDA uint8 tensor")
        _check(load_library().dbp_set_relu_mask(self._h, _ptr(mask)), "dbp_set_relu_mask")

    def last_step(self):
        """(Delta, nnz) of the most recent quantization on this context (synchronises)."""
        d, n = ctypes.c_float(), ctypes.c_longlong()
        _check(load_library().dbp_last_step(self._h, ctypes.byref(d), ctypes.byref(n)), "dbp_last_step")
        return d.value, n.value

    def selftest_bounded_wait(self, cycles: int = 100000):
        """Enqueues the library's wait self-test: a wait that nothing satisfies runs out after
        `cycles` SM clocks and the next last_device_status() reports DBP_ETIMEOUT."""
        _check(load_library().dbp_selftest_bounded_wait(self._h, int(cycles)), "dbp_selftest_bounded_wait")

    def wait_stats(self, reset: bool = True):
        """SM clocks the 3x3 kernels' issuing threads spent waiting, by cause (see dbp_wait_stats)."""
        out = (ctypes.c_ulonglong * 8)()
        _check(load_library().dbp_wait_stats(self._h, out, int(reset)), "dbp_wait_stats")
        return list(out)

    def measure_fma_peak(self) -> float:
        """fp32 FMA throughput of the device in TFLOP/s (dependent FMA chains on every lane)."""
        v = ctypes.c_double()
        _check(load_library().dbp_measure_fma_peak(self._h, ctypes.byref(v)), "dbp_measure_fma_peak")
        return v.value

    def join(self):
        """Orders every dW left running by DBP_DW_ASYNC calls into the context's stream."""
        _check(load_library().dbp_join(self._h), "dbp_join")

    def set_crossover(self, crossover: float):
        """Density above which layers the dense tensor-core path supports use it."""
        _check(load_library().dbp_set_crossover(self._h, float(crossover)), "dbp_set_crossover")

    def profile_enable(self, on: bool = True):
        _check(load_library().dbp_profile_enable(self._h, int(bool(on))), "dbp_profile_enable")

    def profile_select(self, kinds=None):
        """Time only the named kernel kinds while profiling is on (None: all kinds)."""
        mask = 0xFFFFFFFF if kinds is None else sum(1 << KERNEL_KINDS.index(k) for k in kinds)
        _check(load_library().dbp_profile_select(self._h, mask), "dbp_profile_select")

    def profile_read(self):
        """{kernel kind: (milliseconds, launches)} since the previous read."""
        out = {}
        for i, name in enumerate(KERNEL_KINDS):
            ms, n = ctypes.c_double(), ctypes.c_longlong()
            _check(load_library().dbp_profile_read(self._h, i, ctypes.byref(ms), ctypes.byref(n)),
                   "dbp_profile_read")
            out[name] = (ms.value, n.value)
        return out

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            load_library().dbp_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class SparseGradient:
    """Device arrays of a `dbp_sparse` (bitmap, offsets, packed int8 codes, Delta, nnz)."""

    def __init__(self, numel: int, device: int = 0):
        lib = load_library()
        b, o, v = ctypes.c_size_t(), ctypes.c_size_t(), ctypes.c_size_t()
        _check(lib.dbp_sparse_bytes(int(numel), ctypes.byref(b), ctypes.byref(o), ctypes.byref(v)),
               "dbp_sparse_bytes")
        dev = torch.device("cuda", device)
        self.numel = int(numel)
        self.bitmap = torch.empty(b.value // 4, dtype=torch.int32, device=dev)
        self.offsets = torch.empty(o.value // 2, dtype=torch.int16, device=dev)
        self.values = torch.empty(v.value, dtype=torch.int8, device=dev)
        self.delta = torch.zeros(1, dtype=torch.float32, device=dev)
        self.nnz = torch.zeros(1, dtype=torch.int64, device=dev)
        self._c = _Sparse(self.bitmap.data_ptr(), self.offsets.data_ptr(), self.values.data_ptr(),
                          self.delta.data_ptr(), self.nnz.data_ptr(), self.numel)

    def c(self):
        return ctypes.byref(self._c)


def nsd_quantize(ctx: Context, delta: torch.Tensor, seed: int, scale: float,
                 delta_in: Optional[torch.Tensor] = None,
                 out: Optional[SparseGradient] = None) -> SparseGradient:
    """Algorithm 1: (codes, Delta, nnz) of `delta` as a SparseGradient."""
    _dev(delta, "delta")
    out = out or SparseGradient(delta.numel(), ctx.device)
    _check(load_library().nsd_quantize(ctx._h, _ptr(delta), _dtype_code(delta), delta.numel(),
                                       int(seed) & (2 ** 64 - 1), float(scale), _ptr(delta_in),
                                       out.c()), "nsd_quantize")
    return out


def nsd_decode_dense(ctx: Context, q: SparseGradient, shape=None) -> torch.Tensor:
    codes = torch.empty(q.numel, dtype=torch.int8, device=q.values.device)
    _check(load_library().nsd_decode_dense(ctx._h, q.c(), _ptr(codes)), "nsd_decode_dense")
    return codes if shape is None else codes.view(shape)


def _outputs(need, shape, dtype, device):
    return torch.empty(shape, dtype=dtype, device=device) if need else None


def dithered_linear_backward(ctx: Context, delta, X, W, seed: int, scale: float, *,
                             delta_in=None, q_out: Optional[SparseGradient] = None,
                             need_dW=True, need_dX=True, need_db=False, flags: int = 0):
    """delta [B,N], X [B,K], W [N,K] -> dict(dW [N,K] fp32, dX [B,K], db [N] fp32)."""
    _dev(delta, "delta"), _dev(X, "X"), _dev(W, "W")
    B, N = delta.shape
    K = X.shape[1]
    assert X.shape == (B, K) and W.shape == (N, K) and X.dtype == delta.dtype == W.dtype
    dev = delta.device
    dx_dtype = torch.float32 if (flags & DBP_DX_F32) else delta.dtype
    dW = _outputs(need_dW, (N, K), torch.float32, dev)
    dX = _outputs(need_dX, (B, K), dx_dtype, dev)
    db = _outputs(need_db, (N,), torch.float32, dev)
    _check(load_library().dithered_linear_backward(
        ctx._h, _ptr(delta), _ptr(X), _ptr(W), _dtype_code(delta), B, N, K,
        int(seed) & (2 ** 64 - 1), float(scale), _ptr(delta_in),
        q_out.c() if q_out is not None else None, _ptr(dW), _ptr(dX), _ptr(db), int(flags)),
        "dithered_linear_backward")
    return {"dW": dW, "dX": dX, "db": db}


def dithered_conv_backward(ctx: Context, delta, X, W, seed: int, scale: float, *,
                           delta_in=None, q_out: Optional[SparseGradient] = None,
                           need_dW=True, need_dX=True, need_db=False, flags: int = 0,
                           stride: int = 1, pad: Optional[int] = None):
    """delta [B,Cout,H/stride,W/stride], X [B,Cin,H,W], W [Cout,Cin,k,k] (NCHW) -> dict(dW, dX, db)."""
    _dev(delta, "delta"), _dev(X, "X"), _dev(W, "W")
    B, Co = delta.shape[:2]
    Ci, k = X.shape[1], W.shape[2]
    H, Wd = X.shape[2], X.shape[3]
    if stride not in (1, 2) or X.shape[0] != B or W.shape != (Co, Ci, k, k) or \
            (H % stride, Wd % stride) != (0, 0) or tuple(delta.shape[2:]) != (H // stride, Wd // stride):
        raise ValueError("shapes of delta, X and W do not belong to one layer")
    assert X.dtype == delta.dtype == W.dtype
    pad = (k - 1) // 2 if pad is None else pad
    dev = delta.device
    dx_dtype = torch.float32 if (flags & DBP_DX_F32) else delta.dtype
    dW = _outputs(need_dW, (Co, Ci, k, k), torch.float32, dev)
    dX = _outputs(need_dX, (B, Ci, H, Wd), dx_dtype, dev)
    db = _outputs(need_db, (Co,), torch.float32, dev)
    _check(load_library().dithered_conv_backward(
        ctx._h, _ptr(delta), _ptr(X), _ptr(W), _dtype_code(delta), B, Ci, Co, H, Wd, k, stride, pad,
        int(seed) & (2 ** 64 - 1), float(scale), _ptr(delta_in),
        q_out.c() if q_out is not None else None, _ptr(dW), _ptr(dX), _ptr(db), int(flags)),
        "dithered_conv_backward")
    return {"dW": dW, "dX": dX, "db": db}


def _host(t: Optional[torch.Tensor], name):
    if t is not None and (t.is_cuda or not t.is_contiguous()):
        raise ValueError(f"{name} must be a contiguous host tensor")
    return t


def dithered_linear_backward_host(ctx: Context, delta, X, W, seed, scale, dW, dX, db=None,
                                  flags: int = 0):
    """Host tensors in and out (pinned memory recommended); returns (Delta, nnz)."""
    for n, t in (("delta", delta), ("X", X), ("W", W), ("dW", dW), ("dX", dX), ("db", db)):
        _host(t, n)
    B, N = delta.shape
    K = X.shape[1]
    d, nnz = ctypes.c_float(), ctypes.c_longlong()
    _check(load_library().dithered_linear_backward_host(
        ctx._h, _ptr(delta), _ptr(X), _ptr(W), _dtype_code(delta), B, N, K,
        int(seed) & (2 ** 64 - 1), float(scale), _ptr(dW), _ptr(dX), _ptr(db), int(flags),
        ctypes.byref(d), ctypes.byref(nnz)), "dithered_linear_backward_host")
    return d.value, nnz.value


def dithered_conv_backward_host(ctx: Context, delta, X, W, seed, scale, dW, dX, db=None,
                                flags: int = 0, stride: int = 1):
    for n, t in (("delta", delta), ("X", X), ("W", W), ("dW", dW), ("dX", dX), ("db", db)):
        _host(t, n)
    B, Co = delta.shape[:2]
    Ci, k = X.shape[1], W.shape[2]
    H, Wd = X.shape[2], X.shape[3]
    if tuple(delta.shape[2:]) != (H // stride, Wd // stride):
        raise ValueError("shapes of delta and X do not belong to one layer")
    d, nnz = ctypes.c_float(), ctypes.c_longlong()
    _check(load_library().dithered_conv_backward_host(
        ctx._h, _ptr(delta), _ptr(X), _ptr(W), _dtype_code(delta), B, Ci, Co, H, Wd, k, int(stride),
        (k - 1) // 2, int(seed) & (2 ** 64 - 1), float(scale), _ptr(dW), _ptr(dX), _ptr(db),
        int(flags), ctypes.byref(d), ctypes.byref(nnz)), "dithered_conv_backward_host")
    return d.value, nnz.value


def relu_backward(ctx: Context, delta_a: torch.Tensor, mask_u8: torch.Tensor) -> torch.Tensor:
    out = torch.empty_like(delta_a)
    _check(load_library().dbp_relu_backward(ctx._h, _ptr(delta_a), _ptr(mask_u8), _ptr(out),
                                            delta_a.numel()), "dbp_relu_backward")
    return out


def maxpool2x2_backward(ctx: Context, g: torch.Tensor, argmax_i8: torch.Tensor) -> torch.Tensor:
    B, C, h, w = g.shape
    out = torch.empty((B, C, 2 * h, 2 * w), dtype=g.dtype, device=g.device)
    _check(load_library().dbp_maxpool2x2_backward(ctx._h, _ptr(g), _ptr(argmax_i8), _ptr(out),
                                                  B * C, h, w), "dbp_maxpool2x2_backward")
    return out


def nsd_step_size_noalloc(delta: torch.Tensor, scale: float, out: torch.Tensor,
                          stream: Optional[torch.cuda.Stream] = None, numel: Optional[int] = None) -> None:
    """Delta = scale * std(delta) written to the one-element device tensor `out`, through the
    library's allocation-free entry point: no Context, no workspace. The caller owns `delta`
    and `out`; nothing is allocated here either. `numel` overrides delta.numel() (used to
    probe the size limit without a large tensor)."""
    _dev(delta, "delta"), _dev(out, "out")
    if out.dtype != torch.float32 or out.numel() < 1:
        raise ValueError("out must hold one float32")
    if out.device != delta.device:
        raise ValueError("delta and out must live on the same GPU")
    # the C call runs on the current device with that device's scratch array
    with torch.cuda.device(delta.device):
        s = stream if stream is not None else torch.cuda.current_stream()
        _check(load_library().nsd_step_size_noalloc(
            _ptr(delta), _dtype_code(delta), delta.numel() if numel is None else int(numel), float(scale),
            _ptr(out), ctypes.c_void_p(s.cuda_stream)), "nsd_step_size_noalloc")


def kernel_launches() -> int:
    """Kernels the library has launched in this process so far."""
    return int(load_library().dbp_kernel_launches())


def layer_seed(seed: int, layer: int) -> int:
    """Seed of layer `layer` of a network whose backward pass was given `seed` (C: dbp_layer_seed)."""
    return int(load_library().dbp_layer_seed(int(seed) & (2 ** 64 - 1), int(layer)))


def network_backward(ctx: Context, kinds, Xs, Ws, relu_masks, pool_argmax, delta_out, scale: float,
                     seed: int, keep_delta_z: bool = False, first_layer_dX: bool = False,
                     with_sparse: bool = True, flags: int = 0):
    """Dithered backward pass of a feed-forward network (device tensors, forward order):
    for l = L..1: delta_z = delta_a (.) relu'(z); NSD; dW_l, and delta_a of the layer below
    from the QUANTIZED gradient; 2x2 max-pool routing where a pool follows layer l-1.
    Returns one dict per layer with dW, dX (None for layer 0 unless asked), Delta, nnz, and
    optionally the delta_z that was quantized and its SparseGradient. with_sparse=False asks for
    no sparse structure (Delta and nnz are then None; the library runs its leaner quantizer)."""
    L = len(kinds)
    res = [None] * L
    delta_a = delta_out
    for l in range(L - 1, -1, -1):
        # nobody asks for delta_z: the mask is folded into the call (small linear layers never write delta_z at all)
        fold = relu_masks[l] is not None and not keep_delta_z and not with_sparse and delta_a.dtype == torch.float32
        if fold:
            if delta_a.numel() != relu_masks[l].numel():
                raise ValueError("mask must have one byte per element of delta")
            ctx.set_relu_mask(relu_masks[l])
            dz = delta_a
        else:
            dz = delta_a if relu_masks[l] is None else relu_backward(ctx, delta_a, relu_masks[l])
        q = SparseGradient(dz.numel(), ctx.device) if with_sparse else None
        fn = dithered_linear_backward if kinds[l] == "linear" else dithered_conv_backward
        need_dx = l > 0 or first_layer_dX
        r = fn(ctx, dz, Xs[l], Ws[l], layer_seed(seed, l), scale, q_out=q,
               need_dX=need_dx, flags=flags)
        r.update(Delta=q.delta if q else None, nnz=q.nnz if q else None)
        if keep_delta_z:
            r.update(delta_z=dz, q=q)
        res[l] = r
        if l > 0:
            g = r["dX"]
            if kinds[l] == "linear" and kinds[l - 1] == "conv":
                B, C = relu_masks[l - 1].shape[:2]
                shp = pool_argmax[l - 1].shape if pool_argmax[l - 1] is not None else relu_masks[l - 1].shape
                g = g.view(B, C, shp[2], shp[3])
            if pool_argmax[l - 1] is not None:
                g = maxpool2x2_backward(ctx, g, pool_argmax[l - 1])
            delta_a = g
    return res


def average_weight_gradients(grads, group=None) -> None:
    """The exchange step of the data-parallel form (Section 3.6): every rank's weight gradients are replaced, in
    place, by their mean over the ranks of `group` (the parameter server's average followed by its broadcast, as
    one all-reduce). `grads`: this rank's dW tensors (fp32, one device). They travel as one flat bucket, so the
    collective's launch cost is paid once per step, not once per layer. With one rank it does nothing.
    Plumbing only: `torch.distributed` (NCCL between GPUs) moves and adds the data."""
    import torch.distributed as dist
    grads = [g for g in grads if g is not None]
    if not grads or not dist.is_available() or not dist.is_initialized():
        return
    world = dist.get_world_size(group)
    if world == 1:
        return
    if any(g.dtype != torch.float32 or g.device != grads[0].device for g in grads):
        raise ValueError("weight gradients must be float32 tensors on one device")
    bucket = torch.cat([g.reshape(-1) for g in grads])
    dist.all_reduce(bucket, op=dist.ReduceOp.SUM, group=group)
    bucket.div_(world)
    off = 0
    for g in grads:
        n = g.numel()
        g.copy_(bucket[off:off + n].view_as(g))
        off += n
