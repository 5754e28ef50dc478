"""Dithered backward products in fp64 (test infrastructure).

The method reaches exactly the dense products with the quantized gradient
delta~ = q * Delta (sparsity only skips zeros), so the oracle is the plain definition:

  linear (row-major batch form of Eqs. (qda), (qdw)):
      dX[b,k] = sum_j delta~[b,j] W[j,k]          (delta_a^{l-1} = W^T delta~_z)
      dW[j,k] = sum_b delta~[b,j] X[b,k]          (delta_W = delta~_z a^T)
      db[j]   = sum_b delta~[b,j]
  convolution ("analogous for convolutional layers", Section 3): cross-correlation,
  stride 1, zero padding p = (k-1)/2, NCHW,
      z[b,co,y,x]      = sum_{ci,ky,kx} W[co,ci,ky,kx] X[b,ci,y+ky-p,x+kx-p]
      dW[co,ci,ky,kx]  = sum_{b,y,x} delta~[b,co,y,x] X[b,ci,y+ky-p,x+kx-p]
      dX[b,ci,y',x']   = sum_{co,ky,kx} delta~[b,co,y'-ky+p,x'-kx+p] W[co,ci,ky,kx]

Each routine can also return S = sum |term| per output, the scale of the elementwise
error bound |err| <= tol * S.
"""
import numpy as np


def _dq(codes, Delta):
    return np.asarray(codes, dtype=np.float64) * float(np.float32(Delta))


def linear_backward(codes, Delta, X, W, with_abs=False):
    """codes [B,N] int, X [B,K], W [N,K] -> dict(dW [N,K], dX [B,K], db [N]) in fp64."""
    d = _dq(codes, Delta)
    X = np.asarray(X, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    out = {"dW": d.T @ X, "dX": d @ W, "db": d.sum(axis=0)}
    if with_abs:
        a = np.abs(d)
        out["S_dW"] = a.T @ np.abs(X)
        out["S_dX"] = a @ np.abs(W)
        out["S_db"] = a.sum(axis=0)
    return out


def _pad_hw(a, p):
    return np.pad(a, ((0, 0), (0, 0), (p, p), (p, p)))


def conv_forward(X, W):
    """z = W * X (cross-correlation, stride 1, pad (k-1)/2), fp64."""
    X = np.asarray(X, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    B, Ci, H, Wd = X.shape
    Co, Ci2, k, k2 = W.shape
    assert Ci == Ci2 and k == k2 and k % 2 == 1
    p = (k - 1) // 2
    Xp = _pad_hw(X, p)
    z = np.zeros((B, Co, H, Wd))
    for ky in range(k):
        for kx in range(k):
            z += np.einsum("bchw,oc->bohw", Xp[:, :, ky:ky + H, kx:kx + Wd], W[:, :, ky, kx],
                           optimize=True)
    return z


def conv_backward(codes, Delta, X, W, with_abs=False):
    """codes [B,Co,H,W], X [B,Ci,H,W], W [Co,Ci,k,k] -> dict(dW, dX, db) in fp64."""
    d = _dq(codes, Delta)
    X = np.asarray(X, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    B, Co, H, Wd = d.shape
    _, Ci, _, _ = X.shape
    k = W.shape[2]
    assert W.shape == (Co, Ci, k, k) and k % 2 == 1 and X.shape == (B, Ci, H, Wd)
    p = (k - 1) // 2

    def both(dd, XX, WW):
        Xp = _pad_hw(XX, p)
        dp = _pad_hw(dd, p)
        dW = np.zeros((Co, Ci, k, k))
        dX = np.zeros((B, Ci, H, Wd))
        for ky in range(k):
            for kx in range(k):
                # dW[co,ci,ky,kx] = sum_{b,y,x} d[b,co,y,x] X[b,ci,y+ky-p,x+kx-p]
                dW[:, :, ky, kx] = np.einsum("bohw,bchw->oc", dd,
                                             Xp[:, :, ky:ky + H, kx:kx + Wd], optimize=True)
                # dX[b,ci,y',x'] += sum_co d[b,co,y'-ky+p,x'-kx+p] W[co,ci,ky,kx]
                # padded index of d: (y'-ky+p)+p = y' + (2p-ky)
                oy, ox = 2 * p - ky, 2 * p - kx
                dX += np.einsum("bohw,oc->bchw", dp[:, :, oy:oy + H, ox:ox + Wd],
                                WW[:, :, ky, kx], optimize=True)
        return dW, dX

    dW, dX = both(d, X, W)
    out = {"dW": dW, "dX": dX, "db": d.sum(axis=(0, 2, 3))}
    if with_abs:
        sW, sX = both(np.abs(d), np.abs(X), np.abs(W))
        out["S_dW"], out["S_dX"] = sW, sX
        out["S_db"] = np.abs(d).sum(axis=(0, 2, 3))
    return out


# ---- brute force on tiny shapes: the definitions as nested loops, no library contraction ----

def linear_backward_bruteforce(codes, Delta, X, W):
    D = float(np.float32(Delta))
    B, N = np.shape(codes)
    K = np.shape(X)[1]
    dW = [[0.0] * K for _ in range(N)]
    dX = [[0.0] * K for _ in range(B)]
    db = [0.0] * N
    for b in range(B):
        for j in range(N):
            t = float(codes[b][j]) * D
            db[j] += t
            for k in range(K):
                dW[j][k] += t * float(X[b][k])
                dX[b][k] += t * float(W[j][k])
    return {"dW": np.array(dW), "dX": np.array(dX), "db": np.array(db)}


def conv_backward_bruteforce(codes, Delta, X, W):
    D = float(np.float32(Delta))
    codes = np.asarray(codes)
    X = np.asarray(X, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    B, Co, H, Wd = codes.shape
    Ci = X.shape[1]
    k = W.shape[2]
    p = (k - 1) // 2
    dW = np.zeros((Co, Ci, k, k))
    dX = np.zeros((B, Ci, H, Wd))
    db = np.zeros(Co)
    for b in range(B):
        for co in range(Co):
            for y in range(H):
                for x in range(Wd):
                    t = float(codes[b, co, y, x]) * D
                    if t == 0.0:
                        continue
                    db[co] += t
                    for ci in range(Ci):
                        for ky in range(k):
                            for kx in range(k):
                                yy, xx = y + ky - p, x + kx - p
                                if 0 <= yy < H and 0 <= xx < Wd:
                                    # forward term z[b,co,y,x] += W[co,ci,ky,kx] X[b,ci,yy,xx]
                                    dW[co, ci, ky, kx] += t * X[b, ci, yy, xx]
                                    dX[b, ci, yy, xx] += t * W[co, ci, ky, kx]
    return {"dW": dW, "dX": dX, "db": db}


# ---- single outputs of the same definitions (for full-size tensors, where the whole product
# ---- in fp64 would take minutes): each value is the defining sum written out for one index.

def _shifted_dot(q, x, ky, kx, p):
    """sum_{b,y,x} q[b,y,x] * x[b,y+ky-p,x+kx-p] with zero padding, and the sum of |terms|."""
    B, H, Wd = q.shape
    dy, dx = ky - p, kx - p
    y0, y1 = max(0, -dy), min(H, H - dy)
    x0, x1 = max(0, -dx), min(Wd, Wd - dx)
    if y0 >= y1 or x0 >= x1:
        return 0.0, 0.0
    t = q[:, y0:y1, x0:x1] * x[:, y0 + dy:y1 + dy, x0 + dx:x1 + dx]
    return float(t.sum()), float(np.abs(t).sum())


def conv_dW_entry(codes, Delta, X, co, ci, ky, kx, k):
    """(dW[co,ci,ky,kx], sum |terms|) from the definition for a k x k kernel, padding (k-1)/2;
    codes [B,Co,H,W], X [B,Ci,H,W]."""
    D = float(np.float32(Delta))
    q = np.asarray(codes[:, co], dtype=np.float64) * D
    x = np.asarray(X[:, ci], dtype=np.float64)
    return _shifted_dot(q, x, ky, kx, (k - 1) // 2)


def conv_dX_entry(codes, Delta, W, b, ci, y, x):
    """(dX[b,ci,y,x], sum |terms|): sum_{co,ky,kx} delta~[b,co,y-ky+p,x-kx+p] W[co,ci,ky,kx]."""
    D = float(np.float32(Delta))
    Co, _, k, _ = W.shape
    p = (k - 1) // 2
    H, Wd = codes.shape[2], codes.shape[3]
    tot = 0.0
    tot_abs = 0.0
    for ky in range(k):
        for kx in range(k):
            yy, xx = y - ky + p, x - kx + p
            if 0 <= yy < H and 0 <= xx < Wd:
                t = np.asarray(codes[b, :, yy, xx], dtype=np.float64) * D * np.asarray(W[:, ci, ky, kx], dtype=np.float64)
                tot += float(t.sum())
                tot_abs += float(np.abs(t).sum())
    return tot, tot_abs


# ---- strided convolution (the down-sampling layers of residual networks): the same
# ---- definitions with the input sampled every `stride` positions,
#   z[b,co,y,x]      = sum_{ci,ky,kx} W[co,ci,ky,kx] X[b,ci,s*y+ky-p,s*x+kx-p],  p = (k-1)/2,
#   Ho = (H + 2p - k) // s + 1,  Wo likewise,
#   dW[co,ci,ky,kx]  = sum_{b,y,x} delta~[b,co,y,x] X[b,ci,s*y+ky-p,s*x+kx-p]
#   dX[b,ci,y',x']   = sum over the (co,ky,kx,y,x) with s*y+ky-p = y', s*x+kx-p = x' of
#                      delta~[b,co,y,x] W[co,ci,ky,kx]

def strided_out_size(H, k, stride):
    return (H + 2 * ((k - 1) // 2) - k) // stride + 1


def conv_forward_strided(X, W, stride):
    X = np.asarray(X, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    B, Ci, H, Wd = X.shape
    Co, _, k, _ = W.shape
    p, s = (k - 1) // 2, int(stride)
    Ho, Wo = strided_out_size(H, k, s), strided_out_size(Wd, k, s)
    Xp = _pad_hw(X, p)
    z = np.zeros((B, Co, Ho, Wo))
    for ky in range(k):
        for kx in range(k):
            xs = Xp[:, :, ky:ky + s * (Ho - 1) + 1:s, kx:kx + s * (Wo - 1) + 1:s]
            z += np.einsum("bchw,oc->bohw", xs, W[:, :, ky, kx], optimize=True)
    return z


def conv_backward_strided(codes, Delta, X, W, stride, with_abs=False):
    """codes [B,Co,Ho,Wo], X [B,Ci,H,W], W [Co,Ci,k,k] -> dict(dW, dX, db) in fp64."""
    d = _dq(codes, Delta)
    X = np.asarray(X, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    B, Co, Ho, Wo = d.shape
    _, Ci, H, Wd = X.shape
    k = W.shape[2]
    p, s = (k - 1) // 2, int(stride)
    assert W.shape == (Co, Ci, k, k) and k % 2 == 1
    assert Ho == strided_out_size(H, k, s) and Wo == strided_out_size(Wd, k, s)

    def both(dd, XX, WW):
        Xp = _pad_hw(XX, p)
        dXp = np.zeros_like(Xp)
        dW = np.zeros((Co, Ci, k, k))
        for ky in range(k):
            for kx in range(k):
                ys = slice(ky, ky + s * (Ho - 1) + 1, s)      # padded rows s*y + ky
                xs = slice(kx, kx + s * (Wo - 1) + 1, s)
                dW[:, :, ky, kx] = np.einsum("bohw,bchw->oc", dd, Xp[:, :, ys, xs], optimize=True)
                dXp[:, :, ys, xs] += np.einsum("bohw,oc->bchw", dd, WW[:, :, ky, kx], optimize=True)
        return dW, dXp[:, :, p:p + H, p:p + Wd]

    dW, dX = both(d, X, W)
    out = {"dW": dW, "dX": dX, "db": d.sum(axis=(0, 2, 3))}
    if with_abs:
        sW, sX = both(np.abs(d), np.abs(X), np.abs(W))
        out["S_dW"], out["S_dX"] = sW, sX
        out["S_db"] = np.abs(d).sum(axis=(0, 2, 3))
    return out


def conv_backward_strided_bruteforce(codes, Delta, X, W, stride):
    D = float(np.float32(Delta))
    codes = np.asarray(codes)
    X = np.asarray(X, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    B, Co, Ho, Wo = codes.shape
    _, Ci, H, Wd = X.shape
    k = W.shape[2]
    p, s = (k - 1) // 2, int(stride)
    dW = np.zeros((Co, Ci, k, k))
    dX = np.zeros((B, Ci, H, Wd))
    db = np.zeros(Co)
    for b in range(B):
        for co in range(Co):
            for y in range(Ho):
                for x in range(Wo):
                    t = float(codes[b, co, y, x]) * D
                    if t == 0.0:
                        continue
                    db[co] += t
                    for ci in range(Ci):
                        for ky in range(k):
                            for kx in range(k):
                                yy, xx = s * y + ky - p, s * x + kx - p
                                if 0 <= yy < H and 0 <= xx < Wd:
                                    dW[co, ci, ky, kx] += t * X[b, ci, yy, xx]
                                    dX[b, ci, yy, xx] += t * W[co, ci, ky, kx]
    return {"dW": dW, "dX": dX, "db": db}
