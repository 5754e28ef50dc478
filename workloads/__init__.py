"""Seeded synthetic inputs for the dithered-backprop layer shapes.

This module only *makes inputs* (activations X, weights W, preactivation gradients delta,
forward passes that produce the ReLU masks and the output-layer gradient of whole networks).
It holds none of the method's arithmetic (no quantizer, no backward product) and is the one
module that both the CUDA tests/bench and the CPU oracle's tests draw from, so that the two
sides read the same bytes.

The tensors stand in for the MNIST / CIFAR / ImageNet workloads of the paper's experiments:
same shapes and batch sizes, value distributions chosen to match what such layers see
(post-ReLU half-normal activations with ~50 % zeros, He/LeCun-initialised weights,
Laplace-like gradients masked by a ReLU derivative). Uniform numbers come from NumPy's PCG64
stream; every other distribution is derived here by inverse CDF / Box-Muller.
"""
from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np

# --------------------------------------------------------------------------- streams


def _rng(seed: int, tensor_id: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([int(seed), int(tensor_id)]))


def uniform01(seed, tensor_id, n) -> np.ndarray:
    """fp64 uniforms in (0,1) (0 excluded so that logs are finite)."""
    u = _rng(seed, tensor_id).random(int(n))
    return np.maximum(u, 2.0 ** -53)


def normal(seed, tensor_id, n, sigma=1.0) -> np.ndarray:
    """Box-Muller on two uniform streams."""
    n = int(n)
    m = (n + 1) // 2
    u = uniform01(seed, tensor_id, 2 * m)
    r = np.sqrt(-2.0 * np.log(u[:m]))
    th = 2.0 * np.pi * u[m:]
    z = np.concatenate([r * np.cos(th), r * np.sin(th)])[:n]
    return z * sigma


def laplace(seed, tensor_id, n, b=1.0) -> np.ndarray:
    """Inverse CDF of Laplace(0, b)."""
    u = uniform01(seed, tensor_id, n) - 0.5
    return -b * np.sign(u) * np.log1p(-2.0 * np.abs(u) + 2.0 ** -60)


def bernoulli(seed, tensor_id, n, p=0.5) -> np.ndarray:
    return _rng(seed, tensor_id).random(int(n)) < p


# --------------------------------------------------------------------------- bf16 helpers


def f32_to_bf16_bits(a) -> np.ndarray:
    """Round fp32 to bfloat16 (nearest even); returns the 16-bit patterns (uint16)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(bits) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def round_to_bf16(a) -> np.ndarray:
    """fp32 array holding bf16-representable values."""
    return bf16_bits_to_f32(f32_to_bf16_bits(a)).reshape(np.shape(a))


# --------------------------------------------------------------------------- single layers


@dataclass
class Layer:
    """One layer's backward inputs. kind 'linear': delta [B,N], X [B,K], W [N,K].
    kind 'conv': delta [B,Cout,H/stride,W/stride], X [B,Cin,H,W], W [Cout,Cin,k,k] (NCHW,
    pad (k-1)/2). Arrays are fp32; with dtype 'bf16' their values are bf16-representable."""
    name: str
    kind: str
    delta: np.ndarray
    X: np.ndarray
    W: np.ndarray
    scale: float
    seed: int = 0
    dtype: str = "f32"
    k: int = 1
    stride: int = 1

    @property
    def dense_flops(self) -> float:
        """2 flops per MAC, both products."""
        if self.kind == "linear":
            B, N = self.delta.shape
            return 4.0 * B * N * self.X.shape[1]
        B, Co, H, Wd = self.delta.shape
        return 4.0 * B * H * Wd * Co * self.X.shape[1] * self.k * self.k


def _cast(a, dtype):
    a = np.asarray(a, dtype=np.float32)
    return round_to_bf16(a) if dtype == "bf16" else a


def linear_layer(B, N, K, *, data_seed, b_laplace=1e-3, keep=0.5, scale=2.0, seed=0,
                 dtype="f32", name=None) -> Layer:
    X = uniform01(data_seed, 1, B * K).reshape(B, K)
    W = normal(data_seed, 2, N * K, sigma=(1.0 / K) ** 0.5).reshape(N, K)
    d = laplace(data_seed, 3, B * N, b=b_laplace) * bernoulli(data_seed, 4, B * N, keep)
    return Layer(name or f"linear_B{B}_{K}to{N}", "linear", _cast(d.reshape(B, N), dtype),
                 _cast(X, dtype), _cast(W, dtype), scale, seed, dtype, 1)


def conv_layer(B, Cin, Cout, H, Wd, k, *, data_seed, b_laplace=1e-4, keep=0.5, scale=2.0,
               seed=0, dtype="f32", name=None, stride=1) -> Layer:
    nX = B * Cin * H * Wd
    X = np.maximum(normal(data_seed, 1, nX), 0.0).reshape(B, Cin, H, Wd)   # post-ReLU
    W = normal(data_seed, 2, Cout * Cin * k * k, sigma=(2.0 / (Cin * k * k)) ** 0.5)
    W = W.reshape(Cout, Cin, k, k)                                          # He init
    Ho, Wo = H // stride, Wd // stride                                      # even H, W for stride 2
    nd = B * Cout * Ho * Wo
    d = laplace(data_seed, 3, nd, b=b_laplace) * bernoulli(data_seed, 4, nd, keep)
    tag = f"_s{stride}" if stride != 1 else ""
    return Layer(name or f"conv{k}x{k}{tag}_B{B}_{Cin}to{Cout}_{H}x{Wd}", "conv",
                 _cast(d.reshape(B, Cout, Ho, Wo), dtype), _cast(X, dtype), _cast(W, dtype),
                 scale, seed, dtype, k, stride)


def config1(batch=128) -> Layer:
    """Single linear layer backward, fp32: 784 -> 300, Delta = 2 std(delta), seed 0."""
    return linear_layer(batch, 300, 784, data_seed=1001, b_laplace=1e-3, scale=2.0,
                        name="cfg1_linear_784to300")


def config3(batch=128, channels=64, hw=32) -> Layer:
    """Single 3x3 conv layer backward, fp32: 64 -> 64 channels at 32x32."""
    return conv_layer(batch, channels, channels, hw, hw, 3, data_seed=1003, b_laplace=1e-4,
                      scale=2.0, name="cfg3_conv3x3_64to64_32x32")


# ResNet-50 bottleneck layer set (stride-1 shapes): (name, Cin, Cout, HW, k, multiplicity).
# Stage width w in {64,128,256,512} at {56,28,14,7}^2 with {3,4,6,3} blocks: every block has
# 1x1 reduce (4w->w; the first block of a stage reduces from the previous stage's width),
# 3x3 (w->w) and 1x1 expand (w->4w).
RESNET50_SET = [
    ("s1_reduce_first", 64, 64, 56, 1, 1), ("s1_reduce", 256, 64, 56, 1, 2),
    ("s1_conv3x3", 64, 64, 56, 3, 3), ("s1_expand", 64, 256, 56, 1, 3),
    ("s2_reduce_first", 256, 128, 56, 1, 1), ("s2_reduce", 512, 128, 28, 1, 3),
    ("s2_conv3x3", 128, 128, 28, 3, 4), ("s2_expand", 128, 512, 28, 1, 4),
    ("s3_reduce_first", 512, 256, 28, 1, 1), ("s3_reduce", 1024, 256, 14, 1, 5),
    ("s3_conv3x3", 256, 256, 14, 3, 6), ("s3_expand", 256, 1024, 14, 1, 6),
    ("s4_reduce_first", 1024, 512, 14, 1, 1), ("s4_reduce", 2048, 512, 7, 1, 2),
    ("s4_conv3x3", 512, 512, 7, 3, 3), ("s4_expand", 512, 2048, 7, 1, 3),
]


# The stride-2 layers of the same network (torchvision's placement: the stride sits on the 3x3 layer of a
# stage's first block and on its 1x1 shortcut projection): (name, Cin, Cout, input HW, k).
RESNET50_STRIDED = [
    ("s2_conv3x3_down", 128, 128, 56, 3), ("s2_shortcut", 256, 512, 56, 1),
    ("s3_conv3x3_down", 256, 256, 28, 3), ("s3_shortcut", 512, 1024, 28, 1),
    ("s4_conv3x3_down", 512, 512, 14, 3), ("s4_shortcut", 1024, 2048, 14, 1),
]


def resnet50_strided_layer(idx, batch=64, scale=5.0, dtype="bf16") -> Layer:
    name, ci, co, hw, k = RESNET50_STRIDED[idx]
    return conv_layer(batch, ci, co, hw, hw, k, data_seed=2005 + 16 * idx, b_laplace=1e-4,
                      scale=scale, dtype=dtype, name=name, stride=2)


def config5_layer(idx, batch=64, scale=5.0, dtype="bf16") -> Layer:
    """One shape of the ResNet-50 ImageNet-shaped set: bf16 storage, Delta = 5 std(delta)
    (about 90 % zeros after quantization for a Laplace gradient with a 50 % ReLU mask)."""
    name, ci, co, hw, k, _ = RESNET50_SET[idx]
    return conv_layer(batch, ci, co, hw, hw, k, data_seed=1005 + 16 * idx, b_laplace=1e-4,
                      scale=scale, dtype=dtype, name="cfg5_" + name)


# --------------------------------------------------------------------------- whole networks


@dataclass
class Chain:
    """A feed-forward network after its forward pass: per layer (in forward order) the input
    activation, the weight, the ReLU derivative mask of its output (None for the last layer)
    and whether a 2x2 max-pool follows (with the flat argmax index of each pooled value)."""
    name: str
    kinds: List[str]
    X: List[np.ndarray]
    W: List[np.ndarray]
    relu_mask: List[Optional[np.ndarray]]
    pool_argmax: List[Optional[np.ndarray]]
    delta_out: np.ndarray
    scale: float
    seed: int = 0
    extra: Dict = field(default_factory=dict)


def _softmax_minus_onehot(logits, labels):
    z = logits.astype(np.float64)
    z = z - z.max(axis=1, keepdims=True)
    p = np.exp(z)
    p /= p.sum(axis=1, keepdims=True)
    p[np.arange(len(labels)), labels] -= 1.0
    return (p / len(labels)).astype(np.float32)       # mean-reduced cross-entropy


def mlp_chain(batch=256, dims=(784, 300, 100, 10), *, data_seed=1002, scale=2.0) -> Chain:
    """LeNet-300-100-shaped MLP: W ~ N(0, 1/fan_in), zero bias, inputs U(0,1), random labels."""
    a = uniform01(data_seed, 1, batch * dims[0]).reshape(batch, dims[0]).astype(np.float32)
    Xs, Ws, masks = [], [], []
    L = len(dims) - 1
    for l in range(L):
        W = normal(data_seed, 10 + l, dims[l + 1] * dims[l], sigma=(1.0 / dims[l]) ** 0.5)
        W = W.reshape(dims[l + 1], dims[l]).astype(np.float32)
        z = (a.astype(np.float64) @ W.astype(np.float64).T).astype(np.float32)
        Xs.append(a)
        Ws.append(W)
        if l < L - 1:
            masks.append(z > 0)
            a = np.maximum(z, 0.0).astype(np.float32)
        else:
            masks.append(None)
    labels = (uniform01(data_seed, 2, batch) * dims[-1]).astype(np.int64) % dims[-1]
    return Chain("mlp_" + "_".join(map(str, dims)), ["linear"] * L, Xs, Ws, masks, [None] * L,
                 _softmax_minus_onehot(z, labels), scale)


VGG16_CIFAR = [64, 64, "M", 128, 128, "M", 256, 256, 256, "M", 512, 512, 512, "M",
               512, 512, 512, "M"]


def vgg_chain(batch=128, cfg=None, hw=32, in_ch=3, classes=10, *, data_seed=1004,
              scale=2.0, device="cpu", k=3, name="vgg16_cifar") -> Chain:
    """VGG-16 (CIFAR variant, no batch-norm): k x k convs (3x3 unless asked) + ReLU, 2x2 max-pool after each
    stage, one fully-connected classifier; He-initialised weights, N(0,1) input, random
    labels. The forward pass runs through torch (on `device`) -- it only makes inputs."""
    import torch
    import torch.nn.functional as F
    cfg = VGG16_CIFAR if cfg is None else cfg
    a = torch.from_numpy(normal(data_seed, 1, batch * in_ch * hw * hw)
                         .reshape(batch, in_ch, hw, hw).astype(np.float32)).to(device)
    kinds, Xs, Ws, masks, pools = [], [], [], [], []
    c, li = in_ch, 0
    i = 0
    while i < len(cfg):
        co = cfg[i]
        W = normal(data_seed, 10 + li, co * c * k * k, sigma=(2.0 / (c * k * k)) ** 0.5)
        W = torch.from_numpy(W.reshape(co, c, k, k).astype(np.float32)).to(device)
        z = F.conv2d(a, W, padding=(k - 1) // 2)
        kinds.append("conv")
        Xs.append(a.cpu().numpy())
        Ws.append(W.cpu().numpy())
        masks.append((z > 0).cpu().numpy())
        a = torch.relu(z)
        if i + 1 < len(cfg) and cfg[i + 1] == "M":
            B_, C_, H_, W_ = a.shape
            win = a.reshape(B_, C_, H_ // 2, 2, W_ // 2, 2).permute(0, 1, 2, 4, 3, 5)
            win = win.reshape(B_, C_, H_ // 2, W_ // 2, 4)
            am = win.argmax(dim=-1)            # first maximum in row-major window order
            pools.append(am.cpu().numpy().astype(np.int8))
            a = win.gather(-1, am.unsqueeze(-1)).squeeze(-1)
            i += 1
        else:
            pools.append(None)
        c = co
        li += 1
        i += 1
    feat = a.reshape(batch, -1)
    Wfc = normal(data_seed, 10 + li, classes * feat.shape[1], sigma=(2.0 / feat.shape[1]) ** 0.5)
    Wfc = torch.from_numpy(Wfc.reshape(classes, feat.shape[1]).astype(np.float32)).to(device)
    logits = feat @ Wfc.T
    kinds.append("linear")
    Xs.append(feat.cpu().numpy())
    Ws.append(Wfc.cpu().numpy())
    masks.append(None)
    pools.append(None)
    labels = (uniform01(data_seed, 2, batch) * classes).astype(np.int64) % classes
    return Chain(name, kinds, Xs, Ws, masks, pools,
                 _softmax_minus_onehot(logits.cpu().numpy(), labels), scale,
                 extra={"feat_shape": tuple(a.shape)})
