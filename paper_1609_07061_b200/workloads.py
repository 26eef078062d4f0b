"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds NO arithmetic of the method (no sign, no quantiser, no
packing): it only draws random real / integer tensors with the shapes and value
distributions of the paper's networks, so that the CUDA library and the CPU
oracle can be fed byte-identical inputs.  The paper's data sets and trained
weights are not available; these tensors stand in for them.

Every workload owns one ``torch.Generator`` on the CPU, seeded with
``seed * 1000 + stream``; tensors are drawn in the fixed order
inputs -> weights (layer by layer) -> thresholds.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Tuple

import torch


def _gen(seed: int, stream: int = 0) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed * 1000 + stream)
    return g


def _normal(g, *shape) -> torch.Tensor:
    return torch.randn(*shape, generator=g, dtype=torch.float32)


def _uniform_pm1(g, *shape) -> torch.Tensor:
    return torch.rand(*shape, generator=g, dtype=torch.float32) * 2.0 - 1.0


def _thresholds(g, n: int, lo: int = -64, hi: int = 64) -> torch.Tensor:
    return torch.randint(lo, hi + 1, (n,), generator=g, dtype=torch.int32)


@dataclass
class FcLayer:
    """One fully-connected binary layer: fp32 activations and weights to be sign-binarised."""
    X: torch.Tensor  # [M, K] fp32
    W: torch.Tensor  # [K, N] fp32


def fc_single(M: int = 100, K: int = 4096, N: int = 4096, seed: int = 0) -> FcLayer:
    """Single 4096-unit binary layer at the paper's MNIST minibatch size of 100."""
    g = _gen(seed)
    X = _normal(g, M, K)
    W = _uniform_pm1(g, K, N)
    return FcLayer(X, W)


@dataclass
class MlpWorkload:
    """MNIST-shaped binarised MLP (Algorithm 4): 8-bit inputs, +-1 weights, integer thresholds."""
    X: torch.Tensor                     # [M, dims[0]] uint8
    Ws: List[torch.Tensor]              # fp32 [dims[l], dims[l+1]], to be sign-binarised
    Ts: List[torch.Tensor]              # int32 [dims[l+1]] for the hidden layers
    dims: Tuple[int, ...] = field(default=(784, 4096, 4096, 4096, 10))


def mnist_mlp(M: int = 10000, dims: Tuple[int, ...] = (784, 4096, 4096, 4096, 10), seed: int = 1,
              stream: int = 0) -> MlpWorkload:
    """784-4096-4096-4096-10 MLP over a test-set-sized batch of 28x28 8-bit images.

    ``stream`` selects an independent batch with the SAME weights and thresholds
    (used to give every data-parallel rank its own shard): weights and thresholds
    always come from stream 0, inputs from ``stream``.
    """
    gw = _gen(seed, 0)
    X0 = torch.randint(0, 256, (M, dims[0]), generator=gw, dtype=torch.uint8)
    Ws = [_uniform_pm1(gw, dims[l], dims[l + 1]) for l in range(len(dims) - 1)]
    Ts = [_thresholds(gw, dims[l + 1]) for l in range(len(dims) - 2)]
    if stream == 0:
        X = X0
    else:
        gx = _gen(seed, stream)
        X = torch.randint(0, 256, (M, dims[0]), generator=gx, dtype=torch.uint8)
    return MlpWorkload(X, Ws, Ts, tuple(dims))


@dataclass
class KbitFcWorkload:
    """AlexNet-FC-shaped layers: k-bit unsigned activations on [lo, hi], +-1 weights."""
    Xs: List[torch.Tensor]              # fp32 [M, K_l], one per layer (layers are independent)
    Ws: List[torch.Tensor]              # fp32 [K_l, N_l]
    bits: int = 2
    lo: float = 0.0
    hi: float = 1.0


def alexnet_fc(M: int = 256, shapes=((9216, 4096), (4096, 4096), (4096, 1000)), seed: int = 2,
               bits: int = 2) -> KbitFcWorkload:
    g = _gen(seed)
    Xs = [torch.relu(_normal(g, M, k)) for (k, _) in shapes]
    Ws = [_uniform_pm1(g, k, n) for (k, n) in shapes]
    return KbitFcWorkload(Xs, Ws, bits, 0.0, 1.0)


@dataclass
class ConvWorkload:
    """CIFAR-style binary 3x3 'same' convolution followed by a per-channel threshold."""
    X: torch.Tensor   # [B, C, H, W] fp32
    W: torch.Tensor   # [Cout, C, KH, KW] fp32
    T: torch.Tensor   # [Cout] int32
    stride: int = 1
    pad: int = 1


def cifar_conv(B: int = 128, C: int = 256, H: int = 16, W: int = 16, Cout: int = 256, KH: int = 3,
               KW: int = 3, seed: int = 3) -> ConvWorkload:
    g = _gen(seed)
    X = _normal(g, B, C, H, W)
    Wt = _uniform_pm1(g, Cout, C, KH, KW)
    T = _thresholds(g, Cout)
    return ConvWorkload(X, Wt, T, 1, 1)


@dataclass
class ConvNetWorkload:
    """The CIFAR-10 ConvNet of Table 7: 8-bit RGB images, three pairs of 3x3 'same' convolutions
    (the second of each pair followed by 2x2 max-pooling), then fully connected layers."""
    X: torch.Tensor                     # [B, 3, H, W] uint8
    conv_W: List[torch.Tensor]          # fp32 [Cout, C, 3, 3], to be sign-binarised
    conv_pool: List[bool]               # 2x2 max-pooling after this convolution
    fc_W: List[torch.Tensor]            # fp32 [K, N]; the first reads the feature map in (h, w, c) order
    Ts: List[torch.Tensor]              # int32 thresholds, one per layer but the last
    flips: List[torch.Tensor]           # uint8 0/1 per channel, same layers


def cifar_convnet(B: int = 128, H: int = 32, W: int = 32, widths: Tuple[int, ...] = (128, 128, 256, 256, 512, 512),
                  fc: Tuple[int, ...] = (1024, 1024, 10), in_ch: int = 3, seed: int = 5, stream: int = 0,
                  flip_share: float = 0.25, thr: int = 64) -> ConvNetWorkload:
    """Weights, thresholds and flips come from stream 0, the images from ``stream``.  Thresholds are uniform in [-thr, thr]
    (narrow layers need a small thr to keep the bits data dependent); those of the pooled layers are centred near the typical maximum of four sums (about sqrt(K)) so that the bits stay mixed."""
    gw = _gen(seed, 0)
    X = torch.randint(0, 256, (B, in_ch, H, W), generator=gw, dtype=torch.uint8)
    conv_W, conv_pool, Ts, flips = [], [], [], []
    c, h, w = in_ch, H, W
    for i, co in enumerate(widths):
        conv_W.append(_uniform_pm1(gw, co, c, 3, 3))
        pool = (i % 2 == 1)
        conv_pool.append(pool)
        shift = int(round((9 * c) ** 0.5)) if pool else 0
        Ts.append(_thresholds(gw, co, -thr, thr) + shift)
        flips.append((torch.rand(co, generator=gw) < flip_share).to(torch.uint8))
        c = co
        if pool:
            h, w = h // 2, w // 2
    k = c * h * w
    fc_W = []
    for j, n in enumerate(fc):
        fc_W.append(_uniform_pm1(gw, k, n))
        if j < len(fc) - 1:
            Ts.append(_thresholds(gw, n, -thr, thr))
            flips.append((torch.rand(n, generator=gw) < flip_share).to(torch.uint8))
        k = n
    if stream != 0:
        X = torch.randint(0, 256, (B, in_ch, H, W), generator=_gen(seed, stream), dtype=torch.uint8)
    return ConvNetWorkload(X, conv_W, conv_pool, fc_W, Ts, flips)


def square_gemm(n: int, seed: int = 4) -> FcLayer:
    """Square binary GEMM M=N=K=n with N(0,1) operands (the paper timed 8192^3)."""
    g = _gen(seed, n)
    A = _normal(g, n, n)
    B = _normal(g, n, n)
    return FcLayer(A, B)


@dataclass
class LstmGateWorkload:
    """4-bit x 4-bit gate matmul of a recurrent layer: values on 16 uniform levels of [-1, 1]."""
    X: torch.Tensor   # [M, K] fp32, each value -1 + 2 q / 15
    W: torch.Tensor   # [K, N] fp32, same level set
    bits: int = 4
    lo: float = -1.0
    hi: float = 1.0


def lstm_gate(M: int = 700, K: int = 2048, N: int = 4096, seed: int = 4, bits: int = 4) -> LstmGateWorkload:
    g = _gen(seed, 1)
    L = (1 << bits) - 1
    qx = torch.randint(0, L + 1, (M, K), generator=g, dtype=torch.int32)
    qw = torch.randint(0, L + 1, (K, N), generator=g, dtype=torch.int32)
    X = (-1.0 + 2.0 * qx.to(torch.float32) / float(L)).to(torch.float32)
    W = (-1.0 + 2.0 * qw.to(torch.float32) / float(L)).to(torch.float32)
    return LstmGateWorkload(X, W, bits, -1.0, 1.0)


def binary_ops_mlp(M: int, dims: Tuple[int, ...], in_bits: int = 8) -> Dict[str, float]:
    """Operation counts of one MLP pass: 2*M*N*K per 1-bit plane product (bookkeeping only)."""
    per_layer = []
    for l in range(len(dims) - 1):
        planes = in_bits if l == 0 else 1
        per_layer.append(2.0 * M * dims[l + 1] * dims[l] * planes)
    return {"per_layer": per_layer, "total": float(sum(per_layer))}
