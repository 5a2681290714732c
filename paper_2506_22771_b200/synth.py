"""Seeded synthetic inputs shaped like the paper's workloads (Sec. V-A: MNIST-style MLP data,
CIFAR-style CNN data).  Serves the oracle tests, the GPU parity tests and the benchmark alike,
and holds none of the method's arithmetic: it only draws numbers, writes the one-hot label
into the input (the positive / negative set generation of Alg. 1, sample generation; Sec. III) and scales
each sample to the length the first layer expects (the layer-1 input arrives length-normalised).

Nothing here is real MNIST / CIFAR-10 data: only their shapes and value ranges are used.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List

import numpy as np

F32 = np.float32


@dataclass
class LayerCfg:
    kind: int          # 0 linear, 1 conv3x3 (stride 1, pad 1, NHWC), 2 conv1x1 (pointwise, NHWC)
    K: int
    N: int
    theta: float
    lr: float
    tau: float
    H: int = 1
    Wd: int = 1
    Cin: int = 0
    eps: float = 1e-8
    stride: int = 1    # conv3x3 only
    momentum: float = 0.0   # heavy-ball coefficient of the update (0: plain SGD); Adam: beta1
    optimizer: int = 0      # 0 SGD / heavy ball, 1 Adam
    beta2: float = 0.999
    adam_eps: float = 1e-8
    pool: int = 1           # 2: 2x2 max pooling of the normalised output before the next layer
    skip_from: int = -1     # >= 0: the input of that layer is added to this layer's normalised output (residual block)
    skip_scale: float = 1.0


@dataclass
class Workload:
    name: str
    B: int                       # positives per batch = negatives per batch
    layers: List[LayerCfg]
    in_shape: tuple              # per-sample input shape
    data: str                    # "uniform01" | "normal"
    weights: str                 # "kaiming_uniform" | "normal_1_over_k"
    steps: int
    lam_per_step: float = 0.0    # look-ahead lambda increment per step (0: vanilla)
    greedy: bool = False         # train layers one after another (config 2)


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed & 0xFFFFFFFFFFFFFFFF, stream]))


def _mlp(widths, theta=None, lr=0.03):
    out = []
    for K, N in zip(widths[:-1], widths[1:]):
        out.append(LayerCfg(0, K, N, float(N if theta is None else theta), lr, float(np.sqrt(N))))
    return out


def workload(name: str) -> Workload:
    """The five benchmark configurations (sizes only; data are drawn by make_*)."""
    if name == "tiny_mlp":          # config 1
        return Workload(name, 64, _mlp([784, 500, 500]), (784,), "uniform01", "kaiming_uniform", 10)
    if name == "mlp_greedy":        # config 2
        return Workload(name, 1024, _mlp([784, 2000, 2000, 2000, 2000]), (784,), "uniform01",
                        "kaiming_uniform", 58, greedy=True)
    if name == "mlp_lookahead":     # config 3
        return Workload(name, 4096, _mlp([784, 2000, 2000, 2000, 2000]), (784,), "uniform01",
                        "kaiming_uniform", 200, lam_per_step=0.001)
    if name == "cnn":               # config 4
        chans = [3, 64, 128, 256]
        # theta = number of outputs per sample (goodness is a sum over C_out*H*W activities); the
        # step size is the MLP one divided by the H*W positions a filter's gradient sums over
        layers = [LayerCfg(1, 9 * ci, co, float(co * 1024), 0.03 / 1024.0, float(np.sqrt(co * 1024)),
                           H=32, Wd=32, Cin=ci) for ci, co in zip(chans[:-1], chans[1:])]
        return Workload(name, 256, layers, (32, 32, 3), "normal", "kaiming_uniform", 50)
    if name == "separable":         # beyond the five configurations: one inverted-residual-style block (without the
        # skip connection) of the paper's mobile models at CIFAR size: pointwise 32 -> 192, depthwise 3x3 on 192
        # channels, pointwise 192 -> 64, all 32 x 32; theta and step size as for the CNN workload
        hw = 32 * 32
        mk = lambda kind, K, N, cin: LayerCfg(kind, K, N, float(N * hw), 0.03 / hw, float(np.sqrt(N * hw)), H=32, Wd=32, Cin=cin)
        layers = [mk(2, 32, 192, 32), mk(3, 9, 192, 192), mk(2, 192, 64, 192)]
        return Workload(name, 256, layers, (32, 32, 32), "normal", "kaiming_uniform", 50)
    if name == "roofline":          # config 5
        return Workload(name, 16384, [LayerCfg(0, 8192, 8192, 4096.0, 0.03, float(np.sqrt(8192)))],
                        (8192,), "normal", "normal_1_over_k", 100)
    raise KeyError(name)


def scaled(w: Workload, B: int = None, width_div: int = 1) -> Workload:
    """A smaller copy of a workload (fewer rows and/or narrower layers) for parity tests."""
    layers = []
    for l in w.layers:
        first = l is w.layers[0]
        per = l.H * l.Wd
        ratio = l.theta / float(l.N * per)          # theta relative to the layer's output size
        if l.kind == 0:
            K = l.K if first else max(8, l.K // width_div)
            N = max(8, l.N // width_div)
            layers.append(LayerCfg(0, K, N, ratio * N, l.lr, float(np.sqrt(N))))
        else:
            Cin = l.Cin if first else max(4, l.Cin // width_div)
            N = max(4, l.N // width_div)
            layers.append(LayerCfg(1, 9 * Cin, N, ratio * N * per, l.lr, float(np.sqrt(N * per)),
                                   H=l.H, Wd=l.Wd, Cin=Cin))
    return Workload(w.name + "_scaled", B or w.B, layers, w.in_shape, w.data, w.weights, w.steps,
                    w.lam_per_step, w.greedy)


def make_weights(w: Workload, seed: int) -> List[np.ndarray]:
    """Random-init FP32 weights [N,K] per layer (conv: [N,3,3,Cin] flattened to [N,9*Cin])."""
    out = []
    for i, l in enumerate(w.layers):
        g = _rng(seed, 1000 + i)
        if w.weights == "kaiming_uniform":
            bound = np.sqrt(6.0 / l.K)
            Wt = g.uniform(-bound, bound, size=(l.N, l.K))
        else:
            Wt = g.normal(0.0, np.sqrt(1.0 / l.K), size=(l.N, l.K))
        out.append(np.ascontiguousarray(Wt.astype(F32)))
    return out


def _draw_labelled(w: Workload, seed: int, batch_index: int, B: int):
    """B raw samples (float64), their labels and one wrong label each."""
    g = _rng(seed, 2000 + batch_index)
    n_in = int(np.prod(w.in_shape))
    if w.data == "uniform01":
        base = g.random((B, n_in), dtype=np.float64)
    else:
        base = g.normal(0.0, 1.0, size=(B, n_in))
    label = g.integers(0, 10, size=B)
    wrong = (label + g.integers(1, 10, size=B)) % 10
    return base, label, wrong


def make_raw(w: Workload, seed: int, batch_index: int = 0, B: int = None):
    """The labelled samples make_batch builds its batch from: (samples [B, n_in] FP32, labels [2, B] INT32 with
    row 0 the true and row 1 the wrong label, label stride = distance in values between two label places)."""
    B = B or w.B
    base, label, wrong = _draw_labelled(w, seed, batch_index, B)
    stride = 1 if len(w.in_shape) == 1 else int(w.in_shape[-1])
    return np.ascontiguousarray(base.astype(F32)), np.stack([label, wrong]).astype(np.int32), stride


def make_batch(w: Workload, seed: int, batch_index: int = 0, B: int = None) -> np.ndarray:
    """One batch [2B, *in_shape] FP32: rows 0..B-1 positive (true label), B..2B-1 negative (a
    random wrong label), label written one-hot into the first 10 entries (CNN: channel 0, row 0,
    pixels 0..9), each sample scaled to length tau0 = sqrt(number of input values)."""
    B = B or w.B
    base, label, wrong = _draw_labelled(w, seed, batch_index, B)
    n_in = base.shape[1]
    x = np.concatenate([base, base], axis=0).reshape((2 * B,) + tuple(w.in_shape))
    for p, lab in enumerate((label, wrong)):
        rows = np.arange(B) + p * B
        if len(w.in_shape) == 1:
            x[rows, :10] = 0.0
            x[rows, lab] = 1.0
        else:
            x[rows, 0, :10, 0] = 0.0
            x[rows, 0, lab, 0] = 1.0
    flat = x.reshape(2 * B, -1)
    norm = np.sqrt((flat ** 2).sum(axis=1, keepdims=True))
    flat *= np.sqrt(float(n_in)) / (norm + 1e-8)
    return np.ascontiguousarray(x.astype(F32))


def make_candidates(w: Workload, seed: int, B: int, n_classes: int = 10, batch_index: int = 0):
    """Candidate batch for classification [n_classes*B, *in_shape] FP32: row c*B + b is sample b with
    candidate label c written one-hot into it (same places as make_batch), each row scaled to length
    sqrt(number of input values).  Also returns the B drawn labels (random: the data carry no class
    structure, they only have the right shape)."""
    g = _rng(seed, 3000 + batch_index)
    n_in = int(np.prod(w.in_shape))
    if w.data == "uniform01":
        base = g.random((B, n_in), dtype=np.float64)
    else:
        base = g.normal(0.0, 1.0, size=(B, n_in))
    label = g.integers(0, n_classes, size=B)
    x = np.tile(base, (n_classes, 1)).reshape((n_classes * B,) + tuple(w.in_shape))
    for c in range(n_classes):
        rows = np.arange(B) + c * B
        if len(w.in_shape) == 1:
            x[rows, :n_classes] = 0.0
            x[rows, c] = 1.0
        else:
            x[rows, 0, :n_classes, 0] = 0.0
            x[rows, 0, c, 0] = 1.0
    flat = x.reshape(n_classes * B, -1)
    norm = np.sqrt((flat ** 2).sum(axis=1, keepdims=True))
    flat *= np.sqrt(float(n_in)) / (norm + 1e-8)
    return np.ascontiguousarray(x.astype(F32)), label.astype(np.int32)
