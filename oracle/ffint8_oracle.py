"""CPU oracle for the FF-INT8 per-layer train step.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain restatement of what the CUDA library computes.  Only the
tests, the smoke check and the benchmark's CPU-baseline leg may import it; the product
path never does, and this module imports nothing from the CUDA package.

Every function follows one passage of the FF-INT8 paper (cited per function).  Where the
paper leaves arithmetic unspecified, the function implements the written numerics contract
of this project (one correctly rounded IEEE operation at a time, in a stated order, no
fused multiply-add), so that the INT8 tensors it produces have exactly one correct bit
pattern.  numpy float32/float64 ufuncs are individually correctly rounded and never
contracted, which is what makes numpy a suitable language for that contract.

Notation (paper, Sec. IV-B and Algorithm 1): A / X = layer input, W = weights, Y = neuron
activity, G = goodness = ||y||^2, theta = threshold, g^Y = dH = dL/dY, g^W = dW.
Rows 0..B-1 of every batch tensor are the positive set, rows B..2B-1 the negative set.

Pins (tests/test_oracle_*.py): hand-computed tiny layers, closed forms of Eq. 1-2,
brute-force loops, finite differences of the unquantised loss, quantiser error bounds,
library cross-checks (float64 conv2d).  Parity unpinned: the look-ahead *gradient* (Eq. 4)
is a reading of the paper (scalar-coefficient look-ahead); only its closed form, its
lambda=0 and single-layer reductions are pinned.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

F32 = np.float32
F64 = np.float64

ROUND_NEAREST = 0
ROUND_STOCHASTIC = 1

ROLE_X = 0   # hash stream of the layer-input quantiser
ROLE_W = 1   # hash stream of the weight quantiser
ROLE_DH = 2  # hash stream of the output-gradient quantiser

KIND_LINEAR = 0
KIND_CONV3X3 = 1
KIND_CONV1X1 = 2
KIND_DWCONV3X3 = 3

_M64 = (1 << 64) - 1


# --------------------------------------------------------------------------------------
# Layer description
# --------------------------------------------------------------------------------------
@dataclass
class LayerSpec:
    """One FF layer.  linear: X [2B,K] -> Y [2B,N].  conv3x3 (stride 1, zero pad 1, NHWC):
    X [2B,H,W,Cin] -> Y [2B,H,W,N] with K = 9*Cin and weights [N,3,3,Cin] flattened to [N,K].
    conv1x1 (pointwise, NHWC): X [2B,H,W,Cin] -> Y [2B,H,W,N] with K = Cin and weights [N,Cin].
    dwconv3x3 (depthwise: every channel has its own 3x3 filter; stride 1 or 2, zero pad 1, NHWC):
    X [2B,H,W,C] -> Y [2B,Ho,Wo,C] with N = Cin = C, K = 9 and weights [C,3,3] flattened to [C,9]."""
    kind: int
    K: int
    N: int
    theta: float
    lr: float
    tau: float            # length-normalisation target norm of the NEXT layer's input
    eps: float = 1e-8
    H: int = 1
    Wd: int = 1
    Cin: int = 0
    round_x: int = ROUND_STOCHASTIC
    round_w: int = ROUND_NEAREST
    round_dh: int = ROUND_STOCHASTIC
    seed: int = 0
    index: int = 0        # position of the layer in the network (feeds the rounding hash)
    stride: int = 1       # conv3x3 only: 1 or 2 (output (H-1)//stride + 1 by (Wd-1)//stride + 1)
    momentum: float = 0.0 # heavy-ball coefficient of the update; 0 = plain SGD (Adam: beta1)
    optimizer: int = 0    # 0 = SGD / heavy ball, 1 = Adam
    beta2: float = 0.999  # Adam only
    adam_eps: float = 1e-8
    pool: int = 1         # 2: the normalised output is max-pooled 2x2 (stride 2) before it feeds the next layer
    skip_from: int = -1   # >= 0: the (normalised, float32) INPUT of layer skip_from of the same call is added to this
                          # layer's normalised output before it feeds the next layer (a residual block's skip path)
    skip_scale: float = 1.0   # weight of the skip path

    @property
    def out_hw(self):
        if self.kind in (KIND_CONV3X3, KIND_DWCONV3X3):
            return (self.H - 1) // self.stride + 1, (self.Wd - 1) // self.stride + 1
        return self.H, self.Wd

    @property
    def rows_per_sample(self) -> int:
        """Output positions per sample."""
        if self.kind == KIND_LINEAR:
            return 1
        ho, wo = self.out_hw
        return ho * wo


# --------------------------------------------------------------------------------------
# Symmetric uniform quantiser with nearest / stochastic rounding  (Sec. IV; Sec. IV-B)
# --------------------------------------------------------------------------------------
def absmax(x: np.ndarray) -> np.float32:
    """Per-tensor max |x| (the SUQ range, Sec. IV).  Exact: max involves no rounding."""
    x = np.asarray(x, dtype=F32)
    if x.size == 0:
        return F32(0.0)
    if not np.all(np.isfinite(x)):
        raise FloatingPointError("non-finite value in a tensor to be quantised")
    return F32(np.max(np.abs(x)))


TINY_RANGE = F32(2.0 ** -100)


def scale_pair(a: np.float32):
    """SUQ scale s = a/127 and its reciprocal factor inv = 127/a, each ONE float32 division.
    A zero tensor quantises to all zeros: s = 1, inv = 0.  So does a tensor whose range is below
    2^-100 (127/a would leave the float32 range for subnormal a; such a gradient carries nothing)."""
    a = F32(a)
    if a < TINY_RANGE:
        return F32(1.0), F32(0.0)
    return F32(a / F32(127.0)), F32(F32(127.0) / a)


def _splitmix64(x: int) -> int:
    """SplitMix64 output function (Steele/Lea/Flood; public-domain reference by Vigna)."""
    x = (x + 0x9E3779B97F4A7C15) & _M64
    z = x
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def rounding_key(seed: int, role: int, layer: int, step: int):
    """Two 32-bit keys for one (seed, tensor role, layer, step) quantiser call."""
    s0 = _splitmix64(seed & _M64)
    s1 = _splitmix64(s0 ^ ((role & 0xFF) | ((layer & 0xFFFFFF) << 8)))
    s2 = _splitmix64(s1 ^ (step & _M64))
    return s2 & 0xFFFFFFFF, (s2 >> 32) & 0xFFFFFFFF


def rounding_uniform(idx: np.ndarray, k0: int, k1: int) -> np.ndarray:
    """u in [0,1) with 16 random bits for each linear element index (counter-based, so the
    value does not depend on how the tensor is tiled or which thread handles the element).
    One 32-bit hash serves the element pair (2j, 2j+1): low half for the even index, high half
    for the odd one."""
    idx = idx.astype(np.uint64)
    h = (idx >> np.uint64(1)).astype(np.uint32) ^ np.uint32(k0)
    h = h * np.uint32(0x9E3779B1)
    h = h ^ (h >> np.uint32(15))
    h = (h + np.uint32(k1)) * np.uint32(0x85EBCA6B)
    h = h ^ (h >> np.uint32(13))
    h = h * np.uint32(0xC2B2AE35)
    h = h ^ (h >> np.uint32(16))
    half = np.where((idx & np.uint64(1)) == 0, h & np.uint32(0xFFFF), h >> np.uint32(16))
    return half.astype(F32) * F32(2.0 ** -16)


def quantize(x: np.ndarray, a: np.float32, mode: int, key=None, idx0: int = 0,
             u: Optional[np.ndarray] = None) -> np.ndarray:
    """SUQ to INT8 in [-127,127], zero point 0 (Sec. IV).  t = x*inv (one multiply), then
    nearest-even (rint) or stochastic rounding floor(t+u) (Sec. IV-B, Gupta et al.), then clip.
    `idx0` is the linear index of x.flat[0] inside the whole tensor (for per-pass slices);
    `u` overrides the hash (used by the hand-computed pins)."""
    x = np.asarray(x, dtype=F32)
    if x.size >= 1 << 32:
        raise ValueError("tensor too large for 32-bit rounding counters")
    _, inv = scale_pair(a)
    t = x * inv
    if mode == ROUND_NEAREST:
        q = np.rint(t)
    else:
        if u is None:
            idx = (np.arange(x.size, dtype=np.uint64) + np.uint64(idx0)).reshape(x.shape)
            u = rounding_uniform(idx, key[0], key[1])
        q = np.floor(t + np.asarray(u, dtype=F32))
    return np.clip(q, -127.0, 127.0).astype(np.int8)


def quantize_two_pass(x: np.ndarray, B: int, mode: int, key, joint: bool = False):
    """Quantise the positive rows [0,B) and the negative rows [B,2B) with separate per-tensor
    scales (Sec. IV-B runs the quantised workflow once per set).  Returns q, (a_pos, a_neg).
    joint: one range for the whole tensor (both entries of the returned pair are that range) - for batches whose
    halves are not a positive and a negative set (the candidate batch of `predict`)."""
    q = np.empty(x.shape, dtype=np.int8)
    per_row = int(np.prod(x.shape[1:])) if x.ndim > 1 else 1
    a = []
    whole = absmax(x) if joint else None
    for p in range(2):
        sl = slice(p * B, (p + 1) * B)
        ap = whole if joint else absmax(x[sl])
        q[sl] = quantize(x[sl], ap, mode, key, idx0=p * B * per_row)
        a.append(ap)
    return q, (a[0], a[1])


# --------------------------------------------------------------------------------------
# INT8 MAC with INT32 accumulation  (Sec. IV-B)
# --------------------------------------------------------------------------------------
def _check_i32(acc64: np.ndarray) -> np.ndarray:
    if acc64.size and np.max(np.abs(acc64)) >= 2.0 ** 31:
        raise OverflowError("INT32 accumulator range exceeded")
    return acc64.astype(np.int32)


def _matmul_exact(a_i8: np.ndarray, b_i8: np.ndarray) -> np.ndarray:
    """a @ b for INT8 operands as an exact integer result.  The float64 library matmul is the
    step: every product and partial sum is an integer below 2^53, so no rounding occurs."""
    return a_i8.astype(F64) @ b_i8.astype(F64)


def int8_gemm_nt(xq: np.ndarray, wq: np.ndarray, row_chunk: int = 4096) -> np.ndarray:
    """acc[m,n] = sum_k xq[m,k]*wq[n,k], INT8 x INT8 -> INT32 (dense layer, Sec. IV-B)."""
    M = xq.shape[0]
    out = np.empty((M, wq.shape[0]), dtype=np.int32)
    wt = wq.astype(F64).T
    for m0 in range(0, M, row_chunk):
        out[m0:m0 + row_chunk] = _check_i32(xq[m0:m0 + row_chunk].astype(F64) @ wt)
    return out


def int8_gemm_tn(dhq: np.ndarray, xq: np.ndarray) -> np.ndarray:
    """accW[n,k] = sum_m dhq[m,n]*xq[m,k]  (g^W = g^Y^T A as an INT8 MAC, Sec. IV-B)."""
    return _check_i32(_matmul_exact(dhq.T, xq))


def _pad_hw(xq: np.ndarray) -> np.ndarray:
    return np.pad(xq, ((0, 0), (1, 1), (1, 1), (0, 0)))


def int8_conv3x3(xq: np.ndarray, wq: np.ndarray, stride: int = 1) -> np.ndarray:
    """acc[b,i,j,co] = sum_{r,s,ci} xq[b,stride*i+r-1,stride*j+s-1,ci]*wq[co,r,s,ci], zero padding 1
    (the convolutional form of Sec. IV-B's INT8 MAC).  xq NHWC int8, wq [Cout,3,3,Cin] int8."""
    Bn, H, Wd, Cin = xq.shape
    Cout = wq.shape[0]
    Ho, Wo = (H - 1) // stride + 1, (Wd - 1) // stride + 1
    xp = _pad_hw(xq)
    acc = np.zeros((Bn * Ho * Wo, Cout), dtype=F64)
    for r in range(3):
        for s in range(3):
            win = xp[:, r:r + stride * (Ho - 1) + 1:stride, s:s + stride * (Wo - 1) + 1:stride, :].reshape(-1, Cin)
            acc += _matmul_exact(win, wq[:, r, s, :].T)
    return _check_i32(acc).reshape(Bn, Ho, Wo, Cout)


def int8_conv3x3_wgrad(dhq: np.ndarray, xq: np.ndarray, stride: int = 1) -> np.ndarray:
    """accW[co,r,s,ci] = sum_{b,i,j} dhq[b,i,j,co]*xq[b,stride*i+r-1,stride*j+s-1,ci] (weight gradient of
    the convolution above; there is no input gradient in FF, Sec. IV-B)."""
    Bn, H, Wd, Cin = xq.shape
    _, Ho, Wo, Cout = dhq.shape
    xp = _pad_hw(xq)
    d2 = dhq.reshape(-1, Cout)
    out = np.empty((Cout, 3, 3, Cin), dtype=np.int32)
    for r in range(3):
        for s in range(3):
            win = xp[:, r:r + stride * (Ho - 1) + 1:stride, s:s + stride * (Wo - 1) + 1:stride, :].reshape(-1, Cin)
            out[:, r, s, :] = _check_i32(_matmul_exact(d2.T, win))
    return out


def int8_dwconv3x3(xq: np.ndarray, wq: np.ndarray, stride: int = 1) -> np.ndarray:
    """Depthwise 3x3 MAC: acc[b,i,j,c] = sum_{r,s} xq[b,stride*i+r-1,stride*j+s-1,c]*wq[c,r,s], zero
    padding 1 - the convolutional MAC of Sec. IV-B with one filter per
    channel and no sum over channels (the depthwise layers of the paper's MobileNetV2 / EfficientNet
    models, Table II).  xq NHWC int8, wq [C,3,3] int8; exact in int64, checked against INT32."""
    Bn, H, Wd, C = xq.shape
    Ho, Wo = (H - 1) // stride + 1, (Wd - 1) // stride + 1
    xp = _pad_hw(xq).astype(np.int64)
    acc = np.zeros((Bn, Ho, Wo, C), dtype=np.int64)
    for r in range(3):
        for s in range(3):
            acc += xp[:, r:r + stride * (Ho - 1) + 1:stride, s:s + stride * (Wo - 1) + 1:stride, :] * wq[:, r, s].astype(np.int64)
    return _check_i32(acc)


def int8_dwconv3x3_wgrad(dhq: np.ndarray, xq: np.ndarray, stride: int = 1) -> np.ndarray:
    """accW[c,r,s] = sum_{b,i,j} dhq[b,i,j,c]*xq[b,stride*i+r-1,stride*j+s-1,c] (weight gradient of the
    depthwise MAC; no input gradient, Sec. IV-B)."""
    Bn, H, Wd, C = xq.shape
    _, Ho, Wo, _ = dhq.shape
    xp = _pad_hw(xq).astype(np.int64)
    d = dhq.astype(np.int64)
    out = np.empty((C, 3, 3), dtype=np.int64)
    for r in range(3):
        for s in range(3):
            win = xp[:, r:r + stride * (Ho - 1) + 1:stride, s:s + stride * (Wo - 1) + 1:stride, :]
            out[:, r, s] = (d * win).sum(axis=(0, 1, 2))
    return _check_i32(out)


# --------------------------------------------------------------------------------------
# Epilogue: dequantise, ReLU, goodness, length normalisation  (Sec. III; Alg. 1, goodness step)
# --------------------------------------------------------------------------------------
def dequant_relu(acc: np.ndarray, c_rows: np.ndarray) -> np.ndarray:
    """y = max(0, float(acc) * c) with c = s_x*s_w of the row's pass; int->float conversion and
    the multiply are each one rounding."""
    accf = acc.astype(F32)
    c = c_rows.reshape((-1,) + (1,) * (acc.ndim - 1)).astype(F32)
    return np.maximum(F32(0.0), accf * c)


def goodness(acc: np.ndarray, c_rows: np.ndarray):
    """G = ||y||^2 per sample (the sum of the squared activities of the layer, Sec. III; Alg. 1, goodness step),
    evaluated as the exact integer S = sum relu(acc)^2 scaled once: G = float(double(S)*c*c).
    Also returns S and the per-sample max of relu(acc) (used for the absmax short-cuts)."""
    n = acc.shape[0]
    relu = np.maximum(acc.reshape(n, -1), 0).astype(np.uint64)
    approx = (relu.astype(F64) ** 2).sum(axis=1)
    if approx.size and approx.max() >= 2.0 ** 63:
        raise OverflowError("goodness integer sum exceeds 64 bits")
    S = (relu * relu).sum(axis=1, dtype=np.uint64)
    c64 = c_rows.astype(F64)
    G = (S.astype(F64) * (c64 * c64)).astype(F32)
    rowmax = relu.max(axis=1).astype(np.int32) if relu.shape[1] else np.zeros(n, np.int32)
    return G, S, rowmax


def length_normalise(y: np.ndarray, G: np.ndarray, tau: float, eps: float) -> np.ndarray:
    """Next layer's input x = y * tau/(||y|| + eps) with ||y|| = sqrt(G) (FF length
    normalisation of Forward-Forward, Hinton 2022; the paper itself is silent on it).  One sqrt, one add,
    one divide per sample; one multiply per element."""
    r = F32(tau) / (np.sqrt(G.astype(F32)) + F32(eps))
    return y * r.reshape((-1,) + (1,) * (y.ndim - 1)).astype(F32)


def maxpool2x2(x: np.ndarray) -> np.ndarray:
    """2x2 max pooling with stride 2 over the two spatial axes of an NHWC tensor (odd trailing rows /
    columns are dropped): the down-sampling step of the convolutional models the paper trains (Table II).
    In FF it sits between a layer's normalised output and the next layer's input; nothing is differentiated
    through it because no input gradient exists (Sec. IV-B).  A maximum involves no rounding."""
    n, h, w, c = x.shape
    ho, wo = h // 2, w // 2
    out = np.empty((n, ho, wo, c), dtype=x.dtype)
    for i in range(ho):
        for j in range(wo):
            out[:, i, j, :] = np.maximum(np.maximum(x[:, 2 * i, 2 * j, :], x[:, 2 * i, 2 * j + 1, :]),
                                         np.maximum(x[:, 2 * i + 1, 2 * j, :], x[:, 2 * i + 1, 2 * j + 1, :]))
    return out


# --------------------------------------------------------------------------------------
# FF loss, sigma and the look-ahead coefficient  (Eq. 1-4; Alg. 1, loss and update steps)
# --------------------------------------------------------------------------------------
_LOG2E = F64(1.4426950408889634)            # nearest double to 1/ln 2
_LN2_HI = F64(6.93147180369123816490e-01)   # ln 2 split so that n*LN2_HI is exact
_LN2_LO = F64(1.90821492927058770002e-10)
_EXP_DEG = 13


def exp_nonpos(v: np.ndarray) -> np.ndarray:
    """e^v for v <= 0 in float64 by a fixed recipe (clamp at -700; n = rint(v/ln2);
    r = (v - n*LN2_HI) - n*LN2_LO; degree-13 Taylor polynomial by Horner with separate
    multiply and add; scale by 2^n).  A recipe instead of libm so that any two
    implementations agree bit for bit."""
    v = np.maximum(np.asarray(v, dtype=F64), F64(-700.0))
    n = np.rint(v * _LOG2E)
    r = (v - n * _LN2_HI) - n * _LN2_LO
    fact = 1
    coef = []
    for k in range(_EXP_DEG + 1):
        fact = fact * k if k > 0 else 1
        coef.append(F64(1.0) / F64(fact))
    p = np.full_like(r, coef[_EXP_DEG])
    for k in range(_EXP_DEG - 1, -1, -1):
        p = p * r
        p = p + coef[k]
    return np.ldexp(p, n.astype(np.int64))


def sigmoid_spec(x: np.ndarray) -> np.ndarray:
    """sigma(x) = 1/(1+e^-x) from e = e^{-|x|}: x >= 0 -> 1/(1+e), else e/(1+e)."""
    x = np.asarray(x, dtype=F64)
    e = exp_nonpos(-np.abs(x))
    d = F64(1.0) + e
    return np.where(x >= 0, F64(1.0) / d, e / d)


def ff_loss_terms(G: np.ndarray, theta: float, B: int):
    """Per-sample loss and dL/dG.  Positive rows (Eq. 1): L = log(1+e^{-(G-theta)}),
    dL/dG = -sigma(-(G-theta)).  Negative rows (Eq. 2): L = log(1+e^{G-theta}),
    dL/dG = +sigma(G-theta)."""
    z = G.astype(F64) - F64(F32(theta))
    sign = np.concatenate([-np.ones(B), np.ones(B)])        # -1 positive set, +1 negative set
    arg = sign * z                                          # L = softplus(arg)
    L = np.maximum(arg, 0.0) + np.log1p(np.exp(-np.abs(arg)))
    gprime = sign * sigmoid_spec(arg)
    return L, gprime


def lookahead_loss_coef(G_layers: Sequence[np.ndarray], thetas: Sequence[float], B: int,
                        lam: float):
    """Loss of the current layer (first entry) with the look-ahead term over the later layers
    (Eq. 3):  L_new = L_1 + lambda*(L_2+...+L_final), averaged over the 2B samples, and the
    per-sample coefficient of Eq. 4 under the scalar-coefficient reading:
        coef_m = (g'_1,m + lambda * sum_{j>1} g'_j,m) / (2B),   g'_j = dL_j/dG_j,
    so that dH = 2*coef*Y.  All of it in float64, coef rounded once to float32."""
    M = 2 * B
    lam64 = F64(F32(lam))
    L0, g0 = ff_loss_terms(G_layers[0], thetas[0], B)
    Lsum = np.zeros(M, dtype=F64)
    gsum = np.zeros(M, dtype=F64)
    for Gj, tj in zip(G_layers[1:], thetas[1:]):
        Lj, gj = ff_loss_terms(Gj, tj, B)
        Lsum = Lsum + Lj
        gsum = gsum + gj
    inv_m = F64(1.0) / F64(M)
    coef = ((g0 + lam64 * gsum) * inv_m).astype(F32)
    loss = float(np.sum(L0 + lam64 * Lsum) * inv_m) if M else 0.0
    return loss, coef


# --------------------------------------------------------------------------------------
# One layer: forward, loss/gradient, update  (Fig. 4 dataflow, Sec. IV-B)
# --------------------------------------------------------------------------------------
@dataclass
class LayerState:
    """Everything one layer produces during a step (all of it compared against the GPU)."""
    Xq: np.ndarray = None
    Wq: np.ndarray = None
    a_x: tuple = None          # (absmax pos, absmax neg) of the layer input
    a_w: np.float32 = None
    acc: np.ndarray = None     # int32 forward accumulator
    Y: np.ndarray = None
    S: np.ndarray = None       # exact integer sum of relu(acc)^2 per sample
    rowmax: np.ndarray = None
    G: np.ndarray = None
    Xnext: np.ndarray = None
    loss: float = None
    coef: np.ndarray = None
    a_dh: tuple = None
    dHq: np.ndarray = None
    accW: np.ndarray = None    # [2, N, K] int32, pass-separated
    W_new: np.ndarray = None
    dW: np.ndarray = None      # dequantised weight gradient (float32)
    M_new: np.ndarray = None   # momentum buffer after the update (None for plain SGD)
    V_new: np.ndarray = None   # Adam's second-moment buffer after the update


def _pass_rows(v_pos, v_neg, B):
    return np.concatenate([np.full(B, v_pos, dtype=F32), np.full(B, v_neg, dtype=F32)])


def add_skip(xhat: np.ndarray, skip: np.ndarray, scale: float) -> np.ndarray:
    """Output of a residual block: z = xhat + scale*skip, element by element (one float32 multiply, one float32 add).
    xhat is the last layer's length-normalised output, skip the block's (length-normalised) input, so both have a
    fixed length per sample and their sum carries no goodness of either on to the next layer.  The paper trains
    residual networks (Sec. IV-C: the look-ahead exists so that the layers of such a block are trained together;
    Table II) but does not say how the sum is formed in FF training; this reading keeps every layer's own goodness
    ||y||^2 (Sec. III) untouched - the skip path changes what the NEXT layer sees, nothing else - and needs no
    reduction whose order is free.  No gradient passes through it (there is no input gradient, Sec. IV-B)."""
    xhat = np.asarray(xhat, dtype=F32)
    skip = np.asarray(skip, dtype=F32)
    if xhat.size != skip.size or xhat.shape[0] != skip.shape[0]:
        raise ValueError("skip tensor and layer output differ in shape")
    return xhat + F32(scale) * skip.reshape(xhat.shape)


def layer_forward(spec: LayerSpec, X: np.ndarray, W: np.ndarray, B: int, step: int,
                  skip: Optional[np.ndarray] = None, joint_range: bool = False) -> LayerState:
    """Quantise A and W, INT8 MAC, dequantise + ReLU, goodness, normalised output (+ the skip path, if any).
    joint_range: the input is quantised with one range for all 2B rows instead of one per set."""
    st = LayerState()
    X = np.asarray(X, dtype=F32)
    W = np.asarray(W, dtype=F32)
    st.Xq, st.a_x = quantize_two_pass(X, B, spec.round_x,
                                      rounding_key(spec.seed, ROLE_X, spec.index, step), joint_range)
    st.a_w = absmax(W)
    st.Wq = quantize(W, st.a_w, spec.round_w, rounding_key(spec.seed, ROLE_W, spec.index, step))
    if spec.kind == KIND_LINEAR:
        st.acc = int8_gemm_nt(st.Xq, st.Wq)
    elif spec.kind == KIND_CONV1X1:
        # pointwise convolution: the dense MAC of Sec. IV-B applied at every position
        st.acc = int8_gemm_nt(st.Xq.reshape(-1, spec.K), st.Wq).reshape(st.Xq.shape[:3] + (spec.N,))
    elif spec.kind == KIND_DWCONV3X3:
        st.acc = int8_dwconv3x3(st.Xq, st.Wq.reshape(spec.N, 3, 3), spec.stride)
    else:
        st.acc = int8_conv3x3(st.Xq, st.Wq.reshape(spec.N, 3, 3, spec.Cin), spec.stride)
    s_w, _ = scale_pair(st.a_w)
    c_rows = _pass_rows(scale_pair(st.a_x[0])[0] * s_w, scale_pair(st.a_x[1])[0] * s_w, B)
    st.Y = dequant_relu(st.acc, c_rows)
    st.G, st.S, st.rowmax = goodness(st.acc, c_rows)
    st.Xnext = length_normalise(st.Y, st.G, spec.tau, spec.eps)
    if spec.pool == 2:
        if spec.kind == KIND_LINEAR or spec.out_hw[0] % 2 or spec.out_hw[1] % 2:
            raise ValueError("pooling needs a spatial layer with even output extents")
        st.Xnext = maxpool2x2(st.Xnext)
    if skip is not None:
        if spec.pool == 2:
            raise ValueError("a pooled output takes no skip path")
        st.Xnext = add_skip(st.Xnext, skip, spec.skip_scale)
    return st


def layer_loss_grad(spec: LayerSpec, st: LayerState, B: int, G_later: Sequence[np.ndarray],
                    theta_later: Sequence[float], lam: float, step: int) -> LayerState:
    """Loss (Eq. 1-3), g^Y = dH = 2*coef*Y, and its INT8 quantisation per pass (Sec. IV-B)."""
    st.loss, st.coef = lookahead_loss_coef([st.G] + list(G_later),
                                           [spec.theta] + list(theta_later), B, lam)
    k2 = F32(2.0) * st.coef
    dH = k2.reshape((-1,) + (1,) * (st.Y.ndim - 1)) * st.Y
    st.dHq, st.a_dh = quantize_two_pass(dH, B, spec.round_dh,
                                        rounding_key(spec.seed, ROLE_DH, spec.index, step))
    return st


def sgd_momentum(W: np.ndarray, M: np.ndarray, g: np.ndarray, lr: float, mu: float):
    """Heavy-ball SGD (Polyak): m <- mu*m + g, W <- W - lr*m, each operation one float32 rounding.
    The paper names no optimiser for its weight update (Sec. IV-B; Alg. 1, update step); plain
    SGD is mu = 0, this is the usual next choice.  Returns (W_new, M_new)."""
    M_new = F32(mu) * np.asarray(M, dtype=F32) + np.asarray(g, dtype=F32)
    return np.asarray(W, dtype=F32) - F32(lr) * M_new, M_new


def _pow_int(x: float, n: int) -> float:
    """x**n for n >= 0 by square-and-multiply from the low bit up, every product one float64 rounding
    (a fixed order, so that any two implementations agree bit for bit)."""
    r, p = F64(1.0), F64(x)
    while n > 0:
        if n & 1:
            r = r * p
        n >>= 1
        if n:
            p = p * p
    return r


def adam_update(W, M, V, g, lr: float, beta1: float, beta2: float, eps: float, t: int):
    """Adam (Kingma & Ba 2015, Algorithm 1) for update number t >= 1, the other usual choice where the paper
    only says that the weights are updated (Sec. IV-B; Alg. 1, update step):
        m = beta1*m + (1-beta1)*g;  v = beta2*v + (1-beta2)*g*g;
        W -= lr * (m*c1) / (sqrt(v*c2) + eps),   c_i = float32(1/(1 - beta_i^t)).
    float32 throughout, one rounding per operation in the order written (1-beta_i is one float32
    subtraction); the bias corrections come from float64 powers by _pow_int.  Returns (W_new, M_new, V_new)."""
    b1, b2 = F32(beta1), F32(beta2)
    g = np.asarray(g, dtype=F32)
    M_new = b1 * np.asarray(M, dtype=F32) + (F32(1.0) - b1) * g
    V_new = b2 * np.asarray(V, dtype=F32) + (F32(1.0) - b2) * (g * g)
    c1 = F32(F64(1.0) / (F64(1.0) - _pow_int(F64(b1), t)))
    c2 = F32(F64(1.0) / (F64(1.0) - _pow_int(F64(b2), t)))
    upd = (M_new * c1) / (np.sqrt(V_new * c2) + F32(eps))
    return np.asarray(W, dtype=F32) - F32(lr) * upd, M_new, V_new


def layer_update(spec: LayerSpec, st: LayerState, W: np.ndarray, B: int, M: Optional[np.ndarray] = None,
                 V: Optional[np.ndarray] = None, step: int = 0) -> LayerState:
    """g^W per pass as an INT8 MAC, dequantised and applied as plain SGD (Sec. IV-B; Alg. 1,
    update step):  g = float(accP)*cP + float(accN)*cN,  W <- W - lr*g.  With spec.momentum != 0 the
    update is heavy-ball SGD on the momentum buffer M (zeros when None), see sgd_momentum."""
    W = np.asarray(W, dtype=F32)
    accW = []
    for p in range(2):
        sl = slice(p * B, (p + 1) * B)
        if spec.kind == KIND_LINEAR:
            accW.append(int8_gemm_tn(st.dHq[sl], st.Xq[sl]))
        elif spec.kind == KIND_CONV1X1:
            accW.append(int8_gemm_tn(st.dHq[sl].reshape(-1, spec.N), st.Xq[sl].reshape(-1, spec.K)))
        elif spec.kind == KIND_DWCONV3X3:
            accW.append(int8_dwconv3x3_wgrad(st.dHq[sl], st.Xq[sl], spec.stride).reshape(spec.N, 9))
        else:
            accW.append(int8_conv3x3_wgrad(st.dHq[sl], st.Xq[sl], spec.stride).reshape(spec.N, spec.K))
    st.accW = np.stack(accW)
    cP = scale_pair(st.a_dh[0])[0] * scale_pair(st.a_x[0])[0]
    cN = scale_pair(st.a_dh[1])[0] * scale_pair(st.a_x[1])[0]
    st.dW = st.accW[0].astype(F32) * cP + st.accW[1].astype(F32) * cN
    if spec.optimizer == 1:   # Adam; update number t = step + 1
        z = np.zeros_like(W)
        st.W_new, st.M_new, st.V_new = adam_update(W, z if M is None else M, z if V is None else V, st.dW, spec.lr,
                                                   spec.momentum, spec.beta2, spec.adam_eps, step + 1)
    elif spec.momentum != 0.0:
        st.W_new, st.M_new = sgd_momentum(W, np.zeros_like(W) if M is None else M, st.dW, spec.lr, spec.momentum)
    else:
        st.W_new = W - F32(spec.lr) * st.dW
    return st


def train_step(specs: List[LayerSpec], Ws: List[np.ndarray], X: np.ndarray, B: int, lam: float,
               step: int, Ms: Optional[List[np.ndarray]] = None, Vs: Optional[List[np.ndarray]] = None,
               first_trained: int = 0) -> List[LayerState]:
    """Body of Algorithm 1's epoch loop: one INT8 forward through all k layers with the
    pre-update weights, goodness of every layer, then for each layer its loss from the G's
    and its INT8 gradient and update.  lambda is the caller's (the algorithm starts it at zero
    and raises it once per epoch).  With one layer and lambda = 0 this is the vanilla step.  Ms: the
    layers' momentum buffers (only read by layers with momentum != 0).
    first_trained > 0: the layers before it are frozen - they take part in the forward only (their
    states carry no coef, dHq or W_new).  This is one step of the layer-by-layer schedule of Sec. III,
    where a layer is trained on the output of the already trained layers before it."""
    states = []
    inputs = [X]                       # inputs[l] = float32 input of layer l (the skip paths' sources)
    for spec, W in zip(specs, Ws):
        if spec.skip_from >= len(inputs):
            raise ValueError("skip_from must name this layer or an earlier one")
        skip = inputs[spec.skip_from] if spec.skip_from >= 0 else None
        st = layer_forward(spec, inputs[-1], W, B, step, skip)
        states.append(st)
        inputs.append(st.Xnext)
    for l, (spec, W) in enumerate(zip(specs, Ws)):
        if l < first_trained:
            continue
        later = list(range(l + 1, len(specs)))
        layer_loss_grad(spec, states[l], B, [states[j].G for j in later],
                        [specs[j].theta for j in later], lam, step)
        layer_update(spec, states[l], W, B, None if Ms is None else Ms[l], None if Vs is None else Vs[l], step)
    return states


def greedy_epoch(specs: List[LayerSpec], Ws: List[np.ndarray], batches, B: int, on_step=None) -> List[np.ndarray]:
    """Layer-by-layer training (Sec. III: a layer is trained to the end, then its successor): phase l runs
    over every batch once and trains layer l alone (lambda = 0) on the INT8 forward of layers 0..l-1 as
    their own phases left them.  `batches` is a sequence of batches (anything with len() and [i]); the
    step counter that keys the stochastic rounding runs on through the phases: t = l*len(batches) + i.
    on_step(l, i, states) sees every step.  Returns the trained weights."""
    Ws = [np.asarray(W, dtype=F32) for W in Ws]
    n = len(batches)
    for l in range(len(specs)):
        for i in range(n):
            states = train_step(specs[:l + 1], Ws[:l + 1], batches[i], B, 0.0, l * n + i, first_trained=l)
            Ws[l] = states[l].W_new
            if on_step is not None:
                on_step(l, i, states)
    return Ws


# --------------------------------------------------------------------------------------
# Classification with a trained network  (Sec. III: goodness is high for positive data)
# --------------------------------------------------------------------------------------
def predict(specs: List[LayerSpec], Ws: List[np.ndarray], X_cand: np.ndarray, B: int, n_classes: int,
            step: int, first_counted: int = 0):
    """Label of each of B samples by goodness.  The paper reports accuracy but does not spell the
    procedure out; this is the Forward-Forward one its Sec. III builds on: a sample is presented
    once per candidate label (label written one-hot into the input, exactly as for the positive
    set), every candidate runs through the INT8 forward of all layers, the goodness of the layers
    from `first_counted` on is added up, and the label with the largest total wins (lowest label
    on ties).  X_cand [n_classes*B, ...]: row c*B + b is sample b with candidate label c, already
    length-normalised.  Every layer input of the candidate batch is quantised with ONE per-tensor range (the
    candidates of a sample must be compared under the same quantisation step, whichever label they carry); the
    rows are still processed as two halves, so n_classes*B is even.
    Returns (pred [B] int32, scores [n_classes, B] float32, per-layer LayerStates)."""
    if n_classes <= 0 or (n_classes * B) % 2:
        raise ValueError("n_classes must be positive and n_classes*B even")
    half = n_classes * B // 2
    inputs = [np.asarray(X_cand, dtype=F32)]
    states = []
    for spec, W in zip(specs, Ws):
        skip = inputs[spec.skip_from] if spec.skip_from >= 0 else None
        st = layer_forward(spec, inputs[-1], W, half, step, skip, joint_range=True)
        states.append(st)
        inputs.append(st.Xnext)
    total = np.zeros(n_classes * B, dtype=F32)
    for st in states[first_counted:]:
        total = total + st.G.astype(F32)          # float32 additions in layer order
    scores = total.reshape(n_classes, B)
    pred = np.argmax(scores, axis=0).astype(np.int32)   # first maximum = lowest label
    return pred, scores, states


# --------------------------------------------------------------------------------------
# Positive / negative (and candidate) batches by label embedding  (Sec. III; Alg. 1, sample generation)
# --------------------------------------------------------------------------------------
def embed_labels(x: np.ndarray, labels: np.ndarray, n_classes: int, label_stride: int = 1, on_value: float = 1.0,
                 tau0: float = 0.0, eps: float = 1e-8) -> np.ndarray:
    """Batches made from B raw samples by writing a label into each (Sec. III: the true label gives the
    positive sample, a wrong one the negative; Alg. 1, sample generation).  x [B, n] float32, labels [sets, B]:
    output row s*B + b is sample b with labels[s, b] written one-hot over its n_classes label places
    (flat positions 0, label_stride, 2*label_stride, ...: the place of the label holds on_value, the
    others zero).  The wrong labels are drawn by the caller and passed in.  With tau0 > 0 every row is
    then scaled to length tau0: r = tau0 / (float32(sqrt(sum of squares in float64)) + eps), one
    float32 multiply per element (the first layer's input arrives length-normalised like every other
    layer's).  Labels outside [0, n_classes) are an error."""
    x = np.asarray(x, dtype=F32)
    labels = np.asarray(labels)
    B, n = x.shape
    sets = labels.shape[0]
    if labels.shape != (sets, B):
        raise ValueError("labels must be [sets, B]")
    if (labels < 0).any() or (labels >= n_classes).any():
        raise ValueError("label outside [0, n_classes)")
    if n_classes <= 0 or label_stride <= 0 or (n_classes - 1) * label_stride >= n:
        raise ValueError("label places do not fit the sample")
    out = np.empty((sets * B, n), dtype=F32)
    for s_ in range(sets):
        for b_ in range(B):
            v = x[b_].copy()
            v[0:n_classes * label_stride:label_stride] = F32(0.0)
            v[int(labels[s_, b_]) * label_stride] = F32(on_value)
            if tau0 > 0.0:
                ss = np.sum(v.astype(F64) * v.astype(F64))
                r = F32(tau0) / (F32(np.sqrt(ss)) + F32(eps))
                v = v * F32(r)
            out[s_ * B + b_] = v
    return out


# --------------------------------------------------------------------------------------
# Unquantised float64 model of one layer (for the finite-difference pin only)
# --------------------------------------------------------------------------------------
def fp64_layer_loss(spec: LayerSpec, X: np.ndarray, W: np.ndarray, B: int) -> float:
    """Mean over the 2B samples of Eq. 1 / Eq. 2 with G = ||relu(X W^T)||^2, no quantisation."""
    X = np.asarray(X, dtype=F64)
    W = np.asarray(W, dtype=F64)
    if spec.kind in (KIND_LINEAR, KIND_CONV1X1):
        Y = np.maximum(X @ W.T, 0.0)
    elif spec.kind == KIND_DWCONV3X3:
        xp = np.pad(X, ((0, 0), (1, 1), (1, 1), (0, 0)))
        w3 = W.reshape(spec.N, 3, 3)
        Ho, Wo = spec.out_hw
        st = spec.stride
        Y = np.zeros((X.shape[0], Ho, Wo, spec.N))
        for r in range(3):
            for s in range(3):
                Y += xp[:, r:r + st * (Ho - 1) + 1:st, s:s + st * (Wo - 1) + 1:st, :] * w3[:, r, s]
        Y = np.maximum(Y, 0.0)
    else:
        xp = np.pad(X, ((0, 0), (1, 1), (1, 1), (0, 0)))
        w4 = W.reshape(spec.N, 3, 3, spec.Cin)
        Ho, Wo = spec.out_hw
        st = spec.stride
        Y = np.zeros((X.shape[0], Ho, Wo, spec.N))
        for r in range(3):
            for s in range(3):
                Y += xp[:, r:r + st * (Ho - 1) + 1:st, s:s + st * (Wo - 1) + 1:st, :] @ w4[:, r, s, :].T
        Y = np.maximum(Y, 0.0)
    G = (Y.reshape(2 * B, -1) ** 2).sum(axis=1)
    z = G - spec.theta
    sign = np.concatenate([-np.ones(B), np.ones(B)])
    arg = sign * z
    return float(np.mean(np.maximum(arg, 0.0) + np.log1p(np.exp(-np.abs(arg)))))
