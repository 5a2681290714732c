"""Pins of the CPU oracle against things other than itself: hand-computed fixtures, closed
forms of Eq. 1-3, brute-force loops, finite differences, library routines, error bounds.
CPU only."""
import math
import os

import numpy as np
import pytest

from oracle import ffint8_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")
F32 = np.float32


def _rows(name):
    out = []
    for line in open(os.path.join(GOLD, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            out.append(line.split())
    return out


def _spec(K, N, theta=None, kind=0, H=1, Wd=1, Cin=0, rnd=O.ROUND_NEAREST, lr=0.03, index=0, seed=3):
    per = H * Wd
    return O.LayerSpec(kind, K, N, float(theta if theta is not None else N * per), lr,
                       float(np.sqrt(N * per)), 1e-8, H, Wd, Cin, rnd, O.ROUND_NEAREST, rnd, seed, index)


# ------------------------------------------------------------------ quantiser (Sec. IV)
def test_quant_nearest_hand_example():
    rows = _rows("quant_nearest_2x3.txt")
    x = np.array([float(r[0]) for r in rows], dtype=F32)
    q = np.array([int(r[1]) for r in rows], dtype=np.int8)
    a = O.absmax(x)
    assert a == F32(2.0)
    assert np.array_equal(O.quantize(x, a, O.ROUND_NEAREST), q)


def test_quant_stochastic_hand_example():
    rows = _rows("quant_stochastic_1x6.txt")
    x = np.array([float(r[0]) for r in rows], dtype=F32)
    u = np.array([float(r[1]) for r in rows], dtype=F32)
    q = np.array([int(r[2]) for r in rows], dtype=np.int8)
    assert np.array_equal(O.quantize(x, F32(4.0), O.ROUND_STOCHASTIC, u=u), q)


def test_quant_error_bounds_and_range():
    g = np.random.default_rng(0)
    x = g.normal(size=5000).astype(F32)
    a = O.absmax(x)
    s, _ = O.scale_pair(a)
    q = O.quantize(x, a, O.ROUND_NEAREST)
    err = np.abs(x.astype(np.float64) - float(s) * q.astype(np.float64))
    assert err.max() <= float(s) / 2 * (1 + 1e-5)                 # |x - s q| <= s/2
    assert abs(int(q[np.argmax(np.abs(x))])) == 127               # absmax element -> +-127
    assert q.min() >= -127 and q.max() <= 127
    qs = O.quantize(x, a, O.ROUND_STOCHASTIC, key=O.rounding_key(1, 0, 0, 0))
    errs = np.abs(x.astype(np.float64) - float(s) * qs.astype(np.float64))
    assert errs.max() < float(s) * (1 + 1e-5)                     # |x - s q| < s
    assert np.array_equal(O.quantize(x, a, O.ROUND_STOCHASTIC, u=np.zeros_like(x)),
                          np.clip(np.floor(x * O.scale_pair(a)[1]), -127, 127).astype(np.int8))


def test_quant_zero_tensor_and_idempotence():
    z = np.zeros((3, 4), dtype=F32)
    assert O.absmax(z) == 0 and not O.quantize(z, O.absmax(z), O.ROUND_NEAREST).any()
    assert not O.quantize(z, O.absmax(z), O.ROUND_STOCHASTIC, key=(1, 2)).any()
    g = np.random.default_rng(1)
    x = g.uniform(-3, 3, size=1000).astype(F32)
    x[0] = 3.0
    a = O.absmax(x)
    s, _ = O.scale_pair(a)
    q = O.quantize(x, a, O.ROUND_NEAREST)
    xr = (s * q.astype(F32)).astype(F32)
    assert np.array_equal(O.quantize(xr, O.absmax(xr), O.ROUND_NEAREST), q)


def test_quant_rejects_nonfinite():
    with pytest.raises(FloatingPointError):
        O.absmax(np.array([1.0, np.inf], dtype=F32))
    with pytest.raises(FloatingPointError):
        O.absmax(np.array([np.nan], dtype=F32))


def test_stochastic_rounding_is_unbiased():
    # E[q] = t for every element (the property the paper takes stochastic rounding for)
    x = np.array([0.013, -0.4, 0.77, 0.5001, -0.9999, 1.0], dtype=F32)
    a = O.absmax(x)
    t = x.astype(np.float64) * 127.0
    acc = np.zeros_like(t)
    n = 20000
    for seed in range(n):
        acc += O.quantize(x, a, O.ROUND_STOCHASTIC, key=O.rounding_key(seed, 0, 0, 0))
    assert np.max(np.abs(acc / n - t)) < 4 * 0.5 / math.sqrt(n)


def test_rounding_hash_statistics_and_splitmix_vectors():
    # SplitMix64 reference outputs for state 1234567 (published test vector of the generator)
    s = 1234567
    want = [6457827717110365317, 3203168211198807973, 9817491932198370423]
    got = [O._splitmix64((s + i * 0x9E3779B97F4A7C15) & ((1 << 64) - 1)) for i in range(3)]
    assert got == want
    k = O.rounding_key(5, O.ROLE_X, 2, 9)
    u = O.rounding_uniform(np.arange(1 << 20, dtype=np.uint64), *k)
    assert u.dtype == F32 and u.min() >= 0.0 and u.max() < 1.0
    assert abs(float(u.mean()) - 0.5) < 2e-3
    hist = np.bincount((u * 64).astype(int), minlength=64)
    chi2 = float(((hist - u.size / 64) ** 2 / (u.size / 64)).sum())
    assert chi2 < 130                                   # 63 dof; p ~ 1e-6
    assert abs(np.corrcoef(u[:-1], u[1:])[0, 1]) < 5e-3  # neighbouring counters uncorrelated
    # different role / layer / step give different streams
    for other in (O.rounding_key(5, O.ROLE_DH, 2, 9), O.rounding_key(5, O.ROLE_X, 3, 9),
                  O.rounding_key(5, O.ROLE_X, 2, 10), O.rounding_key(6, O.ROLE_X, 2, 9)):
        v = O.rounding_uniform(np.arange(4096, dtype=np.uint64), *other)
        assert abs(np.corrcoef(u[:4096], v)[0, 1]) < 0.06


# ------------------------------------------------------------------ INT8 MAC (Sec. IV-B)
def _brute_gemm_nt(a, b):
    M, K = a.shape
    N = b.shape[0]
    out = [[0] * N for _ in range(M)]
    for m in range(M):
        for n in range(N):
            s = 0
            for k in range(K):
                s += int(a[m, k]) * int(b[n, k])
            out[m][n] = s
    return np.array(out, dtype=np.int64)


@pytest.mark.parametrize("M,N,K", [(3, 5, 33), (1, 1, 1), (7, 2, 27), (16, 9, 64)])
def test_gemm_against_brute_force(M, N, K):
    g = np.random.default_rng(M * 100 + N * 10 + K)
    a = g.integers(-127, 128, size=(M, K)).astype(np.int8)
    b = g.integers(-127, 128, size=(N, K)).astype(np.int8)
    assert np.array_equal(O.int8_gemm_nt(a, b, row_chunk=2), _brute_gemm_nt(a, b))
    # weight-gradient orientation: accW[n,k] = sum_m d[m,n] x[m,k]
    d = g.integers(-127, 128, size=(M, N)).astype(np.int8)
    want = _brute_gemm_nt(np.ascontiguousarray(d.T), np.ascontiguousarray(a.T))
    assert np.array_equal(O.int8_gemm_tn(d, a), want)


def test_gemm_extreme_values_exact_and_overflow_check():
    K = 8192
    a = np.full((2, K), 127, dtype=np.int8)
    b = np.full((3, K), -127, dtype=np.int8)
    assert np.all(O.int8_gemm_nt(a, b) == -127 * 127 * K)
    g = np.random.default_rng(3)
    a = g.integers(-127, 128, size=(64, 1000)).astype(np.int8)
    b = g.integers(-127, 128, size=(48, 1000)).astype(np.int8)
    want = np.einsum("mk,nk->mn", a.astype(np.int64), b.astype(np.int64))
    assert np.array_equal(O.int8_gemm_nt(a, b), want)
    big = np.full((1, 140000), 127, dtype=np.int8)      # 127*127*140000 > 2^31
    with pytest.raises(OverflowError):
        O.int8_gemm_nt(big, big)


def _brute_conv(x, w):
    Bn, H, Wd, Cin = x.shape
    Cout = w.shape[0]
    out = np.zeros((Bn, H, Wd, Cout), dtype=np.int64)
    for b in range(Bn):
        for h in range(H):
            for ww in range(Wd):
                for co in range(Cout):
                    s = 0
                    for r in range(3):
                        for t in range(3):
                            hh, wx = h + r - 1, ww + t - 1
                            if 0 <= hh < H and 0 <= wx < Wd:
                                for ci in range(Cin):
                                    s += int(x[b, hh, wx, ci]) * int(w[co, r, t, ci])
                    out[b, h, ww, co] = s
    return out


def _brute_wgrad(d, x):
    Bn, H, Wd, Cin = x.shape
    Cout = d.shape[-1]
    out = np.zeros((Cout, 3, 3, Cin), dtype=np.int64)
    for co in range(Cout):
        for r in range(3):
            for t in range(3):
                for ci in range(Cin):
                    s = 0
                    for b in range(Bn):
                        for h in range(H):
                            for ww in range(Wd):
                                hh, wx = h + r - 1, ww + t - 1
                                if 0 <= hh < H and 0 <= wx < Wd:
                                    s += int(d[b, h, ww, co]) * int(x[b, hh, wx, ci])
                    out[co, r, t, ci] = s
    return out


def test_conv_against_brute_force_and_library():
    g = np.random.default_rng(11)
    x = g.integers(-127, 128, size=(2, 4, 5, 3)).astype(np.int8)
    w = g.integers(-127, 128, size=(4, 3, 3, 3)).astype(np.int8)
    d = g.integers(-127, 128, size=(2, 4, 5, 4)).astype(np.int8)
    assert np.array_equal(O.int8_conv3x3(x, w), _brute_conv(x, w))
    assert np.array_equal(O.int8_conv3x3_wgrad(d, x), _brute_wgrad(d, x))
    torch = pytest.importorskip("torch")
    x = g.integers(-127, 128, size=(3, 8, 8, 16)).astype(np.int8)
    w = g.integers(-127, 128, size=(24, 3, 3, 16)).astype(np.int8)
    tx = torch.from_numpy(x.astype(np.float64)).permute(0, 3, 1, 2)
    tw = torch.from_numpy(w.astype(np.float64)).permute(0, 3, 1, 2)
    want = torch.nn.functional.conv2d(tx, tw, padding=1).permute(0, 2, 3, 1).numpy()
    assert np.array_equal(O.int8_conv3x3(x, w).astype(np.float64), want)


# ------------------------------------------------------------------ epilogue / goodness
def test_tiny_layer_hand_example():
    vals = {r[0]: np.array([int(v) for v in r[1:]]) for r in _rows("tiny_layer.txt")}
    X = np.array([[1, 0.5], [-0.25, 0.5]], dtype=F32)
    W = np.array([[1, -1], [0.5, 0.25]], dtype=F32)
    st = O.layer_forward(_spec(2, 2), X, W, 1, 0)
    assert np.array_equal(st.Xq.ravel(), vals["Xq"])
    assert np.array_equal(st.Wq.ravel(), vals["Wq"])
    assert np.array_equal(st.acc.ravel(), vals["acc"])
    assert np.array_equal(st.S, vals["S"].astype(np.uint64))
    assert np.array_equal(st.rowmax, vals["rowmax"])
    c = (1.0 / 127) ** 2
    assert np.allclose(st.Y, [[8001 * c, 10176 * c], [0, 0]], rtol=1e-6)
    assert np.allclose(st.G, [167566977 * c * c, 0.0], rtol=1e-6)
    nrm = np.sqrt(167566977.0) * c
    assert np.allclose(st.Xnext[0], np.array([8001, 10176]) * c * np.sqrt(2.0) / nrm, rtol=1e-6)
    assert not st.Xnext[1].any()


def test_goodness_zero_input_and_fp64_sum():
    g = np.random.default_rng(5)
    W = g.normal(size=(40, 30)).astype(F32)
    st = O.layer_forward(_spec(30, 40), np.zeros((6, 30), F32), W, 3, 0)
    assert not st.G.any() and not st.Y.any() and not st.Xnext.any()
    X = g.normal(size=(6, 30)).astype(F32)
    st = O.layer_forward(_spec(30, 40), X, W, 3, 0)
    ref = (st.Y.astype(np.float64) ** 2).sum(axis=1)
    assert np.allclose(st.G, ref, rtol=1e-6)
    nrm = np.sqrt((st.Xnext.astype(np.float64) ** 2).sum(axis=1))
    assert np.allclose(nrm, np.sqrt(40.0), rtol=1e-5)             # normalised to length tau


def test_dequantised_forward_tracks_float_layer():
    g = np.random.default_rng(6)
    X = g.normal(size=(8, 256)).astype(F32)
    W = (g.normal(size=(64, 256)) / 16).astype(F32)
    st = O.layer_forward(_spec(256, 64), X, W, 4, 0)
    ref = np.maximum(X.astype(np.float64) @ W.astype(np.float64).T, 0)
    assert np.abs(st.Y - ref).max() < 0.05 * np.abs(ref).max()


# ------------------------------------------------------------------ loss (Eq. 1-3)
def test_loss_closed_forms():
    theta = 2.0
    G = np.array([0.0, 1.0, 2.0, 5.0, 0.0, 1.0, 2.0, 5.0], dtype=F32)
    L, gp = O.ff_loss_terms(G, theta, 4)
    z = G.astype(np.float64) - theta
    assert np.allclose(L[:4], np.log(1 + np.exp(-z[:4])), rtol=1e-14)      # Eq. 1
    assert np.allclose(L[4:], np.log(1 + np.exp(z[4:])), rtol=1e-14)       # Eq. 2
    assert math.isclose(L[2], math.log(2), rel_tol=1e-15) and math.isclose(L[6], math.log(2), rel_tol=1e-15)
    assert gp[2] == -0.5 and gp[6] == 0.5                                   # sigma(0) = 1/2
    assert np.allclose(gp[:4], -1 / (1 + np.exp(z[:4])), rtol=1e-14)
    assert np.allclose(gp[4:], 1 / (1 + np.exp(-z[4:])), rtol=1e-14)
    # symmetry L_pos(G) = L_neg(2 theta - G)
    Gs = np.array([0.5, 3.0, 3.5, 1.0], dtype=F32)
    Ls, _ = O.ff_loss_terms(Gs, theta, 2)
    assert math.isclose(Ls[0], Ls[2], rel_tol=1e-14) and math.isclose(Ls[1], Ls[3], rel_tol=1e-14)
    # asymptotes without overflow
    Gb = np.array([1e6, 0.0, 1e6, 0.0], dtype=F32)
    Lb, gb = O.ff_loss_terms(Gb, 1000.0, 2)
    assert np.all(np.isfinite(Lb)) and Lb[0] == 0.0 and math.isclose(Lb[2], 1e6 - 1000.0)
    assert math.isclose(Lb[1], 1000.0) and gb[1] == -1.0 and gb[2] == 1.0 and abs(gb[0]) < 1e-300
    # derivative of the loss by finite differences of the closed form
    for G0, pos in [(1.3, True), (2.9, False), (7.0, True)]:
        f = (lambda v: math.log1p(math.exp(-(v - theta)))) if pos else (lambda v: math.log1p(math.exp(v - theta)))
        fd = (f(G0 + 1e-6) - f(G0 - 1e-6)) / 2e-6
        arr = np.array([G0, G0], dtype=np.float64)
        _, gq = O.ff_loss_terms(arr, theta, 1)
        assert math.isclose(gq[0 if pos else 1], fd, rel_tol=1e-6)


def test_exp_and_sigmoid_recipe_accuracy():
    v = -np.concatenate([np.linspace(0, 50, 200001), np.linspace(50, 700, 20001)])
    got = O.exp_nonpos(v)
    want = np.exp(v)
    ulp = np.abs(got - want) / np.spacing(want)
    assert ulp.max() <= 2.0
    assert O.exp_nonpos(np.array([0.0]))[0] == 1.0
    assert O.exp_nonpos(np.array([-1e9]))[0] == O.exp_nonpos(np.array([-700.0]))[0] > 0
    x = np.linspace(-40, 40, 100001)
    s = O.sigmoid_spec(x)
    assert np.allclose(s, 1 / (1 + np.exp(-x)), rtol=1e-15, atol=0)
    assert np.allclose(s + O.sigmoid_spec(-x), 1.0, atol=2e-16)


def test_lookahead_loss_and_coef_closed_form():
    g = np.random.default_rng(8)
    B = 5
    Gs = [g.uniform(0, 6, size=2 * B).astype(F32) for _ in range(3)]
    th = [2.0, 3.0, 2.5]
    lam = 0.125
    loss, coef = O.lookahead_loss_coef(Gs, th, B, lam)
    per = [O.ff_loss_terms(G, t, B) for G, t in zip(Gs, th)]
    want_loss = np.mean(per[0][0] + lam * (per[1][0] + per[2][0]))          # Eq. 3
    assert math.isclose(loss, want_loss, rel_tol=1e-14)
    want_coef = (per[0][1] + lam * (per[1][1] + per[2][1])) / (2 * B)       # Eq. 4, scalar reading
    assert np.allclose(coef, want_coef, rtol=1e-6)
    # lambda = 0 and "no later layer" both reduce to the vanilla coefficient, bit for bit
    _, c0 = O.lookahead_loss_coef(Gs, th, B, 0.0)
    _, c1 = O.lookahead_loss_coef(Gs[:1], th[:1], B, 0.7)
    assert np.array_equal(c0, c1)
    assert np.all(c0[:B] <= 0) and np.all(c0[B:] >= 0)     # raise G on positives, lower on negatives


# ------------------------------------------------------------------ gradient (Sec. IV-B)
def _analytic_grad(spec, X, W, B):
    """dW of the unquantised mean loss through the oracle's own coefficient and dH = 2*coef*Y."""
    X64, W64 = X.astype(np.float64), W.astype(np.float64)
    Y = np.maximum(X64 @ W64.T, 0)
    G = (Y ** 2).sum(axis=1)
    z = G - spec.theta
    sign = np.concatenate([-np.ones(B), np.ones(B)])
    coef = sign * O.sigmoid_spec(sign * z) / (2 * B)
    return (2 * coef[:, None] * Y).T @ X64


def test_gradient_matches_finite_differences_fp64():
    g = np.random.default_rng(9)
    B, K, N = 3, 6, 5
    X = g.normal(size=(2 * B, K)).astype(F32)
    W = (g.normal(size=(N, K)) * 0.4).astype(F32)
    spec = _spec(K, N, theta=2.0)
    ana = _analytic_grad(spec, X, W, B)
    fd = np.zeros_like(ana)
    h = 1e-6
    for n in range(N):
        for k in range(K):
            Wp, Wm = W.astype(np.float64).copy(), W.astype(np.float64).copy()
            Wp[n, k] += h
            Wm[n, k] -= h
            fd[n, k] = (O.fp64_layer_loss(spec, X, Wp, B) - O.fp64_layer_loss(spec, X, Wm, B)) / (2 * h)
    assert np.allclose(ana, fd, rtol=1e-5, atol=1e-8)
    # the oracle's coefficient equals the one used above (float32-rounded)
    st = O.layer_forward(spec, X, W, B, 0)
    O.layer_loss_grad(spec, st, B, [], [], 0.0, 0)
    z = st.G.astype(np.float64) - 2.0
    sign = np.concatenate([-np.ones(B), np.ones(B)])
    assert np.allclose(st.coef, sign * O.sigmoid_spec(sign * z) / (2 * B), rtol=1e-6)


@pytest.mark.parametrize("kind", [0, 1])
def test_int8_gradient_tracks_fp64_gradient(kind):
    """The whole quantised chain (dH -> INT8 -> INT8 MAC -> dequantise) must point the way the
    finite-difference-checked gradient points: catches sign, transposition and scale mistakes."""
    g = np.random.default_rng(10 + kind)
    if kind == 0:
        B, K, N = 32, 96, 48
        spec = _spec(K, N, theta=float(N))
        X = g.normal(size=(2 * B, K)).astype(F32)
        W = (g.normal(size=(N, K)) * np.sqrt(2.0 / K)).astype(F32)
    else:
        B, H, Cin, N = 4, 6, 8, 8
        K = 9 * Cin
        spec = _spec(K, N, theta=float(N * H * H), kind=1, H=H, Wd=H, Cin=Cin)
        X = g.normal(size=(2 * B, H, H, Cin)).astype(F32)
        W = (g.normal(size=(N, K)) * np.sqrt(2.0 / K)).astype(F32)
    st = O.layer_forward(spec, X, W, B, 0)
    O.layer_loss_grad(spec, st, B, [], [], 0.0, 0)
    O.layer_update(spec, st, W, B)
    # float64 gradient of the unquantised loss by central differences on a sample of entries
    idx = [(int(g.integers(spec.N)), int(g.integers(spec.K))) for _ in range(40)]
    h = 1e-5
    fd = []
    for n, k in idx:
        Wp, Wm = W.astype(np.float64).copy(), W.astype(np.float64).copy()
        Wp[n, k] += h
        Wm[n, k] -= h
        fd.append((O.fp64_layer_loss(spec, X, Wp, B) - O.fp64_layer_loss(spec, X, Wm, B)) / (2 * h))
    fd = np.array(fd)
    got = np.array([st.dW[n, k] for n, k in idx], dtype=np.float64)
    cos = float(got @ fd / (np.linalg.norm(got) * np.linalg.norm(fd)))
    assert cos > 0.98
    assert 0.8 < np.linalg.norm(got) / np.linalg.norm(fd) < 1.25
    assert np.array_equal(st.W_new, W - F32(spec.lr) * st.dW)


def test_absmax_shortcuts_hold_bitwise():
    """max|dH| and max|Xnext| per pass equal the values obtained from the per-sample max of
    relu(acc) alone (rounded multiplication by a fixed factor is monotone)."""
    g = np.random.default_rng(12)
    B, K, N = 16, 64, 40
    spec = _spec(K, N, rnd=O.ROUND_STOCHASTIC)
    X = g.normal(size=(2 * B, K)).astype(F32)
    W = (g.normal(size=(N, K)) / 8).astype(F32)
    st = O.layer_forward(spec, X, W, B, 3)
    O.layer_loss_grad(spec, st, B, [], [], 0.0, 3)
    s_w = O.scale_pair(st.a_w)[0]
    r = F32(spec.tau) / (np.sqrt(st.G) + F32(spec.eps))
    for p in range(2):
        sl = slice(p * B, (p + 1) * B)
        c = O.scale_pair(st.a_x[p])[0] * s_w
        ymax = st.rowmax[sl].astype(F32) * c
        k2 = F32(2.0) * st.coef[sl]
        assert np.max(np.abs(k2 * ymax)) == st.a_dh[p]
        assert np.max(ymax * r[sl]) == O.absmax(st.Xnext[sl])


# ------------------------------------------------------------------ update / step
def test_update_hand_example_and_fixed_points():
    spec = _spec(2, 2, theta=0.5, lr=0.5)
    X = np.array([[1, 0.5], [-0.25, 0.5]], dtype=F32)
    W = np.array([[1, -1], [0.5, 0.25]], dtype=F32)
    st = O.layer_forward(spec, X, W, 1, 0)
    O.layer_loss_grad(spec, st, 1, [], [], 0.0, 0)
    O.layer_update(spec, st, W, 1)
    # negative row has Y = 0 -> dH = 0 -> its pass contributes nothing
    assert not st.dHq[1].any() and not st.accW[1].any() and st.a_dh[1] == 0
    # positive row: dH = 2*coef*y, |dH| max at y = 10176*c -> dHq = [-100 (rint(-99.86)), -127]
    assert np.array_equal(st.dHq[0], [-100, -127])
    assert np.array_equal(st.accW[0], [[-100 * 127, -100 * 64], [-127 * 127, -127 * 64]])
    G0 = 167566977 / 127.0 ** 4
    coef = -1 / (1 + math.exp(G0 - 0.5)) / 2
    dH1 = 2 * coef * 10176 / 127.0 ** 2
    dW = np.array(st.accW[0], dtype=np.float64) * (abs(dH1) / 127) * (1 / 127)
    assert np.allclose(st.dW, dW, rtol=1e-5)
    assert np.allclose(st.W_new, W - 0.5 * dW, rtol=1e-6)
    # lr = 0 leaves W untouched; so does a zero gradient
    spec0 = _spec(2, 2, theta=0.5, lr=0.0)
    st0 = O.layer_update(spec0, O.layer_loss_grad(spec0, O.layer_forward(spec0, X, W, 1, 0), 1, [], [], 0.0, 0), W, 1)
    assert np.array_equal(st0.W_new, W)
    Xz = np.zeros_like(X)
    stz = O.layer_update(spec, O.layer_loss_grad(spec, O.layer_forward(spec, Xz, W, 1, 0), 1, [], [], 0.0, 0), W, 1)
    assert np.array_equal(stz.W_new, W)


def _net(g, widths, B, rnd=O.ROUND_STOCHASTIC):
    specs = [_spec(K, N, rnd=rnd, index=i) for i, (K, N) in enumerate(zip(widths[:-1], widths[1:]))]
    Ws = [(g.normal(size=(s.N, s.K)) * np.sqrt(2.0 / s.K)).astype(F32) for s in specs]
    X = g.normal(size=(2 * B, widths[0])).astype(F32)
    return specs, Ws, X


def test_train_step_reductions_and_determinism():
    g = np.random.default_rng(13)
    B = 8
    specs, Ws, X = _net(g, [20, 24, 16, 12], B)
    a = O.train_step(specs, Ws, X, B, 0.0, 4)
    b = O.train_step(specs, Ws, X, B, 0.0, 4)
    for sa, sb in zip(a, b):                                  # run-to-run identity
        assert np.array_equal(sa.W_new, sb.W_new) and np.array_equal(sa.dHq, sb.dHq)
    # lambda = 0: every layer's step equals the stand-alone (vanilla) step on the same input
    x = X
    for l, spec in enumerate(specs):
        st = O.layer_forward(spec, x, Ws[l], B, 4)
        O.layer_loss_grad(spec, st, B, [], [], 0.0, 4)
        O.layer_update(spec, st, Ws[l], B)
        assert np.array_equal(st.W_new, a[l].W_new) and np.array_equal(st.dHq, a[l].dHq)
        assert st.loss == a[l].loss
        x = st.Xnext
    # lambda > 0 changes every layer but the last; all G's come from the pre-update forward
    c = O.train_step(specs, Ws, X, B, 0.5, 4)
    assert np.array_equal(c[-1].W_new, a[-1].W_new)
    assert not np.array_equal(c[0].coef, a[0].coef)
    for sa, sc in zip(a, c):
        assert np.array_equal(sa.G, sc.G) and np.array_equal(sa.Xq, sc.Xq)
    # Eq. 3 from the per-layer vanilla losses
    lam32 = float(F32(0.5))
    per = [O.ff_loss_terms(s.G, sp.theta, B)[0] for s, sp in zip(a, specs)]
    assert math.isclose(c[0].loss, float(np.mean(per[0] + lam32 * (per[1] + per[2]))), rel_tol=1e-12)
    # different step index -> different stochastic rounding, same scales
    d = O.train_step(specs, Ws, X, B, 0.0, 5)
    assert d[0].a_x == a[0].a_x and not np.array_equal(d[0].Xq, a[0].Xq)


def test_tiny_range_is_treated_as_zero_tensor():
    # a subnormal range would make 127/a overflow; below 2^-100 the tensor quantises to zeros
    x = np.array([1e-40, -3e-41, 0.0], dtype=F32)
    a = O.absmax(x)
    assert a > 0 and O.scale_pair(a) == (F32(1.0), F32(0.0))
    assert not O.quantize(x, a, O.ROUND_NEAREST).any()
    assert not O.quantize(x, a, O.ROUND_STOCHASTIC, key=(3, 4)).any()
    b = F32(2.0 ** -99)
    s, inv = O.scale_pair(b)
    assert np.isfinite(inv) and s == b / F32(127.0)


# --------------------------------------------------------------------------------------
# Classification by goodness, and the direction of learning
# --------------------------------------------------------------------------------------
def test_predict_hand_example_and_tie_rule():
    # one linear layer with identity-like weights, nearest rounding, B = 2 samples, 2 candidate labels:
    # sample 0 is longer along unit 0 under label 0, sample 1 gives both labels the same goodness (tie -> 0)
    spec = O.LayerSpec(O.KIND_LINEAR, 2, 2, theta=1.0, lr=0.0, tau=1.0, round_x=0, round_w=0, round_dh=0)
    W = np.eye(2, dtype=np.float32)
    X = np.array([[1.0, 0.0],     # label 0, sample 0
                  [1.0, 1.0],     # label 0, sample 1
                  [0.5, 0.0],     # label 1, sample 0
                  [1.0, 1.0]],    # label 1, sample 1  (both halves have range 1, so the tie is exact)
                 dtype=np.float32)
    pred, scores, states = O.predict([spec], [W], X, B=2, n_classes=2, step=0)
    assert scores.shape == (2, 2)
    assert scores[0, 0] > scores[1, 0] and scores[0, 1] == scores[1, 1]
    assert pred.tolist() == [0, 0]
    # scores are the goodness of the only layer
    assert np.array_equal(scores.reshape(-1), states[0].G)
    # with two layers and first_counted = 1 only the second layer counts
    spec2 = O.LayerSpec(O.KIND_LINEAR, 2, 2, theta=1.0, lr=0.0, tau=1.0, round_x=0, round_w=0, round_dh=0, index=1)
    _, s2, st2 = O.predict([spec, spec2], [W, W], X, 2, 2, 0, first_counted=1)
    assert np.array_equal(s2.reshape(-1), st2[1].G)
    _, s01, st01 = O.predict([spec, spec2], [W, W], X, 2, 2, 0, first_counted=0)
    assert np.array_equal(s01.reshape(-1), (st01[0].G + st01[1].G).astype(np.float32))


def test_predict_compares_all_candidates_under_one_quantisation_step():
    """The candidate batch is quantised with one range per tensor: the scores of a sample's candidates then do not
    depend on where a candidate sits in the batch.  With nearest rounding (no element counters involved) a
    permutation of the candidate labels permutes the scores exactly; with one range per half it would not."""
    g = np.random.default_rng(5)
    K, N, C, B = 24, 16, 6, 5
    specs = [O.LayerSpec(O.KIND_LINEAR, K, N, float(N), 0.0, float(np.sqrt(N)), round_x=0, round_w=0, round_dh=0, index=0),
             O.LayerSpec(O.KIND_LINEAR, N, N, float(N), 0.0, float(np.sqrt(N)), round_x=0, round_w=0, round_dh=0, index=1)]
    Ws = [g.normal(size=(N, K)).astype(F32) * 0.3, g.normal(size=(N, N)).astype(F32) * 0.3]
    X = g.normal(size=(C, B, K)).astype(F32)
    X[3] *= 4.0                                    # one candidate with a much larger range than the others
    _, scores, states = O.predict(specs, Ws, X.reshape(C * B, K), B, C, step=0)
    perm = np.array([4, 0, 3, 5, 1, 2])
    _, scores_p, _ = O.predict(specs, Ws, X[perm].reshape(C * B, K), B, C, step=0)
    assert np.array_equal(scores_p, scores[perm])
    assert states[0].a_x[0] == states[0].a_x[1] == O.absmax(X)
    # the per-half ranges of a training batch do depend on the placement (the case the classification must avoid)
    a = O.layer_forward(specs[0], X.reshape(C * B, K), Ws[0], C * B // 2, 0)
    b = O.layer_forward(specs[0], X[perm].reshape(C * B, K), Ws[0], C * B // 2, 0)
    assert a.a_x != b.a_x
    # an odd number of classes is fine as long as the rows split into two halves
    pred, sc, _ = O.predict(specs, Ws, X[:5, :4].reshape(20, K), 4, 5, step=0)
    assert sc.shape == (5, 4) and pred.shape == (4,)
    with pytest.raises(ValueError):
        O.predict(specs, Ws, X[:5, :3].reshape(15, K), 3, 5, step=0)


def test_int8_ff_training_learns_and_predicts_separable_classes():
    """End-to-end direction check of the whole oracle: FF-INT8 training (positive set = true label, negative
    set = wrong label, Eq. 1 / Eq. 2, INT8 gradients) followed by classification by goodness must learn
    class-dependent synthetic data: a flipped sign anywhere (loss, gradient, update, argmax) keeps the
    accuracy at chance."""
    K, N, C, B = 64, 64, 10, 64
    g = np.random.default_rng(0)
    patterns = g.normal(size=(C, K))

    def draw(gen, n):
        lab = gen.integers(0, C, size=n)
        return patterns[lab] + 0.5 * gen.normal(size=(n, K)), lab

    def embed(base, lab):
        x = base.copy()
        x[:, :C] = 0.0
        x[np.arange(len(lab)), lab] = 1.0
        return (x * np.sqrt(K) / np.sqrt((x ** 2).sum(1, keepdims=True))).astype(np.float32)

    specs = [O.LayerSpec(O.KIND_LINEAR, K, N, theta=float(N), lr=0.03, tau=float(np.sqrt(N)), seed=3, index=0),
             O.LayerSpec(O.KIND_LINEAR, N, N, theta=float(N), lr=0.03, tau=float(np.sqrt(N)), seed=3, index=1)]
    Ws = [(g.uniform(-1, 1, size=(N, K)) * np.sqrt(6 / K)).astype(np.float32),
          (g.uniform(-1, 1, size=(N, N)) * np.sqrt(6 / N)).astype(np.float32)]

    def accuracy(weights):
        base, lab = draw(np.random.default_rng(999), 200)
        Xc = np.concatenate([embed(base, np.full(200, c)) for c in range(C)])
        pred, _, _ = O.predict(specs, weights, Xc, 200, C, step=0)
        return float((pred == lab).mean())

    assert accuracy(Ws) < 0.3
    for step in range(40):
        base, lab = draw(g, B)
        wrong = (lab + g.integers(1, C, size=B)) % C
        X = np.concatenate([embed(base, lab), embed(base, wrong)])
        Ws = [st.W_new for st in O.train_step(specs, Ws, X, B, 0.0, step)]
    assert accuracy(Ws) > 0.9


# --------------------------------------------------------------------------------------
# Layer-by-layer (greedy) schedule, Sec. III
# --------------------------------------------------------------------------------------
def test_frozen_layers_only_forward_and_the_trained_layer_sees_their_output():
    g = np.random.default_rng(21)
    B = 6
    specs, Ws, X = _net(g, [20, 24, 16, 12], B)
    for first in range(3):
        full = O.train_step(specs, Ws, X, B, 0.25, 9)
        part = O.train_step(specs, Ws, X, B, 0.25, 9, first_trained=first)
        for l, (a, b) in enumerate(zip(full, part)):
            # the forward is the same whatever is trained
            assert np.array_equal(a.Xq, b.Xq) and np.array_equal(a.G, b.G) and np.array_equal(a.Xnext, b.Xnext)
            if l < first:
                assert b.coef is None and b.dHq is None and b.W_new is None and b.loss is None
            else:  # a trained layer's step does not depend on whether earlier layers are trained too
                assert np.array_equal(a.W_new, b.W_new) and np.array_equal(a.dHq, b.dHq) and a.loss == b.loss
    # one trained layer at the end, lambda = 0: the stand-alone step on the frozen layers' normalised output
    x = X
    for l in range(2):
        x = O.layer_forward(specs[l], x, Ws[l], B, 9).Xnext
    alone = O.train_step([specs[2]], [Ws[2]], x, B, 0.0, 9)[0]
    part = O.train_step(specs, Ws, X, B, 0.0, 9, first_trained=2)[2]
    assert np.array_equal(alone.W_new, part.W_new) and np.array_equal(alone.Xq, part.Xq)


def test_greedy_epoch_trains_one_layer_per_phase_on_trained_predecessors():
    g = np.random.default_rng(22)
    B, nb = 6, 3
    specs, W0, _ = _net(g, [20, 24, 16], B)
    batches = [g.normal(size=(2 * B, 20)).astype(F32) for _ in range(nb)]
    seen = []
    Wt = O.greedy_epoch(specs, W0, batches, B, lambda l, i, st: seen.append((l, i, st)))
    assert [(l, i) for l, i, _ in seen] == [(l, i) for l in range(2) for i in range(nb)]
    # the same schedule written out by hand: phase 0 on the raw batches, phase 1 on the forward of the TRAINED layer 0
    W = [w.copy() for w in W0]
    for i in range(nb):
        W[0] = O.train_step([specs[0]], [W[0]], batches[i], B, 0.0, i)[0].W_new
    assert np.array_equal(W[0], Wt[0]) and not np.array_equal(W0[0], Wt[0])
    for i in range(nb):
        x = O.layer_forward(specs[0], batches[i], W[0], B, nb + i).Xnext
        W[1] = O.train_step([specs[1]], [W[1]], x, B, 0.0, nb + i)[0].W_new
    assert np.array_equal(W[1], Wt[1])
    # had phase 1 run on the untrained layer 0 the result would differ (the case the schedule must not be)
    Wu = W0[1].copy()
    for i in range(nb):
        x = O.layer_forward(specs[0], batches[i], W0[0], B, nb + i).Xnext
        Wu = O.train_step([specs[1]], [Wu], x, B, 0.0, nb + i)[0].W_new
    assert not np.array_equal(Wu, Wt[1])
    # layer 0 is left alone during phase 1
    for l, i, st in seen:
        if l == 1:
            assert st[0].W_new is None


# --------------------------------------------------------------------------------------
# Skip path of a residual block
# --------------------------------------------------------------------------------------
def test_skip_path_hand_example_and_neutral_cases():
    # z = xhat + scale*skip, one float32 multiply and one float32 add per element
    xhat = np.array([[0.0, 1.5, 0.25], [2.0, 0.0, 0.0]], dtype=F32)
    skip = np.array([[1.0, -0.5, 4.0], [0.125, 3.0, -1.0]], dtype=F32)
    assert np.array_equal(O.add_skip(xhat, skip, 0.5), np.array([[0.5, 1.25, 2.25], [2.0625, 1.5, -0.5]], dtype=F32))
    assert np.array_equal(O.add_skip(xhat, skip, 1.0), xhat + skip)
    # each operation rounds on its own: 0.1f*3 is not 0.3f, and the sum rounds again
    a, b = np.array([[1.0]], dtype=F32), np.array([[3.0]], dtype=F32)
    want = F32(F32(1.0) + F32(F32(0.1) * F32(3.0)))
    assert O.add_skip(a, b, 0.1)[0, 0] == want
    # a zero weight or a zero tensor changes nothing, bit for bit (xhat >= 0, so no signed zero can appear)
    assert np.array_equal(O.add_skip(xhat, skip, 0.0).view(np.uint32), xhat.view(np.uint32))
    assert np.array_equal(O.add_skip(xhat, np.zeros_like(skip), 0.7).view(np.uint32), xhat.view(np.uint32))
    # a spatial output takes the flat skip tensor of the same size
    assert O.add_skip(xhat.reshape(2, 1, 1, 3), skip, 1.0).shape == (2, 1, 1, 3)
    with pytest.raises(ValueError):
        O.add_skip(xhat, skip[:, :2], 1.0)


def test_residual_block_changes_only_what_the_next_layer_sees():
    g = np.random.default_rng(31)
    B = 6
    specs, Ws, X = _net(g, [20, 24, 20, 12], B)           # layer 1 maps back to the width of the block's input
    plain = O.train_step(specs, Ws, X, B, 0.25, 3)
    specs[1].skip_from, specs[1].skip_scale = 0, 1.0      # block = layers 0..1, skip from the block's input
    res = O.train_step(specs, Ws, X, B, 0.25, 3)
    for l in (0, 1):   # the block's own layers: same input codes, same goodness
        assert np.array_equal(plain[l].Xq, res[l].Xq) and np.array_equal(plain[l].G, res[l].G)
    assert np.array_equal(plain[1].Y, res[1].Y)
    # what leaves the block is the normalised output plus the block's input
    assert np.array_equal(res[1].Xnext, plain[1].Xnext + X)
    assert not np.array_equal(plain[2].Xq, res[2].Xq)
    assert np.array_equal(res[2].Xq, O.quantize_two_pass(res[1].Xnext, B, specs[2].round_x,
                                                         O.rounding_key(specs[2].seed, O.ROLE_X, 2, 3))[0])
    # lengths: both summands have a fixed length per sample, so the sum lies between their difference and their sum
    n_out = np.sqrt((res[1].Xnext.astype(np.float64) ** 2).sum(1))
    n_a = np.sqrt((plain[1].Xnext.astype(np.float64) ** 2).sum(1))
    n_b = np.sqrt((X.astype(np.float64) ** 2).sum(1))
    assert np.all(n_out <= (n_a + n_b) * (1 + 1e-6)) and np.all(n_out >= np.abs(n_a - n_b) * (1 - 1e-6))
    # weight 0 is the plain network, bit for bit
    specs[1].skip_scale = 0.0
    zero = O.train_step(specs, Ws, X, B, 0.25, 3)
    for a, b in zip(plain, zero):
        assert np.array_equal(a.W_new, b.W_new) and np.array_equal(a.Xq, b.Xq)
    # the look-ahead coefficient of the block's layers sees the goodness of the layer AFTER the block, which the skip
    # path changed: with lambda > 0 their gradient codes differ from the plain network's, with lambda = 0 they do not
    specs[1].skip_scale = 1.0
    res0 = O.train_step(specs, Ws, X, B, 0.0, 3)
    plain0 = O.train_step([O.LayerSpec(**{**s.__dict__, "skip_from": -1}) for s in specs], Ws, X, B, 0.0, 3)
    for l in (0, 1):
        assert np.array_equal(res0[l].dHq, plain0[l].dHq) and np.array_equal(res0[l].W_new, plain0[l].W_new)
    assert not np.array_equal(res[0].coef, plain[0].coef)
    # a skip source must be this layer's input or an earlier one, and the sizes must agree
    specs[1].skip_from = 2
    with pytest.raises(ValueError):
        O.train_step(specs, Ws, X, B, 0.0, 3)
    specs[1].skip_from = 1
    with pytest.raises(ValueError):
        O.train_step(specs, Ws, X, B, 0.0, 3)      # layer 1's input has 24 values, its output 20


def test_skip_path_in_a_convolutional_block():
    g = np.random.default_rng(32)
    B, H, C = 2, 4, 8
    specs = [_spec(9 * C, C, kind=O.KIND_CONV3X3, H=H, Wd=H, Cin=C, rnd=O.ROUND_STOCHASTIC, index=i) for i in range(2)]
    specs[1].skip_from = 0
    Ws = [(g.normal(size=(C, 9 * C)) * 0.2).astype(F32) for _ in specs]
    X = g.normal(size=(2 * B, H, H, C)).astype(F32)
    st = O.train_step(specs, Ws, X, B, 0.0, 0)
    no = O.layer_forward(specs[1], st[0].Xnext, Ws[1], B, 0)
    assert st[1].Xnext.shape == X.shape and np.array_equal(st[1].Xnext, no.Xnext + X)
    specs[1].pool = 2
    with pytest.raises(ValueError):
        O.train_step(specs, Ws, X, B, 0.0, 0)


# --------------------------------------------------------------------------------------
# Pointwise convolution
# --------------------------------------------------------------------------------------
def test_conv1x1_equals_centre_tap_of_conv3x3():
    """A 1x1 convolution is a 3x3 convolution whose only non-zero tap is the centre one: the whole train
    step of the pointwise layer must reproduce the (brute-force-pinned) 3x3 layer with embedded weights,
    and its weight gradient must equal the centre tap of the 3x3 one."""
    g = np.random.default_rng(11)
    B, H, Wd, Cin, N = 2, 5, 6, 7, 9
    X = g.normal(size=(2 * B, H, Wd, Cin)).astype(F32)
    W1 = g.normal(size=(N, Cin)).astype(F32) * 0.3
    W3 = np.zeros((N, 3, 3, Cin), dtype=F32)
    W3[:, 1, 1, :] = W1
    theta, tau = float(N * H * Wd) / 2, float(np.sqrt(N * H * Wd))
    s1 = O.LayerSpec(O.KIND_CONV1X1, Cin, N, theta, 0.05, tau, H=H, Wd=Wd, Cin=Cin, seed=4)
    s3 = O.LayerSpec(O.KIND_CONV3X3, 9 * Cin, N, theta, 0.05, tau, H=H, Wd=Wd, Cin=Cin, seed=4)
    a = O.train_step([s1], [W1], X, B, 0.0, 5)[0]
    b = O.train_step([s3], [W3.reshape(N, -1)], X, B, 0.0, 5)[0]
    assert np.array_equal(a.Xq, b.Xq) and a.a_w == b.a_w
    assert np.array_equal(a.Wq, b.Wq.reshape(N, 3, 3, Cin)[:, 1, 1, :])
    assert np.array_equal(a.acc, b.acc) and np.array_equal(a.Y, b.Y) and np.array_equal(a.G, b.G)
    assert np.array_equal(a.coef, b.coef) and np.array_equal(a.dHq, b.dHq) and a.loss == b.loss
    assert np.array_equal(a.accW, b.accW.reshape(2, N, 3, 3, Cin)[:, :, 1, 1, :])
    assert np.array_equal(a.W_new, b.W_new.reshape(N, 3, 3, Cin)[:, 1, 1, :])
    assert a.Y.shape == (2 * B, H, Wd, N) and s1.rows_per_sample == H * Wd


def test_conv1x1_gradient_matches_finite_differences():
    g = np.random.default_rng(12)
    B, H, Wd, Cin, N = 2, 3, 3, 4, 5
    X = g.normal(size=(2 * B, H, Wd, Cin))
    W = g.normal(size=(N, Cin)) * 0.4
    spec = O.LayerSpec(O.KIND_CONV1X1, Cin, N, float(N * H * Wd) / 2, 0.0, 1.0, H=H, Wd=Wd, Cin=Cin)
    # analytic dL/dW of the unquantised layer: dH = 2*coef*Y with coef = dL/dG / (2B), dW = dH^T X over positions
    Y = np.maximum(X @ W.T, 0.0)
    G = (Y.reshape(2 * B, -1) ** 2).sum(1)
    _, gp = O.ff_loss_terms(G.astype(F32), spec.theta, B)
    coef = gp / (2 * B)
    dH = 2.0 * coef[:, None, None, None] * Y
    dW = dH.reshape(-1, N).T @ X.reshape(-1, Cin)
    eps = 1e-6
    for (n, k) in [(0, 0), (2, 3), (4, 1)]:
        Wp, Wm = W.copy(), W.copy()
        Wp[n, k] += eps
        Wm[n, k] -= eps
        fd = (O.fp64_layer_loss(spec, X, Wp, B) - O.fp64_layer_loss(spec, X, Wm, B)) / (2 * eps)
        assert abs(fd - dW[n, k]) <= 1e-4 * max(1.0, abs(fd)), (n, k, fd, dW[n, k])


# --------------------------------------------------------------------------------------
# Strided 3x3 convolution
# --------------------------------------------------------------------------------------
def test_strided_conv_is_the_subsampled_stride1_conv_and_matches_brute_force():
    g = np.random.default_rng(21)
    for (H, Wd) in [(6, 8), (5, 7)]:                      # even and odd extents
        x = g.integers(-127, 128, size=(2, H, Wd, 3)).astype(np.int8)
        w = g.integers(-127, 128, size=(4, 3, 3, 3)).astype(np.int8)
        full = O.int8_conv3x3(x, w)                      # pinned by brute force above
        half = O.int8_conv3x3(x, w, stride=2)
        assert half.shape == (2, (H - 1) // 2 + 1, (Wd - 1) // 2 + 1, 4)
        assert np.array_equal(half, full[:, ::2, ::2, :])
        # weight gradient: brute force over the strided windows
        d = g.integers(-127, 128, size=half.shape).astype(np.int8)
        got = O.int8_conv3x3_wgrad(d, x, stride=2)
        want = np.zeros((4, 3, 3, 3), dtype=np.int64)
        Ho, Wo = half.shape[1:3]
        for b in range(2):
            for i in range(Ho):
                for j in range(Wo):
                    for r in range(3):
                        for t in range(3):
                            hh, ww = 2 * i + r - 1, 2 * j + t - 1
                            if 0 <= hh < H and 0 <= ww < Wd:
                                want[:, r, t, :] += np.outer(d[b, i, j].astype(np.int64), x[b, hh, ww].astype(np.int64))
        assert np.array_equal(got, want)


def test_strided_conv_gradient_matches_finite_differences():
    g = np.random.default_rng(22)
    B, H, Wd, Cin, N = 1, 5, 6, 2, 3
    spec = O.LayerSpec(O.KIND_CONV3X3, 9 * Cin, N, 10.0, 0.0, 1.0, H=H, Wd=Wd, Cin=Cin, stride=2)
    X = g.normal(size=(2 * B, H, Wd, Cin))
    W = g.normal(size=(N, 9 * Cin)) * 0.3
    Ho, Wo = spec.out_hw
    assert (Ho, Wo) == (3, 3) and spec.rows_per_sample == 9
    # analytic gradient of the unquantised layer through the oracle's own integer routines is not possible;
    # use the float formula: dW[n,r,s,ci] = sum dH[b,i,j,n] * xpad[b,2i+r,2j+s,ci]
    xp = np.pad(X, ((0, 0), (1, 1), (1, 1), (0, 0)))
    w4 = W.reshape(N, 3, 3, Cin)
    Y = np.zeros((2 * B, Ho, Wo, N))
    for r in range(3):
        for s in range(3):
            Y += xp[:, r:r + 2 * (Ho - 1) + 1:2, s:s + 2 * (Wo - 1) + 1:2, :] @ w4[:, r, s, :].T
    Y = np.maximum(Y, 0.0)
    G = (Y.reshape(2 * B, -1) ** 2).sum(1)
    _, gp = O.ff_loss_terms(G.astype(F32), spec.theta, B)
    dH = 2.0 * (gp / (2 * B))[:, None, None, None] * Y
    dW = np.zeros((N, 3, 3, Cin))
    for r in range(3):
        for s in range(3):
            win = xp[:, r:r + 2 * (Ho - 1) + 1:2, s:s + 2 * (Wo - 1) + 1:2, :]
            dW[:, r, s, :] = dH.reshape(-1, N).T @ win.reshape(-1, Cin)
    dW = dW.reshape(N, -1)
    eps = 1e-6
    for (n, k) in [(0, 0), (1, 7), (2, 17)]:
        Wp, Wm = W.copy(), W.copy()
        Wp[n, k] += eps
        Wm[n, k] -= eps
        fd = (O.fp64_layer_loss(spec, X, Wp, B) - O.fp64_layer_loss(spec, X, Wm, B)) / (2 * eps)
        assert abs(fd - dW[n, k]) <= 1e-4 * max(1.0, abs(fd)), (n, k, fd, dW[n, k])


# ---- label embedding (positive / negative / candidate batches; Sec. III, Alg. 1, sample generation) ------------
def test_embed_labels_hand_example():
    x = np.array([[9.0, 9.0, 9.0, 3.0, 4.0]], dtype=np.float32)          # 3 label places, then the data
    got = O.embed_labels(x, np.array([[2], [0]]), n_classes=3)
    assert np.array_equal(got, np.array([[0, 0, 1, 3, 4], [1, 0, 0, 3, 4]], dtype=np.float32))
    # scaled to length 13: |(0,0,12,3,4)| = 13 exactly, so r = 13/(13+0) = 1 and nothing changes
    got = O.embed_labels(x, np.array([[2]]), n_classes=3, on_value=12.0, tau0=13.0, eps=0.0)
    assert np.array_equal(got, np.array([[0, 0, 12, 3, 4]], dtype=np.float32))
    # label places two apart (a channels-last image: channel 0 of the first pixels)
    x = np.arange(1, 9, dtype=np.float32).reshape(1, 8)
    got = O.embed_labels(x, np.array([[1]]), n_classes=3, label_stride=2, on_value=5.0)
    assert np.array_equal(got, np.array([[0, 2, 5, 4, 0, 6, 7, 8]], dtype=np.float32))


def test_embed_labels_matches_the_batch_generator_and_has_unit_invariants():
    from paper_2506_22771_b200 import synth
    # the input generator builds its batches the same way from its own base samples (float64, then cast):
    # rebuild one of its batches from those base samples and compare
    w = synth.workload("tiny_mlp")
    B, n = 16, int(np.prod(w.in_shape))
    raw, labels, stride = synth.make_raw(w, 7, B=B)
    base, (label, wrong) = raw.astype(np.float64), labels
    want = synth.make_batch(w, 7, B=B).reshape(2 * B, n)
    got = O.embed_labels(raw, labels, 10, label_stride=stride, tau0=float(np.sqrt(n)))
    assert np.allclose(got, want, rtol=2e-6, atol=0.0)
    # invariants: length tau0, label places one-hot, data entries of both sets parallel to the raw sample
    assert np.allclose(np.sqrt((got.astype(np.float64) ** 2).sum(1)), np.sqrt(n), rtol=1e-6)
    hot = got[:, :10] != 0
    assert (hot.sum(1) == 1).all() and (hot.argmax(1) == np.concatenate([label, wrong])).all()
    ratio = got[:, 10:] / np.concatenate([base, base])[:, 10:].astype(np.float32)
    assert np.allclose(ratio, ratio[:, :1], rtol=1e-6)
    with pytest.raises(ValueError):
        O.embed_labels(base.astype(np.float32), np.full((1, B), 10), 10)


# ---- heavy-ball variant of the update (Alg. 1, update step names no optimiser) ----------------------------
def test_sgd_momentum_hand_example_and_closed_form():
    # powers of two: every product and sum is exact in float32
    W, M = np.array([1.0, -2.0], np.float32), np.array([0.5, 0.0], np.float32)
    g = np.array([0.25, 1.0], np.float32)
    W1, M1 = O.sgd_momentum(W, M, g, lr=0.5, mu=0.5)
    assert np.array_equal(M1, np.array([0.5, 1.0], np.float32))          # 0.5*0.5 + 0.25 ; 0 + 1
    assert np.array_equal(W1, np.array([0.75, -2.5], np.float32))        # 1 - 0.5*0.5 ; -2 - 0.5*1
    W2, M2 = O.sgd_momentum(W1, M1, g, lr=0.5, mu=0.5)
    assert np.array_equal(M2, np.array([0.5, 1.5], np.float32)) and np.array_equal(W2, np.array([0.5, -3.25], np.float32))
    # constant gradient from m = 0: m_t = g (1 - mu^t)/(1 - mu), W_t = W_0 - lr * sum_{i<=t} m_i
    mu, lr, gg = 0.9, 0.01, np.float32(0.3)
    Wt, Mt = np.zeros(1, np.float32), np.zeros(1, np.float32)
    for t in range(1, 51):
        Wt, Mt = O.sgd_momentum(Wt, Mt, np.array([gg]), lr, mu)
        m_closed = 0.3 * (1 - mu ** t) / (1 - mu)
        w_closed = -lr * 0.3 * (t - mu * (1 - mu ** t) / (1 - mu)) / (1 - mu)
        assert abs(Mt[0] - m_closed) < 1e-5 and abs(Wt[0] - w_closed) < 1e-5
    # mu = 0 is plain SGD bit for bit
    g3 = np.random.default_rng(0).normal(size=7).astype(np.float32)
    W3 = np.random.default_rng(1).normal(size=7).astype(np.float32)
    assert np.array_equal(O.sgd_momentum(W3, np.ones(7, np.float32), g3, 0.03, 0.0)[0], W3 - np.float32(0.03) * g3)


def test_layer_update_with_momentum_carries_the_buffer():
    from paper_2506_22771_b200 import synth
    w = synth.scaled(synth.workload("tiny_mlp"), B=8, width_div=8)
    l = w.layers[0]
    plain = O.LayerSpec(l.kind, l.K, l.N, l.theta, l.lr, l.tau, seed=3)
    heavy = O.LayerSpec(l.kind, l.K, l.N, l.theta, l.lr, l.tau, seed=3, momentum=0.75)
    W0 = synth.make_weights(w, 3)[0]
    X = synth.make_batch(w, 3)
    a = O.train_step([plain], [W0], X, w.B, 0.0, 0)[0]
    b = O.train_step([heavy], [W0], X, w.B, 0.0, 0)[0]
    # from a zero buffer the first heavy-ball step is the plain step and leaves m = g
    assert np.array_equal(a.W_new, b.W_new) and np.array_equal(b.M_new, b.dW) and a.M_new is None
    b2 = O.train_step([heavy], [b.W_new], X, w.B, 0.0, 1, Ms=[b.M_new])[0]
    a2 = O.train_step([plain], [b.W_new], X, w.B, 0.0, 1)[0]
    assert np.array_equal(b2.dW, a2.dW)                                   # same gradient, different step
    assert np.array_equal(b2.M_new, np.float32(0.75) * b.dW + b2.dW)
    assert np.array_equal(b2.W_new, b.W_new - np.float32(l.lr) * b2.M_new)
    assert not np.array_equal(b2.W_new, a2.W_new)


# --------------------------------------------------------------------------------------
# Depthwise 3x3 convolution
# --------------------------------------------------------------------------------------
def test_depthwise_conv_is_the_full_conv_with_one_filter_per_channel():
    g = np.random.default_rng(31)
    for stride, (H, Wd) in [(1, (5, 6)), (2, (5, 6)), (2, (4, 7))]:
        C = 5
        x = g.integers(-127, 128, size=(3, H, Wd, C)).astype(np.int8)
        w = g.integers(-127, 128, size=(C, 3, 3)).astype(np.int8)
        # the full convolution (pinned by brute force) whose filter for output channel c looks at input channel c only
        wfull = np.zeros((C, 3, 3, C), dtype=np.int8)
        for c in range(C):
            wfull[c, :, :, c] = w[c]
        got = O.int8_dwconv3x3(x, w, stride)
        assert np.array_equal(got, O.int8_conv3x3(x, wfull, stride))
        # weight gradient: the matching entries of the full convolution's gradient
        d = g.integers(-127, 128, size=got.shape).astype(np.int8)
        full_grad = O.int8_conv3x3_wgrad(d, x, stride)                   # [C,3,3,C]
        want = np.stack([full_grad[c, :, :, c] for c in range(C)])
        assert np.array_equal(O.int8_dwconv3x3_wgrad(d, x, stride), want)


def test_depthwise_conv_brute_force_single_output():
    x = np.zeros((1, 3, 3, 2), dtype=np.int8)
    x[0, :, :, 0] = np.arange(1, 10).reshape(3, 3)
    x[0, :, :, 1] = -1
    w = np.zeros((2, 3, 3), dtype=np.int8)
    w[0] = np.arange(9, 0, -1).reshape(3, 3)
    w[1, 1, 1] = 7
    acc = O.int8_dwconv3x3(x, w)
    assert acc[0, 1, 1, 0] == sum((i + 1) * (9 - i) for i in range(9))   # centre: all nine taps
    assert acc[0, 0, 0, 0] == 1 * 5 + 2 * 4 + 4 * 2 + 5 * 1              # corner: the four taps inside the image
    assert np.all(acc[0, :, :, 1] == -7)                                  # channel 1 never sees channel 0


def test_depthwise_gradient_matches_finite_differences():
    g = np.random.default_rng(32)
    for stride in (1, 2):
        B, H, Wd, C = 1, 4, 5, 3
        spec = O.LayerSpec(O.KIND_DWCONV3X3, 9, C, 6.0, 0.0, 1.0, H=H, Wd=Wd, Cin=C, stride=stride)
        X = g.normal(size=(2 * B, H, Wd, C))
        W = g.normal(size=(C, 9)) * 0.5
        Ho, Wo = spec.out_hw
        xp = np.pad(X, ((0, 0), (1, 1), (1, 1), (0, 0)))
        w3 = W.reshape(C, 3, 3)
        wins = {(r, s): xp[:, r:r + stride * (Ho - 1) + 1:stride, s:s + stride * (Wo - 1) + 1:stride, :]
                for r in range(3) for s in range(3)}
        Y = np.maximum(sum(wins[r, s] * w3[:, r, s] for r in range(3) for s in range(3)), 0.0)
        G = (Y.reshape(2 * B, -1) ** 2).sum(1)
        _, gp = O.ff_loss_terms(G.astype(F32), spec.theta, B)
        dH = 2.0 * (gp / (2 * B))[:, None, None, None] * Y
        eps = 1e-6
        for (c, r, s) in [(0, 0, 0), (1, 1, 1), (2, 2, 0), (1, 0, 2)]:
            dW = (dH * wins[r, s])[..., c].sum()
            Wp, Wm = W.copy(), W.copy()
            Wp[c, r * 3 + s] += eps
            Wm[c, r * 3 + s] -= eps
            fd = (O.fp64_layer_loss(spec, X, Wp, B) - O.fp64_layer_loss(spec, X, Wm, B)) / (2 * eps)
            assert abs(fd - dW) <= 1e-4 * max(1.0, abs(fd)), (stride, c, r, s, fd, dW)


def test_depthwise_layer_step_descends_and_chains():
    # a depthwise layer between two pointwise layers (the separable block of the paper's mobile models): the INT8
    # gradient of the depthwise layer correlates with the float64 gradient of the unquantised loss
    g = np.random.default_rng(33)
    B, H, Wd, C = 4, 6, 6, 8
    spec = O.LayerSpec(O.KIND_DWCONV3X3, 9, C, float(C * H * Wd) / 2, 0.01, float(np.sqrt(C * H * Wd)), H=H, Wd=Wd, Cin=C,
                       seed=5)
    X = g.normal(size=(2 * B, H, Wd, C)).astype(F32)
    W = (g.normal(size=(C, 9)) * 0.5).astype(F32)
    st = O.train_step([spec], [W], X, B, 0.0, 0)[0]
    assert st.acc.shape == (2 * B, H, Wd, C) and st.accW.shape == (2, C, 9) and st.W_new.shape == (C, 9)
    fd = np.zeros_like(W, dtype=np.float64)
    eps = 1e-5
    for idx in np.ndindex(*W.shape):
        Wp, Wm = W.astype(np.float64), W.astype(np.float64)
        Wp[idx] += eps
        Wm[idx] -= eps
        fd[idx] = (O.fp64_layer_loss(spec, X, Wp, B) - O.fp64_layer_loss(spec, X, Wm, B)) / (2 * eps)
    cos = float((st.dW * fd).sum() / (np.linalg.norm(st.dW) * np.linalg.norm(fd)))
    assert cos > 0.98, cos


# ---- Adam variant of the update ------------------------------------------------------------------------
def test_pow_int_and_adam_hand_example():
    assert O._pow_int(0.5, 0) == 1.0 and O._pow_int(0.5, 10) == 2.0 ** -10 and O._pow_int(3.0, 5) == 243.0
    assert abs(O._pow_int(0.999, 1000) - 0.999 ** 1000) < 1e-13      # ten roundings of relative size 2^-53, amplified by the squarings
    # first update from zero buffers: m*c1 = g and v*c2 = g*g, so the step is lr*g/(|g|+eps) whatever the betas.
    # Powers of two keep every operation exact: beta1 = 0.5, beta2 = 0.75, g = 2, eps = 2 -> step = lr*2/4
    W1, M1, V1 = O.adam_update(np.array([1.0], np.float32), np.zeros(1, np.float32), np.zeros(1, np.float32),
                               np.array([2.0], np.float32), lr=0.5, beta1=0.5, beta2=0.75, eps=2.0, t=1)
    assert M1[0] == 1.0 and V1[0] == 1.0 and W1[0] == 0.75
    # second update with the same gradient: m = 1.5, v = 1.75, c1 = 1/(1-0.25) = 4/3, c2 = 1/(1-0.5625) = 16/7
    W2, M2, V2 = O.adam_update(W1, M1, V1, np.array([2.0], np.float32), lr=0.5, beta1=0.5, beta2=0.75, eps=2.0, t=2)
    assert M2[0] == 1.5 and V2[0] == 1.75
    want = 0.75 - 0.5 * (1.5 * (4.0 / 3.0)) / (np.sqrt(1.75 * 16.0 / 7.0) + 2.0)      # = 0.75 - 0.5*2/4
    assert abs(W2[0] - want) < 1e-6 and abs(want - 0.5) < 1e-12


def test_adam_constant_gradient_and_sign_invariance():
    # constant gradient: bias-corrected moments equal g and g^2 at every step, so W moves by lr*g/(|g|+eps) per step
    g = np.array([0.3, -0.02, 5.0], np.float32)
    W, M, V = np.zeros(3, np.float32), np.zeros(3, np.float32), np.zeros(3, np.float32)
    for t in range(1, 41):
        W, M, V = O.adam_update(W, M, V, g, lr=0.01, beta1=0.9, beta2=0.999, eps=1e-8, t=t)
        assert np.allclose(W, -0.01 * t * np.sign(g), rtol=2e-5, atol=0.0), (t, W)
    # the step does not depend on the gradient's scale (up to eps), unlike SGD's
    Wa = O.adam_update(np.zeros(1, np.float32), np.zeros(1, np.float32), np.zeros(1, np.float32), np.array([1e-3], np.float32),
                       0.1, 0.9, 0.999, 1e-12, 1)[0]
    Wb = O.adam_update(np.zeros(1, np.float32), np.zeros(1, np.float32), np.zeros(1, np.float32), np.array([1e+3], np.float32),
                       0.1, 0.9, 0.999, 1e-12, 1)[0]
    assert np.allclose(Wa, Wb, rtol=1e-6) and np.allclose(Wa, -0.1, rtol=1e-6)


def test_layer_update_with_adam_carries_both_buffers():
    from paper_2506_22771_b200 import synth
    w = synth.scaled(synth.workload("tiny_mlp"), B=8, width_div=8)
    l = w.layers[0]
    spec = O.LayerSpec(l.kind, l.K, l.N, l.theta, 0.001, l.tau, seed=3, momentum=0.9, optimizer=1, beta2=0.99, adam_eps=1e-6)
    W0 = synth.make_weights(w, 3)[0]
    X = synth.make_batch(w, 3)
    a = O.train_step([spec], [W0], X, w.B, 0.0, 0)[0]
    nz = a.dW != 0
    g64 = a.dW[nz].astype(np.float64)                                                  # first step: lr * g / (|g| + eps)
    assert np.allclose((W0 - a.W_new)[nz], 0.001 * g64 / (np.abs(g64) + 1e-6), rtol=1e-3, atol=1e-9)
    b = O.train_step([spec], [a.W_new], X, w.B, 0.0, 1, Ms=[a.M_new], Vs=[a.V_new])[0]
    Wn, Mn, Vn = O.adam_update(a.W_new, a.M_new, a.V_new, b.dW, 0.001, 0.9, 0.99, 1e-6, 2)
    assert np.array_equal(b.W_new, Wn) and np.array_equal(b.M_new, Mn) and np.array_equal(b.V_new, Vn)


# ---- 2x2 max pooling between layers ----------------------------------------------------------------------
def test_maxpool2x2_hand_example_and_reshape_identity():
    x = np.arange(2 * 4 * 4 * 1, dtype=np.float32).reshape(2, 4, 4, 1)
    x[0, 1, 0, 0] = 99.0
    got = O.maxpool2x2(x)
    assert got.shape == (2, 2, 2, 1)
    assert got[0, :, :, 0].tolist() == [[99.0, 7.0], [13.0, 15.0]] and got[1, :, :, 0].tolist() == [[21.0, 23.0], [29.0, 31.0]]
    # against the reshape form of the same definition, with odd extents (the trailing row / column is dropped)
    g = np.random.default_rng(41)
    y = g.normal(size=(3, 7, 9, 5)).astype(np.float32)
    want = y[:, :6, :8, :].reshape(3, 3, 2, 4, 2, 5).max(axis=(2, 4))
    assert np.array_equal(O.maxpool2x2(y), want)
    # pooling commutes with a positive per-sample factor (so it can be taken before or after the normalisation)
    r = np.float32(0.37)
    assert np.array_equal(O.maxpool2x2(y * r), O.maxpool2x2(y) * r)


def test_pooled_layer_output_keeps_the_range_and_feeds_a_smaller_next_layer():
    from paper_2506_22771_b200 import synth
    H = Wd = 12
    specs = [O.LayerSpec(O.KIND_CONV3X3, 27, 8, float(8 * H * Wd), 0.01, float(np.sqrt(8 * H * Wd)), H=H, Wd=Wd, Cin=3, seed=2,
                         pool=2),
             O.LayerSpec(O.KIND_CONV3X3, 72, 4, float(4 * 36), 0.01, float(np.sqrt(4 * 36)), H=H // 2, Wd=Wd // 2, Cin=8, seed=2,
                         index=1)]
    w = synth.Workload("p", 3, [synth.LayerCfg(1, 27, 8, 1.0, 0.01, 1.0, H=H, Wd=Wd, Cin=3),
                                synth.LayerCfg(1, 72, 4, 1.0, 0.01, 1.0, H=H // 2, Wd=Wd // 2, Cin=8)], (H, Wd, 3), "normal",
                       "kaiming_uniform", 1)
    Ws = synth.make_weights(w, 2)
    X = synth.make_batch(w, 2)
    st = O.train_step(specs, Ws, X, w.B, 0.5, 0)
    full = O.length_normalise(st[0].Y, st[0].G, specs[0].tau, specs[0].eps)
    assert st[0].Xnext.shape == (6, 6, 6, 8) and np.array_equal(st[0].Xnext, O.maxpool2x2(full))
    # the maximum survives max pooling (outputs are >= 0), so the next layer's quantiser range is the unpooled one
    assert st[1].a_x == (O.absmax(full[:3]), O.absmax(full[3:]))
    assert st[1].Y.shape == (6, 6, 6, 4) and st[1].W_new.shape == (4, 72)
