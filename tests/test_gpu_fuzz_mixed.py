"""Seeded random parity sweep over everything a layer stack can combine: dense, 3x3 (stride 1 / 2),
pointwise and depthwise layers, pooling, skip paths of residual blocks, the three update rules, every rounding mode, look-ahead weights,
every contraction route, replayed launches and data-parallel shards - each case against the oracle, bit
for bit, for two or three steps."""
import numpy as np
import pytest

from paper_2506_22771_b200 import binding as ffb
from paper_2506_22771_b200 import synth
from tests.test_gpu_data_parallel import _run_dp
from tests.test_gpu_parity import _run_and_compare

pytestmark = pytest.mark.gpu

ROUTES = [(ffb.FF_GEMM_SIMT, 0), (ffb.FF_GEMM_AUTO, 1), (ffb.FF_GEMM_AUTO, 2), (ffb.FF_GEMM_AUTO, 0)]
RULES = [(0, 0.0, 0.999, 1e-8), (0, 0.5, 0.999, 1e-8), (0, 0.9, 0.999, 1e-8), (1, 0.9, 0.99, 1e-6)]
IMAGES = [(8, 16), (16, 16), (4, 32), (32, 32), (6, 12), (16, 64), (12, 10), (8, 128), (10, 10), (24, 24)]


def _rule(g):
    return dict(zip(("optimizer", "momentum", "beta2", "adam_eps"), RULES[int(g.integers(0, len(RULES)))]))


def _dense_case(g):
    n_layers = int(g.integers(1, 5))
    widths = [int(g.choice([10, 16, 24, 48, 100, 128, 130, 256, 272, 500, 512, 784]))] + \
             [int(g.choice([1, 8, 16, 33, 64, 96, 128, 144, 256, 300, 520])) for _ in range(n_layers)]
    B = int(g.choice([1, 2, 7, 32, 64, 100, 128, 129, 200, 300]))
    layers = []
    for K, N in zip(widths[:-1], widths[1:]):
        o = _rule(g)
        layers.append(synth.LayerCfg(0, K, N, float(N) / 2, 1e-3 if o["optimizer"] else 0.03, float(np.sqrt(N)), **o))
    return synth.Workload("mixed", B, layers, (widths[0],), "uniform01", "kaiming_uniform", 1)


def _spatial_case(g):
    H, Wd = IMAGES[int(g.integers(0, len(IMAGES)))]
    c = cin0 = int(g.choice([3, 4, 8, 16, 64]))
    layers, h, wd = [], H, Wd
    for _ in range(int(g.integers(1, 5))):
        kind = int(g.choice([1, 1, 2, 3]))
        stride = int(g.choice([1, 2])) if kind in (1, 3) and min(h, wd) >= 4 else 1
        co = c if kind == 3 else int(g.choice([6, 16, 48, 64, 128]))
        ho, wo = (h - 1) // stride + 1, (wd - 1) // stride + 1
        pool = 2 if (ho % 2 == 0 and wo % 2 == 0 and min(ho, wo) >= 4 and g.random() < 0.3) else 1
        o = _rule(g)
        layers.append(synth.LayerCfg(kind, {1: 9 * c, 2: c, 3: 9}[kind], co, float(co * ho * wo),
                                     1e-3 if o["optimizer"] else 0.03 / (ho * wo), float(np.sqrt(co * ho * wo)), H=h, Wd=wd, Cin=c,
                                     stride=stride, pool=pool, **o))
        c = co
        h, wd = (ho // 2, wo // 2) if pool == 2 else (ho, wo)
    return synth.Workload("mixed", int(g.choice([1, 2, 3, 5])), layers, (H, Wd, cin0), "normal", "kaiming_uniform", 1)


@pytest.mark.parametrize("case", list(range(64)))
def test_mixed_random_stack(case):
    g = np.random.default_rng(777000 + case)
    w = _dense_case(g) if g.random() < 0.45 else _spatial_case(g)
    rounding = tuple(int(x) for x in g.integers(0, 2, size=3))
    lam = float(g.choice([0.0, 0.25, 1.0]))
    route = ROUTES[int(g.integers(0, len(ROUTES)))]
    mode = int(g.integers(0, 4))          # 0, 2: plain; 1: replayed launches; 3: two data-parallel shards
    if mode == 3 and w.B >= 2:
        _run_dp(w, seed=case + 1, steps=2, lam_per_step=lam, world=2, path=route, rounding=rounding)
    else:
        _run_and_compare(w, seed=case + 1, steps=3 if mode == 1 else 2, lam_per_step=lam, path=route, rounding=rounding,
                         graph=(mode == 1))


def _residual_case(g):
    """A stack that contains one residual block: layers first..last with the input of `first` added to the
    normalised output of `last` (so `last` maps back to the width / shape of the block's input)."""
    if g.random() < 0.5:
        n = int(g.integers(2, 6))
        widths = [int(g.choice([16, 33, 64, 100, 128, 144, 256, 300])) for _ in range(n + 1)]
        first = int(g.integers(0, n - 1))
        last = int(g.integers(first, n))
        widths[last + 1] = widths[first]
        layers = []
        for K, N in zip(widths[:-1], widths[1:]):
            o = _rule(g)
            layers.append(synth.LayerCfg(0, K, N, float(N) / 2, 1e-3 if o["optimizer"] else 0.03, float(np.sqrt(N)), **o))
        w = synth.Workload("res", int(g.choice([1, 7, 64, 129, 200])), layers, (widths[0],), "uniform01", "kaiming_uniform", 1)
    else:
        H, Wd = IMAGES[int(g.integers(0, len(IMAGES)))]
        c = int(g.choice([4, 8, 16, 64]))
        n = int(g.integers(2, 5))
        first = int(g.integers(0, n - 1))
        last = int(g.integers(first, n))
        layers, cin = [], c
        for l in range(n):
            kind = int(g.choice([1, 2, 3]))
            co = cin if (kind == 3 or l == last) else int(g.choice([8, 16, 64]))
            block_in = c if first == 0 else (layers[first].Cin if first < len(layers) else cin)
            if l == last and kind == 3 and cin != block_in:
                kind = 2
            o = _rule(g)
            layers.append(synth.LayerCfg(kind, {1: 9 * cin, 2: cin, 3: 9}[kind], co, float(co * H * Wd),
                                         1e-3 if o["optimizer"] else 0.03 / (H * Wd), float(np.sqrt(co * H * Wd)), H=H, Wd=Wd,
                                         Cin=cin, **o))
            cin = co
        # the block's last layer returns to the channel count of the block's input
        want = c if first == 0 else layers[first].Cin
        ll = layers[last]
        if ll.N != want:
            if ll.kind == 3:
                ll.kind, ll.K = 2, ll.Cin
            ll.N, ll.theta, ll.tau = want, float(want * H * Wd), float(np.sqrt(want * H * Wd))
            if last + 1 < n:
                nx = layers[last + 1]
                nx.Cin = want
                if nx.kind == 3:
                    nx.N, nx.theta, nx.tau = want, float(want * H * Wd), float(np.sqrt(want * H * Wd))
                    for l in range(last + 2, n):      # keep the chain consistent behind a depthwise layer
                        layers[l].Cin = layers[l - 1].N
                        layers[l].K = {1: 9 * layers[l].Cin, 2: layers[l].Cin, 3: 9}[layers[l].kind]
                        if layers[l].kind == 3:
                            layers[l].N = layers[l].Cin
                            layers[l].theta, layers[l].tau = float(layers[l].N * H * Wd), float(np.sqrt(layers[l].N * H * Wd))
                nx.K = {1: 9 * nx.Cin, 2: nx.Cin, 3: 9}[nx.kind]
        w = synth.Workload("res", int(g.choice([1, 2, 3])), layers, (H, Wd, c), "normal", "kaiming_uniform", 1)
    w.layers[last].skip_from = first
    w.layers[last].skip_scale = float(g.choice([1.0, 0.5, -0.75]))
    return w


@pytest.mark.parametrize("case", list(range(24)))
def test_mixed_random_residual_stack(case):
    g = np.random.default_rng(888000 + case)
    w = _residual_case(g)
    rounding = tuple(int(x) for x in g.integers(0, 2, size=3))
    lam = float(g.choice([0.0, 0.25, 1.0]))
    route = ROUTES[int(g.integers(0, len(ROUTES)))]
    graph = bool(g.integers(0, 2))
    _run_and_compare(w, seed=case + 1, steps=3 if graph else 2, lam_per_step=lam, path=route, rounding=rounding, graph=graph)
