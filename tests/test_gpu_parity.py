"""GPU parity tests: the CUDA path (through the C ABI) against the CPU oracle, element by element.
Bit-exact for INT8 / INT32 / index work and, by the arithmetic contract, for every FP32 state
tensor too (tighter than a 1e-5 relative tolerance would be); the loss scalar
is compared at 1e-5 relative."""
import numpy as np
import pytest

from oracle import ffint8_oracle as O
from paper_2506_22771_b200 import binding as ffb
from paper_2506_22771_b200 import synth
from tests.ffharness import GpuNet, compare_layer, specs_and_descs

pytestmark = pytest.mark.gpu

# (contraction path, CTAs per tensor-core tile: 0 = by problem size, 1 = single CTA, 2 = CTA pair)
PATHS = [(ffb.FF_GEMM_SIMT, 0), (ffb.FF_GEMM_AUTO, 1), (ffb.FF_GEMM_AUTO, 2)]
TENSOR_FORMS = [1, 2]


def _gemm_case(M, N, K, trans, path, form=0):
    import torch
    g = np.random.default_rng(M * 7 + N * 3 + K + trans)
    ctx = ffb.Context([ffb.ff_layer_desc(0, 16, 16, 1, 1, 0, 0, 0, 0, 0, 1.0, 0.1, 1.0, 1e-8, 0)], 1, 0)
    ffb.ff_set_gemm_path(ctx.ctx, path)
    ffb.ff_set_tensor_form(ctx.ctx, form)
    if not trans:
        a = g.integers(-127, 128, size=(M, K)).astype(np.int8)
        b = g.integers(-127, 128, size=(N, K)).astype(np.int8)
        want = (a.astype(np.float64) @ b.astype(np.float64).T).astype(np.int64)
    else:
        a = g.integers(-127, 128, size=(K, M)).astype(np.int8)
        b = g.integers(-127, 128, size=(K, N)).astype(np.int8)
        want = (a.astype(np.float64).T @ b.astype(np.float64)).astype(np.int64)
    ta, tb = torch.from_numpy(a).cuda(), torch.from_numpy(b).cuda()
    tc = torch.full((M, N), -7, dtype=torch.int32, device="cuda")
    ffb.ff_int8_gemm(ctx.ctx, ta.data_ptr(), tb.data_ptr(), tc.data_ptr(), M, N, K, trans, 0)
    ffb.ff_poll_status(ctx.ctx, 0)
    got = tc.cpu().numpy()
    ctx.close()
    assert np.array_equal(got, want), (np.argwhere(got != want)[:5], got[got != want][:5], want[got != want][:5])


@pytest.mark.parametrize("M,N,K", [(3, 5, 33), (64, 64, 32), (130, 70, 100), (1, 500, 784)])
@pytest.mark.parametrize("trans", [0, 1])
def test_int8_gemm_simt(M, N, K, trans):
    _gemm_case(M, N, K, trans, ffb.FF_GEMM_SIMT)


@pytest.mark.parametrize("M,N,K", [(128, 256, 128), (128, 256, 512), (256, 512, 1024), (200, 300, 784),
                                   (1000, 2000, 2000), (16, 16, 16), (4096, 2048, 4096),
                                   # one tile column and more tiles than CTA groups: B stays resident in shared memory
                                   (40000, 128, 576), (20000, 96, 1104), (39000, 256, 640),
                                   # tile widths of 224 and 192 columns (the width that fills the last wave best)
                                   (8192, 2000, 256), (4096, 1100, 256)])
@pytest.mark.parametrize("form", TENSOR_FORMS)
def test_int8_gemm_tensor_forward_orientation(M, N, K, form):
    _gemm_case(M, N, K, 0, ffb.FF_GEMM_TENSOR, form)


@pytest.mark.parametrize("M,N,K", [(128, 256, 128), (128, 256, 512), (256, 512, 1000), (208, 304, 77),
                                   (2000, 784, 1024), (16, 16, 3), (2048, 4096, 4096)])
@pytest.mark.parametrize("form", TENSOR_FORMS)
def test_int8_gemm_tensor_weight_gradient_orientation(M, N, K, form):
    _gemm_case(M, N, K, 1, ffb.FF_GEMM_TENSOR, form)


def _run_and_compare(w, seed, steps, lam_per_step, path, rounding=(1, 0, 1), chain=True, check_every=1, graph=False,
                     pad_rows=True, pad_fill=None):
    specs, descs = specs_and_descs(w.layers, seed, *rounding)
    Ws = synth.make_weights(w, seed)
    X = synth.make_batch(w, seed)
    net = GpuNet(descs, w.B, Ws, dumps=True, xnext=True, chain=chain, gemm_path=path, graph=graph, pad_rows=pad_rows,
                 skips=[s.skip_from for s in specs])
    if pad_fill is not None:      # whatever the padding bytes of the pitched rows hold must reach no result
        for b in net.bufs:
            b._Xq_store.fill_(pad_fill)
            b._dHq_store.fill_(pad_fill)
    net.set_input(X)
    Ms = Vs = None
    for step in range(steps):
        lam = lam_per_step * step
        net.train_step(lam, step)
        states = O.train_step(specs, Ws, X, w.B, lam, step, Ms, Vs)
        if step % check_every == 0 or step == steps - 1:
            for l, (st, b, sp) in enumerate(zip(states, net.bufs, specs)):
                compare_layer(st, b, sp, w.B, tag=f"step{step}/layer{l}/")
        Ws = [st.W_new for st in states]
        Ms = [st.M_new for st in states]
        Vs = [st.V_new for st in states]
    if pad_fill is not None:
        for b, d in zip(net.bufs, descs):
            kin = b.Xq.shape[-1]
            assert bool((b._Xq_store[:, kin:] == pad_fill).all()) and bool((b._dHq_store[:, d.N:] == pad_fill).all())
    net.close()


@pytest.mark.parametrize("path", PATHS)
def test_config1_tiny_mlp_ten_steps(path):
    _run_and_compare(synth.workload("tiny_mlp"), seed=11, steps=10, lam_per_step=0.0, path=path)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("rounding", [(0, 0, 0), (1, 1, 1)])
def test_rounding_modes(path, rounding):
    w = synth.scaled(synth.workload("tiny_mlp"), B=24, width_div=4)
    _run_and_compare(w, seed=5, steps=2, lam_per_step=0.0, path=path, rounding=rounding)


@pytest.mark.parametrize("path", PATHS)
def test_config3_lookahead_scaled(path):
    # 4-layer MLP with the look-ahead loss, lambda growing per step; widths cut to keep the oracle fast,
    # several 128x256 tiles plus ragged tails in M (2*200), N (496) and K (784, 496)
    w = synth.scaled(synth.workload("mlp_lookahead"), B=200, width_div=4)
    w.layers[0].N = w.layers[1].K = 496
    w.layers[0].tau = float(np.sqrt(496))
    w.layers[0].theta = 496.0
    _run_and_compare(w, seed=3, steps=3, lam_per_step=0.25, path=path)


@pytest.mark.parametrize("path", PATHS)
def test_config2_greedy_scaled(path):
    # greedy: each layer trained on the frozen forward of the earlier ones = separate single-layer steps
    w = synth.scaled(synth.workload("mlp_greedy"), B=96, width_div=8)
    specs, descs = specs_and_descs(w.layers, 9)
    Ws = synth.make_weights(w, 9)
    x = synth.make_batch(w, 9)
    for l in range(len(specs)):
        net = GpuNet([descs[l]], w.B, [Ws[l]], gemm_path=path)
        net.set_input(x)
        for step in range(2):
            net.train_step(0.0, step)
            st = O.train_step([specs[l]], [Ws[l]], x, w.B, 0.0, step)[0]
            compare_layer(st, net.bufs[0], specs[l], w.B, tag=f"layer{l}/step{step}/")
            Ws[l] = st.W_new
        st = O.layer_forward(specs[l], x, Ws[l], w.B, 99)
        x = st.Xnext
        net.close()


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("graph", [False, True])
def test_greedy_epoch_scaled_with_frozen_layers(path, graph):
    # configuration 2's schedule at reduced width: three batches per phase, phase l trains layer l through
    # ff_train_step_from on the chained INT8 forward of the layers the earlier phases trained; every tensor of the
    # trained layer and the forward tensors of the frozen ones are compared element by element at every step
    w = synth.scaled(synth.workload("mlp_greedy"), B=72, width_div=8)
    specs, descs = specs_and_descs(w.layers, 9)
    Ws = synth.make_weights(w, 9)
    nb = 3
    batches = [synth.make_batch(w, 9, batch_index=i) for i in range(nb)]
    net = GpuNet(descs, w.B, Ws, gemm_path=path, graph=graph)
    ctx = net.ctx.ctx
    frozen_W = {}

    def on_step(l, i, states):
        net.set_input(batches[i])
        ffb.ff_train_step_from(ctx, net.descs_arr, net.bufs_arr, l + 1, l, w.B, 0.0, l * nb + i, 0)
        ffb.ff_poll_status(ctx, 0)
        for j in range(l + 1):
            compare_layer(states[j], net.bufs[j], specs[j], w.B, tag=f"phase{l}/batch{i}/layer{j}/")
        for j in range(l):     # frozen layers keep the weights their own phase left
            assert bool((net.bufs[j].W == frozen_W[j]).all())
        if i == nb - 1:
            frozen_W[l] = net.bufs[l].W.clone()

    O.greedy_epoch(specs, Ws, batches, w.B, on_step)
    net.close()


def test_train_step_from_with_lookahead_over_the_trained_layers():
    # layers 0 frozen, layers 1..3 trained with lambda > 0: each trained layer looks ahead at the layers after it
    w = synth.scaled(synth.workload("mlp_lookahead"), B=40, width_div=8)
    specs, descs = specs_and_descs(w.layers, 6)
    Ws = synth.make_weights(w, 6)
    X = synth.make_batch(w, 6)
    net = GpuNet(descs, w.B, Ws)
    net.set_input(X)
    for step in range(2):
        ffb.ff_train_step_from(net.ctx.ctx, net.descs_arr, net.bufs_arr, len(descs), 1, w.B, 0.3, step, 0)
        ffb.ff_poll_status(net.ctx.ctx, 0)
        states = O.train_step(specs, Ws, X, w.B, 0.3, step, first_trained=1)
        for l, (st, b, sp) in enumerate(zip(states, net.bufs, specs)):
            compare_layer(st, b, sp, w.B, tag=f"step{step}/layer{l}/")
        Ws = [Ws[0]] + [st.W_new for st in states[1:]]
    with pytest.raises(ffb.FFError) as e:
        ffb.ff_train_step_from(net.ctx.ctx, net.descs_arr, net.bufs_arr, len(descs), len(descs), w.B, 0.0, 0, 0)
    assert e.value.code == ffb.FF_ERR_ARG
    net.close()


@pytest.mark.parametrize("path", PATHS)
def test_config4_cnn_scaled(path):
    w = synth.scaled(synth.workload("cnn"), B=2, width_div=4)      # 3 -> 16 -> 32 -> 64 channels, 32x32
    _run_and_compare(w, seed=21, steps=2, lam_per_step=0.0, path=path)


def _conv_workload(chans, H, Wd, B):
    layers = [synth.LayerCfg(1, 9 * ci, co, float(co * H * Wd) / 2, 0.03, float(np.sqrt(co * H * Wd)), H=H, Wd=Wd, Cin=ci)
              for ci, co in zip(chans[:-1], chans[1:])]
    return synth.Workload("conv_case", B, layers, (H, Wd, chans[0]), "normal", "kaiming_uniform", 2)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("chans,H,Wd,B", [((3, 64, 128, 64), 32, 32, 2),     # config 4's channel widths: 64- and 128-byte taps
                                          ((3, 64, 256, 128), 8, 16, 3),     # 8 image rows per 128-position block, odd batch
                                          ((3, 128, 80), 16, 64, 1)])        # ragged Cout, 2 rows per block
def test_conv_tensor_core_shapes(path, chans, H, Wd, B):
    _run_and_compare(_conv_workload(chans, H, Wd, B), seed=31, steps=2, lam_per_step=0.1, path=path)


@pytest.mark.parametrize("form", TENSOR_FORMS)
@pytest.mark.parametrize("cin,cout,hw,B", [(64, 128, 16, 80), (128, 128, 16, 80), (64, 64, 32, 24), (128, 256, 16, 80),
                                           (64, 512, 16, 40), (128, 288, 32, 20)])
def test_conv_layer_with_resident_weights(form, cin, cout, hw, B):
    # more tiles than CTA groups: the forward streams the input as boxes of (tile rows + 2) image rows that serve the
    # three vertical taps each (64- and 128-byte channel chunks; 32- and 16-pixel rows).  The narrow layers keep their
    # INT8 weights in shared memory; the wide ones (last three: one and two tile columns, ragged last column) load the
    # three weight boxes of a stage beside its input box
    layers = [synth.LayerCfg(1, 9 * cin, cout, float(cout * hw * hw) / 2, 0.03 / (hw * hw), float(np.sqrt(cout * hw * hw)), H=hw, Wd=hw,
                             Cin=cin)]
    w = synth.Workload("conv_res", B, layers, (hw, hw, cin), "normal", "kaiming_uniform", 2)
    _run_and_compare(w, seed=8, steps=2, lam_per_step=0.0, path=(ffb.FF_GEMM_TENSOR, form))


@pytest.mark.parametrize("form", TENSOR_FORMS)
@pytest.mark.parametrize("chans", [(64, 128), (128, 256)])
def test_conv_layer_forced_tensor_path(chans, form):
    # FF_GEMM_TENSOR fails instead of falling back, so this proves the tcgen05 implicit-GEMM kernels ran
    _run_and_compare(_conv_workload(chans, 32, 32, 2), seed=33, steps=2, lam_per_step=0.0, path=(ffb.FF_GEMM_TENSOR, form))


@pytest.mark.parametrize("path", PATHS)
def test_config5_roofline_scaled(path):
    w = synth.scaled(synth.workload("roofline"), B=256, width_div=8)   # 8192 -> 1024, theta = N/2
    w.layers[0].K = 1024
    w.in_shape = (1024,)
    _run_and_compare(w, seed=2, steps=2, lam_per_step=0.0, path=path)


def test_separate_calls_equal_train_step():
    w = synth.scaled(synth.workload("tiny_mlp"), B=40, width_div=2)
    w.layers = w.layers[:1]
    specs, descs = specs_and_descs(w.layers, 4)
    Ws = synth.make_weights(w, 4)
    X = synth.make_batch(w, 4)
    net = GpuNet(descs, w.B, Ws)
    net.set_input(X)
    ctx, d, b = net.ctx.ctx, descs[0], net.bufs[0].struct
    ffb.ff_layer_forward(ctx, d, b, w.B, 7, 0)
    ffb.ff_layer_loss_grad(ctx, d, b, w.B, [], [], 0.0, 7, 0)
    ffb.ff_layer_update(ctx, d, b, w.B, 7, 0)
    ffb.ff_poll_status(ctx, 0)
    st = O.train_step(specs, Ws, X, w.B, 0.0, 7)[0]
    compare_layer(st, net.bufs[0], specs[0], w.B)
    net.close()


def test_edge_cases_zero_input_and_nonfinite():
    import torch
    w = synth.scaled(synth.workload("tiny_mlp"), B=8, width_div=4)
    w.layers = w.layers[:1]
    specs, descs = specs_and_descs(w.layers, 1)
    Ws = synth.make_weights(w, 1)
    X = np.zeros((16, 784), dtype=np.float32)
    net = GpuNet(descs, w.B, Ws)
    net.set_input(X)
    net.train_step(0.0, 0)
    st = O.train_step(specs, Ws, X, w.B, 0.0, 0)[0]
    compare_layer(st, net.bufs[0], specs[0], w.B)
    assert not net.bufs[0].G.any() and torch.equal(net.bufs[0].W.cpu(), torch.from_numpy(Ws[0]))
    X[3, 5] = np.inf
    net.set_input(X)
    with pytest.raises(ffb.FFError) as e:
        net.train_step(0.0, 1)
    assert e.value.code == ffb.FF_ERR_NONFINITE
    net.close()


def test_host_side_argument_errors():
    w = synth.scaled(synth.workload("tiny_mlp"), B=8, width_div=4)
    specs, descs = specs_and_descs(w.layers[:1], 1)
    net = GpuNet(descs, w.B, synth.make_weights(w, 1)[:1])
    bad = ffb.ff_layer_desc.from_buffer_copy(descs[0])
    bad.eps = 0.0
    with pytest.raises(ffb.FFError) as e:
        ffb.ff_layer_forward(net.ctx.ctx, bad, net.bufs[0].struct, w.B, 0, 0)
    assert e.value.code == ffb.FF_ERR_ARG
    bad = ffb.ff_layer_desc.from_buffer_copy(descs[0])
    bad.K = 200000
    with pytest.raises(ffb.FFError) as e:
        ffb.ff_layer_forward(net.ctx.ctx, bad, net.bufs[0].struct, w.B, 0, 0)
    assert e.value.code == ffb.FF_ERR_RANGE
    bufs = ffb.ff_layer_bufs.from_buffer_copy(net.bufs[0].struct)
    bufs.Y = net.bufs[0].Y.data_ptr() + 4
    with pytest.raises(ffb.FFError) as e:
        ffb.ff_layer_forward(net.ctx.ctx, descs[0], bufs, w.B, 0, 0)
    assert e.value.code == ffb.FF_ERR_ALIGN
    net.close()


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("first_counted", [0, 1])
def test_predict_matches_oracle(path, first_counted):
    import torch
    n_classes, B = 10, 52                       # 520 candidate rows: several tiles and a ragged tail
    w = synth.scaled(synth.workload("mlp_lookahead"), B=n_classes * B // 2, width_div=4)
    w.layers = w.layers[:3]
    specs, descs = specs_and_descs(w.layers, 6)
    Ws = synth.make_weights(w, 6)
    Xc, _ = synth.make_candidates(w, 6, B, n_classes)
    net = GpuNet(descs, n_classes * B // 2, Ws, dumps=False, xnext=False, chain=True, gemm_path=path)
    net.set_input(Xc)
    scores = torch.zeros(n_classes * B, dtype=torch.float32, device="cuda")
    pred = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    ffb.ff_predict(net.ctx.ctx, net.descs_arr, net.bufs_arr, len(descs), B, n_classes, first_counted,
                   scores.data_ptr(), pred.data_ptr(), 3, 0)
    ffb.ff_poll_status(net.ctx.ctx, 0)
    want_pred, want_scores, states = O.predict(specs, Ws, Xc, B, n_classes, 3, first_counted)
    for l, st in enumerate(states):
        assert np.array_equal(net.bufs[l].G.cpu().numpy().view(np.uint32), st.G.view(np.uint32)), f"G of layer {l}"
        assert np.array_equal(net.bufs[l].Xq.cpu().numpy().reshape(-1), st.Xq.reshape(-1)), f"Xq of layer {l}"
    assert np.array_equal(scores.cpu().numpy().view(np.uint32), want_scores.reshape(-1).view(np.uint32))
    assert np.array_equal(pred.cpu().numpy(), want_pred)
    # weights untouched
    for b, W in zip(net.bufs, Ws):
        assert torch.equal(b.W.cpu(), torch.from_numpy(W))
    for l, st in enumerate(states):          # one range for both halves of the candidate rows
        am = net.bufs[l].absmax.cpu().numpy()
        assert am[0] == am[1] == np.float32(st.a_x[0]) == np.float32(st.a_x[1])
    with pytest.raises(ffb.FFError) as e:
        ffb.ff_predict(net.ctx.ctx, net.descs_arr, net.bufs_arr, len(descs), 1, 9, 0, scores.data_ptr(), pred.data_ptr(), 0, 0)
    assert e.value.code == ffb.FF_ERR_ARG         # 9 candidate rows cannot be split into two halves
    net.close()


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("B,K,N", [(1, 1, 1), (1, 16, 16), (3, 5, 7), (2, 33, 500), (129, 144, 272), (65, 784, 16)])
def test_edge_shapes_dense(path, B, K, N):
    # smallest and ragged shapes: one sample per set, single features, sizes that are no multiple of any tile
    layers = [synth.LayerCfg(0, K, N, float(N) / 2, 0.03, float(np.sqrt(N))),
              synth.LayerCfg(0, N, 24, 12.0, 0.03, float(np.sqrt(24)))]
    w = synth.Workload("edge", B, layers, (K,), "normal", "kaiming_uniform", 2)
    specs, descs = specs_and_descs(w.layers, 41)
    Ws = synth.make_weights(w, 41)
    g = np.random.default_rng(B * 1000 + K)
    X = g.normal(size=(2 * B, K))
    X = (X * np.sqrt(K) / (np.sqrt((X ** 2).sum(1, keepdims=True)) + 1e-8)).astype(np.float32)
    net = GpuNet(descs, B, Ws, gemm_path=path)
    net.set_input(X)
    for step in range(2):
        net.train_step(0.5, step)
        states = O.train_step(specs, Ws, X, B, 0.5, step)
        for l, (st, b, sp) in enumerate(zip(states, net.bufs, specs)):
            compare_layer(st, b, sp, B, tag=f"step{step}/layer{l}/")
        Ws = [st.W_new for st in states]
    net.close()


def test_dead_layer_and_vanishing_gradient():
    # all-negative weights on a non-negative input: every accumulator <= 0, so Y = 0, G = 0, dH = 0 and its
    # range is 0 (all-zero codes); the weights must come back unchanged and the next layer sees zeros
    import torch
    B, K, N = 40, 64, 48
    layers = [synth.LayerCfg(0, K, N, float(N), 0.03, float(np.sqrt(N))), synth.LayerCfg(0, N, 32, 32.0, 0.03, float(np.sqrt(32)))]
    w = synth.Workload("dead", B, layers, (K,), "uniform01", "kaiming_uniform", 1)
    specs, descs = specs_and_descs(w.layers, 2)
    Ws = synth.make_weights(w, 2)
    Ws[0] = -np.abs(Ws[0])
    X = np.abs(synth.make_batch(w, 2))
    net = GpuNet(descs, B, Ws)
    net.set_input(X)
    net.train_step(0.3, 0)
    states = O.train_step(specs, Ws, X, B, 0.3, 0)
    for l, (st, b, sp) in enumerate(zip(states, net.bufs, specs)):
        compare_layer(st, b, sp, B, tag=f"layer{l}/")
    assert not net.bufs[0].Y.any() and not net.bufs[0].G.any() and not net.bufs[0].dHq.any()
    assert torch.equal(net.bufs[0].W.cpu(), torch.from_numpy(Ws[0]))
    net.close()


def _mixed_conv_workload(kinds_chans, H, Wd, B):
    """kinds_chans: list of (kind, Cin, Cout[, stride]); kind 1 = 3x3, 2 = pointwise.  A stride-2 layer
    halves the image for the layers after it."""
    layers = []
    h, w_ = H, Wd
    for spec in kinds_chans:
        kind, ci, co = spec[:3]
        stride = spec[3] if len(spec) > 3 else 1
        K = 9 * ci if kind == 1 else ci
        ho, wo = ((h - 1) // stride + 1, (w_ - 1) // stride + 1) if kind == 1 else (h, w_)
        layers.append(synth.LayerCfg(kind, K, co, float(co * ho * wo) / 2, 0.03 / (ho * wo), float(np.sqrt(co * ho * wo)),
                                     H=h, Wd=w_, Cin=ci, stride=stride))
        h, w_ = ho, wo
    return synth.Workload("mixed_conv", B, layers, (H, Wd, kinds_chans[0][1]), "normal", "kaiming_uniform", 2)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("stack,H,Wd,B", [
    ([(1, 3, 64), (2, 64, 128), (1, 128, 64), (2, 64, 48)], 32, 32, 2),   # 3x3 and pointwise layers alternating
    ([(2, 16, 32), (2, 32, 20)], 8, 16, 3),                                # narrow pointwise layers, ragged Cout
    ([(2, 12, 10)], 4, 12, 5)])                                            # Cin not a multiple of 16: dp4a path
def test_pointwise_convolution_layers(path, stack, H, Wd, B):
    _run_and_compare(_mixed_conv_workload(stack, H, Wd, B), seed=51, steps=2, lam_per_step=0.2, path=path)


SMALL_CIN = [(ci, n) for ci in (1, 2, 3, 4) for n in (16, 32, 64, 128)]


@pytest.mark.parametrize("cin,n", SMALL_CIN)
def test_first_layer_kernels_every_width(cin, n):
    # 3x3 layers with at most four input channels take the direct dp4a kernels (forward and weight gradient) on the
    # default path: every (C_in, width) instantiation, 10 x 12 images (output rows that are not a multiple of four
    # positions only with stride 2 below), three images per set so that the last chunk of 256 positions is ragged,
    # then a second such layer is impossible (C_in > 4) so a pointwise layer closes the stack
    w = _mixed_conv_workload([(1, cin, n), (2, n, 16)], 10, 12, 3)
    _run_and_compare(w, seed=900 + 10 * cin + n, steps=2, lam_per_step=0.3, path=ffb.FF_GEMM_AUTO, rounding=(1, 1, 1))


@pytest.mark.parametrize("cin,n,H,Wd,stride,B", [(3, 64, 32, 32, 1, 5),     # whole chunks, several per block
                                                 (3, 32, 11, 13, 2, 4),    # 6 x 7 outputs: positions of a word in two rows
                                                 (1, 16, 28, 28, 2, 7),    # 14 x 14 outputs
                                                 (4, 128, 9, 10, 1, 2),    # one group of threads per block
                                                 (2, 64, 2, 10, 1, 1)])    # a single ragged chunk
def test_first_layer_kernels_geometries(cin, n, H, Wd, stride, B):
    w = _mixed_conv_workload([(1, cin, n, stride)], H, Wd, B)
    _run_and_compare(w, seed=950 + H, steps=3, lam_per_step=0.0, path=ffb.FF_GEMM_AUTO, graph=(stride == 2))


@pytest.mark.parametrize("optimizer,momentum", [(0, 0.9), (1, 0.9)])
def test_first_layer_weight_gradient_with_optimisers(optimizer, momentum):
    w = _mixed_conv_workload([(1, 3, 32), (1, 32, 32)], 16, 16, 3)
    for l in w.layers:
        l.momentum, l.optimizer = momentum, optimizer
        if optimizer:
            l.beta2, l.adam_eps, l.lr = 0.99, 1e-6, 1e-3
    _run_and_compare(w, seed=970 + optimizer, steps=3, lam_per_step=0.2, path=ffb.FF_GEMM_AUTO)


def _fuzz_cases(n, seed):
    g = np.random.default_rng(seed)
    out = []
    for i in range(n):
        n_layers = int(g.integers(1, 4))
        widths = [int(g.choice([16, 24, 48, 100, 128, 130, 256, 272, 500, 512]))] + \
                 [int(g.choice([8, 16, 33, 64, 96, 128, 144, 256, 300])) for _ in range(n_layers)]
        B = int(g.choice([1, 2, 7, 32, 64, 100, 128, 129, 200]))
        rounding = tuple(int(x) for x in g.integers(0, 2, size=3))
        lam = float(g.choice([0.0, 0.25, 1.0]))
        out.append((i, B, widths, rounding, lam))
    return out


@pytest.mark.parametrize("case", _fuzz_cases(24, 2024), ids=lambda c: f"fuzz{c[0]}")
def test_fuzz_dense_networks(case):
    """Seeded random layer stacks: widths on both sides of every tile and alignment boundary (so both the
    tensor-core and the dp4a kernels and their hand-overs between layers are hit), all rounding modes."""
    i, B, widths, rounding, lam = case
    layers = [synth.LayerCfg(0, K, N, float(N) / 2, 0.03, float(np.sqrt(N))) for K, N in zip(widths[:-1], widths[1:])]
    w = synth.Workload("fuzz", B, layers, (widths[0],), "uniform01", "kaiming_uniform", 1)
    path = PATHS[i % len(PATHS)]
    _run_and_compare(w, seed=100 + i, steps=2, lam_per_step=lam, path=path, rounding=rounding)


@pytest.mark.parametrize("case", list(range(8)), ids=lambda c: f"convfuzz{c}")
def test_fuzz_conv_networks(case):
    g = np.random.default_rng(500 + case)
    H, Wd = [(8, 16), (16, 16), (4, 32), (32, 32), (6, 12), (16, 64), (5, 10), (8, 128)][case]
    chans = [int(g.choice([3, 8, 16]))] + [int(g.choice([16, 48, 64, 128])) for _ in range(int(g.integers(1, 4)))]
    kinds = [1] + [int(g.choice([1, 2])) for _ in chans[2:]]
    stack = [(k, ci, co) for k, ci, co in zip(kinds, chans[:-1], chans[1:])]
    B = int(g.choice([1, 2, 3]))
    _run_and_compare(_mixed_conv_workload(stack, H, Wd, B), seed=600 + case, steps=2, lam_per_step=0.3,
                     path=PATHS[case % len(PATHS)])


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("stack,H,Wd,B", [
    ([(1, 3, 64, 2), (1, 64, 128, 2), (1, 128, 64, 1)], 32, 32, 2),   # 32x32 -> 16x16 -> 8x8: im2col route, then 64- and 128-byte taps
    ([(1, 64, 128, 2)], 64, 64, 1),                                    # one strided layer on the tensor cores, forced below
    ([(1, 16, 32, 2), (2, 32, 24)], 9, 11, 3),                         # odd extents (5x6 outputs): dp4a path, then pointwise
    ([(1, 3, 16, 1), (1, 16, 16, 2)], 16, 16, 2)])
def test_strided_convolution_layers(path, stack, H, Wd, B):
    _run_and_compare(_mixed_conv_workload(stack, H, Wd, B), seed=61, steps=2, lam_per_step=0.2, path=path)


@pytest.mark.parametrize("form", TENSOR_FORMS)
def test_strided_conv_forced_tensor_path(form):
    w = _mixed_conv_workload([(1, 64, 128, 2)], 64, 64, 1)
    _run_and_compare(w, seed=62, steps=2, lam_per_step=0.0, path=(ffb.FF_GEMM_TENSOR, form))


# ---- launch-sequence replay (CUDA graph) of the train step ---------------------------------------
# step 0 runs eagerly, step 1 is captured, steps 2.. are graph launches; the step counter (rounding
# keys) and lambda change every step and must reach the replayed kernels through device memory.
@pytest.mark.parametrize("path", PATHS)
def test_graph_replay_dense_lookahead(path):
    w = synth.scaled(synth.workload("mlp_lookahead"), B=72, width_div=8)
    _run_and_compare(w, seed=31, steps=6, lam_per_step=0.125, path=path, graph=True)


def test_graph_replay_tiny_mlp_all_stochastic():
    _run_and_compare(synth.workload("tiny_mlp"), seed=12, steps=8, lam_per_step=0.0, path=(ffb.FF_GEMM_AUTO, 0),
                     rounding=(1, 1, 1), graph=True)


@pytest.mark.parametrize("path", PATHS)
def test_graph_replay_cnn(path):
    w = synth.scaled(synth.workload("cnn"), B=2, width_div=4)
    _run_and_compare(w, seed=22, steps=4, lam_per_step=0.0, path=path, graph=True)


def test_graph_replay_counts_launches_and_yields_to_profiling():
    w = synth.scaled(synth.workload("mlp_lookahead"), B=40, width_div=8)
    specs, descs = specs_and_descs(w.layers, 4)
    Ws = synth.make_weights(w, 4)
    X = synth.make_batch(w, 4)
    net = GpuNet(descs, w.B, Ws, graph=True)
    net.set_input(X)
    counts = []
    for step in range(7):
        if step == 4:
            ffb.ff_profile_start(net.ctx.ctx)          # profiled steps run kernel by kernel
        before = ffb.ff_launch_count(net.ctx.ctx)
        net.train_step(0.5, step)
        counts.append(ffb.ff_launch_count(net.ctx.ctx) - before)
        if step == 4:
            timed = sum(v[1] for v in ffb.ff_profile_stop(net.ctx.ctx, 0).values())
            assert 0 < timed < counts[-1]               # the step-counter store is launched but not timed
        states = O.train_step(specs, Ws, X, w.B, 0.5, step)
        Ws = [st.W_new for st in states]
    assert len(set(counts)) == 1 and counts[0] > 0, counts   # a replay stands for the same launches
    # steps 0 (first sight) and 1 (capture + first replay) aside, every unprofiled step was a graph launch
    assert ffb.ff_graph_replay_count(net.ctx.ctx) == 5, ffb.ff_last_error(net.ctx.ctx)
    for l, (st, b, sp) in enumerate(zip(states, net.bufs, specs)):
        compare_layer(st, b, sp, w.B, tag=f"layer{l}/")
    # switching the mode off drops the graphs; the eager path continues the same trajectory
    ffb.ff_set_graph_mode(net.ctx.ctx, False)
    net.train_step(0.5, 7)
    states = O.train_step(specs, Ws, X, w.B, 0.5, 7)
    for l, (st, b, sp) in enumerate(zip(states, net.bufs, specs)):
        compare_layer(st, b, sp, w.B, tag=f"eager/layer{l}/")
    net.close()


def test_graph_replay_two_call_shapes_share_a_context():
    # two networks' worth of buffers driven through ONE context, alternating: each call shape gets its own graph
    import torch
    w = synth.scaled(synth.workload("tiny_mlp"), B=16, width_div=2)
    specs, descs = specs_and_descs(w.layers, 8)
    net = GpuNet(descs, w.B, synth.make_weights(w, 8), graph=True)
    other = [ffb.LayerBuffers(d, w.B, net.dev, dumps=True, xnext=True, own_x=(i == 0)) for i, d in enumerate(descs)]
    other_arr = (ffb.ff_layer_bufs * len(descs))(*[b.struct for b in other])
    Wa, Wb = synth.make_weights(w, 8), synth.make_weights(w, 9)
    Xa, Xb = synth.make_batch(w, 8), synth.make_batch(w, 9)
    for b, W in zip(other, Wb):
        b.W.copy_(torch.from_numpy(W))
    net.set_input(Xa)
    other[0].X.copy_(torch.from_numpy(np.ascontiguousarray(Xb)).reshape(other[0].X.shape))
    for step in range(5):
        net.train_step(0.0, step)
        ffb.ff_train_step(net.ctx.ctx, net.descs_arr, other_arr, len(descs), w.B, 0.0, step + 100, 0)
        ffb.ff_poll_status(net.ctx.ctx, 0)
        sa = O.train_step(specs, Wa, Xa, w.B, 0.0, step)
        sb = O.train_step(specs, Wb, Xb, w.B, 0.0, step + 100)
        for l in range(len(specs)):
            compare_layer(sa[l], net.bufs[l], specs[l], w.B, tag=f"a/step{step}/layer{l}/")
            compare_layer(sb[l], other[l], specs[l], w.B, tag=f"b/step{step}/layer{l}/")
        Wa = [st.W_new for st in sa]
        Wb = [st.W_new for st in sb]
    assert ffb.ff_graph_replay_count(net.ctx.ctx) == 8, ffb.ff_last_error(net.ctx.ctx)
    net.close()


# ---- heavy-ball variant of the update: every weight-gradient route carries the momentum buffer ----------
def _with_momentum(w, mu):
    for i, l in enumerate(w.layers):
        l.momentum = mu if i != 1 else 0.0        # one plain layer in between: its buffer must stay untouched / absent
    return w


@pytest.mark.parametrize("path", PATHS)
def test_momentum_dense_lookahead(path):
    w = _with_momentum(synth.scaled(synth.workload("mlp_lookahead"), B=136, width_div=8), 0.875)
    _run_and_compare(w, seed=17, steps=4, lam_per_step=0.25, path=path)
    _run_and_compare(w, seed=17, steps=4, lam_per_step=0.25, path=path, graph=True)


@pytest.mark.parametrize("path", PATHS)
def test_momentum_cnn_and_pointwise(path):
    w = _with_momentum(synth.scaled(synth.workload("cnn"), B=2, width_div=4), 0.5)     # im2col, dp4a / slab routes
    _run_and_compare(w, seed=27, steps=3, lam_per_step=0.0, path=path)
    layers = [synth.LayerCfg(1, 9 * 64, 128, float(128 * 16 * 16) / 2, 0.03 / 1024, float(np.sqrt(128 * 256)), H=16, Wd=16,
                             Cin=64, momentum=0.9),                                   # implicit-GEMM split slabs
              synth.LayerCfg(2, 128, 64, float(64 * 16 * 16) / 2, 0.03 / 256, float(np.sqrt(64 * 256)), H=16, Wd=16, Cin=128,
                             momentum=0.9)]
    w = synth.Workload("conv_mom", 2, layers, (16, 16, 64), "normal", "kaiming_uniform", 2)
    _run_and_compare(w, seed=28, steps=3, lam_per_step=0.0, path=path)


def test_momentum_wide_layer_and_argument_errors():
    # 784 x 1000 weights through the fused tensor-core update (pairs), ragged last column tile
    w = _with_momentum(synth.scaled(synth.workload("mlp_lookahead"), B=130, width_div=2), 0.75)
    w.layers = w.layers[:2]
    w.layers[1].momentum = 0.75
    _run_and_compare(w, seed=19, steps=3, lam_per_step=0.0, path=(ffb.FF_GEMM_AUTO, 0))
    specs, descs = specs_and_descs(w.layers, 1)
    net = GpuNet(descs, w.B, synth.make_weights(w, 1))
    net.bufs_arr[0].Mom = None
    with pytest.raises(ffb.FFError):
        net.train_step(0.0, 0)
    net.descs_arr[0].momentum = 1.5
    with pytest.raises(ffb.FFError):
        net.train_step(0.0, 0)
    net.close()


# ---- Adam variant of the update: sums accumulate in a plane, one update kernel applies the rule ----------
def _with_adam(w, lr, dumps_free_layer=None):
    for l in w.layers:
        l.optimizer, l.momentum, l.beta2, l.adam_eps, l.lr = 1, 0.9, 0.99, 1e-6, lr
    return w


@pytest.mark.parametrize("path", PATHS)
def test_adam_dense_lookahead(path):
    w = _with_adam(synth.scaled(synth.workload("mlp_lookahead"), B=136, width_div=8), 1e-3)
    w.layers[2].optimizer, w.layers[2].momentum = 0, 0.5              # a heavy-ball layer among the Adam ones
    _run_and_compare(w, seed=37, steps=4, lam_per_step=0.25, path=path)
    _run_and_compare(w, seed=37, steps=5, lam_per_step=0.25, path=path, graph=True)   # bias corrections follow the replayed step


@pytest.mark.parametrize("path", PATHS)
def test_adam_convolutions(path):
    w = _with_adam(synth.scaled(synth.workload("cnn"), B=2, width_div=4), 1e-3)         # im2col, dp4a / slab routes
    _run_and_compare(w, seed=38, steps=3, lam_per_step=0.0, path=path)
    layers = [synth.LayerCfg(1, 9 * 64, 128, float(128 * 256), 0.0, float(np.sqrt(128 * 256)), H=16, Wd=16, Cin=64),
              synth.LayerCfg(3, 9, 128, float(128 * 256), 0.0, float(np.sqrt(128 * 256)), H=16, Wd=16, Cin=128),
              synth.LayerCfg(2, 128, 64, float(64 * 256), 0.0, float(np.sqrt(64 * 256)), H=16, Wd=16, Cin=128)]
    w = _with_adam(synth.Workload("conv_adam", 2, layers, (16, 16, 64), "normal", "kaiming_uniform", 2), 1e-3)
    _run_and_compare(w, seed=39, steps=3, lam_per_step=0.5, path=path)


def test_adam_without_dump_buffers_uses_the_workspace():
    # no accW_dump: the sums plane sits at the tail of the workspace; wide first layer takes the 128-bit update kernel
    w = _with_adam(synth.scaled(synth.workload("mlp_lookahead"), B=130, width_div=4), 1e-3)
    w.layers = w.layers[:2]
    specs, descs = specs_and_descs(w.layers, 20)
    Ws = synth.make_weights(w, 20)
    X = synth.make_batch(w, 20)
    net = GpuNet(descs, w.B, Ws, dumps=False, xnext=False)
    net.set_input(X)
    Ms = Vs = None
    for step in range(3):
        net.train_step(0.0, step)
        states = O.train_step(specs, Ws, X, w.B, 0.0, step, Ms, Vs)
        Ws, Ms, Vs = [s.W_new for s in states], [s.M_new for s in states], [s.V_new for s in states]
    for st, b in zip(states, net.bufs):
        for name, got, want in [("W", b.W, st.W_new), ("M", b.Mom, st.M_new), ("V", b.Var, st.V_new)]:
            assert np.array_equal(got.cpu().numpy().view(np.uint32), want.view(np.uint32)), name
    net.bufs_arr[1].Var = None
    with pytest.raises(ffb.FFError):
        net.train_step(0.0, 3)
    net.close()


def test_predict_with_replayed_launches():
    # steps 2.. of a repeated classification call are graph launches; the rounding of the candidates follows the step
    import torch
    n_classes, B = 10, 20
    w = synth.scaled(synth.workload("mlp_lookahead"), B=n_classes * B // 2, width_div=8)
    w.layers = w.layers[:2]
    specs, descs = specs_and_descs(w.layers, 7)
    Ws = synth.make_weights(w, 7)
    Xc, _ = synth.make_candidates(w, 7, B, n_classes)
    net = GpuNet(descs, n_classes * B // 2, Ws, dumps=False, xnext=False, chain=True, graph=True)
    net.set_input(Xc)
    scores = torch.zeros(n_classes * B, dtype=torch.float32, device="cuda")
    pred = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    for step in range(5):
        ffb.ff_predict(net.ctx.ctx, net.descs_arr, net.bufs_arr, len(descs), B, n_classes, 0, scores.data_ptr(), pred.data_ptr(),
                       step, 0)
        ffb.ff_poll_status(net.ctx.ctx, 0)
        want_pred, want_scores, _ = O.predict(specs, Ws, Xc, B, n_classes, step, 0)
        assert np.array_equal(scores.cpu().numpy().view(np.uint32), want_scores.reshape(-1).view(np.uint32)), step
        assert np.array_equal(pred.cpu().numpy(), want_pred), step
    assert ffb.ff_graph_replay_count(net.ctx.ctx) == 4, ffb.ff_last_error(net.ctx.ctx)
    # a train step on the same buffers is a different call shape with a graph of its own
    for step in range(3):
        net.train_step(0.0, step)
    assert ffb.ff_graph_replay_count(net.ctx.ctx) == 6
    net.close()


def test_wide_outputs_many_samples_take_the_per_sample_tiles():
    # 2400 + 2400 samples of 4096 outputs: the output-gradient quantiser (and a normalisation, were there a next
    # layer) takes (sample, tile) pairs per block - more pairs than blocks here; both rounding modes of g^Y
    layers = [synth.LayerCfg(0, 64, 4096, 2048.0, 0.03, float(np.sqrt(4096)))]
    w = synth.Workload("wide_out", 2400, layers, (64,), "uniform01", "kaiming_uniform", 1)
    for rounding in [(1, 0, 1), (1, 0, 0)]:
        _run_and_compare(w, seed=66, steps=2, lam_per_step=0.0, path=(ffb.FF_GEMM_AUTO, 0), rounding=rounding)


def test_graph_cache_evicts_least_recently_used_shapes():
    # 20 call shapes (the same layer with 20 different step sizes) through one context that keeps 16 graphs:
    # every shape still computes the oracle's step, replays resume after a shape was dropped and re-captured
    w = synth.scaled(synth.workload("tiny_mlp"), B=16, width_div=4)
    w.layers = w.layers[:1]
    X = synth.make_batch(w, 3)
    W0 = synth.make_weights(w, 3)
    specs0, descs0 = specs_and_descs(w.layers, 3)
    net = GpuNet(descs0, w.B, W0, graph=True)
    net.set_input(X)
    import torch
    for rnd in range(2):
        for i in range(20):
            lr = 0.01 * (i + 1)
            w.layers[0].lr = lr
            specs, descs = specs_and_descs(w.layers, 3)
            net.descs_arr[0] = descs[0]
            for b, W in zip(net.bufs, W0):
                b.W.copy_(torch.from_numpy(W))
            Ws = W0
            for step in range(3):          # eager, capture, replay
                net.train_step(0.0, step)
                st = O.train_step(specs, Ws, X, w.B, 0.0, step)
                Ws = [s.W_new for s in st]
            compare_layer(st[0], net.bufs[0], specs[0], w.B, tag=f"round{rnd}/shape{i}/")
    # per shape and round: 2 replays (steps 1 and 2); every shape was evicted before its second round (20 > 16)
    assert ffb.ff_graph_replay_count(net.ctx.ctx) == 2 * 20 * 2, ffb.ff_last_error(net.ctx.ctx)
    net.close()


# ---- row pitches of the INT8 tensors -----------------------------------------------------------------------
@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("pad_rows", [False, True])
def test_unaligned_widths_with_and_without_padded_rows(path, pad_rows):
    # widths 784 / 496 / 500: padded to 896 / 512 / 512-byte rows by default, dense rows on request; all rounding stochastic
    w = synth.scaled(synth.workload("mlp_lookahead"), B=136, width_div=4)
    w.layers[0].N = w.layers[1].K = 496
    w.layers[0].tau, w.layers[0].theta = float(np.sqrt(496)), 496.0
    _run_and_compare(w, seed=77, steps=2, lam_per_step=0.5, path=path, rounding=(1, 1, 1), pad_rows=pad_rows)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("momentum", [0.0, 0.9])
def test_padding_bytes_reach_no_result(path, momentum):
    # same widths with the padding of every pitched row preset to a non-zero byte: the contractions may fetch it (their
    # copies span the pitch) but it meets zero-filled weight columns or discarded output rows / columns only
    w = synth.scaled(synth.workload("mlp_lookahead"), B=136, width_div=4)
    w.layers[0].N = w.layers[1].K = 496
    w.layers[0].tau, w.layers[0].theta = float(np.sqrt(496)), 496.0
    for l in w.layers:
        l.momentum = momentum
    _run_and_compare(w, seed=78, steps=2, lam_per_step=0.5, path=path, rounding=(1, 1, 1), pad_fill=-77)


@pytest.mark.parametrize("form", TENSOR_FORMS)
@pytest.mark.parametrize("momentum", [0.0, 0.9])
def test_update_epilogue_edges(form, momentum):
    # weight matrices whose edges cut through the update epilogue's 32 x 32 patches: 144 and 272 rows (warps with 16
    # valid rows and warps wholly outside the matrix), 784 and 272 columns (a last chunk of 16 columns), several
    # tiles per CTA on the first layer; plain SGD moves W as TMA patches, momentum takes the load / store form
    widths = [784, 272, 144, 48]
    layers = [synth.LayerCfg(0, K, N, float(N) / 2, 0.03, float(np.sqrt(N)), momentum=momentum)
              for K, N in zip(widths[:-1], widths[1:])]
    w = synth.Workload("edges", 200, layers, (widths[0],), "uniform01", "kaiming_uniform", 1)
    _run_and_compare(w, seed=91, steps=3, lam_per_step=0.25, path=(ffb.FF_GEMM_AUTO, form), rounding=(1, 0, 1))


def test_explicit_row_pitch_and_its_checks():
    import torch
    w = synth.scaled(synth.workload("tiny_mlp"), B=24, width_div=2)      # 784 -> 250 -> 250
    specs, descs = specs_and_descs(w.layers, 5)
    Ws = synth.make_weights(w, 5)
    X = synth.make_batch(w, 5)
    net = GpuNet(descs, w.B, Ws, pad_rows=False)
    # re-point layer 1 at buffers with pitches of its own choosing (the next multiples of 16 bytes and then some)
    K, N, rows = descs[1].K, descs[1].N, 2 * w.B
    ldx, ldd = (K + 31) // 16 * 16, (N + 63) // 16 * 16
    xq = torch.full((rows, ldx), 99, dtype=torch.int8, device="cuda")
    dh = torch.full((rows, ldd), 99, dtype=torch.int8, device="cuda")
    net.bufs_arr[1].Xq, net.bufs_arr[1].ld_xq = xq.data_ptr(), ldx
    net.bufs_arr[1].dHq, net.bufs_arr[1].ld_dhq = dh.data_ptr(), ldd
    net.set_input(X)
    net.train_step(0.0, 0)
    st = O.train_step(specs, Ws, X, w.B, 0.0, 0)
    assert np.array_equal(xq[:, :K].cpu().numpy(), st[1].Xq) and np.array_equal(dh[:, :N].cpu().numpy(), st[1].dHq)
    assert bool((xq[:, K:] == 99).all()) and bool((dh[:, N:] == 99).all())          # padding bytes are never written
    assert np.array_equal(net.bufs[1].W.cpu().numpy().view(np.uint32), st[1].W_new.view(np.uint32))
    for field, bad in [("ld_xq", K // 16 * 16 - 16), ("ld_xq", ldx + 8), ("ld_dhq", ldd + 3)]:
        old = getattr(net.bufs_arr[1], field)
        setattr(net.bufs_arr[1], field, bad)
        with pytest.raises(ffb.FFError):
            net.train_step(0.0, 1)
        setattr(net.bufs_arr[1], field, old)
    net.close()


def test_bounded_wait_runs_out_is_reported_and_leaves_the_context_usable():
    # the wait every role of the contraction kernels uses, run on a barrier nothing arrives on with a 1 ms limit:
    # the kernel returns, the status word says so, and the steps before and after are bit-exact as ever
    import time
    w = synth.scaled(synth.workload("tiny_mlp"), B=40, width_div=2)
    specs, descs = specs_and_descs(w.layers, 4)
    Ws = synth.make_weights(w, 4)
    X = synth.make_batch(w, 4)
    net = GpuNet(descs, w.B, Ws)
    net.set_input(X)
    ctx = net.ctx.ctx
    for step in range(2):
        if step == 1:
            t0 = time.time()
            ffb.ff_selftest_bounded_wait(ctx, 1_000_000, 0)
            with pytest.raises(ffb.FFError) as e:
                ffb.ff_poll_status(ctx, 0)
            assert e.value.code == ffb.FF_ERR_DEVICE_TIMEOUT and "wait" in str(e.value)
            assert time.time() - t0 < 5.0
            ffb.ff_poll_status(ctx, 0)            # reported once, then clear
        net.train_step(0.0, step)
        states = O.train_step(specs, Ws, X, w.B, 0.0, step)
        for l, (st, b, sp) in enumerate(zip(states, net.bufs, specs)):
            compare_layer(st, b, sp, w.B, tag=f"step{step}/layer{l}/")
        Ws = [st.W_new for st in states]
    with pytest.raises(ffb.FFError) as e:
        ffb.ff_selftest_bounded_wait(ctx, 0, 0)
    assert e.value.code == ffb.FF_ERR_ARG
    net.close()


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("graph", [False, True])
def test_residual_block_dense(path, graph):
    # a look-ahead block of three layers whose last one adds the block's input to its normalised output (the skip
    # path of a residual block), followed by a fourth layer that sees the sum; lambda > 0 so that the block's
    # layers look ahead at the layer behind the sum
    w = synth.scaled(synth.workload("mlp_lookahead"), B=72, width_div=8)
    w.layers[0].K = 256                              # the block maps 256 -> 250 -> 250 -> 256
    w.layers[2].N = w.layers[3].K = 256
    w.layers[2].theta, w.layers[2].tau = 256.0, 16.0
    w.layers[2].skip_from, w.layers[2].skip_scale = 0, 0.75
    w.in_shape = (256,)
    specs, descs = specs_and_descs(w.layers, 12)
    Ws = synth.make_weights(w, 12)
    X = synth.make_batch(w, 12)
    net = GpuNet(descs, w.B, Ws, gemm_path=path, graph=graph, skips=[s.skip_from for s in specs])
    net.set_input(X)
    for step in range(3):
        net.train_step(0.3, step)
        states = O.train_step(specs, Ws, X, w.B, 0.3, step)
        for l, (st, b, sp) in enumerate(zip(states, net.bufs, specs)):
            compare_layer(st, b, sp, w.B, tag=f"step{step}/layer{l}/")
        Ws = [st.W_new for st in states]
    net.close()


@pytest.mark.parametrize("path", PATHS)
def test_residual_block_convolutional_with_inner_skip_source(path):
    # conv stack 8 -> 16 -> 16 -> 16 on 12x12 images: layer 2 adds the input of layer 1 (= layer 0's normalised output)
    chans = [8, 16, 16, 16]
    hw = 12
    layers = [synth.LayerCfg(1, 9 * ci, co, float(co * hw * hw), 0.03 / (hw * hw), float(np.sqrt(co * hw * hw)), H=hw, Wd=hw, Cin=ci)
              for ci, co in zip(chans[:-1], chans[1:])]
    layers[2].skip_from = 1
    w = synth.Workload("res_conv", 3, layers, (hw, hw, chans[0]), "normal", "kaiming_uniform", 2)
    specs, descs = specs_and_descs(w.layers, 5)
    Ws = synth.make_weights(w, 5)
    X = synth.make_batch(w, 5)
    net = GpuNet(descs, w.B, Ws, gemm_path=path, skips=[s.skip_from for s in specs])
    net.set_input(X)
    for step in range(2):
        net.train_step(0.0, step)
        states = O.train_step(specs, Ws, X, w.B, 0.0, step)
        for l, (st, b, sp) in enumerate(zip(states, net.bufs, specs)):
            compare_layer(st, b, sp, w.B, tag=f"step{step}/layer{l}/")
        Ws = [st.W_new for st in states]
    net.close()


def test_skip_path_argument_errors():
    w = synth.scaled(synth.workload("tiny_mlp"), B=8, width_div=4)
    w.layers[0].K = w.layers[0].N
    specs, descs = specs_and_descs(w.layers, 1)
    net = GpuNet(descs, w.B, synth.make_weights(w, 1), xnext=False)
    net.bufs[0].struct.Skip = net.bufs[0].X.data_ptr()
    arr = (ffb.ff_layer_bufs * len(descs))(*[b.struct for b in net.bufs])
    with pytest.raises(ffb.FFError) as e:      # the sum has to be written somewhere
        ffb.ff_train_step(net.ctx.ctx, net.descs_arr, arr, len(descs), w.B, 0.0, 0, 0)
    assert e.value.code == ffb.FF_ERR_ARG
    net.close()
