"""Data-parallel train step on the GPU: the batch split by rows over several shards, each with its
own context, buffers and weight replica, must reproduce the whole-batch step of the oracle bit for
bit (per-sample tensors on the shard's rows; ranges, weight-gradient sums and new weights on every
shard).  The shards are driven phase by phase from one process on one device, one after the other
(no kernel of one shard waits for another's), and the arrays the library asks to be combined are
combined with plain tensor maxima / sums standing in for the all-reduce."""
import numpy as np
import pytest

from oracle import ffint8_oracle as O
from paper_2506_22771_b200 import binding as ffb
from paper_2506_22771_b200 import data_parallel as dp
from paper_2506_22771_b200 import synth
from tests.ffharness import GpuNet, compare_layer, shard_state, specs_and_descs

pytestmark = pytest.mark.gpu


class Shard:
    def __init__(self, descs, Ws, B_total, world, rank, path):
        import torch
        self.off, self.B = dp.shard_rows(B_total, world, rank)
        self.net = GpuNet(descs, self.B, Ws, dumps=True, xnext=True, chain=True, gemm_path=path)
        self.table = dp.PointerTable()
        self.table.add_layer_buffers(self.net.bufs)
        self.torch = torch


def _combine(shards, entries_per_shard):
    """Stand-in for the all-reduce: entry i of every shard is replaced by the max / sum over the shards."""
    import torch
    n = len(entries_per_shard[0])
    assert all(len(e) == n for e in entries_per_shard)
    for i in range(n):
        views = [sh.table.view(*ent[i][:3]) for sh, ent in zip(shards, entries_per_shard)]
        kinds = {ent[i][1:] for ent in entries_per_shard}
        assert len(kinds) == 1, kinds            # same count, type and operation on every shard
        stack = torch.stack(views)
        total = stack.max(0).values if entries_per_shard[0][i][3] == ffb.FF_DP_MAX else stack.sum(0)
        if entries_per_shard[0][i][3] == ffb.FF_DP_SUM and stack.dtype == torch.int32:
            assert torch.equal(total.to(torch.int64), stack.to(torch.int64).sum(0))   # no INT32 wrap
        for v in views:
            v.copy_(total)


def _run_dp(w, seed, steps, lam_per_step, world, path, rounding=(1, 0, 1), defer=False):
    """defer: an array is combined only right before the phase that needs it (the latest moment the overlapped
    reducer allows), instead of right behind the phase that listed it."""
    specs, descs = specs_and_descs(w.layers, seed, *rounding)
    Ws = synth.make_weights(w, seed)
    X = synth.make_batch(w, seed)
    shards = [Shard(descs, Ws, w.B, world, r, path) for r in range(world)]
    n = len(descs)
    for sh in shards:
        sh.net.set_input(dp.shard_batch(np.ascontiguousarray(X).reshape(2 * w.B, -1), w.B, sh.off, sh.B))
    Ms = Vs = None
    for step in range(steps):
        lam = lam_per_step * step
        assert ffb.ff_dp_phase_count(n) == 3 * n + 2
        waiting = {}                                  # phase that needs them -> per-shard entry lists
        for phase in range(ffb.ff_dp_phase_count(n)):
            for ents in waiting.pop(phase, []):
                _combine(shards, ents)
            entries = [ffb.ff_dp_train_phase(sh.net.ctx.ctx, sh.net.descs_arr, sh.net.bufs_arr, n, sh.B, w.B, sh.off,
                                             phase, lam, step, 0) for sh in shards]
            assert all(e[4] > phase for ent in entries for e in ent)
            if n + 2 <= phase < 2 * n + 2:            # the INT32 sums of layer l are read by that layer's update phase
                assert [e[4] for e in entries[0]] == [2 * n + 2 + (phase - n - 2)]
            if not defer:
                _combine(shards, entries)
                continue
            for need in sorted({e[4] for e in entries[0]}):
                waiting.setdefault(need, []).append([[e for e in ent if e[4] == need] for ent in entries])
        assert not waiting
        for sh in shards:
            ffb.ff_poll_status(sh.net.ctx.ctx, 0)
        states = O.train_step(specs, Ws, X, w.B, lam, step, Ms, Vs)
        for r, sh in enumerate(shards):
            for l, (st, b, sp) in enumerate(zip(states, sh.net.bufs, specs)):
                compare_layer(shard_state(st, w.B, sh.off, sh.B), b, sp, sh.B, tag=f"step{step}/shard{r}/layer{l}/")
        Ws = [st.W_new for st in states]
        Ms = [st.M_new for st in states]
        Vs = [st.V_new for st in states]
    for sh in shards:
        sh.net.close()


PATHS = [(ffb.FF_GEMM_SIMT, 0), (ffb.FF_GEMM_AUTO, 0)]


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("world", [2, 3])
def test_dp_dense_lookahead_equals_whole_batch(path, world):
    # 4 dense layers with the look-ahead loss; 200 rows per set do not divide evenly over 3 shards
    w = synth.scaled(synth.workload("mlp_lookahead"), B=200, width_div=8)
    _run_dp(w, seed=41, steps=3, lam_per_step=0.25, world=world, path=path)


@pytest.mark.parametrize("rounding", [(0, 0, 0), (1, 1, 1)])
def test_dp_rounding_modes(rounding):
    w = synth.scaled(synth.workload("tiny_mlp"), B=30, width_div=4)
    _run_dp(w, seed=6, steps=2, lam_per_step=0.0, world=4, path=(ffb.FF_GEMM_AUTO, 0), rounding=rounding)


@pytest.mark.parametrize("path", PATHS)
def test_dp_cnn_equals_whole_batch(path):
    w = synth.scaled(synth.workload("cnn"), B=4, width_div=4)
    _run_dp(w, seed=23, steps=2, lam_per_step=0.0, world=2, path=path)


def test_dp_tensor_core_conv_and_odd_sizes():
    # 64 -> 128 channel convolution (implicit-GEMM tensor-core route with split slabs), 3 shards of 1 sample
    layers = [synth.LayerCfg(1, 9 * 64, 128, float(128 * 16 * 16) / 2, 0.03 / 1024, float(np.sqrt(128 * 16 * 16)), H=16, Wd=16,
                             Cin=64)]
    w = synth.Workload("conv_dp", 3, layers, (16, 16, 64), "normal", "kaiming_uniform", 2)
    _run_dp(w, seed=5, steps=2, lam_per_step=0.0, world=3, path=(ffb.FF_GEMM_AUTO, 0))
    # odd feature counts: the element-pair hashing must line up with the unsplit tensor at odd row offsets
    layers = [synth.LayerCfg(0, 13, 7, 7.0, 0.03, float(np.sqrt(7))), synth.LayerCfg(0, 7, 5, 5.0, 0.03, float(np.sqrt(5)))]
    w = synth.Workload("odd_dp", 5, layers, (13,), "normal", "kaiming_uniform", 2)
    _run_dp(w, seed=9, steps=2, lam_per_step=0.5, world=5, path=(ffb.FF_GEMM_AUTO, 0))


def test_dp_wide_layers_take_the_flat_update():
    # 784 x 500 weights: large enough for the 128-bit update kernel and for CTA pairs in the unsplit contraction
    w = synth.scaled(synth.workload("mlp_lookahead"), B=160, width_div=4)
    _run_dp(w, seed=13, steps=2, lam_per_step=0.5, world=2, path=(ffb.FF_GEMM_AUTO, 0))
    _run_dp(w, seed=13, steps=1, lam_per_step=0.5, world=2, path=(ffb.FF_GEMM_AUTO, 1))


def test_dp_with_momentum():
    w = synth.scaled(synth.workload("mlp_lookahead"), B=90, width_div=8)
    for l in w.layers:
        l.momentum = 0.9
    _run_dp(w, seed=14, steps=3, lam_per_step=0.5, world=3, path=(ffb.FF_GEMM_AUTO, 0))


def test_dp_with_adam():
    w = synth.scaled(synth.workload("mlp_lookahead"), B=90, width_div=8)
    for l in w.layers:
        l.optimizer, l.momentum, l.beta2, l.adam_eps, l.lr = 1, 0.9, 0.99, 1e-6, 1e-3
    _run_dp(w, seed=15, steps=3, lam_per_step=0.5, world=3, path=(ffb.FF_GEMM_AUTO, 0))


def test_dp_deferred_reductions_equal_whole_batch():
    # every reduction done at the last moment its needed_by_phase allows: the weight-gradient sums of layer l are
    # combined after the contractions of all later layers have run, as with a reduction overlapped on a side stream
    w = synth.scaled(synth.workload("mlp_lookahead"), B=120, width_div=8)
    _run_dp(w, seed=44, steps=2, lam_per_step=0.25, world=3, path=(ffb.FF_GEMM_AUTO, 0), defer=True)
    w = synth.scaled(synth.workload("cnn"), B=4, width_div=4)
    _run_dp(w, seed=45, steps=2, lam_per_step=0.0, world=2, path=(ffb.FF_GEMM_AUTO, 0), defer=True)


def test_dp_single_shard_equals_train_step():
    # world = 1: the phase sequence with nothing to combine is the ordinary step
    w = synth.scaled(synth.workload("mlp_lookahead"), B=64, width_div=8)
    _run_dp(w, seed=2, steps=2, lam_per_step=0.5, world=1, path=(ffb.FF_GEMM_AUTO, 0))


def test_dp_argument_errors():
    w = synth.scaled(synth.workload("tiny_mlp"), B=8, width_div=4)
    specs, descs = specs_and_descs(w.layers, 1)
    net = GpuNet(descs, 8, synth.make_weights(w, 1), dumps=False)        # no accW_dump
    with pytest.raises(ffb.FFError):
        ffb.ff_dp_train_phase(net.ctx.ctx, net.descs_arr, net.bufs_arr, len(descs), 8, 16, 0, 0, 0.0, 0, 0)
    net.close()
    net = GpuNet(descs, 8, synth.make_weights(w, 1), dumps=True)
    for bad in [dict(B_total=4), dict(row_offset=9), dict(phase=99), dict(phase=-1)]:
        a = dict(B_total=16, row_offset=8, phase=0)
        a.update(bad)
        with pytest.raises(ffb.FFError):
            ffb.ff_dp_train_phase(net.ctx.ctx, net.descs_arr, net.bufs_arr, len(descs), 8, a["B_total"], a["row_offset"],
                                  a["phase"], 0.0, 0, 0)
    net.close()
