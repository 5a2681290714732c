"""Full-size parity: the CUDA path at the full sizes of the five benchmark configurations, in the launch configuration
bench.py times (no parity dumps, no FP32 copy of the normalised output, layers chained on device),
against SHA-256 digests of the CPU oracle's tensors (tests/golden/fullsize_digests.json, written by
tests/golden/make_fullsize_digests.py from oracle/ alone).  Every INT8 tensor, accumulator statistic
and FP32 tensor is compared bit for bit through its digest; the loss scalar at 1e-5 relative."""
import ctypes as C
import hashlib
import json
import os

import numpy as np
import pytest

from paper_2506_22771_b200 import binding as ffb
from paper_2506_22771_b200 import synth
from tests.ffharness import GpuNet, REL_TOL

pytestmark = pytest.mark.gpu

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "fullsize_digests.json")
DIG = json.load(open(GOLDEN)) if os.path.exists(GOLDEN) else {}
TENSORS = ["Xq", "Wq", "Y", "S", "rowmax", "G", "coef", "dHq"]


def _sha(t):
    return hashlib.sha256(t.detach().cpu().contiguous().numpy().tobytes()).hexdigest()


def _check_layer(b, want, tag):
    am = b.absmax.detach().cpu().numpy()
    got_am = [float(np.float32(v)).hex() for v in am[:5]]
    assert got_am == want["absmax"], (tag, "absmax", got_am, want["absmax"])
    for name in TENSORS:
        assert _sha(getattr(b, name)) == want[name], (tag, name, "digest differs from the oracle's")
    assert _sha(b.W) == want["W_new"], (tag, "W_new", "digest differs from the oracle's")
    got = float(b.loss[0])
    assert abs(got - want["loss"]) <= REL_TOL * max(abs(want["loss"]), 1e-30), (tag, "loss", got, want["loss"])


def _descs(w, seed):
    return [ffb.make_desc(l, i, seed) for i, l in enumerate(w.layers)]


@pytest.mark.parametrize("name,graph", [("tiny_mlp", False), ("mlp_lookahead", False), ("cnn", False), ("roofline", False),
                                        ("separable", False), ("tiny_mlp", True), ("mlp_lookahead", True)])
def test_fullsize_train_steps_match_oracle_digests(name, graph):
    if name not in DIG:
        pytest.skip("no digests for this workload in tests/golden/fullsize_digests.json")
    d = DIG[name]
    w = synth.workload(name)
    assert d["B"] == w.B and not d["greedy"]
    net = GpuNet(_descs(w, d["seed"]), w.B, synth.make_weights(w, d["seed"]), dumps=False, xnext=False, chain=True,
                 graph=graph)             # graph: steps 2.. are replays of the launch sequence captured at step 1
    net.set_input(synth.make_batch(w, d["seed"]))
    digested = d.get("digested", list(range(len(d["steps"]))))
    for step in range(d.get("n_steps", len(d["steps"]))):
        net.train_step(w.lam_per_step * step, step)
        if step in digested:                      # long runs: the first steps and every tenth are compared
            for l, want in enumerate(d["steps"][digested.index(step)]):
                _check_layer(net.bufs[l], want, f"{name}/step{step}/layer{l}")
    net.close()


@pytest.mark.parametrize("graph", [False, True])
def test_fullsize_greedy_epoch_matches_oracle_digests(graph):
    """Configuration 2 as stated: 58 distinct batches of 1024 + 1024 samples per phase, four phases; phase l trains
    layer l alone (ff_train_step_from with the earlier layers frozen) on the INT8 forward of the layers its
    predecessors' phases trained, weights carried through all 232 layer-steps.  The oracle's digests of the
    trained layer at the first two, every tenth and the last step of each phase, and of each layer's final
    weights, are compared with the device's."""
    name = "mlp_greedy"
    if name not in DIG or "final_W" not in DIG[name]:
        pytest.skip("no epoch digests for this workload in tests/golden/fullsize_digests.json")
    import torch
    d = DIG[name]
    w = synth.workload(name)
    n_batches = d["n_steps"]
    assert d["B"] == w.B and d["greedy"] and n_batches == w.steps
    net = GpuNet(_descs(w, d["seed"]), w.B, synth.make_weights(w, d["seed"]), dumps=False, xnext=False, chain=True, graph=graph)
    batches = [torch.from_numpy(synth.make_batch(w, d["seed"], batch_index=i)).cuda() for i in range(n_batches)]
    ctx = net.ctx.ctx
    for l in range(len(w.layers)):
        for i in range(n_batches):
            net.bufs[0].X.copy_(batches[i].reshape(net.bufs[0].X.shape))
            ffb.ff_train_step_from(ctx, net.descs_arr, net.bufs_arr, l + 1, l, w.B, 0.0, l * n_batches + i, 0)
            if i in d["digested"]:
                ffb.ff_poll_status(ctx, 0)
                _check_layer(net.bufs[l], d["steps"][l][d["digested"].index(i)], f"{name}/phase{l}/batch{i}")
        ffb.ff_poll_status(ctx, 0)
        assert _sha(net.bufs[l].W) == d["final_W"][l], (name, l, "final weights differ from the oracle's")
    if graph:
        assert ffb.ff_graph_replay_count(ctx) >= len(w.layers) * (n_batches - 2)
    net.close()
