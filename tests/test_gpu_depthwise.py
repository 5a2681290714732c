"""GPU parity of depthwise 3x3 convolution layers against the oracle, bit for bit: alone, inside
separable blocks (pointwise - depthwise - pointwise), with stride 2, with channel counts that are
not multiples of four (scalar kernels), widths that are not multiples of the four outputs a thread
takes, with the heavy-ball update, split over data-parallel shards, and with replayed launches."""
import numpy as np
import pytest

from paper_2506_22771_b200 import binding as ffb
from paper_2506_22771_b200 import synth
from tests.ffharness import GpuNet, specs_and_descs
from tests.test_gpu_data_parallel import _run_dp
from tests.test_gpu_parity import _run_and_compare

pytestmark = pytest.mark.gpu

PATHS = [(ffb.FF_GEMM_SIMT, 0), (ffb.FF_GEMM_AUTO, 0)]


def _dw(C, H, Wd, stride=1, lr=0.03 / 64, momentum=0.0):
    Ho, Wo = (H - 1) // stride + 1, (Wd - 1) // stride + 1
    return synth.LayerCfg(3, 9, C, float(C * Ho * Wo), lr, float(np.sqrt(C * Ho * Wo)), H=H, Wd=Wd, Cin=C, stride=stride,
                          momentum=momentum)


def _pw(Cin, Cout, H, Wd, lr=0.03 / 64):
    return synth.LayerCfg(2, Cin, Cout, float(Cout * H * Wd), lr, float(np.sqrt(Cout * H * Wd)), H=H, Wd=Wd, Cin=Cin)


# (the batch generator writes the label into ten pixels of the first image row: Wd >= 10)
@pytest.mark.parametrize("C,H,Wd,B,stride", [(16, 12, 12, 3, 1), (64, 16, 16, 2, 1), (32, 9, 11, 2, 2), (128, 8, 10, 5, 2),
                                             (8, 5, 13, 2, 1), (6, 10, 10, 2, 1), (3, 12, 12, 2, 2), (1, 10, 10, 1, 1)])
def test_depthwise_layer_alone(C, H, Wd, B, stride):
    w = synth.Workload("dw", B, [_dw(C, H, Wd, stride)], (H, Wd, C), "normal", "kaiming_uniform", 2)
    _run_and_compare(w, seed=40 + C, steps=3, lam_per_step=0.0, path=(ffb.FF_GEMM_AUTO, 0))


@pytest.mark.parametrize("path", PATHS)
def test_separable_block_with_lookahead(path):
    # pointwise 16 -> 64, depthwise 64 (stride 2), pointwise 64 -> 32: the block of the paper's mobile models
    H = Wd = 16
    layers = [_pw(16, 64, H, Wd), _dw(64, H, Wd, stride=2), _pw(64, 32, H // 2, Wd // 2)]
    w = synth.Workload("separable", 4, layers, (H, Wd, 16), "normal", "kaiming_uniform", 2)
    _run_and_compare(w, seed=51, steps=3, lam_per_step=0.5, path=path)
    _run_and_compare(w, seed=51, steps=4, lam_per_step=0.5, path=path, graph=True)


def test_depthwise_all_rounding_modes_and_momentum():
    H = Wd = 12
    w = synth.Workload("dw_mom", 3, [_dw(24, H, Wd, 1, momentum=0.875), _dw(24, H, Wd, 2, momentum=0.5)], (H, Wd, 24), "normal",
                       "kaiming_uniform", 2)
    for rounding in [(0, 0, 0), (1, 1, 1)]:
        _run_and_compare(w, seed=61, steps=3, lam_per_step=0.25, path=(ffb.FF_GEMM_AUTO, 0), rounding=rounding)


def test_depthwise_data_parallel():
    H = Wd = 12
    layers = [_pw(8, 32, H, Wd), _dw(32, H, Wd, 1), _dw(32, H, Wd, 2)]
    w = synth.Workload("dw_dp", 5, layers, (H, Wd, 8), "normal", "kaiming_uniform", 2)
    _run_dp(w, seed=71, steps=2, lam_per_step=0.5, world=2, path=(ffb.FF_GEMM_AUTO, 0))


def test_depthwise_large_enough_for_many_blocks():
    # 2 x 24 images of 32 x 32 x 160: many position chunks per set and two channel-group tiles (one ragged) in the gradient
    w = synth.Workload("dw_big", 24, [_dw(160, 32, 32, 1, lr=0.03 / 1024)], (32, 32, 160), "normal", "kaiming_uniform", 1)
    _run_and_compare(w, seed=81, steps=1, lam_per_step=0.0, path=(ffb.FF_GEMM_AUTO, 0))


def test_depthwise_argument_errors():
    H = Wd = 12
    w = synth.Workload("dw", 2, [_dw(16, H, Wd)], (H, Wd, 16), "normal", "kaiming_uniform", 1)
    specs, descs = specs_and_descs(w.layers, 1)
    net = GpuNet(descs, w.B, synth.make_weights(w, 1))
    for field, bad in [("K", 16), ("N", 8), ("stride", 3)]:
        old = getattr(net.descs_arr[0], field)
        setattr(net.descs_arr[0], field, bad)
        with pytest.raises(ffb.FFError):
            net.train_step(0.0, 0)
        setattr(net.descs_arr[0], field, old)
    net.train_step(0.0, 0)
    net.close()
