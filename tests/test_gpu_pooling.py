"""GPU parity of 2x2 max pooling between layers (a layer's normalised output is pooled before it becomes
the next layer's FP32 / INT8 input) against the oracle, bit for bit."""
import numpy as np
import pytest

from paper_2506_22771_b200 import binding as ffb
from paper_2506_22771_b200 import synth
from tests.ffharness import GpuNet, specs_and_descs
from tests.test_gpu_data_parallel import _run_dp
from tests.test_gpu_parity import _run_and_compare

pytestmark = pytest.mark.gpu

PATHS = [(ffb.FF_GEMM_SIMT, 0), (ffb.FF_GEMM_AUTO, 0)]


def _conv(ci, co, H, Wd, pool=1, stride=1):
    Ho, Wo = (H - 1) // stride + 1, (Wd - 1) // stride + 1
    return synth.LayerCfg(1, 9 * ci, co, float(co * Ho * Wo), 0.03 / (Ho * Wo), float(np.sqrt(co * Ho * Wo)), H=H, Wd=Wd, Cin=ci,
                          stride=stride, pool=pool)


def _dw(C, H, Wd, pool=1):
    return synth.LayerCfg(3, 9, C, float(C * H * Wd), 0.03 / (H * Wd), float(np.sqrt(C * H * Wd)), H=H, Wd=Wd, Cin=C, pool=pool)


def _pw(ci, co, H, Wd, pool=1):
    return synth.LayerCfg(2, ci, co, float(co * H * Wd), 0.03 / (H * Wd), float(np.sqrt(co * H * Wd)), H=H, Wd=Wd, Cin=ci, pool=pool)


@pytest.mark.parametrize("path", PATHS)
def test_conv_pool_stack(path):
    # conv 3->16 (pool) -> conv 16->64 (pool) -> conv 64->32 on 32x32 -> 16x16 -> 8x8; look-ahead over all three
    layers = [_conv(3, 16, 32, 32, pool=2), _conv(16, 64, 16, 16, pool=2), _conv(64, 32, 8, 8)]
    w = synth.Workload("pool3", 3, layers, (32, 32, 3), "normal", "kaiming_uniform", 2)
    _run_and_compare(w, seed=91, steps=3, lam_per_step=0.5, path=path)
    _run_and_compare(w, seed=91, steps=4, lam_per_step=0.5, path=path, graph=True)


@pytest.mark.parametrize("rounding", [(0, 0, 0), (1, 1, 1)])
def test_pool_scalar_channels_and_last_layer(rounding):
    # 6 channels (no four-channel groups), pooled output of the LAST layer (only the FP32 copy exists), strided conv before it
    layers = [_pw(5, 6, 12, 12, pool=2), _dw(6, 6, 6), _conv(6, 10, 6, 6, pool=2, stride=1)]
    w = synth.Workload("pool_odd", 2, layers, (12, 12, 5), "normal", "kaiming_uniform", 2)
    _run_and_compare(w, seed=92, steps=2, lam_per_step=0.25, path=(ffb.FF_GEMM_AUTO, 0), rounding=rounding)


def test_pool_data_parallel():
    layers = [_conv(3, 8, 12, 12, pool=2), _dw(8, 6, 6, pool=2), _pw(8, 12, 3, 3)]
    w = synth.Workload("pool_dp", 5, layers, (12, 12, 3), "normal", "kaiming_uniform", 2)
    _run_dp(w, seed=93, steps=2, lam_per_step=0.5, world=2, path=(ffb.FF_GEMM_AUTO, 0))


def test_pool_argument_errors():
    layers = [_conv(3, 8, 12, 12, pool=2), _conv(8, 8, 6, 6)]
    w = synth.Workload("pool_err", 2, layers, (12, 12, 3), "normal", "kaiming_uniform", 1)
    specs, descs = specs_and_descs(w.layers, 1)
    net = GpuNet(descs, w.B, synth.make_weights(w, 1))
    net.train_step(0.0, 0)
    net.descs_arr[0].pool = 1            # the next layer no longer fits
    with pytest.raises(ffb.FFError):
        net.train_step(0.0, 1)
    net.descs_arr[0].pool = 3
    with pytest.raises(ffb.FFError):
        net.train_step(0.0, 1)
    net.close()
    # odd output extents cannot be pooled
    bad = [_conv(3, 8, 11, 12, pool=2)]
    wb = synth.Workload("pool_err2", 2, bad, (11, 12, 3), "normal", "kaiming_uniform", 1)
    _, d2 = specs_and_descs(wb.layers, 1)
    with pytest.raises(ffb.FFError):
        n2 = GpuNet(d2, wb.B, synth.make_weights(wb, 1))
        n2.train_step(0.0, 0)
