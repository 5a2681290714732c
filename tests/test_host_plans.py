"""Host logic of the library, checked on the CPU: how a weight gradient's contraction is cut.

INT8 x INT8 products accumulated in INT32 (Sec. IV-B) can wrap once a sum covers more than
floor((2^31 - 1) / 127^2) = 133144 products.  A convolution's weight gradient sums over every output position of a
set, so the library cuts the contraction into parts that stay below that length, adds the parts in 64 bits and
reports a total outside INT32 (the GPU tests in test_gpu_range.py check the reporting).  ff_plan_wgrad exposes the
planning arithmetic the launches use; here it is swept over layer shapes, batch sizes and device sizes:
  * no accumulator and no array element ever sums more than 133144 products;
  * the parts cover the contraction;
  * a contraction that is short enough is not cut for safety's sake alone;
  * a workspace too small for the parts safety needs is refused, never silently under-split.
No device is touched."""
import itertools

import pytest

from paper_2506_22771_b200 import binding as ffb
from paper_2506_22771_b200 import synth

SAFE = (2 ** 31 - 1) // (127 * 127)


def _desc(kind, cin, n, h, w, stride=1):
    K = 9 * cin if kind == 1 else cin
    return ffb.make_desc(synth.LayerCfg(kind, K, n, 1.0, 1e-3, 1.0, H=h, Wd=w, Cin=cin, stride=stride), 0, 1)


def _positions(h, w, stride, B):
    ho, wo = (h - 1) // stride + 1, (w - 1) // stride + 1
    return B * ho * wo


def test_safe_length_constant():
    assert SAFE == 133144 and 127 * 127 * SAFE <= 2 ** 31 - 1 < 127 * 127 * (SAFE + 1)


@pytest.mark.parametrize("sm_count", [148, 132, 64, 8])
def test_tensor_core_split_plans_never_exceed_the_safe_length(sm_count):
    seen = 0
    for (cin, n), (h, w), B, stride in itertools.product([(64, 64), (64, 128), (128, 256), (128, 128), (192, 320), (64, 512)],
                                                         [(32, 32), (16, 16), (8, 16), (64, 64), (32, 128)],
                                                         [1, 2, 16, 130, 131, 256, 1024, 5000], [1, 2]):
        d = _desc(1, cin, n, h, w, stride)
        code, pl = ffb.ff_plan_wgrad(d, B, sm_count, ffb.FF_PLAN_TENSOR_SLABS)
        if code == ffb.FF_ERR_ARG:          # the implicit-GEMM kernels do not take this geometry
            continue
        assert code == 0
        seen += 1
        clen = _positions(h, w, stride, B)
        assert 1 <= pl.longest_register_sum <= pl.longest_part_sum <= SAFE, (cin, n, h, w, B, stride)
        assert pl.parts >= 1 and pl.splits >= pl.parts
        assert pl.splits * pl.longest_register_sum >= clen          # the splits cover every position
        assert pl.parts * pl.longest_part_sum >= clen
        assert pl.parts >= -(-clen // SAFE)                          # at least the parts safety needs ...
        if clen <= SAFE // 2:
            assert pl.parts == 1, "a short contraction leaves one array"   # ... and no more arrays than splits demand
    assert seen > 100


@pytest.mark.parametrize("sm_count", [148, 64])
def test_pointwise_split_plans(sm_count):
    for (cin, n), (h, w), B in itertools.product([(64, 128), (128, 64), (256, 256), (32, 48)], [(16, 16), (32, 32), (7, 9)],
                                                 [1, 3, 64, 131, 600, 4000]):
        d = _desc(2, cin, n, h, w)
        code, pl = ffb.ff_plan_wgrad(d, B, sm_count, ffb.FF_PLAN_TENSOR_SLABS)
        if code == ffb.FF_ERR_ARG:
            continue
        assert code == 0
        clen = B * h * w
        assert pl.longest_register_sum <= pl.longest_part_sum <= SAFE
        assert pl.splits * pl.longest_register_sum >= clen and pl.parts * pl.longest_part_sum >= clen


def test_first_layer_plans():
    for cin, n, (h, w), B, stride, sm in itertools.product([1, 2, 3, 4], [16, 32, 64, 128], [(32, 32), (28, 28), (11, 13), (2, 10)],
                                                           [1, 2, 130, 131, 256, 3000], [1, 2], [148, 16]):
        d = _desc(1, cin, n, h, w, stride)
        code, pl = ffb.ff_plan_wgrad(d, B, sm, ffb.FF_PLAN_FIRST_LAYER)
        assert code == 0
        clen = _positions(h, w, stride, B)
        assert pl.longest_register_sum <= pl.longest_part_sum <= SAFE
        assert pl.parts * pl.longest_part_sum >= clen
        assert pl.parts == max(1, -(-(-(-clen // 256)) // (SAFE // 256)))    # chunks of 256 positions, 520 chunks per part
    # other layers are not this route's
    assert ffb.ff_plan_wgrad(_desc(1, 8, 64, 16, 16), 4, 148, ffb.FF_PLAN_FIRST_LAYER)[0] == ffb.FF_ERR_ARG
    assert ffb.ff_plan_wgrad(_desc(1, 3, 48, 16, 16), 4, 148, ffb.FF_PLAN_FIRST_LAYER)[0] == ffb.FF_ERR_ARG


def test_fallback_plans_and_a_workspace_too_small():
    for (kind, cin, n), (h, w), B in itertools.product([(1, 12, 20), (1, 3, 10), (2, 12, 10), (1, 16, 16)], [(32, 32), (9, 11), (64, 64)],
                                                       [1, 5, 131, 700, 2500]):
        d = _desc(kind, cin, n, h, w)
        code, pl = ffb.ff_plan_wgrad(d, B, 148, ffb.FF_PLAN_DP4A_SLABS)
        assert code == 0
        clen = B * h * w
        assert pl.longest_register_sum <= SAFE and pl.longest_part_sum <= SAFE
        assert pl.splits * pl.longest_register_sum >= clen
        need = -(-clen // (SAFE // 32 * 32))
        assert pl.splits >= need
        if need >= 2:
            # room for one slab fewer than safety needs: refused, not under-split
            per_split = 2 * d.N * d.K * 4
            code2, _ = ffb.ff_plan_wgrad(d, B, 148, ffb.FF_PLAN_DP4A_SLABS, workspace_bytes=per_split * (need - 1) + 4096)
            assert code2 == ffb.FF_ERR_WORKSPACE


def test_argument_errors():
    d = _desc(1, 64, 64, 16, 16)
    assert ffb.ff_plan_wgrad(d, 0, 148, ffb.FF_PLAN_TENSOR_SLABS)[0] == ffb.FF_ERR_ARG
    assert ffb.ff_plan_wgrad(d, 4, 0, ffb.FF_PLAN_TENSOR_SLABS)[0] == ffb.FF_ERR_ARG
    assert ffb.ff_plan_wgrad(d, 4, 148, 7)[0] == ffb.FF_ERR_ARG
    lin = ffb.make_desc(synth.LayerCfg(0, 64, 64, 1.0, 1e-3, 1.0), 0, 1)
    assert ffb.ff_plan_wgrad(lin, 4, 148, ffb.FF_PLAN_TENSOR_SLABS)[0] == ffb.FF_ERR_ARG
