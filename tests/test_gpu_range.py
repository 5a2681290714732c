"""INT32 range of the weight-gradient sums (Sec. IV-B: INT8 operands, INT32 accumulation).

A convolution's weight gradient sums over every output position of a set, so its worst case (all codes
+-127) leaves INT32 once a set has more than 133144 positions.  The library cuts such contractions into
parts that cannot wrap, adds the parts in 64 bits and reports a sum outside INT32 as FF_ERR_RANGE through
ff_poll_status (the weight concerned keeps its value); the oracle raises OverflowError for the same
codes.  The cases here call ff_layer_update on INT8 tensors the test writes itself:
  * every code +-127 and a set just below the bound: no error, bit-exact against the oracle;
  * the same just above the bound: FF_ERR_RANGE where the oracle raises, nothing else disturbed;
  * random codes above the bound (the realistic case): no error, bit-exact.
No access leaves its buffer in any of them: the kernels finish and report."""
import numpy as np
import pytest

from oracle import ffint8_oracle as O
from paper_2506_22771_b200 import binding as ffb
from paper_2506_22771_b200 import synth

pytestmark = pytest.mark.gpu

SAFE = (2 ** 31 - 1) // (127 * 127)     # 133144 positions
HW = 32

# (name, kind, Cin, N): routes - tensor-core implicit GEMM slabs, explicit im2col, dp4a, pointwise dense slabs, depthwise
LAYERS = [("conv64", 1, 64, 64), ("conv3", 1, 3, 16), ("conv16", 1, 16, 16), ("pw64", 2, 64, 64), ("dw16", 3, 16, 16)]
PATHS = [ffb.FF_GEMM_AUTO, ffb.FF_GEMM_SIMT]


def _cfg(kind, Cin, N):
    K = {1: 9 * Cin, 2: Cin, 3: 9}[kind]
    return synth.LayerCfg(kind, K, N, 1.0, 2.0 ** -40, 1.0, H=HW, Wd=HW, Cin=Cin)


def _run(kind, Cin, N, B, path, fill, seed=0):
    """ff_layer_update on chosen codes.  Returns (error code or 0, W before, W after, oracle state or None)."""
    import torch
    cfg = _cfg(kind, Cin, N)
    desc = ffb.make_desc(cfg, 0, 1, 0, 0, 0)
    spec = O.LayerSpec(kind, cfg.K, N, 1.0, cfg.lr, 1.0, H=HW, Wd=HW, Cin=Cin, round_x=0, round_w=0, round_dh=0, seed=1)
    ctx = ffb.Context([desc], B, 0)
    ffb.ff_set_gemm_path(ctx.ctx, path)
    b = ffb.LayerBuffers(desc, B, torch.device("cuda:0"), dumps=True)
    g = np.random.default_rng(seed)
    rows = 2 * B * HW * HW
    if fill == "extreme":       # +127 everywhere; the negative set's gradient codes are -127
        xq = np.full((rows, Cin), 127, np.int8)
        dhq = np.full((rows, N), 127, np.int8)
        dhq[rows // 2:] = -127
    else:
        xq = g.integers(-127, 128, size=(rows, Cin)).astype(np.int8)
        dhq = g.integers(-127, 128, size=(rows, N)).astype(np.int8)
    W0 = g.normal(size=(N, cfg.K)).astype(np.float32)
    b.Xq.copy_(torch.from_numpy(xq))
    b.dHq.copy_(torch.from_numpy(dhq))
    b.W.copy_(torch.from_numpy(W0))
    am = np.zeros(ffb.FF_ABSMAX_LEN, np.float32)
    am[[0, 1, 3]] = 127.0                                      # unit scales: the positive set's g^W is the integer sum itself
    am[4] = 63.5                                               # (half scale for the negative set, so the two do not cancel)
    b.absmax.copy_(torch.from_numpy(am))
    ffb.ff_layer_update(ctx.ctx, desc, b.struct, B, 0, 0)
    code = 0
    try:
        ffb.ff_poll_status(ctx.ctx, 0)
    except ffb.FFError as e:
        code = e.code
    ffb.ff_poll_status(ctx.ctx, 0)                             # the status word was cleared by the poll
    W1 = b.W.cpu().numpy()
    accW = b.accW_dump.cpu().numpy()
    st = O.LayerState(Xq=xq.reshape(2 * B, HW, HW, Cin), dHq=dhq.reshape(2 * B, HW, HW, N), a_x=(np.float32(127), np.float32(127)),
                      a_dh=(np.float32(127), np.float32(63.5)))
    try:
        O.layer_update(spec, st, W0, B)
    except OverflowError:
        st = None
    ctx.close()
    return code, W0, W1, accW, st


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("name,kind,Cin,N", LAYERS)
def test_extreme_codes_just_inside_the_range_are_exact(name, kind, Cin, N, path):
    B = SAFE // (HW * HW)                                      # 130 images: 133120 positions per set
    code, W0, W1, accW, st = _run(kind, Cin, N, B, path, "extreme")
    assert code == 0 and st is not None
    assert int(np.abs(st.accW).max()) == 127 * 127 * B * HW * HW   # the centre tap sees every position
    assert np.array_equal(accW, st.accW)
    assert np.array_equal(W1.view(np.uint32), st.W_new.view(np.uint32))


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("name,kind,Cin,N", LAYERS)
def test_extreme_codes_just_outside_the_range_are_reported(name, kind, Cin, N, path):
    B = SAFE // (HW * HW) + 1                                  # 131 images: 134144 positions per set
    code, W0, W1, accW, st = _run(kind, Cin, N, B, path, "extreme")
    assert st is None, "the oracle must refuse these codes (INT32 accumulator range)"
    assert code == ffb.FF_ERR_RANGE
    # the sums that left INT32 are those of the taps that see every position: their weights keep their value and
    # their dumped sums saturate; a corner tap stays in range and is updated
    K = W0.shape[1]
    taps = W0.reshape(N, 9, -1) if kind != 2 else W0.reshape(N, 1, K)
    after = W1.reshape(taps.shape)
    centre = 4 if kind != 2 else 0
    assert np.array_equal(after[:, centre], taps[:, centre])
    sat = accW.reshape((2,) + taps.shape)[:, :, centre]
    assert (sat[0] == 2 ** 31 - 1).all() and (sat[1] == -(2 ** 31 - 1)).all()
    if kind != 2:
        assert not np.array_equal(after[:, 0], taps[:, 0])


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("name,kind,Cin,N", LAYERS)
def test_random_codes_beyond_the_safe_length_are_exact(name, kind, Cin, N, path):
    B = SAFE // (HW * HW) + 6                                  # a contraction the worst case would not allow
    code, W0, W1, accW, st = _run(kind, Cin, N, B, path, "random", seed=3)
    assert code == 0 and st is not None
    assert np.array_equal(accW, st.accW)
    assert np.array_equal(W1.view(np.uint32), st.W_new.view(np.uint32))
