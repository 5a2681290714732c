"""GPU parity of the label-embedding kernel (positive / negative / candidate batches) against the oracle.
Without scaling the rows must be equal bit for bit; with length scaling the sum of squares is reduced
in a different order (FP64), so rows are compared to FP32 rounding (2e-6 relative)."""
import numpy as np
import pytest

from oracle import ffint8_oracle as O
from paper_2506_22771_b200 import binding as ffb

pytestmark = pytest.mark.gpu


def _run(x, labels, n_classes, stride, on, tau0, eps=1e-8):
    import torch
    B, n = x.shape
    sets = labels.shape[0]
    ctx = ffb.Context([ffb.ff_layer_desc(0, 16, 16, 1, 1, 0, 0, 0, 0, 0, 1.0, 0.1, 1.0, 1e-8, 0)], 1, 0)
    tx = torch.from_numpy(x).cuda()
    tl = torch.from_numpy(labels.astype(np.int32)).cuda()
    out = torch.full((sets * B, n), float("nan"), dtype=torch.float32, device="cuda")
    ffb.ff_embed_labels(ctx.ctx, tx.data_ptr(), tl.data_ptr(), B, n, sets, n_classes, stride, on, tau0, eps, out.data_ptr(), 0)
    try:
        ffb.ff_poll_status(ctx.ctx, 0)
    finally:
        res = out.cpu().numpy()
        ctx.close()
    return res


@pytest.mark.parametrize("B,n,n_classes,stride,sets", [(32, 784, 10, 1, 2), (5, 3072, 10, 3, 2), (7, 77, 10, 1, 2),
                                                       (3, 13, 4, 3, 4), (300, 2000, 10, 1, 10), (2, 10, 10, 1, 2)])
@pytest.mark.parametrize("tau0", [0.0, -1.0, 1.0])
def test_embed_labels_matches_oracle(B, n, n_classes, stride, sets, tau0):
    g = np.random.default_rng(B * 1000 + n)
    x = g.normal(size=(B, n)).astype(np.float32)
    labels = g.integers(0, n_classes, size=(sets, B))
    t0 = float(np.sqrt(n)) if tau0 > 0 else tau0
    got = _run(x, labels, n_classes, stride, 1.0, t0)
    want = O.embed_labels(x, labels, n_classes, stride, 1.0, t0)
    if tau0 > 0:
        assert np.allclose(got, want, rtol=2e-6, atol=0.0)
        assert np.array_equal(got == 0, want == 0)
        assert np.mean(got == want) > 0.999          # a different rounding of r would change whole rows
    else:
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_embed_labels_on_value_and_eps():
    g = np.random.default_rng(3)
    x = g.uniform(size=(9, 64)).astype(np.float32)
    labels = g.integers(0, 10, size=(2, 9))
    got = _run(x, labels, 10, 1, 2.5, 8.0, eps=0.5)
    want = O.embed_labels(x, labels, 10, 1, 2.5, 8.0, eps=0.5)
    assert np.allclose(got, want, rtol=2e-6, atol=0.0)


def test_embed_labels_rejects_bad_labels_and_arguments():
    x = np.ones((4, 16), dtype=np.float32)
    labels = np.array([[0, 1, 10, 3], [1, 2, 3, -1]])
    with pytest.raises(ffb.FFError) as e:
        _run(x, labels, 10, 1, 1.0, 0.0)
    assert e.value.code == ffb.FF_ERR_RANGE
    with pytest.raises(ffb.FFError):
        _run(x, np.zeros((2, 4), dtype=np.int64), 10, 2, 1.0, 0.0)      # places 0, 2, ..., 18 do not fit 16 values
