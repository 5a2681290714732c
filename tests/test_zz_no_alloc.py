"""The entry point that allocates nothing (ff_loss_coef_static) against the regular one.

Some users of the library call it from places where device memory cannot be allocated: inside
another framework's memory-pool lock or stream callback, or in a process whose device memory was
given away in full at start-up.  For them the loss / coefficient step exists in a second form
whose partial sums live in a small array built into the library instead of the caller's workspace.
This test runs the regular step (ff_layer_forward + ff_layer_loss_grad) and then the static
form on the same goodness values, twice in a row because the built-in array is shared by every
call and keeps the previous call's contents, and compares what both write: coef and the two g^Y
ranges bit for bit, the loss scalar to 1e-5 relative (the tolerance of the parity tests).  The static
form's outputs are also held against the CPU oracle's loss step on the same inputs (coef, the g^Y
ranges taken over every element of dH, and the loss), so the check does not rest on the regular
entry point alone.

Collected last on purpose (file name): a failure here cannot hide a failure elsewhere under -x.
"""
import numpy as np
import pytest

from oracle import ffint8_oracle as O
from paper_2506_22771_b200 import binding as ffb
from paper_2506_22771_b200 import synth
from tests.ffharness import GpuNet, REL_TOL, specs_and_descs

pytestmark = pytest.mark.gpu


def _bits(t):
    return t.detach().cpu().numpy().view(np.uint32)


@pytest.mark.parametrize("B,lam", [(300, 0.0), (300, 0.5)])
def test_static_loss_matches_workspace_loss_twice(B, lam):
    import torch
    w = synth.scaled(synth.workload("mlp_lookahead"), B=B, width_div=8)
    w.layers = w.layers[:2]
    specs, descs = specs_and_descs(w.layers, 17)
    Ws = synth.make_weights(w, 17)
    net = GpuNet(descs, w.B, Ws, dumps=False, xnext=True, chain=False)
    ctx = net.ctx.ctx
    for call in range(2):                      # two calls in a row: the second sees the first one's leftovers
        X = synth.make_batch(w, 17, batch_index=call)
        net.set_input(X)
        ffb.ff_layer_forward(ctx, descs[0], net.bufs[0].struct, B, call, 0)
        net.bufs[1].X.copy_(net.bufs[0].Xnext)
        ffb.ff_layer_forward(ctx, descs[1], net.bufs[1].struct, B, call, 0)
        b0, b1 = net.bufs[0], net.bufs[1]
        # regular path: scratch in the caller's workspace
        ffb.ff_layer_loss_grad(ctx, descs[0], b0.struct, B, [b1.G.data_ptr()], [descs[1].theta], lam, call, 0)
        ffb.ff_poll_status(ctx, 0)
        want_coef, want_loss, want_a = b0.coef.clone(), float(b0.loss[0]), b0.absmax.clone()
        # static path: same inputs, separate outputs, no context, no workspace
        coef = torch.full_like(b0.coef, -1.0)
        loss = torch.full((4,), -1.0, dtype=torch.float32, device="cuda")
        absmax = b0.absmax.clone()
        absmax[ffb.FF_A_DH_POS:ffb.FF_A_DH_NEG + 1] = -1.0
        ffb.ff_loss_coef_static(b0.G.data_ptr(), descs[0].theta, [b1.G.data_ptr()], [descs[1].theta], lam, B,
                                b0.rowmax.data_ptr(), absmax.data_ptr(), coef.data_ptr(), loss.data_ptr(), 0)
        torch.cuda.synchronize()
        assert np.array_equal(_bits(coef), _bits(want_coef)), f"call {call}: coef differs"
        assert np.array_equal(_bits(absmax), _bits(want_a)), f"call {call}: absmax differs"
        got_loss = float(loss[0])
        assert abs(got_loss - want_loss) <= REL_TOL * max(abs(want_loss), 1e-30), (call, got_loss, want_loss)
        # and against the oracle's loss step, computed from the inputs alone
        st0 = O.layer_forward(specs[0], X, Ws[0], B, call)
        st1 = O.layer_forward(specs[1], st0.Xnext, Ws[1], B, call)
        O.layer_loss_grad(specs[0], st0, B, [st1.G], [specs[1].theta], lam, call)
        assert np.array_equal(_bits(coef), st0.coef.view(np.uint32)), f"call {call}: coef differs from the oracle's"
        got_a = absmax.detach().cpu().numpy()[ffb.FF_A_DH_POS:ffb.FF_A_DH_NEG + 1]
        assert np.array_equal(got_a.view(np.uint32), np.array(st0.a_dh, dtype=np.float32).view(np.uint32)), (call, got_a, st0.a_dh)
        assert abs(got_loss - st0.loss) <= REL_TOL * max(abs(st0.loss), 1e-30), (call, got_loss, st0.loss)
    net.close()


def test_static_loss_rejects_batches_beyond_its_array():
    import torch
    z = torch.zeros(8, device="cuda")
    zi = torch.zeros(8, dtype=torch.int32, device="cuda")
    with pytest.raises(ffb.FFError) as e:
        ffb.ff_loss_coef_static(z.data_ptr(), 1.0, [], [], 0.0, ffb.FF_STATIC_LOSS_MAX_SAMPLES // 2 + 1,
                                zi.data_ptr(), z.data_ptr(), z.data_ptr(), z.data_ptr(), 0)
    assert e.value.code == ffb.FF_ERR_RANGE and "FF_STATIC_LOSS_MAX_SAMPLES" in str(e.value)
