"""Shared helpers of the GPU parity tests: run a step through the C ABI and through the oracle
on the same seeded inputs and compare every tensor (bit-exact for INT8 / INT32 / absmax / S /
rowmax / coef / W, 1e-5 relative for the loss scalar)."""
import ctypes as C

import numpy as np

from oracle import ffint8_oracle as O
from paper_2506_22771_b200 import binding as ffb

REL_TOL = 1e-5   # relative tolerance for order-dependent FP32 scalars (the loss value)


def specs_and_descs(layers, seed, round_x=1, round_w=0, round_dh=1):
    specs, descs = [], []
    for i, l in enumerate(layers):
        specs.append(O.LayerSpec(l.kind, l.K, l.N, l.theta, l.lr, l.tau, l.eps, l.H, l.Wd, l.Cin,
                                 round_x, round_w, round_dh, seed, i, getattr(l, "stride", 1),
                                 getattr(l, "momentum", 0.0), getattr(l, "optimizer", 0), getattr(l, "beta2", 0.999),
                                 getattr(l, "adam_eps", 1e-8), getattr(l, "pool", 1), getattr(l, "skip_from", -1),
                                 getattr(l, "skip_scale", 1.0)))
        descs.append(ffb.make_desc(l, i, seed, round_x, round_w, round_dh))
    return specs, descs


class GpuNet:
    def __init__(self, descs, B, Ws, dumps=True, xnext=True, chain=True, gemm_path=ffb.FF_GEMM_AUTO, graph=False,
                 pad_rows=True, skips=None):
        """skips[l] >= 0: layer l's output takes a skip path from the FP32 input of layer skips[l] (the network input for
        layer 0, else the Xnext of the layer before it)."""
        import torch
        self.torch = torch
        self.dev = torch.device("cuda:0")
        self.B = B
        self.descs = descs
        self.ctx = ffb.Context(descs, B, 0)
        if isinstance(gemm_path, tuple):
            gemm_path, form = gemm_path
            ffb.ff_set_tensor_form(self.ctx.ctx, form)
        ffb.ff_set_gemm_path(self.ctx.ctx, gemm_path)
        if graph:
            ffb.ff_set_graph_mode(self.ctx.ctx, True)
        self.bufs = [ffb.LayerBuffers(d, B, self.dev, dumps=dumps, xnext=xnext, own_x=(i == 0 or not chain), pad_rows=pad_rows)
                     for i, d in enumerate(descs)]
        for b, W in zip(self.bufs, Ws):
            b.W.copy_(torch.from_numpy(W))
        for l, src in enumerate(skips or []):
            if src >= 0:
                t = self.bufs[0].X if src == 0 else self.bufs[src - 1].Xnext
                self.bufs[l].struct.Skip = t.data_ptr()
        self.descs_arr = (ffb.ff_layer_desc * len(descs))(*descs)
        self.bufs_arr = (ffb.ff_layer_bufs * len(descs))(*[b.struct for b in self.bufs])

    def set_input(self, X):
        t = self.torch.from_numpy(np.ascontiguousarray(X)).reshape(self.bufs[0].X.shape)
        self.bufs[0].X.copy_(t)

    def train_step(self, lam, step):
        ffb.ff_train_step(self.ctx.ctx, self.descs_arr, self.bufs_arr, len(self.descs), self.B, lam, step, 0)
        ffb.ff_poll_status(self.ctx.ctx, 0)

    def close(self):
        self.ctx.close()


def _np(t):
    return t.detach().cpu().numpy()


def compare_layer(st: O.LayerState, b, spec, B, check_dumps=True, tag=""):
    """Assert that the GPU buffers of one layer equal the oracle's LayerState."""
    R = spec.rows_per_sample
    rows = 2 * B * R
    eq = lambda name, got, want: _assert_equal(f"{tag}{name}", got, want)
    am = _np(b.absmax)
    eq("a_x", am[0:2], np.array(st.a_x, dtype=np.float32))
    eq("a_w", am[2], np.float32(st.a_w))
    eq("Xq", _np(b.Xq).reshape(-1), st.Xq.reshape(-1))
    eq("Wq", _np(b.Wq).reshape(-1), st.Wq.reshape(-1))
    if check_dumps and b.acc_dump is not None:
        eq("acc", _np(b.acc_dump).reshape(-1), st.acc.reshape(-1))
    eq("S", _np(b.S).astype(np.uint64), st.S)
    eq("rowmax", _np(b.rowmax), st.rowmax)
    eq("Y", _np(b.Y).reshape(-1), st.Y.reshape(-1))
    eq("G", _np(b.G), st.G)
    if b.Xnext is not None:
        eq("Xnext", _np(b.Xnext).reshape(-1), st.Xnext.reshape(-1))
        a_xn = getattr(st, "a_xnext_full", None) or (O.absmax(st.Xnext[:B]), O.absmax(st.Xnext[B:]))
        eq("a_xnext", am[5:7], np.array(a_xn, dtype=np.float32))
    if st.coef is not None:
        eq("coef", _np(b.coef), st.coef)
        eq("a_dh", am[3:5], np.array(st.a_dh, dtype=np.float32))
        eq("dHq", _np(b.dHq).reshape(-1), st.dHq.reshape(-1))
        got_loss = float(_np(b.loss)[0])
        assert abs(got_loss - st.loss) <= REL_TOL * max(abs(st.loss), 1e-30), (tag, "loss", got_loss, st.loss)
    if st.W_new is not None:
        if check_dumps and b.accW_dump is not None:
            eq("accW", _np(b.accW_dump).reshape(-1), st.accW.reshape(-1))
        eq("W_new", _np(b.W).reshape(-1), st.W_new.reshape(-1))
        if st.M_new is not None:
            eq("M_new", _np(b.Mom).reshape(-1), st.M_new.reshape(-1))
        if st.V_new is not None:
            eq("V_new", _np(b.Var).reshape(-1), st.V_new.reshape(-1))


def _assert_equal(name, got, want):
    got = np.asarray(got)
    want = np.asarray(want)
    assert got.shape == want.shape, (name, got.shape, want.shape)
    if got.dtype.kind == "f":
        same = got.view(np.uint32) == want.astype(np.float32).view(np.uint32) if got.ndim else \
            np.float32(got).view(np.uint32) == np.float32(want).view(np.uint32)
    else:
        same = got == want
    if not np.all(same):
        bad = np.flatnonzero(~np.atleast_1d(same))
        i = int(bad[0])
        raise AssertionError(f"{name}: {bad.size} of {same.size} elements differ; first at {i}: "
                             f"got {np.atleast_1d(got)[i]!r} want {np.atleast_1d(want)[i]!r}")


def shard_state(st: O.LayerState, B_total, row_off, B_local):
    """The part of a whole-batch LayerState that the shard holding samples [row_off, row_off + B_local)
    of each set must reproduce: per-sample arrays (first axis = sample) cut to those samples; ranges,
    loss, weight-gradient sums and new weights are those of the whole batch."""
    import copy

    def cut(a):
        if a is None:
            return None
        a = np.asarray(a)
        return np.concatenate([a[row_off:row_off + B_local], a[B_total + row_off:B_total + row_off + B_local]], 0)

    out = copy.copy(st)
    for name in ("Xq", "acc", "Y", "Xnext", "dHq", "S", "rowmax", "G", "coef"):
        setattr(out, name, cut(getattr(st, name)))
    out.a_xnext_full = (O.absmax(st.Xnext[:B_total]), O.absmax(st.Xnext[B_total:]))
    return out
