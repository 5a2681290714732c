"""Thin ctypes binding of libffint8.so: same names as the C ABI (include/ffint8.h), argument
marshalling only.  PyTorch supplies device memory and streams; every step of the path runs in
the library's CUDA kernels.  There is no CPU fallback: a missing library raises."""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

from . import build as _build

FF_OK = 0
FF_ERR_ARG, FF_ERR_ALIGN, FF_ERR_WORKSPACE, FF_ERR_NONFINITE = -1, -2, -3, -4
FF_ERR_RANGE, FF_ERR_DEVICE_TIMEOUT, FF_ERR_CUDA, FF_ERR_UNSUPPORTED_ARCH = -5, -6, -7, -8
FF_LINEAR, FF_CONV3X3, FF_CONV1X1, FF_DWCONV3X3 = 0, 1, 2, 3
FF_ROUND_NEAREST_EVEN, FF_ROUND_STOCHASTIC = 0, 1
FF_OPT_SGD, FF_OPT_ADAM = 0, 1
FF_GEMM_AUTO, FF_GEMM_SIMT, FF_GEMM_TENSOR = 0, 1, 2
FF_A_X_POS, FF_A_X_NEG, FF_A_W, FF_A_DH_POS, FF_A_DH_NEG, FF_A_XNEXT_POS, FF_A_XNEXT_NEG = range(7)
FF_ABSMAX_LEN = 8

EXPORTS = ["ff_create", "ff_destroy", "ff_workspace_bytes", "ff_set_workspace", "ff_set_gemm_path", "ff_set_tensor_form",
           "ff_set_graph_mode", "ff_graph_replay_count", "ff_dp_phase_count", "ff_dp_train_phase",
           "ff_embed_labels",
           "ff_layer_forward", "ff_layer_loss_grad", "ff_layer_update", "ff_train_step", "ff_train_step_from",
           "ff_poll_status", "ff_last_error", "ff_launch_count", "ff_int8_gemm",
           "ff_profile_start", "ff_profile_stop", "ff_loss_coef_static", "ff_predict", "ff_selftest_bounded_wait",
           "ff_plan_wgrad"]
FF_PLAN_TENSOR_SLABS, FF_PLAN_FIRST_LAYER, FF_PLAN_DP4A_SLABS = 0, 1, 2
FF_STATIC_LOSS_MAX_SAMPLES = 65536
FF_K_NAMES = ["absmax", "quantize", "fwd_gemm", "finalize", "normalize", "loss", "dh_quantize",
              "upd_gemm", "raw_gemm", "classify", "dw_fwd", "dw_upd"]


class ff_layer_desc(C.Structure):
    _fields_ = [("kind", C.c_int32), ("K", C.c_int32), ("N", C.c_int32), ("H", C.c_int32),
                ("Wd", C.c_int32), ("Cin", C.c_int32), ("index", C.c_int32),
                ("round_x", C.c_int32), ("round_w", C.c_int32), ("round_dh", C.c_int32),
                ("theta", C.c_float), ("lr", C.c_float), ("tau", C.c_float), ("eps", C.c_float),
                ("seed", C.c_uint64), ("stride", C.c_int32), ("momentum", C.c_float),
                ("optimizer", C.c_int32), ("beta2", C.c_float), ("adam_eps", C.c_float), ("pool", C.c_int32),
                ("skip_scale", C.c_float)]


class ff_layer_bufs(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("W", "X", "Y", "G", "Xnext", "Xq", "Wq", "dHq", "absmax", "S", "rowmax", "coef",
                 "loss", "acc_dump", "accW_dump", "Mom", "Var", "Skip")] + [("ld_xq", C.c_int32), ("ld_dhq", C.c_int32)]


FF_DP_MAX_REDUCE = 96
FF_DP_F32, FF_DP_I32 = 0, 1
FF_DP_MAX, FF_DP_SUM = 0, 1


class ff_dp_reduce(C.Structure):
    _fields_ = [("dev_ptr", C.c_void_p), ("count", C.c_uint64), ("dtype", C.c_int32), ("op", C.c_int32),
                ("needed_by_phase", C.c_int32), ("reserved", C.c_int32)]


class ff_wgrad_plan(C.Structure):
    _fields_ = [("splits", C.c_int32), ("parts", C.c_int32), ("longest_register_sum", C.c_int64),
                ("longest_part_sum", C.c_int64)]


class FFError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"libffint8 error {code}: {msg}")
        self.code = code


_lib = None


def lib_path() -> str:
    return _build.LIB_PATH


def load(build_if_missing: bool = True):
    """Load libffint8.so (building it first when the file is absent and nvcc is there)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_build.LIB_PATH):
        if not build_if_missing:
            raise FileNotFoundError(_build.LIB_PATH)
        _build.build()
    lib = C.CDLL(_build.LIB_PATH)
    vp, i32, u64, f32 = C.c_void_p, C.c_int, C.c_uint64, C.c_float
    lib.ff_create.argtypes = [C.POINTER(vp), i32]
    lib.ff_destroy.argtypes = [vp]
    lib.ff_workspace_bytes.argtypes = [C.POINTER(ff_layer_desc), i32, i32, C.POINTER(C.c_size_t)]
    lib.ff_set_workspace.argtypes = [vp, vp, C.c_size_t]
    lib.ff_set_gemm_path.argtypes = [vp, i32]
    lib.ff_set_tensor_form.argtypes = [vp, i32]
    lib.ff_set_graph_mode.argtypes = [vp, i32]
    lib.ff_embed_labels.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, f32, f32, f32, vp, vp]
    lib.ff_dp_phase_count.argtypes = [i32]
    lib.ff_dp_train_phase.argtypes = [vp, C.POINTER(ff_layer_desc), C.POINTER(ff_layer_bufs), i32, i32, i32, i32, i32, f32,
                                      u64, vp, C.POINTER(ff_dp_reduce), C.POINTER(i32)]
    lib.ff_layer_forward.argtypes = [vp, C.POINTER(ff_layer_desc), C.POINTER(ff_layer_bufs), i32, u64, vp]
    lib.ff_layer_loss_grad.argtypes = [vp, C.POINTER(ff_layer_desc), C.POINTER(ff_layer_bufs), i32,
                                       C.POINTER(vp), C.POINTER(f32), i32, f32, u64, vp]
    lib.ff_layer_update.argtypes = [vp, C.POINTER(ff_layer_desc), C.POINTER(ff_layer_bufs), i32, u64, vp]
    lib.ff_train_step.argtypes = [vp, C.POINTER(ff_layer_desc), C.POINTER(ff_layer_bufs), i32, i32, f32, u64, vp]
    lib.ff_train_step_from.argtypes = [vp, C.POINTER(ff_layer_desc), C.POINTER(ff_layer_bufs), i32, i32, i32, f32, u64, vp]
    lib.ff_poll_status.argtypes = [vp, vp]
    lib.ff_last_error.argtypes = [vp]
    lib.ff_last_error.restype = C.c_char_p
    lib.ff_launch_count.argtypes = [vp]
    lib.ff_launch_count.restype = u64
    lib.ff_graph_replay_count.argtypes = [vp]
    lib.ff_graph_replay_count.restype = u64
    lib.ff_int8_gemm.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp]
    lib.ff_profile_start.argtypes = [vp]
    lib.ff_selftest_bounded_wait.argtypes = [vp, u64, vp]
    lib.ff_plan_wgrad.argtypes = [C.POINTER(ff_layer_desc), i32, i32, i32, u64, C.POINTER(ff_wgrad_plan)]
    lib.ff_predict.argtypes = [vp, C.POINTER(ff_layer_desc), C.POINTER(ff_layer_bufs), i32, i32, i32, i32, vp, vp, u64, vp]
    lib.ff_loss_coef_static.argtypes = [vp, f32, C.POINTER(vp), C.POINTER(f32), i32, f32, i32, vp, vp, vp, vp, vp,
                                        C.c_char_p, C.c_size_t]
    lib.ff_profile_stop.argtypes = [vp, vp, C.POINTER(f32), C.POINTER(C.c_uint32)]
    for name in EXPORTS:
        if name not in ("ff_last_error", "ff_launch_count", "ff_graph_replay_count", "ff_dp_phase_count"):
            getattr(lib, name).restype = i32
    _lib = lib
    return lib


def _check(ctx, code: int):
    if code != FF_OK:
        msg = load().ff_last_error(ctx).decode() if ctx else ""
        raise FFError(code, msg)


def ff_create(device: int = 0):
    ctx = C.c_void_p()
    code = load().ff_create(C.byref(ctx), device)
    if code != FF_OK:
        raise FFError(code, "ff_create failed")
    return ctx


def ff_destroy(ctx):
    load().ff_destroy(ctx)


def ff_workspace_bytes(descs: Sequence[ff_layer_desc], B: int) -> int:
    arr = (ff_layer_desc * len(descs))(*descs)
    out = C.c_size_t()
    _check(None, load().ff_workspace_bytes(arr, len(descs), B, C.byref(out)))
    return out.value


def ff_set_workspace(ctx, dev_ptr: int, nbytes: int):
    _check(ctx, load().ff_set_workspace(ctx, dev_ptr, nbytes))


def ff_set_gemm_path(ctx, path: int):
    _check(ctx, load().ff_set_gemm_path(ctx, path))


def ff_set_tensor_form(ctx, ctas_per_tile: int):
    _check(ctx, load().ff_set_tensor_form(ctx, ctas_per_tile))


def ff_set_graph_mode(ctx, on: bool):
    _check(ctx, load().ff_set_graph_mode(ctx, 1 if on else 0))


def ff_layer_forward(ctx, desc, bufs, B: int, step: int, stream: int = 0):
    _check(ctx, load().ff_layer_forward(ctx, C.byref(desc), C.byref(bufs), B, step, stream))


def ff_layer_loss_grad(ctx, desc, bufs, B: int, G_later: Sequence[int], theta_later: Sequence[float],
                       lam: float, step: int, stream: int = 0):
    n = len(G_later)
    gp = (C.c_void_p * max(n, 1))(*G_later)
    th = (C.c_float * max(n, 1))(*theta_later)
    _check(ctx, load().ff_layer_loss_grad(ctx, C.byref(desc), C.byref(bufs), B, gp, th, n, lam, step, stream))


def ff_layer_update(ctx, desc, bufs, B: int, step: int, stream: int = 0):
    _check(ctx, load().ff_layer_update(ctx, C.byref(desc), C.byref(bufs), B, step, stream))


def ff_train_step(ctx, descs_arr, bufs_arr, n_layers: int, B: int, lam: float, step: int, stream: int = 0):
    """descs_arr / bufs_arr: ctypes arrays (ff_layer_desc * n), (ff_layer_bufs * n)."""
    _check(ctx, load().ff_train_step(ctx, descs_arr, bufs_arr, n_layers, B, lam, step, stream))


def ff_train_step_from(ctx, descs_arr, bufs_arr, n_layers: int, first_trained: int, B: int, lam: float, step: int,
                       stream: int = 0):
    """ff_train_step with the layers before first_trained frozen (forward only)."""
    _check(ctx, load().ff_train_step_from(ctx, descs_arr, bufs_arr, n_layers, first_trained, B, lam, step, stream))


def ff_embed_labels(ctx, x: int, labels: int, B: int, n: int, sets: int, n_classes: int, label_stride: int,
                    on_value: float, tau0: float, eps: float, out: int, stream: int = 0):
    """x / labels / out are device addresses (see include/ffint8.h)."""
    _check(ctx, load().ff_embed_labels(ctx, x, labels, B, n, sets, n_classes, label_stride, on_value, tau0, eps, out,
                                       stream))


def ff_dp_phase_count(n_layers: int) -> int:
    return int(load().ff_dp_phase_count(n_layers))


def ff_dp_train_phase(ctx, descs_arr, bufs_arr, n_layers: int, B_local: int, B_total: int, row_offset: int, phase: int,
                      lam: float, step: int, stream: int = 0):
    """One phase of the data-parallel step.  Returns the arrays to combine over the shards before the
    next phase as a list of (device address, element count, FF_DP_F32 | FF_DP_I32, FF_DP_MAX | FF_DP_SUM, first phase
    that reads the combined array)."""
    red = (ff_dp_reduce * FF_DP_MAX_REDUCE)()
    n = C.c_int(0)
    _check(ctx, load().ff_dp_train_phase(ctx, descs_arr, bufs_arr, n_layers, B_local, B_total, row_offset, phase, lam,
                                         step, stream, red, C.byref(n)))
    return [(int(red[i].dev_ptr), int(red[i].count), int(red[i].dtype), int(red[i].op), int(red[i].needed_by_phase))
            for i in range(n.value)]


def ff_predict(ctx, descs_arr, bufs_arr, n_layers: int, B: int, n_classes: int, first_counted_layer: int, scores: int,
               pred: int, step: int, stream: int = 0):
    """descs_arr / bufs_arr as for ff_train_step; scores / pred are device addresses."""
    _check(ctx, load().ff_predict(ctx, descs_arr, bufs_arr, n_layers, B, n_classes, first_counted_layer, scores, pred,
                                  step, stream))


def ff_poll_status(ctx, stream: int = 0):
    _check(ctx, load().ff_poll_status(ctx, stream))


def ff_plan_wgrad(desc, B: int, sm_count: int, route: int, workspace_bytes: int = 1 << 62):
    """Host arithmetic only (no device): (status code, ff_wgrad_plan)."""
    out = ff_wgrad_plan()
    code = load().ff_plan_wgrad(C.byref(desc), B, sm_count, route, workspace_bytes, C.byref(out))
    return code, out


def ff_selftest_bounded_wait(ctx, limit_ns: int, stream: int = 0):
    _check(ctx, load().ff_selftest_bounded_wait(ctx, limit_ns, stream))


def ff_launch_count(ctx) -> int:
    return int(load().ff_launch_count(ctx))


def ff_last_error(ctx) -> str:
    return load().ff_last_error(ctx).decode()


def ff_graph_replay_count(ctx) -> int:
    return int(load().ff_graph_replay_count(ctx))


def ff_profile_start(ctx):
    _check(ctx, load().ff_profile_start(ctx))


def ff_profile_stop(ctx, stream: int = 0):
    """Returns {kernel kind: (total ms, launches)} for the kinds that were launched."""
    n = len(FF_K_NAMES)
    ms = (C.c_float * n)()
    cnt = (C.c_uint32 * n)()
    _check(ctx, load().ff_profile_stop(ctx, stream, ms, cnt))
    return {FF_K_NAMES[i]: (float(ms[i]), int(cnt[i])) for i in range(n) if cnt[i]}


def ff_loss_coef_static(G: int, theta: float, G_later: Sequence[int], theta_later: Sequence[float], lam: float, B: int,
                        rowmax: int, absmax: int, coef: int, loss: int, stream: int = 0):
    """Loss / coefficient step with the library's built-in scratch array: needs no context and no
    workspace and allocates nothing (for callers that cannot allocate device memory).  Arguments
    are device addresses on the current device."""
    n = len(G_later)
    gp = (C.c_void_p * max(n, 1))(*G_later)
    th = (C.c_float * max(n, 1))(*theta_later)
    buf = C.create_string_buffer(256)
    code = load().ff_loss_coef_static(G, theta, gp, th, n, lam, B, rowmax, absmax, coef, loss, stream, buf, len(buf))
    if code != FF_OK:
        raise FFError(code, buf.value.decode())


def ff_int8_gemm(ctx, A: int, B: int, Cptr: int, M: int, N: int, K: int, trans: int, stream: int = 0):
    _check(ctx, load().ff_int8_gemm(ctx, A, B, Cptr, M, N, K, trans, stream))


# --------------------------------------------------------------------------------------------
# Convenience: device buffers for a stack of layers (torch is used for allocation only)
# --------------------------------------------------------------------------------------------
def make_desc(cfg, index: int, seed: int, round_x=FF_ROUND_STOCHASTIC, round_w=FF_ROUND_NEAREST_EVEN,
              round_dh=FF_ROUND_STOCHASTIC) -> ff_layer_desc:
    """cfg: an object with kind, K, N, H, Wd, Cin, theta, lr, tau, eps (e.g. synth.LayerCfg)."""
    return ff_layer_desc(cfg.kind, cfg.K, cfg.N, cfg.H, cfg.Wd, cfg.Cin, index, round_x, round_w, round_dh,
                         cfg.theta, cfg.lr, cfg.tau, cfg.eps, seed, getattr(cfg, "stride", 1), getattr(cfg, "momentum", 0.0),
                         getattr(cfg, "optimizer", 0), getattr(cfg, "beta2", 0.999), getattr(cfg, "adam_eps", 1e-8),
                         getattr(cfg, "pool", 1), getattr(cfg, "skip_scale", 1.0))


class LayerBuffers:
    """Torch-allocated device tensors of one layer plus the ff_layer_bufs struct pointing at them."""

    def __init__(self, desc: ff_layer_desc, B: int, device, dumps: bool = False, xnext: bool = True,
                 own_x: bool = True, accw: bool = False, pad_rows: bool = True):
        """pad_rows: give the INT8 tensors Xq / dHq of a linear layer whose row length is not a multiple of 128 a
        row pitch that is (the contractions' TMA box rows are then aligned); .Xq / .dHq stay [rows, K] / [rows, N]
        views of the padded storage."""
        import torch
        st = 2 if (desc.kind in (FF_CONV3X3, FF_DWCONV3X3) and desc.stride == 2) else 1
        Rin = desc.H * desc.Wd if desc.kind != FF_LINEAR else 1                    # input rows per sample
        R = ((desc.H - 1) // st + 1) * ((desc.Wd - 1) // st + 1) if desc.kind != FF_LINEAR else 1   # output rows
        kin = desc.Cin if desc.kind != FF_LINEAR else desc.K
        rows, rows_in = 2 * B * R, 2 * B * Rin
        z = lambda shape, dt: torch.zeros(shape, dtype=dt, device=device)
        self.W = z((desc.N, desc.K), torch.float32)
        self.X = z((rows_in, kin), torch.float32) if own_x else None
        self.Y = z((rows, desc.N), torch.float32)
        self.G = z((2 * B,), torch.float32)
        self.Xnext = z((rows // 4 if desc.pool == 2 else rows, desc.N), torch.float32) if xnext else None
        pad = lambda n: (n + 127) // 128 * 128 if (pad_rows and desc.kind == FF_LINEAR and n % 128 and n >= 256) else n
        self.ld_xq, self.ld_dhq = pad(kin), pad(desc.N)
        self._Xq_store, self._dHq_store = z((rows_in, self.ld_xq), torch.int8), z((rows, self.ld_dhq), torch.int8)
        self.Xq, self.dHq = self._Xq_store[:, :kin], self._dHq_store[:, :desc.N]
        self.Wq = z((desc.N, desc.K), torch.int8)
        self.absmax = z((FF_ABSMAX_LEN,), torch.float32)
        self.S = z((2 * B,), torch.int64)
        self.rowmax = z((2 * B,), torch.int32)
        self.coef = z((2 * B,), torch.float32)
        self.loss = z((4,), torch.float32)
        self.acc_dump = z((rows, desc.N), torch.int32) if dumps else None
        self.accW_dump = z((2, desc.N, desc.K), torch.int32) if (dumps or accw) else None
        self.Mom = z((desc.N, desc.K), torch.float32) if (desc.momentum != 0.0 or desc.optimizer == FF_OPT_ADAM) else None
        self.Var = z((desc.N, desc.K), torch.float32) if desc.optimizer == FF_OPT_ADAM else None
        p = lambda t: t.data_ptr() if t is not None else None
        self.struct = ff_layer_bufs(p(self.W), p(self.X), p(self.Y), p(self.G), p(self.Xnext), p(self.Xq),
                                    p(self.Wq), p(self.dHq), p(self.absmax), p(self.S), p(self.rowmax),
                                    p(self.coef), p(self.loss), p(self.acc_dump), p(self.accW_dump), p(self.Mom), p(self.Var),
                                    None, self.ld_xq if self.ld_xq != kin else 0, self.ld_dhq if self.ld_dhq != desc.N else 0)


class Context:
    """ff_ctx plus a torch-allocated workspace."""

    def __init__(self, descs: Sequence[ff_layer_desc], B: int, device_index: int = 0):
        import torch
        self.ctx = ff_create(device_index)
        n = ff_workspace_bytes(descs, B)
        self.workspace = torch.zeros(max(n, 256), dtype=torch.uint8, device=f"cuda:{device_index}")
        ff_set_workspace(self.ctx, self.workspace.data_ptr(), self.workspace.numel())

    def close(self):
        if self.ctx is not None:
            ff_destroy(self.ctx)
            self.ctx = None
