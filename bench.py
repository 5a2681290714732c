#!/usr/bin/env python
"""Benchmark of the FF-INT8 train step (Sec. IV-B / Alg. 1 of the FF-INT8 paper) on B200.

    python bench.py --gpus N --steps K --warmup W [--workload roofline] [--impl reference]

A step is one pass of the whole hot path (quantise -> INT8 GEMM -> goodness -> loss -> dH ->
quantise -> INT8 dW GEMM -> update) over one batch of seeded synthetic input.  The default
workload is the largest single-GPU configuration ("roofline": one 8192 -> 8192 FF layer,
16384 positive + 16384 negative samples), the one the GEMM-roofline target is quoted on.
Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank trains its own replica on its own
batches (no data-path collective: weak scaling); the time is the maximum over ranks.

--impl reference times the CPU oracle (oracle/) on the host cores on a bounded sample of the
same workload; it is a deliberately plain program, not a target.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2506_22771_b200 import synth  # noqa: E402

METRIC = "FF-INT8 train samples/s"
UNIT = "samples/s"
INT8_TO_BF16 = 2.0          # nominal dense tensor ratio (4.5 : 2.25 PFLOP/s)
BURST_SECONDS = 2.0         # timed regions shorter than this are compared with the burst GEMM peak

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from one ncu capture of the
# roofline workload at its full size.  They are reported only while the kernel source is the one that
# was profiled (hash below) and the workload matches; otherwise the key is null.
NCU_TRAFFIC = {
    "source": "paper_2506_22771_b200/csrc/gemm_tc.cuh",
    "sha256": "eaf84a93e525880e0bbfee3cd5fd52077da6694dcbb03a57deb5dee0f41fadba",
    "workload": "roofline", "B": 16384,
    "bytes_per_launch": {"fwd_gemm": 2058.7e6, "upd_gemm": 2868.2e6},
}


def _ncu_traffic(kind: str, workload: str, B: int):
    import hashlib
    t = NCU_TRAFFIC
    try:
        sha = hashlib.sha256(open(os.path.join(ROOT, t["source"]), "rb").read()).hexdigest()
    except OSError:
        return None
    if sha != t["sha256"] or workload != t["workload"] or B != t["B"]:
        return None
    return t["bytes_per_launch"].get(kind)


def _library_int8_gemm(w, B: int, dev):
    """Context for the contraction figures: the vendor library's INT8 GEMM (torch._int_mm -> cuBLASLt) on the shape of
    the last layer's forward contraction, timed with CUDA events right after the bench's own timed regions (so at
    about the same power state; a 20-launch burst all the same).  Not part of the product path."""
    import torch
    l = w.layers[-1]
    M, N, K = 2 * B * l.H * l.Wd, l.N, l.K
    if l.kind != 0 or M % 8 or N % 8 or K % 8 or M * N * 4 > 8e9:
        return None
    try:
        a = torch.randint(-127, 128, (M, K), dtype=torch.int8, device=dev)
        bt = torch.randint(-127, 128, (N, K), dtype=torch.int8, device=dev).t()
        for _ in range(3):
            torch._int_mm(a, bt)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n = 20
        e0.record()
        for _ in range(n):
            torch._int_mm(a, bt)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / n
        return {"shape": [M, N, K], "ms": ms, "tops": 2.0 * M * N * K / (ms * 1e-3) / 1e12,
                "note": "torch._int_mm (cuBLASLt), INT32 output, no epilogue; for comparison only"}
    except Exception as e:  # the comparison is optional
        return {"unavailable": str(e)[:200]}


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_burst": d["bf16_tflops"], "bf16_sustained": d["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t_begin=None, t_end=None):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                pass
        return self.window(t_begin, t_end)

    def window(self, t_begin=None, t_end=None):
        """Statistics of the samples taken between two host times (None: all samples)."""
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for t, r in self.rows:
            if t_begin is not None and not (t_begin <= t <= t_end + 0.05):
                continue
            f = [x.strip() for x in r.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                smax.append(float(f[1]))
                power.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def whole_job_throughput(ms_local: float, units_local: float, device=None):
    """(max over ranks of the local time, units of all ranks / that time).  Uses the default
    process group when one is initialised (NCCL on GPUs, gloo in the CPU tests)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return ms_local, units_local / (ms_local * 1e-3)
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    u = torch.tensor([units_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item()) / (float(t.item()) * 1e-3)


def algorithmic_work(w, B: int):
    """Algorithmic bytes (memory-bound kernels) and INT8 ops (contractions) of ONE train step, per
    kernel kind, from the layer shapes: absmax reads 4 B/element, the quantisers read 4 B and write
    1 B per element, a contraction does 2*rows*N*K operations."""
    out = {k: 0.0 for k in ("absmax", "quantize", "normalize", "dh_quantize", "fwd_gemm", "upd_gemm", "dw_fwd", "dw_upd")}
    for i, l in enumerate(w.layers):
        st = getattr(l, "stride", 1) if l.kind in (1, 3) else 1
        rows = 2 * B * ((l.H - 1) // st + 1) * ((l.Wd - 1) // st + 1)      # output positions of both sets
        kin = l.Cin if l.kind in (1, 3) else l.K
        n_w = l.N * l.K
        n_x = 2 * B * l.H * l.Wd * kin
        n_y = rows * l.N
        out["absmax"] += 4.0 * n_w + (4.0 * n_x if i == 0 else 0.0)
        out["quantize"] += 5.0 * n_w + (5.0 * n_x if i == 0 else 0.0)
        if i + 1 < len(w.layers):
            out["normalize"] += 5.0 * n_y            # reads Y, writes the next layer's INT8 input
        out["dh_quantize"] += 5.0 * n_y
        if l.kind == 3:       # depthwise: streaming kernels, bytes not operations
            out["dw_fwd"] += 1.0 * n_x + 4.0 * n_y
            out["dw_upd"] += 1.0 * n_x + 1.0 * n_y
            continue
        out["fwd_gemm"] += 2.0 * rows * l.N * l.K
        out["upd_gemm"] += 2.0 * rows * l.N * l.K
    return out


def layer_bounds(w, B: int, int8_tops: float, hbm_gbs: float, layers=None):
    """Lower bounds on the time of one step's contractions, per kernel kind, in seconds.  A contraction is bounded
    by the tensor pipe (2*rows*N*K operations at the INT8 peak) AND by HBM (its algorithmic bytes: INT8 operands
    read once, FP32 output written once; the weight gradient reads both INT8 operands of both sets and reads and
    writes the FP32 weights): per layer the larger of the two counts, and the layers add up."""
    out = {}
    for k in ("fwd_gemm", "upd_gemm"):
        out[k] = {"tensor_s": 0.0, "hbm_s": 0.0, "bound_s": 0.0}
    for l in (w.layers if layers is None else layers):
        if l.kind == 3:
            continue
        st = getattr(l, "stride", 1) if l.kind == 1 else 1
        rows = 2 * B * ((l.H - 1) // st + 1) * ((l.Wd - 1) // st + 1)
        kin = l.Cin if l.kind == 1 else l.K
        n_x, n_w, n_y = 2 * B * l.H * l.Wd * kin, l.N * l.K, rows * l.N
        ops = 2.0 * rows * l.N * l.K
        for k, nbytes in (("fwd_gemm", n_x + n_w + 4.0 * n_y), ("upd_gemm", n_y + n_x + 8.0 * n_w)):
            t_t, t_h = ops / (int8_tops * 1e12), nbytes / (hbm_gbs * 1e9)
            out[k]["tensor_s"] += t_t
            out[k]["hbm_s"] += t_h
            out[k]["bound_s"] += max(t_t, t_h)
    return out


def kernel_table(w, B: int, kernel_ms: dict, steps: int, ms_profiled: float, peaks: dict, int8_peak: float, work=None,
                 bounds=None):
    """Per kernel kind: time per step, share, achieved rate against its roofline.  Contractions also carry the
    bound that holds layer by layer (max of tensor time and HBM time) and the fraction of it that was reached."""
    work = work or algorithmic_work(w, B)
    bounds = bounds or layer_bounds(w, B, int8_peak, peaks["hbm_gbs"])
    out = {}
    for k, (tot_ms, n) in kernel_ms.items():
        ent = {"launches_per_step": n / steps, "ms_per_step": tot_ms / steps, "share": tot_ms / ms_profiled}
        if k in work and work[k] > 0 and tot_ms > 0:
            rate = work[k] * steps / (tot_ms * 1e-3)
            if k.endswith("gemm"):
                b = bounds[k]
                ent.update(bound="tensor" if b["tensor_s"] >= b["hbm_s"] else "hbm", achieved=rate / 1e12, unit="TOP/s",
                           frac=rate / 1e12 / int8_peak, tensor_bound_ms=b["tensor_s"] * 1e3, hbm_bound_ms=b["hbm_s"] * 1e3,
                           layerwise_bound_ms=b["bound_s"] * 1e3, frac_of_layerwise_bound=b["bound_s"] * 1e3 / (tot_ms / steps))
            else:
                ent.update(bound="hbm", achieved=rate / 1e9, unit="GB/s", frac=rate / 1e9 / peaks["hbm_gbs"])
        out[k] = ent
    return out


def greedy_work(w, B: int):
    """Algorithmic work of ONE layer-step of the layer-by-layer epoch, averaged over the phases: phase l runs the
    forward of layers 0..l and the loss / gradient / update of layer l alone."""
    n = len(w.layers)
    tot = {k: 0.0 for k in algorithmic_work(w, B)}
    bounds = None
    for l in range(n):
        sub = type(w)(w.name, w.B, w.layers[:l + 1], w.in_shape, w.data, w.weights, w.steps)
        full = algorithmic_work(sub, B)
        last = algorithmic_work(type(w)(w.name, w.B, [w.layers[l]], w.in_shape, w.data, w.weights, w.steps), B)
        for k in tot:
            tot[k] += last[k] if k in ("dh_quantize", "upd_gemm", "dw_upd") else full[k]
    return {k: v / n for k, v in tot.items()}


def _oracle_step_time(w, B_sample: int, steps: int, seed: int = 1):
    """Time the CPU oracle, as it stands, on a bounded sample (B_sample positives + negatives)."""
    from oracle import ffint8_oracle as O
    specs = [O.LayerSpec(l.kind, l.K, l.N, l.theta, l.lr, l.tau, l.eps, l.H, l.Wd, l.Cin, seed=seed, index=i,
                         stride=l.stride) for i, l in enumerate(w.layers)]
    Ws = synth.make_weights(w, seed)
    X = synth.make_batch(w, seed, B=B_sample)
    times = []
    for s in range(steps):
        if w.greedy:    # a step of the layer-by-layer workload is one layer-step: the average over the phases is timed
            t0 = time.perf_counter()
            for l in range(len(specs)):
                st = O.train_step(specs[:l + 1], Ws[:l + 1], X, B_sample, 0.0, s, first_trained=l)
                Ws[l] = st[l].W_new
            times.append((time.perf_counter() - t0) / len(specs))
            continue
        t0 = time.perf_counter()
        st = O.train_step(specs, Ws, X, B_sample, w.lam_per_step * s, s)
        times.append(time.perf_counter() - t0)
        Ws = [x.W_new for x in st]
    try:
        from threadpoolctl import threadpool_info
        cores = max([i.get("num_threads", 1) for i in threadpool_info()] or [1])
    except Exception:
        cores = os.cpu_count() or 1
    return float(np.mean(times)), cores


def cpu_baseline_leg(w, B: int, B_sample: int, budget_s: float):
    """The oracle, as it stands, on the host cores.  Two small probes (B_sample and 2*B_sample rows per set, full layer
    widths) give step time = a + b*rows: a is the per-step work on the weights (range, codes, update), b the work per
    row.  When one FULL step of the workload is projected to fit the budget it is run and reported; otherwise the
    larger probe is reported, with the reason and the projection for the full batch (the probe's samples/s spreads
    the weight work over few rows and so understates the oracle on the full batch)."""
    t0 = time.perf_counter()
    b1 = min(B, B_sample)
    t1, cores = _oracle_step_time(w, b1, 1)
    if b1 == B:
        return {"value": B / t1, "unit": UNIT, "cores": cores, "kind": "oracle", "full_step": True,
                "sample": f"one full step: {B} positive + {B} negative samples, full layer widths"}
    b2 = min(B, 2 * b1)
    t2, _ = _oracle_step_time(w, b2, 1)
    slope = max((t2 - t1) / (b2 - b1), 0.0) if b2 > b1 else t2 / b2
    fixed = max(t2 - slope * b2, 0.0)
    t_full = fixed + slope * B
    left = budget_s - (time.perf_counter() - t0)
    if t_full * 1.3 < left:
        tf, cores = _oracle_step_time(w, B, 1)
        return {"value": B / tf, "unit": UNIT, "cores": cores, "kind": "oracle", "full_step": True,
                "sample": f"one full step: {B} positive + {B} negative samples, full layer widths"}
    return {"value": b2 / t2, "unit": UNIT, "cores": cores, "kind": "oracle", "full_step": False,
            "sample": f"{b2} positive + {b2} negative samples, full layer widths, 1 step (a full step of {B} + {B} rows is "
                      f"projected at {t_full:.0f} s, beyond the {budget_s:.0f} s this leg may take)",
            "projected_full_step": {"seconds": t_full, "value": B / t_full,
                                    "fit": f"step seconds = {fixed:.3f} + {slope:.6f} x rows per set, from probes at {b1} and {b2}"}}


def run_reference(args):
    """Reference arm = the CPU oracle, as it stands, on the host cores.  Each step is a bounded sample of the
    workload (--cpu-sample positives + negatives at full layer widths).  `--warmup` untimed and `--steps` timed steps
    are run when they fit --cpu-budget-s seconds (projected from the first step); a step's cost is dominated by
    quantising and updating the full-width weights, which a smaller sample would not reduce, so when they do not
    fit, fewer steps are timed and the line says how many ("steps" = timed, "steps_requested" = asked for)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = synth.workload(args.workload)
    want, warmup = max(1, args.steps), max(1, args.warmup)
    B_sample = min(w.B, args.cpu_sample)
    t_first, _ = _oracle_step_time(w, B_sample, 1)                 # the first warm-up step, also the probe
    afford = max(1, int(args.cpu_budget_s / max(t_first, 1e-6)))    # steps of any kind that fit the budget
    warm_left = min(warmup - 1, max(0, afford - 2))
    steps = min(want, max(1, afford - 1 - warm_left))
    if warm_left:
        _oracle_step_time(w, B_sample, warm_left)
    t, cores = _oracle_step_time(w, B_sample, steps)
    v = B_sample / t
    sample = (f"{B_sample} positive + {B_sample} negative samples of the {args.workload} workload per step, full layer widths "
              f"(the workload has {w.B} + {w.B}; the per-step work on the weights - range, codes, update - is spread over "
              "this sample's rows only, so the figure understates the oracle on the full batch)")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "steps_requested": want, "warmup": 1 + warm_left, "ms_per_step": t * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": args.workload, "B_pos": B_sample, "B_neg": B_sample},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def run_predict(args, w, world, rank, local, dev):
    """Classification by goodness: every sample is forwarded once per candidate label (10 labels); the
    candidate batch has about as many rows as the workload's training batch."""
    import torch
    import torch.distributed as dist
    from paper_2506_22771_b200 import binding as ffb
    n_classes = 10
    Bp = args.B or (2 * w.B) // n_classes
    half = n_classes * Bp // 2
    seed = 1 + rank
    descs = [ffb.make_desc(l, i, seed) for i, l in enumerate(w.layers)]
    ctx = ffb.Context(descs, half, local)
    ffb.ff_set_graph_mode(ctx.ctx, not args.no_graph)
    bufs = [ffb.LayerBuffers(d, half, dev, dumps=False, xnext=False, own_x=(i == 0)) for i, d in enumerate(descs)]
    for b, W in zip(bufs, synth.make_weights(w, seed)):
        b.W.copy_(torch.from_numpy(W))
    Xc, _ = synth.make_candidates(w, seed, Bp, n_classes)
    bufs[0].X.copy_(torch.from_numpy(Xc).reshape(bufs[0].X.shape))
    descs_arr = (ffb.ff_layer_desc * len(descs))(*descs)
    bufs_arr = (ffb.ff_layer_bufs * len(descs))(*[b.struct for b in bufs])
    scores = torch.zeros(n_classes * Bp, dtype=torch.float32, device=dev)
    pred = torch.zeros(Bp, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream().cuda_stream

    def step(i):
        ffb.ff_predict(ctx.ctx, descs_arr, bufs_arr, len(descs), Bp, n_classes, 0, scores.data_ptr(), pred.data_ptr(), i, stream)

    for i in range(args.warmup):
        step(i)
    ffb.ff_poll_status(ctx.ctx, stream)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        step(i)
    e1.record()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    # per-kernel times from a second pass (the event pairs around every launch would distort the figure above)
    ffb.ff_profile_start(ctx.ctx)
    for i in range(args.steps):
        step(i)
    kernel_ms = ffb.ff_profile_stop(ctx.ctx, stream)
    ffb.ff_poll_status(ctx.ctx, stream)
    ms, value = whole_job_throughput(e0.elapsed_time(e1), Bp * args.steps, dev)
    if rank == 0:
        print(json.dumps({
            "metric": "FF-INT8 classified samples/s (10 candidate labels per sample)", "value": value, "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": {"workload": args.workload, "mode": "predict", "samples": Bp, "candidate_rows": n_classes * Bp,
                       "layers": [[x.K, x.N] for x in w.layers],
                       "launch": "kernel by kernel" if args.no_graph else "captured launch sequence"},
            "kernels": {k: {"ms_per_step": t / args.steps, "launches_per_step": n / args.steps}
                        for k, (t, n) in kernel_ms.items()}}))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


class DeviceWorkload:
    """A workload's context, buffers, weights and input batches on one device, with the step the benchmark times:
    ff_train_step on one resident batch, or - for the layer-by-layer workload - the epoch of ff_train_step_from
    calls over its resident batches (phase l trains layer l on the forward of the layers trained before)."""

    def __init__(self, w, B, seed, dev, local, graph=True, tensor_form=0, accw=False):
        import torch
        from paper_2506_22771_b200 import binding as ffb
        self.ffb, self.torch, self.w, self.B = ffb, torch, w, B
        self.descs = [ffb.make_desc(l, i, seed) for i, l in enumerate(w.layers)]
        self.ctx = ffb.Context(self.descs, B, local)
        ffb.ff_set_tensor_form(self.ctx.ctx, tensor_form)
        ffb.ff_set_graph_mode(self.ctx.ctx, graph)
        self.bufs = [ffb.LayerBuffers(d, B, dev, dumps=False, xnext=False, own_x=(i == 0), accw=accw)
                     for i, d in enumerate(self.descs)]
        for b, W in zip(self.bufs, synth.make_weights(w, seed)):
            b.W.copy_(torch.from_numpy(W))
        self.W0 = [b.W.clone() for b in self.bufs]
        self.n = len(self.descs)
        self.descs_arr = (ffb.ff_layer_desc * self.n)(*self.descs)
        self.bufs_arr = (ffb.ff_layer_bufs * self.n)(*[b.struct for b in self.bufs])
        self.stream = torch.cuda.current_stream().cuda_stream
        n_batches = w.steps if w.greedy else 1
        self.batches = [torch.from_numpy(synth.make_batch(w, seed, batch_index=i, B=B)).reshape(self.bufs[0].X.shape).to(dev)
                        for i in range(n_batches)]
        self.bufs[0].X.copy_(self.batches[0])
        self.steps_per_pass = self.n * n_batches if w.greedy else 1      # layer-steps of one epoch

    def reset_weights(self):
        for b, W in zip(self.bufs, self.W0):
            b.W.copy_(W)

    def step(self, i):
        """Step i of the timed sequence (greedy: layer-step i of the epoch, wrapping around)."""
        ffb, w = self.ffb, self.w
        if not w.greedy:
            ffb.ff_train_step(self.ctx.ctx, self.descs_arr, self.bufs_arr, self.n, self.B, w.lam_per_step * i, i, self.stream)
            return
        nb = len(self.batches)
        i %= self.steps_per_pass
        l, k = divmod(i, nb)
        self.bufs[0].X.copy_(self.batches[k], non_blocking=True)       # device-to-device: the batch is resident
        ffb.ff_train_step_from(self.ctx.ctx, self.descs_arr, self.bufs_arr, l + 1, l, self.B, 0.0, i, self.stream)

    def close(self):
        self.ctx.close()


def measure_extra(name, dev, local, peaks, seconds=0.4, graph=True):
    """A short timed run of another workload (device-resident inputs, same timing rules): ms per step and the
    per-kernel table.  For the layer-by-layer workload a step is one layer-step and whole epochs are timed."""
    import torch
    w = synth.workload(name)
    dw = DeviceWorkload(w, w.B, 1, dev, local, graph=graph)
    ffb = dw.ffb
    per = dw.steps_per_pass
    for i in range(max(3, per if w.greedy else 3)):
        dw.step(i)
    ffb.ff_poll_status(dw.ctx.ctx, dw.stream)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(per):
        dw.step(i)
    e1.record()
    torch.cuda.synchronize()
    probe_ms = e0.elapsed_time(e1) / per
    want = max(per, int(seconds * 1e3 / max(probe_ms, 1e-3)) // per * per)
    # a run never goes beyond the number of steps the workload is defined for (the weights of a long run on one
    # batch drift out of range); longer timing = several runs from the initial weights, each timed on the device
    chunk = per if w.greedy else max(3, min(want, w.steps))
    steps, total_ms = 0, 0.0
    while steps < want:
        dw.reset_weights()
        torch.cuda.synchronize()
        e0.record()
        for i in range(chunk):
            dw.step(i)
        e1.record()
        torch.cuda.synchronize()
        total_ms += e0.elapsed_time(e1)
        steps += chunk
    ms = total_ms / steps
    dw.reset_weights()
    ksteps = min(chunk, max(per, 50 // per * per))
    ffb.ff_profile_start(dw.ctx.ctx)
    e0.record()
    for i in range(ksteps):
        dw.step(i)
    e1.record()
    kernel_ms = ffb.ff_profile_stop(dw.ctx.ctx, dw.stream)
    ms_prof = e0.elapsed_time(e1)
    ffb.ff_poll_status(dw.ctx.ctx, dw.stream)
    int8_peak = INT8_TO_BF16 * peaks["bf16_burst"]
    work = greedy_work(w, w.B) if w.greedy else None
    bounds = None
    if w.greedy:       # bounds of the average layer-step
        n = len(w.layers)
        bounds = {k: {kk: 0.0 for kk in ("tensor_s", "hbm_s", "bound_s")} for k in ("fwd_gemm", "upd_gemm")}
        for l in range(n):
            f = layer_bounds(w, w.B, int8_peak, peaks["hbm_gbs"], w.layers[:l + 1])["fwd_gemm"]
            u = layer_bounds(w, w.B, int8_peak, peaks["hbm_gbs"], [w.layers[l]])["upd_gemm"]
            for kk in f:
                bounds["fwd_gemm"][kk] += f[kk] / n
                bounds["upd_gemm"][kk] += u[kk] / n
    out = {"workload": name, "B_pos": w.B, "B_neg": w.B, "steps": steps, "ms_per_step": ms, "samples_per_s": w.B / (ms * 1e-3),
           "launch": "captured launch sequence" if graph else "kernel by kernel",
           "kernels": kernel_table(w, w.B, kernel_ms, ksteps, ms_prof, peaks, int8_peak, work, bounds)}
    if w.greedy:
        out["note"] = (f"one epoch = {len(w.layers)} phases x {len(dw.batches)} batches; a step is one layer-step "
                       "(forward of the trained layers before it + train step of the phase's layer)")
        out["ms_per_epoch"] = ms * per
    dw.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="roofline")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-sample", type=int, default=256, help="positives per step of the CPU-oracle sample")
    ap.add_argument("--cpu-budget-s", type=float, default=210.0,
                    help="--impl reference: seconds of oracle time that all warm-up and timed steps together may take")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-library-gemm", action="store_true", help="skip the cuBLASLt INT8 GEMM timed for comparison")
    ap.add_argument("--B", type=int, default=0, help="override positives per batch (profiling runs on a smaller case)")
    ap.add_argument("--tensor-form", type=int, default=0, help="CTAs per tensor-core tile: 0 auto, 1, 2")
    ap.add_argument("--no-graph", action="store_true",
                    help="launch every kernel of a step one by one instead of replaying the captured launch sequence")
    ap.add_argument("--data-parallel", action="store_true",
                    help="split ONE batch by rows over the ranks (ff_dp_train_phase + NCCL all-reduce between the phases) "
                         "instead of independent replicas; strong scaling, no end-to-end leg")
    ap.add_argument("--sustained-s", type=float, default=2.0,
                    help="when the timed region is shorter than this, a second region of at least this many seconds gives "
                         "value_sustained (0: skip)")
    ap.add_argument("--cpu-baseline-budget-s", type=float, default=45.0,
                    help="seconds the cpu_baseline leg may take: one full step of the workload if it fits, else a sample")
    ap.add_argument("--no-extra", action="store_true", help="skip the short runs of the other workloads")
    ap.add_argument("--predict", action="store_true",
                    help="time classification by goodness (ff_predict, 10 candidate labels) instead of the train step")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    args.warmup = max(args.warmup, 3)

    import torch
    import torch.distributed as dist
    from paper_2506_22771_b200 import binding as ffb

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device(f"cuda:{local}")
    if world > 1 or args.data_parallel:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29533")
        dist.init_process_group("nccl", device_id=dev, rank=rank, world_size=world)

    w = synth.workload(args.workload)
    if args.predict:
        return run_predict(args, w, world, rank, local, dev)
    B = args.B or w.B
    seed = 1 + rank
    dpar = args.data_parallel
    if dpar:
        # one batch of B_total rows per set, this rank holds rows [row_off, row_off + B); identical replicas
        from paper_2506_22771_b200 import data_parallel as dp
        B_total, seed = B, 1
        row_off, B = dp.shard_rows(B_total, world, rank)
        args.no_e2e = args.no_graph = True
    descs = [ffb.make_desc(l, i, seed) for i, l in enumerate(w.layers)]
    ctx = ffb.Context(descs, B, local)
    ffb.ff_set_tensor_form(ctx.ctx, args.tensor_form)
    ffb.ff_set_graph_mode(ctx.ctx, not args.no_graph)
    bufs = [ffb.LayerBuffers(d, B, dev, dumps=False, xnext=False, own_x=(i == 0), accw=dpar) for i, d in enumerate(descs)]
    Ws = synth.make_weights(w, seed)
    for b, W in zip(bufs, Ws):
        b.W.copy_(torch.from_numpy(W))
    if dpar:
        table = dp.PointerTable()
        table.add_layer_buffers(bufs)
        reducer = dp.OverlappedReducer(table, device=dev)   # INT32 sums reduced on a side stream beside later contractions
        X_all = torch.from_numpy(synth.make_batch(w, seed, B=B_total)).reshape(2 * B_total, -1)
        X_host = dp.shard_batch(X_all, B_total, row_off, B).reshape(bufs[0].X.shape).pin_memory()
        del X_all
    else:
        X_host = torch.from_numpy(synth.make_batch(w, seed, B=B)).reshape(bufs[0].X.shape).pin_memory()
    bufs[0].X.copy_(X_host)
    greedy = bool(w.greedy) and not dpar
    # layer-by-layer workload: its batches stay resident on the device; a step is one layer-step of the epoch
    batches = [torch.from_numpy(synth.make_batch(w, seed, batch_index=i, B=B)).reshape(bufs[0].X.shape).to(dev)
               for i in range(w.steps)] if greedy else []
    epoch_steps = len(descs) * len(batches) if greedy else 1
    if greedy and args.steps % epoch_steps:
        args.steps = max(epoch_steps, args.steps // epoch_steps * epoch_steps)   # whole epochs only
    W0 = [b.W.clone() for b in bufs]
    descs_arr = (ffb.ff_layer_desc * len(descs))(*descs)
    bufs_arr = (ffb.ff_layer_bufs * len(descs))(*[b.struct for b in bufs])
    stream = torch.cuda.current_stream().cuda_stream
    n_layers = len(descs)
    last = n_layers - 1

    def step(i):
        if dpar:
            dp.dp_train_step(ctx.ctx, descs_arr, bufs_arr, n_layers, B, B_total, row_off, w.lam_per_step * i, i,
                             reducer, stream)
        elif greedy:
            l, k = divmod(i % epoch_steps, len(batches))
            bufs[0].X.copy_(batches[k], non_blocking=True)
            ffb.ff_train_step_from(ctx.ctx, descs_arr, bufs_arr, l + 1, l, B, 0.0, i % epoch_steps, stream)
        else:
            ffb.ff_train_step(ctx.ctx, descs_arr, bufs_arr, n_layers, B, w.lam_per_step * i, i, stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def reset_weights():
        for b, W in zip(bufs, W0):
            b.W.copy_(W)

    # ---------------- device-resident timing (value) ----------------
    for i in range(max(args.warmup, epoch_steps if greedy else 0)):   # (layer-by-layer: every phase's launch sequence once)
        step(i)
    ffb.ff_poll_status(ctx.ctx, stream)
    reset_weights()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier()
    l0 = ffb.ff_launch_count(ctx.ctx)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_begin = time.time()
    e0.record()
    for i in range(args.steps):
        step(i)
    e1.record()
    barrier()
    t_value_end = time.time()
    launches = ffb.ff_launch_count(ctx.ctx) - l0
    ms_local = e0.elapsed_time(e1)
    ffb.ff_poll_status(ctx.ctx, stream)
    loss_last = float(bufs[last].loss[0].item())
    ms, value = whole_job_throughput(ms_local, B * args.steps, dev)

    # ---------------- the same K steps again with a CUDA-event pair around every kernel ----------------
    # (a second region, so that the events' cost stays out of `value`; same steps, same state of the device)
    reset_weights()
    barrier()
    t_prof_begin = time.time()
    ffb.ff_profile_start(ctx.ctx)
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2.record()
    for i in range(args.steps):
        step(i)
    e3.record()
    barrier()
    t_end = time.time()
    kernel_ms = ffb.ff_profile_stop(ctx.ctx, stream)
    ms_profiled = e2.elapsed_time(e3)
    ffb.ff_poll_status(ctx.ctx, stream)

    # ---------------- a region long enough for the power cap to settle (value_sustained) ----------------
    # The K-step region above may last a fraction of a second: the clocks are then those of a burst.  This one runs
    # the same steps for at least --sustained-s seconds; its second half alone is timed as well.
    sustained = None
    if args.sustained_s > 0 and ms * 1e-3 < args.sustained_s and not dpar:
        per = ms / args.steps
        n_s = int(np.ceil(args.sustained_s * 1e3 / per))
        n_s = max(2, (n_s + epoch_steps - 1) // epoch_steps * epoch_steps)
        half = n_s // 2 // epoch_steps * epoch_steps or n_s // 2
        reset_weights()
        barrier()
        es = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        t_s0 = time.time()
        es[0].record()
        period = epoch_steps if greedy else max(1, w.steps)   # the run the workload is defined for, repeated from the
        for i in range(n_s):                                   # initial weights (a longer run on one batch drifts out of range)
            if i == half:
                es[1].record()
            if i and i % period == 0:
                reset_weights()
            step(i % period)
        es[2].record()
        barrier()
        t_s1 = time.time()
        ffb.ff_poll_status(ctx.ctx, stream)
        ms_s, value_s = whole_job_throughput(es[0].elapsed_time(es[2]), B * n_s, dev)
        ms_h, value_h = whole_job_throughput(es[1].elapsed_time(es[2]), B * (n_s - half), dev)
        sustained = {"steps": n_s, "seconds": ms_s * 1e-3, "ms_per_step": ms_s / n_s, "value": value_s,
                     "ms_per_step_second_half": ms_h / (n_s - half), "value_second_half": value_h,
                     "window": (t_s0, t_s1)}
    if rank == 0:
        time.sleep(0.1)
        clocks = sampler.stop(t_begin, t_end)
        clocks["regions"] = {"value": sampler.window(t_begin, t_value_end), "per_kernel": sampler.window(t_prof_begin, t_end)}
        if sustained:
            clocks["regions"]["sustained"] = sampler.window(*sustained["window"])
        for name, reg in clocks["regions"].items():      # time x clock: what the region would take at 1 MHz, for comparisons
            per_step = {"value": ms / args.steps, "per_kernel": ms_profiled / args.steps,
                        "sustained": sustained["ms_per_step"] if sustained else None}[name]
            reg["ms_per_step_x_sm_mhz"] = per_step * reg["sm_mhz"] if reg.get("sm_mhz") else None
    else:
        clocks = None
    if sustained:
        sustained.pop("window")

    # the vendor library's INT8 GEMM of the same shape, right after the timed regions (same power state)
    lib_gemm = _library_int8_gemm(w, B, dev) if (world == 1 and rank == 0 and not args.no_library_gemm) else None

    # ---------------- end to end: host buffers, H2D of the step's inputs + D2H of the loss every step ---------
    # What crosses PCIe per step is what a trainer holds on the host: the B labelled samples (FP32) and their
    # true / wrong labels.  The positive / negative batch is built from them on the device (ff_embed_labels),
    # which halves the copy against shipping the finished batch.  The samples of step i+1 are copied (pinned
    # host -> second device buffer, copy stream) while step i computes; every step still waits for its own
    # samples and its loss is read back to the host.
    e2e = None
    if not args.no_e2e:
        reset_weights()
        # one set of labelled samples per distinct batch of the workload (one, or the epoch's batches)
        raws = [synth.make_raw(w, seed, batch_index=i, B=B) for i in range(len(batches) if greedy else 1)]
        label_stride = raws[0][2]
        n_in = raws[0][0].shape[1]
        raw_hosts = [torch.from_numpy(r[0]).pin_memory() for r in raws]
        labels_hosts = [torch.from_numpy(r[1]).pin_memory() for r in raws]
        raw_host, labels_host = raw_hosts[0], labels_hosts[0]
        raw_dev = [torch.empty_like(raw_host, device=dev) for _ in range(2)]
        labels_dev = [torch.empty_like(labels_host, device=dev) for _ in range(2)]
        loss_host = torch.zeros(4, dtype=torch.float32).pin_memory()
        n_e2e = epoch_steps if greedy else max(3, min(args.steps, 10))
        tau0 = float(np.sqrt(n_in))

        def e2e_step(k, i):
            ffb.ff_embed_labels(ctx.ctx, raw_dev[k].data_ptr(), labels_dev[k].data_ptr(), B, n_in, 2, 10, label_stride, 1.0,
                                tau0, 1e-8, bufs[0].X.data_ptr(), stream)
            if greedy:
                l = (i % epoch_steps) // len(batches)
                ffb.ff_train_step_from(ctx.ctx, descs_arr, bufs_arr, l + 1, l, B, 0.0, i % epoch_steps, stream)
                return l
            ffb.ff_train_step(ctx.ctx, descs_arr, bufs_arr, n_layers, B, w.lam_per_step * i, i, stream)
            return last

        for k in (0, 1):           # untimed: both buffer sets hold data, the launch sequence is in its steady form
            raw_dev[k].copy_(raw_host)
            labels_dev[k].copy_(labels_host)
            e2e_step(k, k)
        reset_weights()
        copy_stream = torch.cuda.Stream()
        main = torch.cuda.current_stream()
        ready = [torch.cuda.Event(), torch.cuda.Event()]     # samples landed in raw_dev[k]
        freed = [torch.cuda.Event(), torch.cuda.Event()]     # the step reading raw_dev[k] has finished

        def h2d(k, i):             # the samples of step i: batch (i mod batches)
            j = (i % epoch_steps) % len(raw_hosts)
            raw_dev[k].copy_(raw_hosts[j], non_blocking=True)
            labels_dev[k].copy_(labels_hosts[j], non_blocking=True)
            ready[k].record(copy_stream)

        barrier()
        e0.record()
        with torch.cuda.stream(copy_stream):
            h2d(0, 0)
        for i in range(n_e2e):
            k = i & 1
            if i + 1 < n_e2e:
                with torch.cuda.stream(copy_stream):
                    if i >= 1:
                        copy_stream.wait_event(freed[k ^ 1])
                    h2d(k ^ 1, i + 1)
            main.wait_event(ready[k])
            trained = e2e_step(k, i)
            freed[k].record(main)
            loss_host.copy_(bufs[trained].loss, non_blocking=True)
            main.synchronize()
        e1.record()
        barrier()
        _, e2e_value = whole_job_throughput(e0.elapsed_time(e1), B * n_e2e, dev)
        e2e = {"value": e2e_value, "unit": UNIT,
               "h2d_bytes_per_step": int(raw_host.numel() * 4 + labels_host.numel() * 4),
               "d2h_bytes_per_step": 16, "steps": n_e2e,
               "note": "labelled FP32 samples cross PCIe, the positive / negative batch is built on the device; "
                       "the next step's copy overlaps the current step"}
        del raw_dev

    if rank == 0:
        peaks = _peaks()
        burst = (ms + ms_profiled) * 1e-3 < BURST_SECONDS
        bf16 = peaks["bf16_burst"] if burst else peaks["bf16_sustained"]
        int8_peak = INT8_TO_BF16 * bf16
        g_work = g_bounds = None
        if greedy:                      # work and bounds of the average layer-step of the epoch
            g_work = greedy_work(w, B)
            g_bounds = {k: {kk: 0.0 for kk in ("tensor_s", "hbm_s", "bound_s")} for k in ("fwd_gemm", "upd_gemm")}
            for li in range(n_layers):
                f = layer_bounds(w, B, int8_peak, peaks["hbm_gbs"], w.layers[:li + 1])["fwd_gemm"]
                u = layer_bounds(w, B, int8_peak, peaks["hbm_gbs"], [w.layers[li]])["upd_gemm"]
                for kk in f:
                    g_bounds["fwd_gemm"][kk] += f[kk] / n_layers
                    g_bounds["upd_gemm"][kk] += u[kk] / n_layers
        per_kernel = kernel_table(w, B, kernel_ms, args.steps, ms_profiled, peaks, int8_peak, g_work, g_bounds)
        gemms = [k for k in ("fwd_gemm", "upd_gemm") if k in per_kernel]
        dom = max(gemms, key=lambda k: per_kernel[k]["ms_per_step"])
        names = {"fwd_gemm": "tc_gemm_kernel<FWD> (forward INT8 GEMM + dequant/ReLU/goodness epilogue)",
                 "upd_gemm": "tc_gemm_kernel<UPD> (INT8 dW GEMM of both sets + SGD epilogue)"}
        l = w.layers[-1]
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "strong" if dpar else "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": {"workload": args.workload, "B_pos": B, "B_neg": B,
                       "layers": [[x.K, x.N] for x in w.layers],
                       "parallelism": f"one batch of {B_total} + {B_total} rows split over {world} rank(s), all-reduce of "
                                      "ranges, loss and INT32 weight-gradient sums between phases" if dpar else
                                      "independent replicas",
                       "launch": "kernel by kernel" if args.no_graph else
                       f"captured launch sequence, {ffb.ff_graph_replay_count(ctx.ctx)} graph replays in this run",
                       "l2": "inputs larger than L2 (no flush needed)"
                       if 2 * B * l.H * l.Wd * l.K * 4 > 126e6 else "inputs smaller than L2, not flushed"},
            "clocks": clocks, "gpu_launches": int(launches), "e2e": e2e, "loss_last": loss_last,
            "ms_per_step_with_kernel_events": ms_profiled / args.steps,
            "roofline": {"bound": per_kernel[dom]["bound"], "kernel": names[dom], "achieved": per_kernel[dom]["achieved"],
                         "peak": int8_peak, "unit": "TOP/s", "frac": per_kernel[dom]["frac"],
                         "regime": "burst" if burst else "sustained",
                         "peak_source": f"{INT8_TO_BF16:g} x {peaks['source']} bf16 cuBLAS "
                                        f"{'burst' if burst else 'sustained'} ({bf16} TF/s): the two timed regions lasted "
                                        f"{(ms + ms_profiled) * 1e-3:.2f} s",
                         "frac_of_measured_burst_x2": per_kernel[dom]["achieved"] / (INT8_TO_BF16 * peaks["bf16_burst"]),
                         "frac_of_measured_sustained_x2": per_kernel[dom]["achieved"] / (INT8_TO_BF16 * peaks["bf16_sustained"]),
                         "frac_of_nominal_4500": per_kernel[dom]["achieved"] / 4500.0,
                         "layerwise_bound_ms": per_kernel[dom]["layerwise_bound_ms"],
                         "frac_of_layerwise_bound": per_kernel[dom]["frac_of_layerwise_bound"],
                         "traffic": _ncu_traffic(dom, args.workload, B)},
            "kernels": per_kernel,
            "rows_per_s": 2.0 * value,
        }
        if greedy:
            out["config"]["schedule"] = (f"layer by layer: {n_layers} phases x {len(batches)} distinct batches, phase l trains "
                                         "layer l on the INT8 forward of the layers trained before; a step is one layer-step")
            out["ms_per_epoch"] = ms / args.steps * epoch_steps
        if sustained:
            # the same steps over a region long enough for the power cap to settle; the contraction rates are scaled by
            # the step-time ratio (the step is >= 85 % contractions at the roofline workload)
            out["value_sustained"] = sustained["value"]
            ratio = (ms / args.steps) / sustained["ms_per_step_second_half"]
            sustained["dominant_kernel_tops_scaled"] = per_kernel[dom]["achieved"] * ratio
            sustained["dominant_kernel_frac_of_nominal_4500_scaled"] = per_kernel[dom]["achieved"] * ratio / 4500.0
            out["sustained"] = sustained
        if lib_gemm is not None:
            out["library_int8_gemm"] = lib_gemm
    ctx.close()
    if rank == 0:
        del bufs, batches, W0
        torch.cuda.empty_cache()
        if world == 1 and not args.no_extra and not dpar:
            # the other paper-shaped workloads, a few hundred milliseconds each, so that their figures are measured by
            # the same run: ms per step and every kernel against its roofline
            others = {}
            for name in ("mlp_greedy", "mlp_lookahead", "cnn"):
                if name != args.workload:
                    try:
                        others[name] = measure_extra(name, dev, local, peaks, graph=not args.no_graph)
                    except Exception as e:   # an extra must not lose the main line
                        others[name] = {"unavailable": str(e)[:200]}
            out["other_workloads"] = others
        if not args.no_cpu_baseline and world == 1:
            out["cpu_baseline"] = cpu_baseline_leg(w, B, args.cpu_sample, args.cpu_baseline_budget_s)
        print(json.dumps(out))
    if world > 1 or args.data_parallel:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
