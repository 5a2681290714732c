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
# roofline workload at its full size (profiles/tc_gemm_kernel_roofline_layer.md).  They are reported
# only while the kernel source is the one that was profiled (hash below) and the workload matches.
NCU_TRAFFIC = {
    "source": "paper_2506_22771_b200/csrc/gemm_tc.cuh",
    "sha256": "519324433b4262903f19bc68415dd4d0d3f1446dcaff9f0a18bfbbd486e554c0",
    "workload": "roofline", "B": 16384,
    "bytes_per_launch": {"fwd_gemm": 2630.4e6, "upd_gemm": 2887.3e6},
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
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
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


def _oracle_step_time(w, B_sample: int, steps: int, seed: int = 1):
    """Time the CPU oracle, as it stands, on a bounded sample (B_sample positives + negatives)."""
    from oracle import ffint8_oracle as O
    specs = [O.LayerSpec(l.kind, l.K, l.N, l.theta, l.lr, l.tau, l.eps, l.H, l.Wd, l.Cin, seed=seed, index=i,
                         stride=l.stride) for i, l in enumerate(w.layers)]
    Ws = synth.make_weights(w, seed)
    X = synth.make_batch(w, seed, B=B_sample)
    times = []
    for s in range(steps):
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
    sample = f"{B_sample} positive + {B_sample} negative samples of the {args.workload} workload per step, full layer widths"
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
    for i in range(args.warmup):
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
    launches = ffb.ff_launch_count(ctx.ctx) - l0
    ms_local = e0.elapsed_time(e1)
    ffb.ff_poll_status(ctx.ctx, stream)
    loss_last = float(bufs[last].loss[0].item())
    ms, value = whole_job_throughput(ms_local, B * args.steps, dev)

    # ---------------- the same K steps again with a CUDA-event pair around every kernel ----------------
    # (a second region, so that the events' cost stays out of `value`; same steps, same state of the device)
    reset_weights()
    barrier()
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
    clocks = sampler.stop(t_begin, t_end) if rank == 0 else None
    ffb.ff_poll_status(ctx.ctx, stream)

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
        raw_np, labels_np, label_stride = synth.make_raw(w, seed, B=B)
        n_in = raw_np.shape[1]
        raw_host = torch.from_numpy(raw_np).pin_memory()
        labels_host = torch.from_numpy(labels_np).pin_memory()
        raw_dev = [torch.empty_like(raw_host, device=dev) for _ in range(2)]
        labels_dev = [torch.empty_like(labels_host, device=dev) for _ in range(2)]
        loss_host = torch.zeros(4, dtype=torch.float32).pin_memory()
        n_e2e = max(3, min(args.steps, 10))
        tau0 = float(np.sqrt(n_in))

        def e2e_step(k, i):
            ffb.ff_embed_labels(ctx.ctx, raw_dev[k].data_ptr(), labels_dev[k].data_ptr(), B, n_in, 2, 10, label_stride, 1.0,
                                tau0, 1e-8, bufs[0].X.data_ptr(), stream)
            ffb.ff_train_step(ctx.ctx, descs_arr, bufs_arr, n_layers, B, w.lam_per_step * i, i, stream)

        for k in (0, 1):           # untimed: both buffer sets hold data, the launch sequence is in its steady form
            raw_dev[k].copy_(raw_host)
            labels_dev[k].copy_(labels_host)
            e2e_step(k, k)
        reset_weights()
        copy_stream = torch.cuda.Stream()
        main = torch.cuda.current_stream()
        ready = [torch.cuda.Event(), torch.cuda.Event()]     # samples landed in raw_dev[k]
        freed = [torch.cuda.Event(), torch.cuda.Event()]     # the step reading raw_dev[k] has finished

        def h2d(k):
            raw_dev[k].copy_(raw_host, non_blocking=True)
            labels_dev[k].copy_(labels_host, non_blocking=True)
            ready[k].record(copy_stream)

        barrier()
        e0.record()
        with torch.cuda.stream(copy_stream):
            h2d(0)
        for i in range(n_e2e):
            k = i & 1
            if i + 1 < n_e2e:
                with torch.cuda.stream(copy_stream):
                    if i >= 1:
                        copy_stream.wait_event(freed[k ^ 1])
                    h2d(k ^ 1)
            main.wait_event(ready[k])
            e2e_step(k, i)
            freed[k].record(main)
            loss_host.copy_(bufs[last].loss, non_blocking=True)
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
        work = algorithmic_work(w, B)
        burst = (ms + ms_profiled) * 1e-3 < BURST_SECONDS
        bf16 = peaks["bf16_burst"] if burst else peaks["bf16_sustained"]
        int8_peak = INT8_TO_BF16 * bf16
        per_kernel = {}
        for k, (tot_ms, n) in kernel_ms.items():
            ent = {"launches_per_step": n / args.steps, "ms_per_step": tot_ms / args.steps,
                   "share": tot_ms / ms_profiled}
            if k in work and work[k] > 0 and tot_ms > 0:
                rate = work[k] * args.steps / (tot_ms * 1e-3)
                if k.endswith("gemm"):
                    ent.update(bound="tensor", achieved=rate / 1e12, unit="TOP/s", frac=rate / 1e12 / int8_peak)
                else:
                    ent.update(bound="hbm", achieved=rate / 1e9, unit="GB/s", frac=rate / 1e9 / peaks["hbm_gbs"])
            per_kernel[k] = ent
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
            "roofline": {"bound": "tensor", "kernel": names[dom], "achieved": per_kernel[dom]["achieved"],
                         "peak": int8_peak, "unit": "TOP/s", "frac": per_kernel[dom]["frac"],
                         "peak_source": f"{INT8_TO_BF16:g} x {peaks['source']} bf16 cuBLAS "
                                        f"{'burst' if burst else 'sustained'} ({bf16} TF/s): the two timed regions lasted "
                                        f"{(ms + ms_profiled) * 1e-3:.2f} s",
                         "frac_of_sustained_x2": per_kernel[dom]["achieved"] / (INT8_TO_BF16 * peaks["bf16_sustained"]),
                         "frac_of_nominal_4500": per_kernel[dom]["achieved"] / 4500.0,
                         "traffic": _ncu_traffic(dom, args.workload, B)},
            "kernels": per_kernel,
            "rows_per_s": 2.0 * value,
        }
        if lib_gemm is not None:
            out["library_int8_gemm"] = lib_gemm
        if not args.no_cpu_baseline and world == 1:
            Bs = min(B, args.cpu_sample)
            t, cores = _oracle_step_time(w, Bs, 1)
            out["cpu_baseline"] = {"value": Bs / t, "unit": UNIT, "cores": cores, "kind": "oracle",
                                   "sample": f"{Bs} positive + {Bs} negative samples, full layer widths, 1 step"}
        print(json.dumps(out))
    ctx.close()
    if world > 1 or args.data_parallel:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
