#!/usr/bin/env python
"""Benchmark of the FF-INT8 train step (Sec. IV-B / Alg. 1 of the FF-INT8 paper) on B200.

    python bench.py --gpus N --steps K --warmup W [--workload roofline] [--impl reference]

A step is one pass of the whole hot path (quantise -> INT8 GEMM -> goodness -> loss -> dH ->
quantise -> INT8 dW GEMM -> update) over one batch of seeded synthetic input.  The default
workload is the task's largest single-GPU configuration ("roofline": one 8192 -> 8192 FF layer,
16384 positive + 16384 negative samples), the one the GEMM-roofline target is quoted on.
Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank runs the same per-GPU batch on its
own GPU (independent batches, no data-path collective: weak scaling).

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
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                smax.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def _oracle_step_time(w, B_sample: int, steps: int, seed: int = 1):
    """Time the CPU oracle, as it stands, on a bounded sample (B_sample positives + negatives)."""
    from oracle import ffint8_oracle as O
    specs = [O.LayerSpec(l.kind, l.K, l.N, l.theta, l.lr, l.tau, l.eps, l.H, l.Wd, l.Cin, seed=seed, index=i)
             for i, l in enumerate(w.layers)]
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
    """Reference arm = the CPU oracle on the host cores (bounded sample per step)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = synth.workload(args.workload)
    B_sample = min(w.B, args.cpu_sample)
    for _ in range(args.warmup if args.warmup < 2 else 1):
        _oracle_step_time(w, B_sample, 1)
    steps = max(1, min(args.steps, 3))
    t, cores = _oracle_step_time(w, B_sample, steps)
    v = B_sample / t
    sample = f"{B_sample} positive + {B_sample} negative samples of the {args.workload} workload per step, full layer widths"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int8", "data": "synthetic", "config": {"workload": args.workload, "B": B_sample},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="roofline")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-sample", type=int, default=256, help="positives per step of the CPU-oracle sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--B", type=int, default=0, help="override positives per batch (parity / profiling runs)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = max(args.warmup, 1)

    if args.impl == "reference":
        return run_reference(args)

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
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    w = synth.workload(args.workload)
    B = args.B or w.B
    seed = 1 + rank
    descs = [ffb.make_desc(l, i, seed) for i, l in enumerate(w.layers)]
    ctx = ffb.Context(descs, B, local)
    bufs = [ffb.LayerBuffers(d, B, dev, dumps=False, xnext=False, own_x=(i == 0)) for i, d in enumerate(descs)]
    Ws = synth.make_weights(w, seed)
    for b, W in zip(bufs, Ws):
        b.W.copy_(torch.from_numpy(W))
    X_host = torch.from_numpy(synth.make_batch(w, seed, B=B)).reshape(bufs[0].X.shape).pin_memory()
    bufs[0].X.copy_(X_host)
    W0 = [b.W.clone() for b in bufs]
    descs_arr = (ffb.ff_layer_desc * len(descs))(*descs)
    bufs_arr = (ffb.ff_layer_bufs * len(descs))(*[b.struct for b in bufs])
    stream = torch.cuda.current_stream().cuda_stream
    n_layers = len(descs)

    def step(i):
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
    e0.record()
    for i in range(args.steps):
        step(i)
    e1.record()
    barrier()
    launches = ffb.ff_launch_count(ctx.ctx) - l0
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop() if rank == 0 else None
    ffb.ff_poll_status(ctx.ctx, stream)
    loss_last = float(bufs[0].loss[0].item())

    # ---------------- dominant kernel: the weight-gradient GEMM + update (one launch per call) ---------
    reset_weights()
    step(0)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    evf = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    last = n_layers - 1
    for i in range(args.steps):
        evf[i][0].record()
        ffb.ff_layer_forward(ctx.ctx, descs[0], bufs[0].struct, B, i, stream) if n_layers == 1 else step(i)
        evf[i][1].record()
        if n_layers == 1:
            ffb.ff_layer_loss_grad(ctx.ctx, descs[0], bufs[0].struct, B, [], [], 0.0, i, stream)
        ev[i][0].record()
        ffb.ff_layer_update(ctx.ctx, descs[last], bufs[last].struct, B, stream)
        ev[i][1].record()
    torch.cuda.synchronize()
    upd_ms = float(np.mean([a.elapsed_time(b) for a, b in ev]))
    fwd_ms = float(np.mean([a.elapsed_time(b) for a, b in evf]))
    ffb.ff_poll_status(ctx.ctx, stream)

    # ---------------- end to end: host buffers, H2D of the batch + D2H of the loss every step ---------
    e2e = None
    if not args.no_e2e:
        reset_weights()
        loss_host = torch.zeros(4, dtype=torch.float32).pin_memory()
        n_e2e = max(3, min(args.steps, 10))
        barrier()
        e0.record()
        for i in range(n_e2e):
            bufs[0].X.copy_(X_host, non_blocking=True)
            step(i)
            loss_host.copy_(bufs[last].loss, non_blocking=True)
            torch.cuda.current_stream().synchronize()
        e1.record()
        barrier()
        ms_e2e = e0.elapsed_time(e1)
        e2e_ms = ms_e2e
        if world > 1:
            t = torch.tensor([ms_e2e], device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            e2e_ms = float(t.item())
        e2e = {"value": world * B * n_e2e / (e2e_ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": int(X_host.numel() * 4), "d2h_bytes_per_step": 16, "steps": n_e2e}

    if world > 1:
        t = torch.tensor([ms], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())

    if rank == 0:
        peaks = _peaks()
        l = w.layers[-1]
        R = l.H * l.Wd
        ops = 2.0 * (2 * B * R) * l.N * l.K                      # INT8 ops of the weight-gradient GEMM (2*M*N*K)
        int8_peak = 2.0 * peaks["bf16_sustained"]                # nominal INT8 : bf16 ratio = 2
        ach = ops / (upd_ms * 1e-3) / 1e12
        out = {
            "metric": METRIC, "value": world * B * args.steps / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": {"workload": args.workload, "B_pos": B, "B_neg": B,
                       "layers": [[x.K, x.N] for x in w.layers], "l2": "inputs larger than L2 (no flush needed)"
                       if 2 * B * R * l.K * 4 > 126e6 else "inputs smaller than L2, not flushed"},
            "clocks": clocks, "gpu_launches": int(launches), "e2e": e2e, "loss_last": loss_last,
            "phases_ms": {"forward_all_kernels": fwd_ms, "update_gemm_kernel": upd_ms},
            "roofline": {"bound": "tensor", "kernel": "tc_gemm_kernel<update> (INT8 dW GEMM + SGD epilogue)",
                         "achieved": ach, "peak": int8_peak, "unit": "TOP/s", "frac": ach / int8_peak,
                         "peak_source": f"2 x {peaks['source']} sustained bf16 cuBLAS ({peaks['bf16_sustained']} TF/s)",
                         "frac_of_burst": ach / (2.0 * peaks["bf16_burst"]), "frac_of_nominal_4500": ach / 4500.0,
                         "traffic": None},
        }
        if not args.no_cpu_baseline and world == 1:
            Bs = min(B, args.cpu_sample)
            t, cores = _oracle_step_time(w, Bs, 1)
            out["cpu_baseline"] = {"value": Bs / t, "unit": UNIT, "cores": cores, "kind": "oracle",
                                   "sample": f"{Bs} positive + {Bs} negative samples, full layer widths, 1 step"}
        print(json.dumps(out))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
