"""World-size-2 check (gloo, CPU) of what bench.py does when it runs on more than one GPU: every rank
trains its own replica, the reported time is the maximum over ranks and the reported value is the
samples of ALL ranks divided by that time (no data-path collective)."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms_local = 10.0 + 5.0 * rank          # rank 1 is the slow one
    units_local = 1000.0 * (rank + 1)     # and did more work
    ms, value = bench.whole_job_throughput(ms_local, units_local)
    out[rank] = (ms, value)
    dist.barrier()
    dist.destroy_process_group()


def test_whole_job_throughput_is_total_units_over_slowest_rank():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in range(world):
        ms, value = res[rank]
        assert ms == 15.0
        assert abs(value - 3000.0 / 15e-3) < 1e-6


def test_whole_job_throughput_single_process():
    import bench
    ms, value = bench.whole_job_throughput(4.0, 100.0)
    assert ms == 4.0 and abs(value - 25000.0) < 1e-9


def test_algorithmic_work_of_the_roofline_workload():
    import bench
    from paper_2506_22771_b200 import synth
    w = synth.workload("roofline")
    work = bench.algorithmic_work(w, w.B)
    M, N, K = 2 * w.B, 8192, 8192
    assert work["fwd_gemm"] == 2.0 * M * N * K and work["upd_gemm"] == 2.0 * M * N * K
    assert work["absmax"] == 4.0 * (M * K + N * K) and work["quantize"] == 5.0 * (M * K + N * K)
    assert work["dh_quantize"] == 5.0 * M * N and work["normalize"] == 0.0


# ---- data-parallel step: the plumbing around the library's phases -----------------------------------
def _dp_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2506_22771_b200 import binding as ffb
    from paper_2506_22771_b200 import data_parallel as dp
    # stand-ins for one layer's buffers on this rank: a range vector, a loss share, INT32 weight-gradient sums
    absmax = torch.tensor([0.5 + rank, 3.0 - rank, 0.0, 1.0 + 2 * rank, 0.25, 0.0, 0.0, 0.0])
    loss = torch.tensor([0.125 * (rank + 1), 0.0, 0.0, 0.0])
    accw = torch.arange(24, dtype=torch.int32).reshape(2, 3, 4) * (1 if rank == 0 else -3)
    table = dp.PointerTable([absmax, loss, accw])
    entries = [(absmax.data_ptr(), 2, ffb.FF_DP_F32, ffb.FF_DP_MAX),           # input ranges
               (absmax.data_ptr() + 12, 2, ffb.FF_DP_F32, ffb.FF_DP_MAX),      # dH ranges (elements 3, 4)
               (loss.data_ptr(), 1, ffb.FF_DP_F32, ffb.FF_DP_SUM),
               (accw.data_ptr(), 24, ffb.FF_DP_I32, ffb.FF_DP_SUM)]
    dp.all_reduce_entries(entries, table)
    out[rank] = (absmax.tolist(), loss.tolist(), accw.reshape(-1).tolist())
    dist.barrier()
    dist.destroy_process_group()


def test_dp_reductions_over_two_ranks():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_dp_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        absmax, loss, accw = res[rank]
        assert absmax[:2] == [1.5, 3.0] and absmax[3:5] == [3.0, 0.25]
        assert absmax[2] == 0.0 and absmax[5:] == [0.0, 0.0, 0.0]          # untouched neighbours
        assert loss == [0.375, 0.0, 0.0, 0.0]
        assert accw == [-2 * i for i in range(24)]


def test_shard_rows_cover_the_batch_once():
    from paper_2506_22771_b200 import data_parallel as dp
    for B, world in [(16384, 8), (200, 3), (5, 5), (7, 2)]:
        spans = [dp.shard_rows(B, world, r) for r in range(world)]
        assert spans[0][0] == 0 and sum(n for _, n in spans) == B
        for (o0, n0), (o1, _) in zip(spans, spans[1:]):
            assert o0 + n0 == o1
        assert max(n for _, n in spans) - min(n for _, n in spans) <= 1


def test_shard_batch_takes_the_same_rows_of_both_sets():
    import numpy as np
    from paper_2506_22771_b200 import data_parallel as dp
    B, per, K = 6, 2, 3                       # 2 rows per sample (e.g. positions of a convolution input)
    X = np.arange(2 * B * per * K, dtype=np.float32).reshape(2 * B * per, K)
    got = dp.shard_batch(X, B, 4, 2)
    want = np.concatenate([X[8:12], X[B * per + 8:B * per + 12]], 0)
    assert np.array_equal(got, want)
    assert torch.equal(dp.shard_batch(torch.from_numpy(X), B, 4, 2), torch.from_numpy(want))


def test_pointer_table_rejects_foreign_addresses_and_types():
    import pytest
    from paper_2506_22771_b200 import binding as ffb
    from paper_2506_22771_b200 import data_parallel as dp
    t = torch.zeros(8, dtype=torch.float32)
    table = dp.PointerTable([t])
    assert table.view(t.data_ptr() + 8, 3, ffb.FF_DP_F32).data_ptr() == t.data_ptr() + 8
    with pytest.raises(KeyError):
        table.view(t.data_ptr() + 24, 4, ffb.FF_DP_F32)      # runs past the end
    with pytest.raises(TypeError):
        table.view(t.data_ptr(), 2, ffb.FF_DP_I32)


def test_reference_arm_prints_one_contract_line():
    """`bench.py --impl reference` (the oracle on the host cores) on the small workload: one JSON line with the
    metric, the exact step counts when they fit the time budget, and the oracle named as the baseline."""
    import json
    import subprocess
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny_mlp",
                          "--steps", "4", "--warmup", "2", "--gpus", "1"], capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-500:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "FF-INT8 train samples/s" and d["unit"] == "samples/s"
    assert d["steps"] == 4 and d["steps_requested"] == 4 and d["warmup"] == 2 and d["n_gpus"] == 1
    assert d["higher_is_better"] is True and d["vs_baseline"] is None and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": "samples/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["config"]["workload"] == "tiny_mlp"


def test_reference_arm_other_ranks_do_nothing():
    import subprocess
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny_mlp",
                          "--steps", "1", "--warmup", "1", "--gpus", "2"], capture_output=True, text=True, timeout=300, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""


# ---- the overlapped form: large reductions started behind their phase, waited for where they are needed ----------
def _dp_overlap_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2506_22771_b200 import binding as ffb
    from paper_2506_22771_b200 import data_parallel as dp
    n = 2                                                   # layers of the stand-in network
    absmax = [torch.zeros(8) for _ in range(n)]
    loss = [torch.zeros(4) for _ in range(n)]
    accw = [torch.zeros(2, 3, 5, dtype=torch.int32) for _ in range(n)]
    table = dp.PointerTable(absmax + loss + accw)
    seen = {"update_saw_global_sums": [], "phases": []}

    def local_sums(l, r):                                   # what rank r's contraction of layer l leaves
        return (torch.arange(30, dtype=torch.int32).reshape(2, 3, 5) + 7 * l) * (r + 1)

    def fake_phase(ctx, descs, bufs, n_layers, B_local, B_total, row_off, phase, lam, step, stream=0):
        # the call sequence and the lists of ff_dp_train_phase, on CPU tensors
        seen["phases"].append(phase)
        F, I, MAX, SUM = ffb.FF_DP_F32, ffb.FF_DP_I32, ffb.FF_DP_MAX, ffb.FF_DP_SUM
        if phase == 0:
            absmax[0][0:2] = torch.tensor([1.0 + rank, 2.0 - rank])
            return [(absmax[0].data_ptr(), 2, F, MAX, 1)]
        if phase <= n:
            l = phase - 1
            absmax[l][5:7] = torch.tensor([0.5 * (rank + 1) + l, 3.0 - rank])
            ent = [(absmax[l].data_ptr() + 20, 2, F, MAX, phase + 1)]
            if l + 1 < n:
                absmax[l + 1][0:2] = absmax[l][5:7]
                ent.append((absmax[l + 1].data_ptr(), 2, F, MAX, phase + 1))
            return ent
        if phase == n + 1:
            ent = []
            for l in range(n):
                absmax[l][3:5] = torch.tensor([float(rank + l), 1.0])
                loss[l][0] = 0.25 * (rank + 1) + l
                ent += [(absmax[l].data_ptr() + 12, 2, F, MAX, n + 2), (loss[l].data_ptr(), 1, F, SUM, n + 2)]
            return ent
        if phase < 2 * n + 2:
            l = phase - (n + 2)
            accw[l].copy_(local_sums(l, rank))
            return [(accw[l].data_ptr(), 30, I, SUM, 2 * n + 2 + l)]
        l = phase - (2 * n + 2)
        want = sum(local_sums(l, r) for r in range(world))
        seen["update_saw_global_sums"].append(bool(torch.equal(accw[l], want)))
        return []

    ffb.ff_dp_train_phase, ffb.ff_dp_phase_count = fake_phase, (lambda k: 3 * k + 2)
    red = dp.OverlappedReducer(table)
    dp.dp_train_step(None, None, None, n, 4, 8, 4 * rank, 0.0, 0, red)
    out[rank] = (seen, red.log, [a.tolist() for a in absmax], [x.tolist() for x in loss])
    dist.barrier()
    dist.destroy_process_group()


def test_dp_overlapped_reductions_over_two_ranks():
    world, n = 2, 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_dp_overlap_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        seen, log, absmax, loss = res[rank]
        assert seen["phases"] == list(range(3 * n + 2))
        assert seen["update_saw_global_sums"] == [True, True]          # each update found the sums of the whole batch
        # small reductions at once, the weight-gradient sums of layer l started behind phase n+2+l and waited for
        # right before phase 2n+2+l - i.e. the reduction of layer 0 is in flight while layer 1's sums are computed
        assert log == [("now", 0), ("now", 1), ("now", 2), ("now", 3), ("start", 4), ("start", 5), ("finish", 6),
                       ("finish", 7)]
        assert absmax[0][0:2] == [2.0, 2.0] and absmax[0][5:7] == [1.0, 3.0] and absmax[1][0:2] == [1.0, 3.0]
        assert absmax[0][3:5] == [1.0, 1.0] and absmax[1][3:5] == [2.0, 1.0]
        assert loss[0][0] == 0.75 and loss[1][0] == 2.75
