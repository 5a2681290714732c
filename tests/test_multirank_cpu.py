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
