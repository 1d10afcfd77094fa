"""Host-side logic of bench.py for N > 1 (independent replicas): two gloo ranks on the CPU."""
import io
import os
import sys
import contextlib

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import jq_workloads as W
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, device="cpu")       # the slowest rank's time counts
    value = bench.job_value(W.CFG3, world, ms * 1e-3)
    # ranks draw different caches (the sequence number of the seed is the rank)
    differs = W.seed_of(W.CFG3, layer=3, seq=rank) != W.seed_of(W.CFG3, layer=3, seq=1 - rank)
    out[rank] = (ms, value, differs)
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_time_and_the_summed_work():
    world, port = 2, 29500 + os.getpid() % 1000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        import jq_workloads as W
        for rank in range(world):
            ms, value, differs = out[rank]
            assert ms == 15.0 and differs
            assert abs(value - 2 * W.CFG3.L / 15.0e-3) < 1e-6 * value


def test_reference_arm_runs_on_rank_0_only(monkeypatch):
    import bench
    monkeypatch.setenv("RANK", "1")
    buf = io.StringIO()
    with contextlib.redirect_stdout(buf):
        bench.run_reference(None)          # returns before touching its arguments
    assert buf.getvalue() == ""
