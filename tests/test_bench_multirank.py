"""The N > 1 path of bench.py on CPU: two gloo ranks.  The eviction step does not shard (every
(sequence, KV head) is independent and there is no exchange step), so ranks are replicas; the only
cross-rank logic is the max over ranks of the device time and the whole-job value built from it."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from tests.conftest import ROOT


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = [2.0, 3.5][rank]                         # rank 1 is the slow one
    got = bench.max_over_ranks(ms, world, torch.device("cpu"))
    out[rank] = (got, bench.whole_job_value(1000, world, got))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_report_the_slowest_time_and_the_whole_job_value():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 3.5
    assert res[0][1] == res[1][1] == 2 * 1000 / 3.5e-3


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(1.25, 1, "cpu") == 1.25
    assert bench.whole_job_value(262144, 1, 1.0) == 262144e3


def test_reference_arm_runs_on_rank_zero_only(monkeypatch, capsys):
    import bench
    monkeypatch.setenv("RANK", "1")
    bench.run_reference(bench.argparse.Namespace(workload="tiny", steps=1, warmup=0, gpus=2, resident_layers=1))
    assert capsys.readouterr().out == ""
