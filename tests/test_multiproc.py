"""Host-side multi-rank logic of the benchmark on CPU: two gloo ranks, max-over-ranks timing and the
whole-job throughput formula (every rank owns an independent batch; there is no data-path collective)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    agg = bench.max_over_ranks(ms, torch.device("cpu"))
    dist.barrier()
    out[rank] = (agg, bench.whole_job_mtok_per_s(32768, world, agg))
    dist.destroy_process_group()


def test_two_gloo_ranks_report_the_slowest_time_and_the_whole_job_rate():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    agg, rate = res[0]
    assert agg == 15.0
    assert abs(rate - 2 * 32768 / 15e-3 / 1e6) < 1e-9


def test_single_process_is_identity():
    import bench
    assert bench.max_over_ranks(3.5, torch.device("cpu")) == 3.5
    assert abs(bench.whole_job_mtok_per_s(1000, 1, 1.0) - 1.0) < 1e-12
