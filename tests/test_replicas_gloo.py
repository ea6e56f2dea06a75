"""The N > 1 path of the benchmark is replicas only: no data-path collective, just the timing
protocol (barrier, MAX over the ranks' device times, whole-job rate).  Two gloo ranks on the CPU run
that protocol with different per-rank times and disjoint instance shards."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_18063_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        n_inst = 8
        first = replicas.first_instance(rank, n_inst)
        mine = torch.tensor(list(range(first, first + n_inst)), dtype=torch.int64)
        gathered = [torch.zeros(n_inst, dtype=torch.int64) for _ in range(world)]
        dist.all_gather(gathered, mine)
        dist.barrier()
        ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
        ms_max = replicas.max_over_ranks(ms)
        rate = replicas.whole_job_rate(world, 1000, ms_max)
        out[rank] = (ms_max, rate, [g.tolist() for g in gathered])
    finally:
        dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_disjoint_shards():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in (0, 1):
        ms_max, rate, shards = res[rank]
        assert ms_max == 15.0                        # the same on every rank: the maximum
        assert abs(rate - 2 * 1000 / 15e-3) < 1e-6   # whole job: both ranks' steps over the slowest time
        flat = [i for sh in shards for i in sh]
        assert len(flat) == len(set(flat)) == 16     # the ranks' layer instances do not overlap


def test_single_process_needs_no_process_group():
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.whole_job_rate(1, 100, 50.0) == 2000.0
