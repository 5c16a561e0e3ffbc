"""The multi-GPU path is N independent replicas; its only cross-rank logic (barrier, max time,
summed work, per-rank seeds) is covered here with two gloo ranks on the CPU."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2501_07161_b200 import replicas as R
    R.barrier()
    thr, slow = R.whole_job_throughput(units_local=10.0 * (rank + 1), elapsed_local_s=1.0 + rank)
    seeds = [R.replica_seed(0, r) for r in range(world)]
    out.put((rank, R.world(), R.rank(), thr, slow, R.max_over_ranks(rank), R.sum_over_ranks(1), seeds))
    dist.destroy_process_group()


def test_two_replicas_aggregate_over_gloo():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, world, rk, thr, slow, mx, sm, seeds in res:
        assert world == 2 and rk == rank
        assert slow == 2.0 and thr == (10.0 + 20.0) / 2.0      # total work / slowest rank
        assert mx == 1.0 and sm == 2.0
        assert len(set(seeds)) == 2


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    from paper_2501_07161_b200 import replicas as R
    assert R.world() == 1 and R.rank() == 0
    assert R.whole_job_throughput(8.0, 2.0) == (4.0, 2.0)
