"""World-size-2 check of the benchmark's multi-rank plumbing on CPU (gloo)."""
import os
import socket

import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_01662_b200 import distributed as d


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms_local = 10.0 + 5.0 * rank                 # rank 1 is the slow one
    ms = d.max_over_ranks(ms_local)
    dist.barrier()
    out.put((rank, ms, d.job_throughput(1000, world, ms), list(d.shard_units(7, rank, world))))
    dist.destroy_process_group()


def test_two_ranks_agree_on_the_slowest_time_and_aggregate_throughput():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [15.0, 15.0]                      # max over ranks on both
    assert all(abs(r[2] - 2 * 1000 / 15e-3) < 1e-6 for r in res)     # weak scaling: all ranks' units / slowest time
    assert res[0][3] == [0, 1, 2, 3] and res[1][3] == [4, 5, 6]      # contiguous, disjoint, complete shares


def test_single_process_is_identity():
    assert d.max_over_ranks(3.5) == 3.5
    assert list(d.shard_units(5, 0, 1)) == [0, 1, 2, 3, 4]
    assert d.job_throughput(131072, 1, 500.0) == 262144.0
