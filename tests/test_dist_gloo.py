"""The N > 1 benchmark plumbing on CPU: two gloo ranks agree on the slowest rank's time and on the
whole-job throughput, and draw different input shards."""
import os
import socket

import torch
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    from paper_2412_00876_b200 import dist_util as du
    from paper_2412_00876_b200 import workloads as wl
    assert du.env_world() == (world, rank, rank)
    du.init("gloo")
    du.barrier(sync_cuda=False)
    my_ms = 100.0 + 50.0 * rank                         # rank 1 is the slow one
    slow = du.max_over_ranks(my_ms)
    value = du.job_throughput(units_per_rank=32 * 1024, ms_slowest=slow)
    cfg = wl.CONFIGS[1]
    x = wl.host_normal(cfg, wl.S_X_VIS, (4,), sub=du.shard_seed(rank))
    du.barrier(sync_cuda=False)
    q.put((rank, slow, value, x.tolist()))
    torch.distributed.destroy_process_group()


def test_two_gloo_ranks_agree_on_time_and_throughput():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [150.0, 150.0]                      # max over ranks, same everywhere
    expect = 2 * 32 * 1024 / 0.150
    assert all(abs(r[2] - expect) < 1e-6 for r in res)               # weak scaling: both shards count
    assert res[0][3] != res[1][3]                                     # different shards
