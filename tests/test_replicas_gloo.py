"""The N > 1 path of the benchmark: independent replicas (one batch per rank, no data-path
collective), whole-job throughput over the slowest rank's step time.  Run here as two gloo
ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    from paper_2604_18103_b200 import workloads as wl
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # every rank draws its own batch of the same shape
        w = wl.config2(T=64, seed=bench.rank_seed(1, rank), shape=wl.MINI)
        digest = float(w.tensors["H"].double().sum())
        # the job's step time is the slowest rank's
        mine = 1.0 + rank                    # rank 1 is the slow one
        t = bench.reduce_max_over_ranks(mine, dist, torch.device("cpu"))
        gathered = [None] * world
        dist.all_gather_object(gathered, (digest, w.T, t))
        if rank == 0:
            out.put(gathered)
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_run_independent_batches_and_time_by_the_slowest():
    world, port = 2, 29000 + os.getpid() % 2000
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (d0, T0, t0), (d1, T1, t1) = got
    assert d0 != d1 and T0 == T1 == 64                      # different data, same shape: weak scaling
    assert t0 == t1 == 2.0                                   # both ranks agree on the max
    import bench
    assert bench.whole_job_value(T0, world, t0) == world * T0 / (t0 * 1e-3)
    assert bench.reduce_max_over_ranks(3.5, None, None) == 3.5
