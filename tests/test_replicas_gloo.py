"""The N > 1 path of the benchmark (independent replicas, max-over-ranks timing) with 2 gloo ranks on CPU."""
import os

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2408_08696_b200 import replicas
    replicas.barrier()
    agg = replicas.aggregate(10.0 + 5.0 * rank, 4)          # rank 1 is slower: 15 ms for 4 steps
    q.put((rank, agg, replicas.world()))
    dist.destroy_process_group()


def test_two_replicas_take_the_slowest_time():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, agg, w in res:
        assert w == (rank, 2)
        assert agg["n_ranks"] == 2
        assert abs(agg["ms_per_step"] - 15.0 / 4) < 1e-9
        assert abs(agg["us_per_step_job"] - 15000.0 / 8) < 1e-6
        assert abs(agg["steps_per_s"] - 8 / 0.015) < 1e-6


def test_single_process_is_identity():
    from paper_2408_08696_b200 import replicas
    agg = replicas.aggregate(8.0, 4)
    assert agg["n_ranks"] == 1 and agg["ms_per_step"] == 2.0 and agg["steps_per_s"] == 500.0
