"""The N > 1 path of bench.py on CPU: replicas only, so the only cross-rank step is the final
aggregation (tokens summed, time maximised).  Two gloo ranks check it."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    tokens, e2e_tokens = 100 + 7 * rank, 90 + rank
    ms, e2e_s = 10.0 + 5 * rank, 0.5 - 0.1 * rank
    res = bench.aggregate_replicas(dist, [tokens, e2e_tokens], [ms, e2e_s], "cpu")
    dist.barrier()
    if rank == 0:
        out.put(res)
    dist.destroy_process_group()


def test_replica_aggregation_sums_tokens_and_takes_the_slowest_rank():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    world, port = 2, 29731
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0] == 207 and res[1] == 181          # tokens: sum over ranks
    assert res[2] == 15.0 and abs(res[3] - 0.5) < 1e-12   # time: max over ranks


def test_single_process_aggregation_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_replicas(None, [5, 6], [1.5, 2.5], "cpu") == [5, 6, 1.5, 2.5]
