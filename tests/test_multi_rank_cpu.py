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


def test_gpus_flag_spawns_replicas_through_the_launcher():
    """`python bench.py --gpus 2 ...` with no launcher around it starts two ranks of itself under
    torch.distributed.run (rendezvous on 127.0.0.1).  On a machine without GPUs the arm that can run is
    the reference arm (the CPU oracle): rank 0 works and prints the line, rank 1 exits 0 without work, and
    the line reports the world size the launcher made."""
    import json
    import subprocess
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference", "--workload", "tiny",
           "--steps", "2", "--warmup", "0"]
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=600, env=env, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, out.stdout
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["value"] > 0
    assert rec["config"]["workload"] == "tiny" and rec["cpu_baseline"]["kind"] == "oracle"


def test_replica_command_is_the_documented_launch_line():
    sys.path.insert(0, ROOT)
    import argparse
    import bench
    cmd = bench.replica_command(argparse.Namespace(gpus=4), ["--gpus", "4", "--steps", "3"], 29500)
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"] and "--nproc-per-node=4" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[-4:] == ["--gpus", "4", "--steps", "3"]
