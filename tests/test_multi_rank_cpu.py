"""The multi-GPU mode of the benchmark is N independent replicas (units of the path never exchange
data); the only cross-rank step is the max-over-ranks reduction of the timings and the aggregate
throughput.  Both run here on two gloo ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = [10.0 + 5.0 * rank, 7.0 - rank]            # rank 1 is slower on the first clock, faster on the second
    got = bench.max_over_ranks(mine, torch.device("cpu"), world)
    dist.barrier()
    dist.destroy_process_group()
    q.put((rank, got))


def test_max_over_ranks_and_aggregate_on_two_gloo_ranks():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0] == res[1] == [15.0, 7.0]
    sys.path.insert(0, ROOT)
    import bench
    # two replicas of batch 32 at 20 ms per step: 3200 tokens/s for the whole job
    assert abs(bench.aggregate_throughput(32, 2, 20.0) - 3200.0) < 1e-9
    assert bench.max_over_ranks([3.0], torch.device("cpu"), 1) == [3.0]


def test_gpus_flag_without_a_launcher_starts_that_many_replicas():
    """`bench.py --gpus N` run directly (no WORLD_SIZE in the environment) re-launches itself as N replica
    processes on this node with a loopback rendezvous; the command is checked here, not run."""
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.replica_launch_command(4, ["--gpus", "4", "--steps", "5"])
    assert cmd[1:3] == ["-m", "torch.distributed.run"]
    assert "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert 0 < int(cmd[cmd.index("--master-port") + 1]) < 65536
    assert cmd[-5] == os.path.join(ROOT, "bench.py") and cmd[-4:] == ["--gpus", "4", "--steps", "5"]
