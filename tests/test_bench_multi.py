"""bench.py at N > 1: the path does not shard, so ranks are independent replicas and the job's
number is (tokens of all ranks) / (max over ranks of the device time).  Two gloo ranks on CPU."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    local = [10.0 + 5.0 * rank, 100.0 - 20.0 * rank]          # rank 1 slower on the first, faster on the second
    ms, tokens = bench.aggregate_over_ranks(local, tokens_per_rank=1000, steps=3, dist=dist, device="cpu")
    out[rank] = (ms, tokens)
    dist.barrier()
    dist.destroy_process_group()


def test_replica_aggregation_two_ranks():
    world, port = 2, _free_port()
    with mp.get_context("spawn").Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        ms, tokens = res[rank]
        assert ms == [15.0, 100.0]            # MAX over ranks, per timing
        assert tokens == 2 * 1000 * 3         # tokens of all replicas


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    ms, tokens = bench.aggregate_over_ranks([7.5, 0.0], tokens_per_rank=64, steps=4)
    assert ms == [7.5, 0.0] and tokens == 256


def test_algorithmic_work_matches_the_stated_formula():
    sys.path.insert(0, ROOT)
    import bench
    from workloads import get_config
    cfg = get_config("long")
    w = bench.algorithmic_work(cfg, cfg.seq_lengths(), with_initial_state=True)
    assert w["tokens"] == 10240
    assert w["flops"] == 10240 * 16 * 180224                      # 6Cd_k + 4Cd_v + 6d_kd_v at d = 128
    assert w["bytes"] == 10240 * 16 * 1032 + 2 * 16 * 128 * 128 * 4


def test_bench_starts_its_own_replicas_when_no_launcher_did():
    """`python bench.py --gpus N` without WORLD_SIZE in the environment must start N ranks itself: the command it
    builds is the launcher invocation the driver uses (one node, N processes, rendezvous on 127.0.0.1)."""
    import bench
    cmd = bench.replica_launch_command(4, ["--gpus", "4", "--steps", "2", "--warmup", "3"], port=29555)
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"]
    assert "--nproc-per-node=4" in cmd and cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[cmd.index("--master-port") + 1] == "29555"
    assert cmd[-7].endswith("bench.py") and cmd[-6:] == ["--gpus", "4", "--steps", "2", "--warmup", "3"]
    port = int(bench.replica_launch_command(2, [])[bench.replica_launch_command(2, []).index("--master-port") + 1])
    assert 1024 < port < 65536
