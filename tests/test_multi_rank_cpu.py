"""The N > 1 contract of bench.py ("replicas only": every rank its own batch, no collective on the
data path, job time = slowest rank, job throughput = all ranks' tokens over that time), exercised
with two gloo ranks on the CPU."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2412_19829_b200 import synth

    c = dict(bench.WORKLOADS["gpt2s"])
    seed = bench.replica_seed(c, rank)
    q, _, _ = synth.qkv(1, 1, 8, 64, "bf16", seed)
    # each rank "measures" a different time; everybody must end up with the slowest one
    local = [10.0 + 5.0 * rank, 100.0 - 30.0 * rank]
    got = bench.max_over_ranks(local, dist, "cpu")
    value = bench.job_throughput(world, c["B"] * c["N"], 4, got[0])
    torch.save({"seed": seed, "q0": q.float().sum().item(), "got": got, "value": value},
               os.path.join(out_dir, f"rank{rank}.pt"))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_agree_on_the_slowest_time_and_use_different_data(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    r = [torch.load(tmp_path / f"rank{i}.pt") for i in range(world)]
    assert r[0]["seed"] != r[1]["seed"] and r[0]["q0"] != r[1]["q0"]  # replicas, not copies
    assert r[0]["got"] == r[1]["got"] == [15.0, 100.0]                  # max over ranks, per entry
    import bench

    c = bench.WORKLOADS["gpt2s"]
    expect = 2 * c["B"] * c["N"] * 4 / 15.0e-3  # both ranks' tokens over the slowest rank's time
    assert abs(r[0]["value"] - expect) < 1e-6 * expect and r[0]["value"] == r[1]["value"]


def test_single_rank_needs_no_process_group():
    import bench

    assert bench.max_over_ranks([1.5, 2.5], None, "cpu") == [1.5, 2.5]
    assert bench.job_throughput(1, 1000, 10, 2.0) == 1000 * 10 / 2.0e-3
