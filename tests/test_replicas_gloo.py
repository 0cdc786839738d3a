"""The multi-GPU form of the benchmark is N independent replicas (the path shards over the batch and
has no exchange step): what the ranks share is only the barrier and the max-over-ranks of the step
time.  This checks that host-side logic with two gloo ranks on the CPU."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, out_dir: str):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench

    # each rank "measures" a different step time; every rank must end up with the slowest one
    mine = 2.0 + rank
    slowest = bench.max_over_ranks(mine, world, device="cpu")
    value = bench.aggregate_images_per_s(64, world, slowest)
    seeds = [bench.replica_seed(layer, rank) for layer in range(3)]
    torch.save({"slowest": slowest, "value": value, "seeds": seeds}, os.path.join(out_dir, f"r{rank}.pt"))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_agree_on_the_slowest_step(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    r = [torch.load(os.path.join(tmp_path, f"r{i}.pt")) for i in range(world)]
    assert r[0]["slowest"] == r[1]["slowest"] == 3.0
    assert r[0]["value"] == r[1]["value"] == pytest.approx(2 * 64 / 3.0e-3)
    assert set(r[0]["seeds"]).isdisjoint(r[1]["seeds"])          # replicas draw different batches


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.max_over_ranks(1.25, 1) == 1.25
    assert bench.aggregate_images_per_s(64, 1, 2.0) == pytest.approx(32000.0)
