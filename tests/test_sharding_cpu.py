"""The multi-GPU path shards independent sequences across ranks with no data-path collective.
Host-side logic checked with two gloo ranks on CPU."""
import os

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2410_01699_b200.sharding import gather_token_lists, max_over_ranks, shard_sequences


def test_partition_covers_every_sequence_once():
    for n in (0, 1, 5, 8, 13):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                start, count = shard_sequences(n, world, r)
                seen += list(range(start, start + count))
            assert seen == list(range(n))
            sizes = [shard_sequences(n, world, r)[1] for r in range(world)]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard_sequences(4, 2, 2)


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        n_seq = 5
        start, count = shard_sequences(n_seq, world, rank)
        # stand-in for decoding: a sequence's tokens depend on its GLOBAL id only
        local = [[1000 * (start + i) + t for t in range(3)] for i in range(count)]
        everything = gather_token_lists(local)
        slowest = max_over_ranks(10.0 + rank)
        dist.barrier()
        if rank == 0:
            q.put((everything, slowest))
    finally:
        dist.destroy_process_group()


def test_two_ranks_reproduce_the_single_rank_result():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    everything, slowest = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert everything == [[1000 * s + t for t in range(3)] for s in range(5)]
    assert slowest == 11.0


def test_bench_starts_one_rank_per_gpu_when_no_launcher_did(monkeypatch):
    """`python bench.py --gpus N` without torchrun: bench starts the N ranks itself; every rank gets its
    RANK / LOCAL_RANK / WORLD_SIZE and a rendezvous on 127.0.0.1 (checked with the process spawner and the
    per-rank body replaced by recorders: no GPU involved)."""
    import argparse
    import importlib.util
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    spec = importlib.util.spec_from_file_location("bench_under_test", os.path.join(root, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    seen = []

    def fake_run(args, wl):
        seen.append({k: os.environ[k] for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")})

    def fake_spawn(fn, args=(), nprocs=1, join=True):
        for i in range(nprocs):
            fn(i, *args)

    monkeypatch.setattr(bench, "run_library", fake_run)
    monkeypatch.setattr(mp, "spawn", fake_spawn)
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT"):
        monkeypatch.setenv(k, "unset")   # restored by monkeypatch afterwards
    bench.launch_ranks(argparse.Namespace(gpus=3), None)
    assert [s["RANK"] for s in seen] == ["0", "1", "2"] and [s["LOCAL_RANK"] for s in seen] == ["0", "1", "2"]
    assert all(s["WORLD_SIZE"] == "3" and s["MASTER_ADDR"] == "127.0.0.1" for s in seen)
    assert len({s["MASTER_PORT"] for s in seen}) == 1 and int(seen[0]["MASTER_PORT"]) > 0
