"""The N > 1 path on CPU (gloo, world size 2): row sharding without a data-path collective and the
max-over-ranks timing reduction the benchmark uses."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

from paper_2510_25977_b200 import inputs, sharding


def test_shard_rows_partition():
    for T, world in [(1000, 2), (4096, 8), (130, 4), (1, 2), (0, 3), (257, 2)]:
        blocks = [sharding.shard_rows(T, world, r) for r in range(world)]
        assert blocks[0][0] == 0 and blocks[-1][1] == T
        for (a, b), (c, d) in zip(blocks, blocks[1:]):
            assert b == c and a <= b
        assert all(a % 128 == 0 for a, b in blocks if a < T)
        sizes = [b - a for a, b in blocks]
        assert max(sizes) - min(sizes) <= 128 + 127
    with pytest.raises(ValueError):
        sharding.shard_rows(10, 2, 2)


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import oracle
    T, d, ffn, r = 300, 64, 96, 8
    f = inputs.direct_factors(d, ffn, r, seed=0)          # every rank holds the factors
    X = inputs.activations(T, d, seed=0)
    lo, hi = sharding.shard_rows(T, world, rank)
    Y_local = oracle.svdmlp(X[lo:hi], *f.tensors())       # the single-device forward on this rank's rows
    slowest = sharding.max_over_ranks(10.0 + rank, dist)  # timing reduction: max over ranks
    import bench   # the benchmark's own rank logic: row blocks of one world * T batch at large T, replicas at decode
    assert bench.local_tokens(1024, world, rank, "tensor") == 1024
    blo, bhi = sharding.shard_rows(world * 300, world, rank)
    assert bench.local_tokens(300, world, rank, "tensor") == bhi - blo
    assert bench.local_tokens(8, world, rank, "skinny") == 8
    total = torch.tensor([bench.local_tokens(300, world, rank, "tensor")])
    dist.all_reduce(total)
    assert int(total) == world * 300   # the blocks of all ranks add up to the whole batch
    np.save(os.path.join(out_dir, f"y{rank}.npy"), Y_local)
    np.save(os.path.join(out_dir, f"t{rank}.npy"), np.array([slowest, lo, hi]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_rows_and_reduce_time(tmp_path, oracle):
    world, port = 2, 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    T, d, ffn, r = 300, 64, 96, 8
    f = inputs.direct_factors(d, ffn, r, seed=0)
    X = inputs.activations(T, d, seed=0)
    full = oracle.svdmlp(X, *f.tensors())
    parts = [np.load(tmp_path / f"y{k}.npy") for k in range(world)]
    assert np.array_equal(np.concatenate(parts, axis=0), full)   # rows are independent: bit-identical
    for k in range(world):
        slowest, lo, hi = np.load(tmp_path / f"t{k}.npy")
        assert slowest == 11.0
        assert (lo, hi) == sharding.shard_rows(T, world, k)


def test_bench_gpus_flag_spawns_one_rank_per_gpu():
    """`bench.py --gpus 2` started as a plain process re-launches itself as two ranks (here the reference arm, which
    needs no GPU: rank 0 prints the one JSON line, rank 1 exits 0 without work)."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference", "--steps", "1",
                          "--warmup", "0"], capture_output=True, text=True, timeout=900, cwd=ROOT, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    j = json.loads(lines[0])
    assert j["impl"] == "reference" and j["n_gpus"] == 2 and j["value"] > 0
