"""Tensor-parallel variant (ffn sharded over ranks, one all-reduce of the narrow Zd).

On CPU, two gloo ranks check the partition and the reduction against the oracle: every rank takes its slice of
the factors, the partial Zd of a slice is what the oracle gives for that slice, the all-reduced sum followed by
the last product equals the oracle's full forward.  On one GPU, the shards of a two-way split run one after the
other through the library's two half-forward calls and a device add stands in for the all-reduce.
"""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

from paper_2510_25977_b200 import inputs, tensor_parallel as tp


def test_shard_ffn_partition():
    for ffn, world in [(11008, 2), (14336, 8), (688, 2), (100, 4), (13824, 3)]:
        cuts = [tp.shard_ffn(ffn, world, r) for r in range(world)]
        assert cuts[0][0] == 0 and cuts[-1][1] == ffn
        for (a, b), (c, d) in zip(cuts, cuts[1:]):
            assert b == c and a <= b
        assert all(a % 128 == 0 for a, b in cuts if a < ffn)


def _partial_zd(oracle, X, Ug, Vg, Uu, Vu, Vd):
    """fp64 Zd of one shard from the oracle's own pieces: Zd = H Vd^T with H = SiLU(G) * Up."""
    F = [oracle.to_f64(t) for t in (Ug, Vg, Uu, Vu, Vd)]
    Xd = oracle.to_f64(X)
    G = oracle.svdlinear(Xd, F[0], F[1])
    Up = oracle.svdlinear(Xd, F[2], F[3])
    H = np.vectorize(oracle.silu)(G) * Up
    return H @ F[4].T


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import oracle
    T, d, ffn, r = 9, 64, 300, 8
    f = inputs.direct_factors(d, ffn, r, seed=1)
    X = inputs.activations(T, d, seed=1)
    Ug, Vg, Uu, Vu, Ud, Vd = tp.shard_factors(*f.tensors(), world, rank)
    lo, hi = tp.shard_ffn(ffn, world, rank)
    assert Ug.shape == (hi - lo, r) and Vd.shape == (r, hi - lo) and Vd.is_contiguous()
    zd = torch.from_numpy(_partial_zd(oracle, X, Ug, Vg, Uu, Vu, Vd))
    dist.all_reduce(zd)                                   # the one collective of the variant
    Y = zd.numpy() @ oracle.to_f64(Ud).T                  # every rank finishes on its own
    np.save(os.path.join(out_dir, f"y{rank}.npy"), Y)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_partition_and_all_reduce(tmp_path, oracle):
    world, port = 2, 31500 + os.getpid() % 2000
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    T, d, ffn, r = 9, 64, 300, 8
    f = inputs.direct_factors(d, ffn, r, seed=1)
    X = inputs.activations(T, d, seed=1)
    full = oracle.svdmlp(X, *f.tensors())
    for k in range(world):
        Y = np.load(tmp_path / f"y{k}.npy")
        assert np.abs(Y - full).max() <= 1e-12 * np.abs(full).max()   # a re-association of fp64 sums


@pytest.mark.gpu
@pytest.mark.parametrize("T", [8, 27, 300])
@pytest.mark.parametrize("world", [2, 3])
def test_sharded_handles_on_one_gpu(oracle, T, world):
    import _gpu
    from paper_2510_25977_b200 import binding
    _gpu.require_gpu()
    d, ffn, r = 512, 1408, 64
    f = inputs.direct_factors(d, ffn, r, seed=5, device="cuda")
    X = inputs.activations(T, d, seed=5, device="cuda")
    handles = [binding.svdmlp_create(*tp.shard_factors(*f.tensors(), world, g), max_T=T) for g in range(world)]
    zd = None
    for h in handles:
        part = binding.svdmlp_forward_partial(h, X)
        zd = part if zd is None else zd + part            # stands in for the all-reduce
    for h in handles:                                      # every rank finishes with the same sum
        Y = binding.svdmlp_forward_finish(h, zd)
        torch.cuda.synchronize()
        assert binding.svdmlp_last_device_status(h) == 0
        _gpu.assert_close(Y, oracle.svdmlp(X, *f.tensors()), f"tensor parallel x{world}, T={T}")
    # the two halves on an unsharded handle equal the whole forward, and the handle still serves plain calls
    h = binding.svdmlp_create(*f.tensors(), max_T=T)
    Y2 = binding.svdmlp_forward_finish(h, binding.svdmlp_forward_partial(h, X))
    Y3 = binding.svdmlp_forward(h, X)
    torch.cuda.synchronize()
    ref = oracle.svdmlp(X, *f.tensors())
    _gpu.assert_close(Y2, ref, "partial + finish")
    _gpu.assert_close(Y3, ref, "plain forward after the halves")
    for hh in handles + [h]:
        binding.svdmlp_destroy(hh)
