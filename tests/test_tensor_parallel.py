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


@pytest.mark.gpu
@pytest.mark.parametrize("T", [8, 27, 300])
@pytest.mark.parametrize("world", [2, 4])
def test_exchange_by_the_librarys_own_kernels(oracle, T, world):
    """svdmlp_forward_partial_push / svdmlp_forward_finish_gather with every rank's buffers on this one device: the
    ranks' calls run one after the other on one stream, so no kernel ever waits for a later one.  Three steps in a
    row use both halves of the two-deep receive buffers; every rank must produce the same bits (all sum the same
    slots in the same order) and match the oracle."""
    import _gpu
    from paper_2510_25977_b200 import binding
    _gpu.require_gpu()
    d, ffn, r = 512, 1408, 64
    f = inputs.direct_factors(d, ffn, r, seed=6, device="cuda")
    handles = [binding.svdmlp_create(*tp.shard_factors(*f.tensors(), world, g), max_T=T) for g in range(world)]
    ex = tp.Exchange(binding, world, T, r)
    try:
        for step in range(3):
            X = inputs.activations(T, d, seed=60 + step, device="cuda")
            Ys = tp.forward_all_ranks_on_one_device(binding, handles, X, ex)
            torch.cuda.synchronize()
            for h in handles:
                assert binding.svdmlp_last_device_status(h) == 0
            for Y in Ys[1:]:
                assert torch.equal(Y, Ys[0])
            _gpu.assert_close(Ys[0], oracle.svdmlp(X, *f.tensors()), f"exchange x{world}, T={T}, step {step + 1}")
        assert all(int(v) == 3 for fl in ex.flags for v in fl.tolist())
    finally:
        for h in handles:
            binding.svdmlp_destroy(h)


@pytest.mark.gpu
def test_exchange_gather_gives_up_when_a_peer_never_pushes():
    """Failure detection without a fault: rank 1 never pushes step 1, rank 0's gather waits out its (shortened) limit,
    sets the status word and returns; the context stays usable and a later complete step succeeds."""
    import _gpu
    from paper_2510_25977_b200 import binding
    _gpu.require_gpu()
    d, ffn, r, T, world = 256, 768, 32, 8, 2
    f = inputs.direct_factors(d, ffn, r, seed=7, device="cuda")
    X = inputs.activations(T, d, seed=7, device="cuda")
    handles = [binding.svdmlp_create(*tp.shard_factors(*f.tensors(), world, g), max_T=T) for g in range(world)]
    ex = tp.Exchange(binding, world, T, r)
    try:
        binding.svdmlp_tp_wait_limit_ns(handles[0], 20_000_000)          # 20 ms
        binding.svdmlp_forward_partial_push(handles[0], X, ex.peers(0), 1)
        binding.svdmlp_forward_finish_gather(handles[0], ex.recv[0], ex.flags[0], world, 1, T)
        torch.cuda.synchronize()
        assert binding.svdmlp_last_device_status(handles[0]) == -7
        assert binding.svdmlp_last_device_status(handles[0]) == 0        # cleared by the read
        ex.step = 1                                                      # step 1 is lost; both ranks go on with step 2
        Ys = tp.forward_all_ranks_on_one_device(binding, handles, X, ex)
        torch.cuda.synchronize()
        assert binding.svdmlp_last_device_status(handles[0]) == 0 and torch.equal(Ys[0], Ys[1])
        assert torch.isfinite(Ys[0].float()).all()
    finally:
        for h in handles:
            binding.svdmlp_destroy(h)


def test_exchange_argument_checks():
    from paper_2510_25977_b200 import binding, build
    build.build()
    L = binding.lib()
    assert L.svdmlp_tp_recv_bytes(2, 8, 32) == 2 * 2 * 8 * 32 * 4
    assert L.svdmlp_tp_recv_bytes(9, 8, 32) == 0 and L.svdmlp_tp_recv_bytes(0, 8, 32) == 0
    assert L.svdmlp_forward_partial_push(None, None, 1, None, 1, None) == -1
    assert L.svdmlp_forward_finish_gather(None, None, None, 2, 1, 1, None, None) == -1
