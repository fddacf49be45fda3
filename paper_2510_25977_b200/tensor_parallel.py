"""Tensor parallelism over ffn for the factored MLP (host logic; the kernels are those of the single-GPU path).

Shard g of G holds the rows Ug[F_g], Uu[F_g] and the columns Vd[:, F_g] of a contiguous slice F_g of ffn,
and Vg, Vu, Ud whole.  Every rank computes the narrow first projection redundantly, its slice of H and its
partial fp32 Zd_g = H[:, F_g] Vd[:, F_g]^T; one all-reduce of Zd[T, r_down] (fp32, r_down / d of the bytes an
all-reduce of Y would move) and every rank finishes Y = Zd Ud^T on its own.
"""
from __future__ import annotations


def shard_ffn(ffn: int, world: int, rank: int, align: int = 128) -> tuple[int, int]:
    """Slice [begin, end) of ffn for `rank`: whole `align`-column tiles, sizes differing by at most one tile."""
    if ffn < 0 or world <= 0 or not (0 <= rank < world):
        raise ValueError("bad shard request")
    tiles = (ffn + align - 1) // align
    base, extra = divmod(tiles, world)
    first = rank * base + min(rank, extra)
    count = base + (1 if rank < extra else 0)
    return min(ffn, first * align), min(ffn, (first + count) * align)


def shard_factors(Ug, Vg, Uu, Vu, Ud, Vd, world: int, rank: int):
    """The six factor tensors of one shard, contiguous (Vd's column slice is copied)."""
    lo, hi = shard_ffn(Ug.shape[0], world, rank)
    return (Ug[lo:hi].contiguous(), Vg, Uu[lo:hi].contiguous(), Vu, Ud, Vd[:, lo:hi].contiguous())


def forward(binding, handle, X, dist=None, Y=None, stream=None):
    """One tensor-parallel forward on this rank: partial Zd, all-reduce (NCCL through torch.distributed), finish."""
    Zd = binding.svdmlp_forward_partial(handle, X, stream=stream)
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(Zd)
    return binding.svdmlp_forward_finish(handle, Zd, Y, stream=stream)


class Exchange:
    """Receive buffers and flag words for the library's own exchange (svdmlp_forward_partial_push /
    svdmlp_forward_finish_gather).  `ranks_on_this_device` > 0 builds the buffers of ALL ranks on the current device:
    the single-GPU form used by the tests, where the ranks' calls run one after the other on one stream (a push
    never waits, so nothing can block).  Across GPUs every process allocates its own pair and passes the peers'
    mapped addresses (peer access, IPC handles or symmetric memory) to `binding.tp_peers` itself."""

    def __init__(self, binding, world: int, max_T: int, r_down: int, device="cuda"):
        import torch
        n = binding.svdmlp_tp_recv_bytes(world, max_T, r_down) // 4
        self.world = world
        self.recv = [torch.zeros(n, dtype=torch.float32, device=device) for _ in range(world)]
        self.flags = [torch.zeros(world, dtype=torch.int64, device=device) for _ in range(world)]
        self.step = 0
        self._binding = binding

    def peers(self, rank: int):
        return self._binding.tp_peers(rank, [t.data_ptr() for t in self.recv], [t.data_ptr() for t in self.flags])


def forward_all_ranks_on_one_device(binding, handles, X, ex: Exchange, stream=None):
    """One tensor-parallel step with every rank's handle on this device: all pushes, then all gathers.  Returns the G
    outputs (they are equal up to nothing: every rank sums the same G slots in the same order)."""
    ex.step += 1
    T = X.shape[0]
    for g, h in enumerate(handles):
        binding.svdmlp_forward_partial_push(h, X, ex.peers(g), ex.step, stream=stream)
    return [binding.svdmlp_forward_finish_gather(h, ex.recv[g], ex.flags[g], ex.world, ex.step, T, stream=stream)
            for g, h in enumerate(handles)]
