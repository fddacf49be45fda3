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
