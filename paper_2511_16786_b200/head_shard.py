"""The compression pass with the KV heads of every layer split over the ranks (one process per GPU).

Scoring, selection and gathering are independent per (layer, sequence, head).  The one coupling is
the energy ratio of Eq. 12, which sums over all heads of a layer: each rank produces the four energy
sums of its own heads, one all-reduce (SUM) of the float64 [L, B, 4] array makes them whole, and every
rank then computes the same budgets.  A few kilobytes per prefill, latency-bound; "nccl" on GPUs,
"gloo" on CPU (used by the tests).
"""
from __future__ import annotations

import torch


def shard_heads(num_heads: int, world: int, rank: int):
    """[h0, h1): the contiguous block of KV heads rank `rank` owns; blocks differ by at most one head."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError("bad rank/world")
    base, extra = divmod(num_heads, world)
    h0 = rank * base + min(rank, extra)
    return h0, h0 + base + (1 if rank < extra else 0)


def allreduce_energy(energy: torch.Tensor, dist) -> torch.Tensor:
    """Sums the per-rank energy arrays [L, B, 4] in place over all ranks (no-op without a group)."""
    if dist is not None:
        dist.all_reduce(energy, op=dist.ReduceOp.SUM)
    return energy


class HeadShardedCompressor:
    """`Compressor` on this rank's heads with the energy exchange between scoring and allocation.
    K_layers/V_layers passed to `compress` hold only the local heads: [T, h1 - h0, d]."""

    def __init__(self, dist, rank: int, world: int, num_layers: int, num_heads: int, head_dim: int, cu_seqlens,
                 dtype, rho: float, gamma: float = 0.2, min_keep: int = 1, device: int = 0, **kw):
        from .binding import Compressor
        self.dist = dist
        self.h0, self.h1 = shard_heads(num_heads, world, rank)
        if self.h1 == self.h0:
            raise ValueError("more ranks than KV heads")
        # the energies must be complete in stream order before the exchange reads them
        self.local = Compressor(num_layers, self.h1 - self.h0, head_dim, cu_seqlens, dtype, rho, gamma, min_keep,
                                device=device, score_overlap=False, **kw)

    def compress(self, K_layers, V_layers):
        c = self.local
        c.score(K_layers, V_layers)
        allreduce_energy(c.energy, self.dist)       # on the current stream, after the scoring kernels
        c.allocate()
        c.select_compact(K_layers, V_layers)

    def close(self):
        self.local.close()
