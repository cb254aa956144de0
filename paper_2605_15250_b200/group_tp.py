"""Group-axis tensor parallelism of the GQA path (Sec. 3.2, "Merging grouped heads to a latent head":
W^UK, W^UV stay indexed by the group j, so the GQA path keeps the group axis that MLA loses once its
up-projections are absorbed).

Rank r of `world` owns the groups [r*g/world, (r+1)*g/world) and their h_q/world query heads.  It keeps
its groups' slices of W^UK / W^UV, expands the (replicated) latent cache into K_C, V for its groups only,
and reads the shared 64-wide k^R from the latent cache's tail: no K/V element is stored twice across
ranks except k^R.  The attention of a rank needs nothing from the others -- the only exchange of the
layer is the all-reduce after W^O, which is outside the decode path -- so this module contains index
arithmetic and no collective.  Every rank-local problem is an ordinary GQLA problem with dims
(h_q/world, g/world, d_h, r_kv, d_r), which the library takes as it is.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

from .decoder import GqlaDecoder


@dataclass(frozen=True)
class GroupShard:
    rank: int
    world: int
    h_q: int  # global head count
    g: int    # global group count

    def __post_init__(self):
        if self.world < 1 or not 0 <= self.rank < self.world:
            raise ValueError("rank outside the world")
        if self.g % self.world != 0 or self.h_q % self.g != 0:
            raise ValueError("the group count must be a multiple of the world size (and h_q of g)")

    @property
    def g_local(self) -> int:
        return self.g // self.world

    @property
    def h_local(self) -> int:
        return self.h_q // self.world

    @property
    def groups(self) -> slice:
        return slice(self.rank * self.g_local, (self.rank + 1) * self.g_local)

    @property
    def heads(self) -> slice:
        """Heads of the rank's groups: head i belongs to group i // (h_q/g), so they are contiguous."""
        return slice(self.rank * self.h_local, (self.rank + 1) * self.h_local)

    def cache_elems_per_token(self, d_h: int, d_r: int) -> int:
        """Expanded-cache elements a rank stores per token: its groups' K_C and V, plus the shared k^R."""
        return 2 * self.g_local * d_h + d_r

    def slice_weights(self, w: torch.Tensor) -> torch.Tensor:
        """W^UK or W^UV [g, r_kv, d_h] -> the rank's [g/world, r_kv, d_h] (a contiguous view)."""
        return w[self.groups]

    def slice_queries(self, q: torch.Tensor) -> torch.Tensor:
        """q [B, s_q, h_q, d] -> the rank's heads, copied to a contiguous tensor."""
        return q[:, :, self.heads].contiguous()


def shard_decoder(shard: GroupShard, d_h: int, r_kv: int, d_r: int, w_uk: torch.Tensor, w_uv: torch.Tensor,
                  cache: torch.Tensor, seq_start: torch.Tensor, seqlens: torch.Tensor, scale: float) -> GqlaDecoder:
    """The rank's decoder: local dims, its weight slices, the replicated latent cache."""
    return GqlaDecoder(shard.h_local, shard.g_local, d_h, r_kv, d_r, shard.slice_weights(w_uk), shard.slice_weights(w_uv),
                       cache, seq_start, seqlens, scale)


def gather_heads(parts: list[torch.Tensor]) -> torch.Tensor:
    """Outputs [B, s_q, h_q/world, d] of ranks 0..world-1 -> [B, s_q, h_q, d] (what W^O's input would be
    if it were not sharded along the same axis)."""
    return torch.cat(parts, dim=2)
