"""Multi-GPU host logic: one process per GPU, the (sequence, KV head) units of a job sharded over the ranks.

Every unit of the SubGen cache is independent in update, prefill and query (Algorithm 1 is stated for one stream;
nothing couples heads or sequences), so ranks never exchange cache data. A job is cut either by sequence (every
rank serves some sequences with all their heads) or by KV head (every rank serves some KV heads, and the query
heads that share them, of every sequence). Each rank creates a handle for its shard with the unit numbering of the
whole job (`unit_stride`, `unit_offset` of the configuration), so that every Philox draw, and with it every sampled
index, is the one the unsharded job would take. The only data that ever crosses ranks is the step's output
[B, H, d], gathered where the next layer wants it replicated (`gather_outputs`), and, when timing, a barrier and a
MAX reduction of the measured time.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import torch


@dataclass(frozen=True)
class Shard:
    """What one rank serves of a job with B sequences, H query heads and Hkv KV heads per sequence."""
    rank: int
    world: int
    B: int
    H: int
    Hkv: int
    b0: int
    b1: int            # sequences [b0, b1)
    h0: int
    h1: int            # KV heads [h0, h1)

    @property
    def G(self) -> int:
        return self.H // self.Hkv

    @property
    def B_local(self) -> int:
        return self.b1 - self.b0

    @property
    def Hkv_local(self) -> int:
        return self.h1 - self.h0

    @property
    def H_local(self) -> int:
        return self.Hkv_local * self.G

    @property
    def empty(self) -> bool:
        return self.B_local == 0 or self.Hkv_local == 0

    @property
    def unit_stride(self) -> int:
        """Units per sequence in the whole job's numbering."""
        return self.Hkv

    @property
    def unit_offset(self) -> int:
        """Whole-job index of this shard's unit (local sequence 0, local KV head 0)."""
        return self.b0 * self.Hkv + self.h0

    def unit_id(self, seq_local: int, kvhead_local: int) -> int:
        """Whole-job unit index (the Philox counter's unit field) of a local unit."""
        return seq_local * self.unit_stride + self.unit_offset + kvhead_local

    def handle_kwargs(self) -> dict:
        """Shape and unit numbering of this shard's handle (keyword arguments of binding.SubGen besides d, delta, ...)."""
        return dict(B=self.B_local, H=self.H_local, Hkv=self.Hkv_local, unit_stride=self.unit_stride, unit_offset=self.unit_offset)

    # slices of whole-job tensors --------------------------------------------------------------
    def q_rows(self, q: torch.Tensor) -> torch.Tensor:
        """[B, H, ...] -> this shard's [B_local, H_local, ...] (query heads follow their KV heads)."""
        return q[self.b0:self.b1, self.h0 * self.G:self.h1 * self.G].contiguous()

    def kv_rows(self, k: torch.Tensor) -> torch.Tensor:
        """[B, Hkv, ...] -> this shard's [B_local, Hkv_local, ...] (new tokens [B, Hkv, d] or prompts [B, Hkv, n, d])."""
        return k[self.b0:self.b1, self.h0:self.h1].contiguous()


def partition(B: int, H: int, Hkv: int, world: int, mode: str = "auto") -> List[Shard]:
    """Cut a job over `world` ranks. mode "sequence": contiguous runs of sequences whose sizes differ by at most one
    (ranks beyond B get nothing); "head": Hkv / world KV heads each (world must divide Hkv); "auto": by sequence when
    every rank gets one, else by head."""
    if world < 1 or B < 1 or Hkv < 1 or H % Hkv:
        raise ValueError("need world >= 1, B >= 1, Hkv >= 1 and H a multiple of Hkv")
    if mode == "auto":
        mode = "sequence" if B >= world or Hkv % world else "head"
    if mode == "sequence":
        base, extra = divmod(B, world)
        out, b0 = [], 0
        for r in range(world):
            b1 = b0 + base + (1 if r < extra else 0)
            out.append(Shard(r, world, B, H, Hkv, b0, b1, 0, Hkv))
            b0 = b1
        return out
    if mode == "head":
        if Hkv % world:
            raise ValueError("head sharding needs the number of ranks to divide Hkv")
        per = Hkv // world
        return [Shard(r, world, B, H, Hkv, 0, B, r * per, (r + 1) * per) for r in range(world)]
    raise ValueError("mode must be 'auto', 'sequence' or 'head'")


def scatter_outputs(full: torch.Tensor, shard: Shard, out_local: torch.Tensor) -> None:
    """Write a shard's [B_local, H_local, d] output into its place in the whole job's [B, H, d]."""
    if not shard.empty:
        full[shard.b0:shard.b1, shard.h0 * shard.G:shard.h1 * shard.G] = out_local


def gather_outputs(out_local: torch.Tensor, shards: Sequence[Shard], rank: int, dist=None) -> torch.Tensor:
    """All ranks' step outputs as the whole job's [B, H, d] on every rank (the one exchange a sharded layer needs).

    Shards may differ in size (sequence mode with B not a multiple of the world size), so every rank contributes a
    buffer padded to the largest shard and the rows are put in place from the partition. Without a process group the
    call expects a single shard and returns its output."""
    me = shards[rank]
    d = out_local.shape[-1]
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        if len(shards) != 1:
            raise ValueError("several shards need a process group")
        return out_local
    rows = max(s.B_local * s.H_local for s in shards)
    mine = torch.zeros(rows, d, dtype=out_local.dtype, device=out_local.device)
    if not me.empty:
        mine[: me.B_local * me.H_local] = out_local.reshape(-1, d)
    parts = [torch.empty_like(mine) for _ in shards]
    dist.all_gather(parts, mine)
    full = torch.empty(me.B, me.H, d, dtype=out_local.dtype, device=out_local.device)
    for s, p in zip(shards, parts):
        scatter_outputs(full, s, p[: s.B_local * s.H_local].reshape(s.B_local, s.H_local, d))
    return full


# ---- benchmark helpers (weak scaling: every rank serves a batch of its own) ---------------------------------
def rank_workload(w, rank: int):
    """The batch of sequences rank `rank` serves: same shape, its own seeded data."""
    return w.scaled(data_seed=w.data_seed + 7919 * int(rank))


def max_over_ranks(value: float, dist=None, device: Optional[str] = None) -> float:
    """MAX of a host scalar over all ranks (identity without a process group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_steps_per_s(world: int, steps_per_rank: int, slowest_ms: float) -> float:
    """Whole-job throughput: every rank advanced its batch by steps_per_rank steps within slowest_ms."""
    return world * steps_per_rank / (slowest_ms * 1e-3)
