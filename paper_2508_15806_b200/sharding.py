"""KV-head sharding of the compression step over several GPUs (one process per GPU, torch.distributed).

Every (sequence, KV head) segment of a layer is an independent problem through scoring, pooling, selection and
gather (Algorithm 3 runs per head), and the budgets are a deterministic function of a small replicated table
(Algorithm 2).  A tensor-parallel attention layer already holds its own KV heads' Q, K and V on each GPU, so each
rank compresses its heads with the ordinary entry points and no tensor data crosses NVLink.  The one thing a rank
cannot know alone is where its segments sit in the layer-wide packed cache: that takes the kept-row counts of the
other ranks' heads -- n_seqs * n_kv_heads int32 values per layer, exchanged with one all-gather (NCCL on GPUs, gloo
in the CPU tests).  This module holds that host logic; the kernels are the library's.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch


def head_range(n_kv_heads: int, rank: int, world: int) -> Tuple[int, int]:
    """The contiguous KV heads [h0, h1) of `rank`: as even as possible, the first ranks take the larger shares."""
    assert 0 <= rank < world and n_kv_heads >= 1
    base, extra = divmod(n_kv_heads, world)
    h0 = rank * base + min(rank, extra)
    return h0, h0 + base + (1 if rank < extra else 0)


def shard_inputs(q_win: torch.Tensor, k: torch.Tensor, v: torch.Tensor, budgets_row: torch.Tensor, h0: int, h1: int):
    """Views (no copies) of one layer's tensors restricted to KV heads [h0, h1) and their query heads.

    q_win [n_seqs, w, n_q_heads, d], k / v [T, n_kv_heads, d], budgets_row [n_kv_heads].  The library takes strided
    tensors, so a rank that holds the whole layer (tests) and a rank that holds only its heads (tensor parallelism)
    call it the same way.
    """
    G = q_win.shape[2] // k.shape[1]
    return q_win[:, :, h0 * G:h1 * G, :], k[:, h0:h1, :], v[:, h0:h1, :], budgets_row[h0:h1].contiguous()


def local_kept(offsets_local: torch.Tensor, n_seqs: int, n_heads_local: int) -> torch.Tensor:
    """Rows kept per (sequence, local head), int32 [n_seqs, n_heads_local], from a rank's own offsets array."""
    o = offsets_local.to(torch.int64)
    return (o[1:] - o[:-1]).reshape(n_seqs, n_heads_local).to(torch.int32)


def stitch(kept_per_rank: Sequence[torch.Tensor]) -> Tuple[torch.Tensor, List[torch.Tensor]]:
    """Layer-wide offsets from every rank's kept counts.

    kept_per_rank[r] is int32 [n_seqs, heads of rank r] (ranks in head order).  Returns (offsets int64
    [n_seqs * n_kv_heads + 1] in the library's segment order s * n_kv_heads + h, and per rank an int64
    [n_seqs, heads of rank r] tensor with the first row of each of its segments in the layer-wide packed cache).
    """
    kept = torch.cat([x.to(torch.int64) for x in kept_per_rank], dim=1)              # [n_seqs, n_kv_heads]
    flat = kept.reshape(-1)
    offsets = torch.zeros(flat.numel() + 1, dtype=torch.int64)
    offsets[1:] = torch.cumsum(flat, dim=0)
    starts = offsets[:-1].reshape(kept.shape)
    bases, h = [], 0
    for x in kept_per_rank:
        bases.append(starts[:, h:h + x.shape[1]].clone())
        h += x.shape[1]
    return offsets, bases


def all_gather_kept(kept_local: torch.Tensor, group=None) -> List[torch.Tensor]:
    """All ranks' kept counts (the only exchange of the head-sharded step).  Ranks may hold different numbers of heads:
    the counts travel padded to the largest share."""
    import torch.distributed as dist
    world = dist.get_world_size(group)
    n_seqs, n_loc = kept_local.shape
    sizes = [torch.zeros(1, dtype=torch.int64, device=kept_local.device) for _ in range(world)]
    dist.all_gather(sizes, torch.tensor([n_loc], dtype=torch.int64, device=kept_local.device), group=group)
    width = int(max(int(s.item()) for s in sizes))
    padded = torch.zeros(n_seqs, width, dtype=torch.int32, device=kept_local.device)
    padded[:, :n_loc] = kept_local
    out = [torch.empty_like(padded) for _ in range(world)]
    dist.all_gather(out, padded, group=group)
    return [o[:, :int(s.item())].cpu() for o, s in zip(out, sizes)]
