"""Context-parallel compression of ONE long sequence (Sec. 3.4, Eq. 7-8; Algorithm 3): the per-rank call sequence of
the slkv_cp_* entry points with the collectives between them.

The history keys are split over the ranks by contiguous ranges; the last rank also holds the window rows.  Every step
of the arithmetic runs in the library's kernels; this module slices the rank's views, allocates its buffers and calls
the three kinds of collective the method needs per layer:
    all-gather of the rows' local log-sum-exps   [n_q_heads, window] float32
    3 x all-reduce (sum) of a radix histogram    [n_kv_heads, 2048] int32
    all-gather of the tie counts                 [n_kv_heads] int32
`comm` is anything with rank, world, all_gather(tensor) -> [world, ...] and all_reduce_sum(tensor) (in place):
DistComm wraps torch.distributed (NCCL for CUDA tensors, gloo for CPU tensors); tests emulate several ranks on one GPU
with a thread-and-barrier comm of their own.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import torch

from . import binding as B


def key_ranges(seq_len: int, window: int, world: int) -> List[Tuple[int, int]]:
    """History positions [b, e) of every rank: the n_hist = seq_len - window history keys in `world` near-equal
    contiguous shares (the first n_hist % world ranks hold one more); the last rank also holds the window rows."""
    n_hist = max(seq_len - window, 0)
    base, extra = divmod(n_hist, world)
    out, b = [], 0
    for r in range(world):
        e = b + base + (1 if r < extra else 0)
        out.append((b, e))
        b = e
    return out


class DistComm:
    """torch.distributed as the communicator (one process per GPU; NCCL moves CUDA tensors, gloo CPU tensors)."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self._dist, self._group = dist, group
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)

    def all_gather(self, t: torch.Tensor) -> torch.Tensor:
        out = torch.empty(self.world * t.numel(), dtype=t.dtype, device=t.device)
        self._dist.all_gather_into_tensor(out, t.contiguous().reshape(-1), group=self._group)
        return out.reshape((self.world,) + tuple(t.shape))

    def all_reduce_sum(self, t: torch.Tensor) -> torch.Tensor:
        self._dist.all_reduce(t, op=self._dist.ReduceOp.SUM, group=self._group)
        return t


@dataclass
class RankShard:
    """What one rank holds of a layer: q_win [1, window, n_q_heads, d]; k, v [rows, n_kv_heads, d] = the history
    positions [begin - margin_left, end + margin_right) and, on the last rank, the window rows behind them."""
    rank: int
    world: int
    seq_len: int
    window: int
    begin: int
    end: int
    margin_left: int
    margin_right: int
    q_win: torch.Tensor
    k: torch.Tensor
    v: torch.Tensor

    @property
    def last(self) -> bool:
        return self.rank == self.world - 1

    @property
    def own(self) -> int:
        return self.end - self.begin


def shard_of(q_win: torch.Tensor, k: torch.Tensor, v: torch.Tensor, window: int, pool_kernel: int, rank: int,
             world: int) -> RankShard:
    """The rank's views of a whole sequence's q_win [1, w, Hq, d], k, v [seq_len, Hkv, d] (for callers and tests that
    hold the whole sequence; a context-parallel prefill already holds each rank's rows and fills RankShard itself)."""
    seq_len = k.shape[0]
    n_hist = max(seq_len - window, 0)
    b, e = key_ranges(seq_len, window, world)[rank]
    ml = min(pool_kernel // 2, b)
    mr = 0 if rank == world - 1 else min(pool_kernel // 2, n_hist - e)
    hi = seq_len if rank == world - 1 else e + mr
    return RankShard(rank, world, seq_len, window, b, e, ml, mr, q_win, k[b - ml:hi], v[b - ml:hi])


def compress_rank(shard: RankShard, budgets_row: torch.Tensor, pool_kernel: int, comm, pool_mode: int = B.SLKV_POOL_MAX,
                  softmax_domain: int = B.SLKV_HISTORY, score_path: int = B.SLKV_PATH_AUTO, stream=None) -> dict:
    """One layer on one rank.  budgets_row: CUDA int32 [n_kv_heads], the layer's budgets (the same on every rank).
    Returns this rank's packed rows: k_out, v_out [capacity, d], offsets [n_kv_heads + 1] (local), kept_idx (positions
    in the whole sequence), status, pooled (the rank's scores, margins included) and lse (the merged row statistics)."""
    sh = shard
    assert sh.seq_len >= sh.window and comm.world == sh.world and comm.rank == sh.rank
    dev = sh.k.device
    w, hkv, hq, d = sh.window, sh.k.shape[1], sh.q_win.shape[2], sh.k.shape[2]
    f32, i32 = dict(dtype=torch.float32, device=dev), dict(dtype=torch.int32, device=dev)
    n_win = w if sh.last else 0
    status = torch.zeros(1, **i32)
    cu_dev1 = torch.zeros(2, **i32)              # one sequence: the library's tables are inline, this is never read

    def params_for(k_rows: torch.Tensor, history_only: bool) -> B.SlkvParams:
        p = B.make_params(sh.q_win, k_rows, None, w, pool_kernel, pool_mode, score_path, softmax_domain, B.SLKV_LSE_LOG2)
        p.history_only = 1 if history_only else 0
        return p

    # 1. the rows' log-sum-exp over the keys this rank owns (the last rank's range is an ordinary sequence tail)
    k_own = sh.k[sh.margin_left:sh.margin_left + sh.own + n_win]
    lse_local = torch.full((1, hq, w), float("-inf"), **f32)
    if sh.own > 0 or (sh.last and softmax_domain == B.SLKV_ALL_CAUSAL):
        p_own = params_for(k_own, not sh.last)
        cu = [0, k_own.shape[0]]
        ws = torch.empty(max(B.slkv_workspace_bytes(p_own, cu), 256), dtype=torch.uint8, device=dev)
        B.slkv_row_lse(p_own, sh.q_win, k_own, cu_dev1, cu, lse_local, ws, status, stream)
    # 2. merged over the ranks
    lse = torch.empty(1, hq, w, **f32)
    p_any = params_for(sh.k, not sh.last)
    B.slkv_cp_merge_lse(p_any, comm.all_gather(lse_local.reshape(hq, w)), lse, stream)
    # 3. pooled scores of the owned rows and the neighbours' margins
    n_ext = sh.margin_left + sh.own + sh.margin_right
    pooled = torch.zeros(hkv * max(n_ext, 1), **f32)
    if n_ext > 0:
        cu = [0, sh.k.shape[0]]
        ws = torch.empty(max(B.slkv_workspace_bytes(p_any, cu), 256), dtype=torch.uint8, device=dev)
        B.slkv_score(p_any, sh.q_win, sh.k, cu_dev1, cu, pooled, ws, status, stream, lse=lse)
    # 4. every head's threshold: radix descent on histograms summed over the ranks
    prefix, need = torch.zeros(hkv, **i32), torch.zeros(hkv, **i32)
    B.slkv_cp_select_init(budgets_row, w, sh.seq_len, prefix, need, stream)
    hist = torch.empty(hkv, 2048, **i32)
    hist_own = hist
    for level in range(3):
        B.slkv_cp_histogram(pooled, hkv, max(n_ext, 1), sh.margin_left, sh.own, level, prefix, hist, stream)
        if level == 2:
            hist_own = hist.clone()
        comm.all_reduce_sum(hist)
        B.slkv_cp_descend(hist, level, prefix, need, stream)
    # 5. ties in rank order, then this rank's packed rows
    ties = torch.empty(hkv, **i32)
    B.slkv_cp_local_ties(hist_own, prefix, ties, stream)
    ties_all = comm.all_gather(ties)
    cap = hkv * (sh.own + n_win)
    out = dict(k_out=torch.zeros(max(cap, 1), d, dtype=sh.k.dtype, device=dev),
               v_out=torch.zeros(max(cap, 1), d, dtype=sh.k.dtype, device=dev),
               offsets=torch.zeros(hkv + 1, **i32), kept_idx=torch.full((max(cap, 1),), -1, **i32), status=status,
               pooled=pooled, lse=lse, capacity=cap)
    ws = torch.empty(max(B.slkv_cp_workspace_bytes(hkv, sh.own, max(cap, 1)), 256), dtype=torch.uint8, device=dev)
    B.slkv_cp_emit(p_any, sh.k, sh.v, sh.k.shape[0], pooled, max(n_ext, 1), sh.margin_left, sh.own, sh.begin, prefix,
                   need, ties_all, sh.rank, n_win, sh.seq_len - n_win, out["k_out"], out["v_out"], out["offsets"],
                   out["kept_idx"], ws, status, stream)
    out["keep_alive"] = (ws, hist, hist_own, ties_all, prefix, need, lse_local)
    return out


def stitch_heads(per_rank: Sequence[dict], n_kv_heads: int) -> List[dict]:
    """Per KV head, the whole sequence's packed cache from the ranks' outputs (rank order = position order): for
    callers that bring the ranks' rows together, and for tests.  Returns [{"kept_idx", "k", "v"}] per head."""
    heads = []
    for h in range(n_kv_heads):
        idx, ks, vs = [], [], []
        for o in per_rank:
            a, b = int(o["offsets"][h]), int(o["offsets"][h + 1])
            idx.append(o["kept_idx"][a:b])
            ks.append(o["k_out"][a:b])
            vs.append(o["v_out"][a:b])
        heads.append(dict(kept_idx=torch.cat(idx), k=torch.cat(ks), v=torch.cat(vs)))
    return heads
