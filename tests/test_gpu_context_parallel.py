"""GPU parity: one sequence compressed with its history keys split over several ranks (Sec. 3.4, Eq. 7-8; Algorithm 3)
against the oracle's result for the whole sequence.

One GPU: the ranks are host threads with a stream each; their collectives are a barrier and a shared list (no kernel
waits for another: every exchange is host-side, between launches).  The same per-rank code runs under torch.distributed.
"""
import threading

import numpy as np
import pytest
import torch

from oracle import slkv_oracle as O
from paper_2508_15806_b200 import binding as B
from paper_2508_15806_b200 import context_parallel as CP
import parity as P

pytestmark = pytest.mark.gpu

DEV = torch.device("cuda:0")


class ThreadComm:
    """`world` ranks in one process: all_gather = publish, barrier, read; all_reduce = gather and add."""

    class Shared:
        def __init__(self, world):
            self.world, self.barrier, self.slots = world, threading.Barrier(world, timeout=120), [None] * world

    def __init__(self, shared, rank):
        self.s, self.rank, self.world = shared, rank, shared.world

    def all_gather(self, t):
        torch.cuda.current_stream().synchronize()        # the value is complete before another rank's stream reads it
        self.s.slots[self.rank] = t
        self.s.barrier.wait()
        out = torch.stack([x for x in self.s.slots])
        torch.cuda.current_stream().synchronize()
        self.s.barrier.wait()                             # nobody overwrites a slot that is still being read
        return out

    def all_reduce_sum(self, t):
        t.copy_(self.all_gather(t.clone()).sum(0).to(t.dtype))
        return t


def run_ranks(world, q, k, v, budgets_row, w, p, **kw):
    shared = ThreadComm.Shared(world)
    outs, errors = [None] * world, []
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    bud = torch.tensor(list(budgets_row), dtype=torch.int32, device=DEV)
    torch.cuda.synchronize()

    def worker(r):
        try:
            torch.cuda.set_device(0)
            with torch.cuda.stream(torch.cuda.Stream()):
                shard = CP.shard_of(qd, kd, vd, w, p, r, world)
                outs[r] = CP.compress_rank(shard, bud, p, ThreadComm(shared, r), **kw)
                torch.cuda.current_stream().synchronize()
        except Exception as e:                              # noqa: BLE001 - reported in the main thread
            errors.append((r, e))
            shared.barrier.abort()

    threads = [threading.Thread(target=worker, args=(r,)) for r in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=300)
    assert not errors, errors
    torch.cuda.synchronize()
    return outs


def as_one_layer(outs, world, seq_len, w, p, n_kv):
    """The ranks' outputs in the layout of a single-GPU call: pooled per head over the whole history, offsets,
    kept_idx, k_out, v_out with segment h = head h."""
    pooled = []
    for h in range(n_kv):
        parts = []
        for r, o in enumerate(outs):
            b, e = CP.key_ranges(seq_len, w, world)[r]
            ml = min(p // 2, b)
            n_hist = seq_len - w
            mr = 0 if r == world - 1 else min(p // 2, n_hist - e)
            n_ext = ml + (e - b) + mr
            row = o["pooled"][:n_kv * max(n_ext, 1)].reshape(n_kv, max(n_ext, 1))[h]
            parts.append(row[ml:ml + (e - b)])
        pooled.append(torch.cat(parts))
    heads = CP.stitch_heads(outs, n_kv)
    offsets = np.cumsum([0] + [int(hd["kept_idx"].numel()) for hd in heads])
    return {"pooled": torch.cat(pooled).cpu().numpy(), "offsets": offsets.astype(np.int64),
            "kept_idx": torch.cat([hd["kept_idx"] for hd in heads]).cpu().numpy().astype(np.int64),
            "k_out": torch.cat([hd["k"] for hd in heads]).cpu(), "v_out": torch.cat([hd["v"] for hd in heads]).cpu()}


def rand_seq(Hq, Hkv, w, L, seed, d=128, dtype=torch.bfloat16, scale=1.2):
    g = torch.Generator().manual_seed(seed)
    q = (torch.randn(1, w, Hq, d, generator=g) * scale).to(dtype)
    k = (torch.randn(L, Hkv, d, generator=g) * scale).to(dtype)
    v = torch.randn(L, Hkv, d, generator=g).to(dtype)
    return q, k, v


CASES = [
    # Hq, Hkv, w, L, d, dtype, path, p, pool, domain, worlds
    (8, 2, 32, 6000, 128, torch.bfloat16, B.SLKV_PATH_TENSOR, 7, B.SLKV_POOL_MAX, B.SLKV_HISTORY, (1, 2, 3, 4)),
    (8, 2, 32, 3333, 128, torch.bfloat16, B.SLKV_PATH_TENSOR, 5, B.SLKV_POOL_MAX, B.SLKV_ALL_CAUSAL, (2, 5)),
    (8, 2, 64, 2500, 128, torch.bfloat16, B.SLKV_PATH_TENSOR, 7, B.SLKV_POOL_AVG, B.SLKV_HISTORY, (3,)),     # R = 256
    (8, 8, 16, 1500, 64, torch.float32, B.SLKV_PATH_SIMT, 5, B.SLKV_POOL_MAX, B.SLKV_HISTORY, (3,)),
    (8, 8, 16, 700, 64, torch.float32, B.SLKV_PATH_SIMT, 9, B.SLKV_POOL_AVG, B.SLKV_ALL_CAUSAL, (2, 4)),
]


@pytest.mark.parametrize("Hq,Hkv,w,L,d,dtype,path,p,pool,domain,worlds", CASES)
def test_ranks_together_match_the_oracle_on_the_whole_sequence(Hq, Hkv, w, L, d, dtype, path, p, pool, domain, worlds):
    q, k, v = rand_seq(Hq, Hkv, w, L, seed=L + w, d=d, dtype=dtype)
    cu = [0, L]
    # budgets: below the window (keeps the window only), ordinary ones, one above the sequence length (keeps all)
    bud = [w - 3, w + 40] + [w + 100 + 57 * h for h in range(Hkv - 2)]
    bud[-1] = L + 10 if Hkv > 2 else bud[-1]
    ref = P.oracle_pooled(q, k, cu, w, p, pool, domain)
    for world in worlds:
        outs = run_ranks(world, q, k, v, bud, w, p, pool_mode=pool, softmax_domain=domain, score_path=path)
        assert all(int(o["status"].item()) == 0 for o in outs)
        gpu = as_one_layer(outs, world, L, w, p, Hkv)
        P.assert_pooled_close(gpu["pooled"], ref, cu, Hkv, w)
        P.assert_selection_valid(gpu, ref, cu, bud, w, k, v)


def test_more_ranks_than_a_short_history_has_keys():
    # 3 history keys over 5 ranks: two ranks own nothing, the last one owns only the window rows
    Hq, Hkv, w, L, p = 8, 2, 32, 35, 5
    q, k, v = rand_seq(Hq, Hkv, w, L, seed=7)
    bud = [w + 1, w + 2]
    ref = P.oracle_pooled(q, k, [0, L], w, p)
    outs = run_ranks(5, q, k, v, bud, w, p, score_path=B.SLKV_PATH_TENSOR)
    gpu = as_one_layer(outs, 5, L, w, p, Hkv)
    P.assert_pooled_close(gpu["pooled"], ref, [0, L], Hkv, w)
    P.assert_selection_valid(gpu, ref, [0, L], bud, w, k, v)


@pytest.mark.parametrize("seed", range(6))
def test_selection_is_exact_on_given_scores_with_many_ties(seed):
    # the select-and-pack steps alone, fed with scores of few distinct values: the kept set must be exactly the k
    # largest with ties to the lowest positions, whatever the split (ranks run one after the other here; sums and
    # gathers of the tiny tables are done by the test, as a communicator would)
    rng = np.random.default_rng(seed)
    n_kv, w, d = 3, 8, 64
    world = int(rng.integers(1, 6))
    n_hist = int(rng.integers(50, 9000))
    L = n_hist + w
    scores = rng.choice(np.array([0.0, 0.25, 0.5, 1.0, 3.0, 1e-30, 7.5], dtype=np.float32), size=(n_kv, n_hist))
    if seed % 2:
        scores = rng.random((n_kv, n_hist)).astype(np.float32)
        m = scores[:, 1::3].shape[1]
        scores[:, 0:3 * m:3] = scores[:, 1::3]                              # duplicates among distinct values
    budgets = [w + int(rng.integers(0, n_hist + 1)), w - 2, L + 5]
    k = torch.randn(L, n_kv, d, device=DEV)
    v = torch.randn(L, n_kv, d, device=DEV)
    q = torch.zeros(1, w, n_kv, d, device=DEV)
    bud = torch.tensor(budgets, dtype=torch.int32, device=DEV)
    ranges = CP.key_ranges(L, w, world)
    i32 = dict(dtype=torch.int32, device=DEV)
    st = []
    for r, (b, e) in enumerate(ranges):
        ml, mr = min(2, b), (0 if r == world - 1 else min(2, n_hist - e))
        ext = np.zeros((n_kv, max(ml + e - b + mr, 1)), dtype=np.float32)
        ext[:, :ml + e - b + mr] = scores[:, b - ml:e + mr]
        prefix, need = torch.zeros(n_kv, **i32), torch.zeros(n_kv, **i32)
        B.slkv_cp_select_init(bud, w, L, prefix, need)
        st.append(dict(b=b, e=e, ml=ml, mr=mr, pooled=torch.from_numpy(ext).to(DEV).contiguous(), prefix=prefix,
                       need=need, hist=torch.empty(n_kv, 2048, **i32)))
    for level in range(3):
        for s in st:
            B.slkv_cp_histogram(s["pooled"], n_kv, s["pooled"].shape[1], s["ml"], s["e"] - s["b"], level, s["prefix"],
                                s["hist"])
            if level == 2:
                s["own"] = s["hist"].clone()
        total = torch.stack([s["hist"] for s in st]).sum(0).to(torch.int32)
        for s in st:
            B.slkv_cp_descend(total, level, s["prefix"], s["need"])
    ties_all = torch.stack([B.slkv_cp_local_ties(s["own"], s["prefix"], torch.empty(n_kv, **i32)) for s in st]).contiguous()
    kept = [[] for _ in range(n_kv)]
    for r, s in enumerate(st):
        last = r == world - 1
        lo, hi = s["b"] - s["ml"], (L if last else s["e"] + s["mr"])
        kr, vr = k[lo:hi].contiguous(), v[lo:hi].contiguous()
        p = B.make_params(q, kr, vr, w, 5)
        p.history_only = 0 if last else 1
        cap = n_kv * (s["e"] - s["b"] + (w if last else 0))
        o = dict(k=torch.zeros(max(cap, 1), d, device=DEV), v=torch.zeros(max(cap, 1), d, device=DEV),
                 off=torch.zeros(n_kv + 1, **i32), idx=torch.full((max(cap, 1),), -1, **i32), status=torch.zeros(1, **i32))
        ws = torch.empty(max(B.slkv_cp_workspace_bytes(n_kv, s["e"] - s["b"], max(cap, 1)), 256), dtype=torch.uint8, device=DEV)
        B.slkv_cp_emit(p, kr, vr, kr.shape[0], s["pooled"], s["pooled"].shape[1], s["ml"], s["e"] - s["b"], s["b"],
                       s["prefix"], s["need"], ties_all, r, w if last else 0, L - w, o["k"], o["v"], o["off"], o["idx"],
                       ws, o["status"])
        torch.cuda.synchronize()
        assert int(o["status"].item()) == 0
        for h in range(n_kv):
            a, bb = int(o["off"][h]), int(o["off"][h + 1])
            idx = o["idx"][a:bb].cpu().numpy()
            kept[h].append(idx)
            assert torch.equal(o["k"][a:bb], k[idx, h]) and torch.equal(o["v"][a:bb], v[idx, h])     # bit copies
    for h in range(n_kv):
        kh, nw = O.kept_counts(L, budgets[h], w)
        want = np.concatenate([O.select_topk(scores[h].astype(np.float64), kh), np.arange(L - nw, L)])
        assert np.array_equal(np.concatenate(kept[h]), want), (h, world, n_hist)


@pytest.mark.parametrize("path,dtype,d,w,Hq,Hkv", [(B.SLKV_PATH_TENSOR, torch.bfloat16, 128, 32, 8, 2),
                                                   (B.SLKV_PATH_SIMT, torch.float32, 64, 16, 8, 8)])
def test_history_only_rows_score_as_the_history_of_a_longer_sequence(path, dtype, d, w, Hq, Hkv):
    # K holds history rows only (history_only = 1): same votes, pooled scores and row log-sum-exps as the oracle gives
    # for a sequence of those rows followed by `w` window rows (which the history-only softmax never reads as keys)
    n, p = 1777, 5
    q, k, _ = rand_seq(Hq, Hkv, w, n, seed=3, d=d, dtype=dtype)
    k_padded = torch.cat([k, torch.zeros(w, Hkv, d, dtype=dtype)])
    cu_pad = [0, n + w]
    ref = P.oracle_pooled(q, k_padded, cu_pad, w, p)
    ref_lse = O.row_lse(P.to_np64(q), P.to_np64(k_padded), cu_pad, w, "history")
    qd, kd = q.to(DEV), k.to(DEV)
    prm = B.make_params(qd, kd, None, w, p, B.SLKV_POOL_MAX, path)
    prm.history_only = 1
    cu = [0, n]
    assert B.slkv_pooled_elems(prm, cu) == Hkv * n
    ws = torch.empty(B.slkv_workspace_bytes(prm, cu), dtype=torch.uint8, device=DEV)
    cu_dev = torch.tensor(cu, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    pooled = torch.full((Hkv * n,), float("nan"), dtype=torch.float32, device=DEV)
    lse = torch.empty(1, Hq, w, dtype=torch.float32, device=DEV)
    B.slkv_score(prm, qd, kd, cu_dev, cu, pooled, ws, status)
    B.slkv_row_lse(prm, qd, kd, cu_dev, cu, lse, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    P.assert_pooled_close(pooled.cpu().numpy(), ref, cu_pad, Hkv, w)
    assert np.allclose(lse.cpu().numpy().astype(np.float64), np.asarray(ref_lse).reshape(1, Hq, w), rtol=0, atol=2e-4)
    # the same scores when the caller hands the log-sum-exps over
    pooled2 = torch.full_like(pooled, float("nan"))
    B.slkv_score(prm, qd, kd, cu_dev, cu, pooled2, ws, status, lse=lse)
    torch.cuda.synchronize()
    P.assert_pooled_close(pooled2.cpu().numpy(), ref, cu_pad, Hkv, w)
