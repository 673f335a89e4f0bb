"""Helpers for the GPU-vs-oracle parity tests: run the CUDA path through the C ABI, compare by the rules.

Rules (tolerances written here, used by every parity test):
  budgets, offsets        bit-exact
  pooled scores           |gpu - oracle| <= REL_TOL * oracle + ABS_FLOOR   (fp32 accumulate of bf16/fp32 inputs)
  kept index sets         identical up to the tolerance band at each head's k-th score: with tau = the
                          oracle's k-th largest pooled score, every position whose oracle score exceeds
                          tau (1 + REL_TOL) must be kept, every kept position must score >= tau (1 - REL_TOL),
                          and the count must be exactly k; indices ascending; window suffix present
  gathered K / V rows     bit copies of the input rows at the GPU's own kept indices
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from oracle import slkv_oracle as O
from paper_2508_15806_b200 import binding as B

REL_TOL = 1e-3
ABS_FLOOR = 1e-30


def to_np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().to(torch.float32).numpy().astype(np.float64)


def to_np_bits(t: torch.Tensor) -> np.ndarray:
    """Exact values as float32 (bf16 -> fp32 is exact) for bit comparisons of gathered rows."""
    return t.detach().cpu().to(torch.float32).numpy()


def lse_to_dev(lse, units: int = B.SLKV_LSE_LN) -> Optional[torch.Tensor]:
    """Host row log-sum-exps (natural log, numpy fp64 with NaN where a sequence has no history) -> CUDA fp32 in `units`."""
    if lse is None:
        return None
    a = np.nan_to_num(np.asarray(lse, dtype=np.float64), nan=0.0)
    if units == B.SLKV_LSE_LOG2:
        a = a / np.log(2.0)
    return torch.tensor(a, dtype=torch.float32, device="cuda:0").contiguous()


def gpu_compress(q_win, k, v, cu: Sequence[int], budgets_row: Sequence[int], window: int, pool_kernel: int,
                 pool_mode: int = B.SLKV_POOL_MAX, score_path: int = B.SLKV_PATH_AUTO,
                 capacity: Optional[int] = None, want_pooled: bool = True, domain: int = B.SLKV_HISTORY,
                 lse=None, lse_units: int = B.SLKV_LSE_LN) -> Dict[str, object]:
    """Runs slkv_compress on cuda:0 with host tensors q_win, k, v; returns host results."""
    dev = torch.device("cuda:0")
    qd, kd, vd = q_win.to(dev), k.to(dev), v.to(dev)
    params = B.make_params(qd, kd, vd, window, pool_kernel, pool_mode, score_path, domain, lse_units)
    cu = [int(x) for x in cu]
    n_seg = (len(cu) - 1) * k.shape[1]
    cap = B.slkv_packed_rows_upper_bound(params, cu) if capacity is None else capacity
    cu_dev = torch.tensor(cu, dtype=torch.int32, device=dev)
    bud = torch.tensor(list(budgets_row), dtype=torch.int32, device=dev)
    k_out = torch.full((max(cap, 1), k.shape[2]), 0, dtype=k.dtype, device=dev)[:cap]
    v_out = torch.full((max(cap, 1), k.shape[2]), 0, dtype=k.dtype, device=dev)[:cap]
    offsets = torch.full((n_seg + 1,), -1, dtype=torch.int32, device=dev)
    kept = torch.full((max(cap, 1),), -1, dtype=torch.int32, device=dev)[:cap]
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    ws = B.new_workspace(params, cu, dev)
    n_pool = B.slkv_pooled_elems(params, cu)
    pooled = torch.full((max(n_pool, 1),), float("nan"), dtype=torch.float32, device=dev) if want_pooled else None
    B.slkv_compress(params, qd, kd, vd, cu_dev, cu, bud, k_out, v_out, offsets, kept, ws, pooled, status,
                    lse=lse_to_dev(lse, lse_units))
    launches = B.slkv_last_launch_count()
    torch.cuda.synchronize()
    return {"offsets": offsets.cpu().numpy().astype(np.int64), "kept_idx": kept.cpu().numpy().astype(np.int64),
            "k_out": k_out.cpu(), "v_out": v_out.cpu(), "status": int(status.item()),
            "pooled": None if pooled is None else pooled[:n_pool].cpu().numpy(), "launches": launches}


def gpu_score(q_win, k, cu: Sequence[int], window: int, pool_kernel: int, pool_mode: int = B.SLKV_POOL_MAX,
              score_path: int = B.SLKV_PATH_AUTO, domain: int = B.SLKV_HISTORY, lse=None,
              lse_units: int = B.SLKV_LSE_LN) -> np.ndarray:
    dev = torch.device("cuda:0")
    qd, kd = q_win.to(dev), k.to(dev)
    params = B.make_params(qd, kd, None, window, pool_kernel, pool_mode, score_path, domain, lse_units)
    cu = [int(x) for x in cu]
    cu_dev = torch.tensor(cu, dtype=torch.int32, device=dev)
    ws = B.new_workspace(params, cu, dev)
    n_pool = B.slkv_pooled_elems(params, cu)
    pooled = torch.full((max(n_pool, 1),), float("nan"), dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    lse_dev = lse if isinstance(lse, torch.Tensor) else lse_to_dev(lse, lse_units)
    B.slkv_score(params, qd, kd, cu_dev, cu, pooled, ws, status, lse=lse_dev)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return pooled[:n_pool].cpu().numpy()


def gpu_row_lse(q_win, k, cu: Sequence[int], window: int, score_path: int = B.SLKV_PATH_AUTO,
                domain: int = B.SLKV_HISTORY, lse_units: int = B.SLKV_LSE_LN) -> torch.Tensor:
    """slkv_row_lse on cuda:0: CUDA float32 [n_seqs, n_q_heads, window] (rows of sequences without history: NaN)."""
    dev = torch.device("cuda:0")
    qd, kd = q_win.to(dev), k.to(dev)
    params = B.make_params(qd, kd, None, window, 1, B.SLKV_POOL_MAX, score_path, domain, lse_units)
    cu = [int(x) for x in cu]
    cu_dev = torch.tensor(cu, dtype=torch.int32, device=dev)
    ws = B.new_workspace(params, cu, dev)
    out = torch.full((q_win.shape[0], q_win.shape[2], window), float("nan"), dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    B.slkv_row_lse(params, qd, kd, cu_dev, cu, out, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return out


def split_pooled(flat: np.ndarray, cu: Sequence[int], n_kv_heads: int, window: int) -> List[np.ndarray]:
    """Ragged pooled array -> list per sequence of [n_kv_heads, n_hist]."""
    out, o = [], 0
    for s in range(len(cu) - 1):
        nh = max(int(cu[s + 1]) - int(cu[s]) - window, 0)
        out.append(flat[o:o + n_kv_heads * nh].reshape(n_kv_heads, nh))
        o += n_kv_heads * nh
    assert o == len(flat)
    return out


def assert_pooled_close(gpu_flat: np.ndarray, oracle_pooled: List[np.ndarray], cu, n_kv_heads, window) -> float:
    got = split_pooled(gpu_flat.astype(np.float64), cu, n_kv_heads, window)
    worst = 0.0
    for g, o in zip(got, oracle_pooled):
        assert g.shape == o.shape
        if o.size == 0:
            continue
        assert np.all(np.isfinite(g))
        err = np.abs(g - o)
        bound = REL_TOL * np.abs(o) + ABS_FLOOR
        bad = err > bound
        assert not bad.any(), f"pooled mismatch at {np.argwhere(bad)[:5].tolist()}: max rel {np.max(err / (np.abs(o) + ABS_FLOOR)):.3e}"
        worst = max(worst, float(np.max(err / (np.abs(o) + ABS_FLOOR))))
    return worst


def assert_selection_valid(gpu: Dict[str, object], oracle_pooled: List[np.ndarray], cu, budgets_row, window: int,
                           k_in: torch.Tensor, v_in: torch.Tensor) -> Dict[str, int]:
    """Offsets bit-exact, kept sets valid by the band rule, rows bit-exact.  Returns counters."""
    n_kv = k_in.shape[1]
    offs, idx_all = gpu["offsets"], gpu["kept_idx"]
    exp_off = [0]
    for s in range(len(cu) - 1):
        n = int(cu[s + 1]) - int(cu[s])
        for h in range(n_kv):
            kh, nw = O.kept_counts(n, int(budgets_row[h]), window)
            exp_off.append(exp_off[-1] + kh + nw)
    assert offs.tolist() == exp_off, "offsets differ from the oracle's"
    kb, vb = to_np_bits(k_in), to_np_bits(v_in)
    ko, vo = to_np_bits(gpu["k_out"]), to_np_bits(gpu["v_out"])
    stats = {"segments": 0, "identical": 0, "band_swaps": 0}
    for s in range(len(cu) - 1):
        t0 = int(cu[s]); n = int(cu[s + 1]) - t0
        for h in range(n_kv):
            seg = s * n_kv + h
            a, b = int(offs[seg]), int(offs[seg + 1])
            idx = idx_all[a:b]
            kh, nw = O.kept_counts(n, int(budgets_row[h]), window)
            assert len(idx) == kh + nw
            assert np.all(np.diff(idx) > 0), "kept indices must ascend"
            assert idx[kh:].tolist() == list(range(n - nw, n)), "window suffix missing"
            hist = idx[:kh]
            if kh:
                assert hist.min() >= 0 and hist.max() < n - nw
            sc = oracle_pooled[s][h]
            ref = O.select_topk(sc, kh)
            stats["segments"] += 1
            if np.array_equal(ref, hist):
                stats["identical"] += 1
            else:
                tau = np.sort(sc)[::-1][kh - 1]
                must = np.nonzero(sc > tau * (1 + REL_TOL))[0]
                assert np.isin(must, hist).all(), "a position clearly above the k-th score was dropped"
                assert np.all(sc[hist] >= tau * (1 - REL_TOL)), "a position clearly below the k-th score was kept"
                stats["band_swaps"] += int(len(set(hist.tolist()) ^ set(ref.tolist())) // 2)
            # gathered rows: bit copies of the source rows at the GPU's own indices
            assert np.array_equal(ko[a:b], kb[t0 + idx, h, :]), "K rows differ"
            assert np.array_equal(vo[a:b], vb[t0 + idx, h, :]), "V rows differ"
    return stats


def oracle_pooled(q_win, k, cu, window, pool_kernel, pool_mode=B.SLKV_POOL_MAX, domain: int = B.SLKV_HISTORY,
                  lse=None) -> List[np.ndarray]:
    votes = O.window_votes(to_np64(q_win), to_np64(k), cu, window,
                           "all_causal" if domain == B.SLKV_ALL_CAUSAL else "history", lse)
    return [O.pool(vt, pool_kernel, "max" if pool_mode == B.SLKV_POOL_MAX else "avg") for vt in votes]


def check_compress(q_win, k, v, cu, budgets_row, window, pool_kernel, pool_mode=B.SLKV_POOL_MAX,
                   score_path=B.SLKV_PATH_AUTO, pooled_ref=None, domain: int = B.SLKV_HISTORY, lse=None):
    """Full parity of one layer: returns (gpu result, stats).  `lse` (natural log, host fp64) goes to both sides."""
    gpu = gpu_compress(q_win, k, v, cu, budgets_row, window, pool_kernel, pool_mode, score_path, domain=domain, lse=lse)
    assert gpu["status"] == 0
    ref = pooled_ref if pooled_ref is not None else oracle_pooled(q_win, k, cu, window, pool_kernel, pool_mode, domain,
                                                                 lse)
    worst = assert_pooled_close(gpu["pooled"], ref, cu, k.shape[1], window)
    stats = assert_selection_valid(gpu, ref, cu, budgets_row, window, k, v)
    stats["pooled_max_rel_err"] = worst
    return gpu, stats
