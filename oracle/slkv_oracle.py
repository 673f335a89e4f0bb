"""CPU oracle for the SurfaceLogicKV prefill KV-compression step.  TEST INFRASTRUCTURE ONLY.

Plain, slow, fp64 numpy written from the paper; it shares no code with the CUDA library and must never
be imported by the product path (only tests, the smoke check and the bench's CPU-baseline leg use it).
A numpy matmul / stable sort serves as a step where the definition is a matrix product / an ordering;
there is no blocking, fusion or reordering beyond what the definitions state.

What follows which passage of the paper:
  head_weights          Algorithm 2's weight (0.01 + L_i) * S_ij of every head; S_ij over the grand sum (the
                        algorithm) or over the layer's sum (the prose under Eq. 6).
  alloc_paper_literal   Eq. 6 / Algorithm 2 in the paper's parameters (b_c, beta), with its own rounding.
  alloc_budgets         the same weights, normalised so that the dynamic parts sum to the dynamic pool exactly
                        (largest-remainder rounding): Sec. 3.3 itself says that the printed formula is not a
                        normalisation.  Options: the prose's head normaliser, a per-head cap with the excess
                        handed on (the paper has no cap), Algorithm 2's own rounding.
  row_lse               Eq. 3-4's row normaliser over Eq. 7's key set (the log of the softmax denominator).
  window_votes          Eq. 7 / Algorithm 3 line 6: softmax over the history keys of Q_window H^T / sqrt(d_k)
                        (Eq. 3-4 fix the scale and the softmax axis), then -- the paper does not say how the
                        w rows are reduced -- summed over the window rows and averaged over a GQA group.
  pool                  not in the paper (it defers to prior work): max / mean over an odd window, stride 1.
  select_topk           Eq. 8 / Algorithm 3 lines 7-8: the C - window best history entries.
  compress              Algorithm 3 as a whole: early-out, window always kept, Concat(history', window).
  behavior_scores       Algorithm 1 (SF_sc, LG_sc, INF_sc of one attention row).

Pins (tests/test_oracle_*.py): brute-force attention from Eq. 4 in pure Python loops, votes summing to w,
closed forms for equal keys / one dominant key, permutation equivariance, box response of max pooling,
exhaustive pure-Python sort for selection, Hamilton apportionment in exact rationals, the closed form
sum of Algorithm 2's literal dynamic parts, the (b_c, beta) <-> (fixed, total) mapping at the paper's
beta = 1.351, Algorithm 1 against the harmonic-mean identity and the consistency of Tables 6-8.
Parity unpinned: the *choices* the paper leaves open (pool type, softmax over history only vs. all causal
keys, global vs. within-layer head normaliser) are readings, each behind a flag; no printed value fixes them.
"""
from __future__ import annotations

import math
from typing import List, Sequence, Tuple

import numpy as np

LAYER_FLOOR = 0.01          # Sec. 3.3: minimum layer budget


class OracleError(ValueError):
    def __init__(self, code: str, msg: str = ""):
        super().__init__(f"{code}: {msg}")
        self.code = code


# ----------------------------------------------------------------------------------------------
# Stage 2: budgets
# ----------------------------------------------------------------------------------------------
def paper_fixed_and_pool(b_c: float, beta: float, n_layers: int, n_heads: int) -> Tuple[float, float]:
    """Algorithm 2 lines 1-2: b_fixed = b_c (1 - 1/beta), B_total = (b_c / beta) L H."""
    return b_c * (1.0 - 1.0 / beta), (b_c / beta) * n_layers * n_heads


def head_weights(inf: np.ndarray, within_layer: bool = False) -> List[float]:
    """Algorithm 2's dynamic-budget weight of every head, flat in (layer, head) order:
    (0.01 + L_i / L_s) * S_ij, with L_i the layer's INF_sc sum, L_s the grand sum and S_ij the head's share --
    of the grand sum as the algorithm prints it (S_ij = inf_ij / L_s), or of its own layer's sum as the prose
    under Eq. 6 describes it (within_layer: S_ij = inf_ij / L_i; an all-zero layer shares evenly).  All-zero INF_sc
    gives every head the weight 1.  Separately rounded fp64 operations, sums in index order."""
    x = np.asarray(inf, dtype=np.float32).astype(np.float64)
    L, H = x.shape
    N = L * H
    La = [0.0] * L
    for i in range(L):
        acc = 0.0
        for j in range(H):
            acc = acc + float(x[i][j])
        La[i] = acc
    Ls = 0.0
    for i in range(L):
        Ls = Ls + La[i]
    if not (Ls > 0.0):
        return [1.0] * N
    wgt = [0.0] * N
    for i in range(L):
        lw = LAYER_FLOOR + La[i] / Ls                            # 0.01 + L_{i,h}
        for j in range(H):
            if within_layer:
                share = float(x[i][j]) / La[i] if La[i] > 0.0 else 1.0 / H
            else:
                share = float(x[i][j]) / Ls                      # S_{j,h}
            wgt[i * H + j] = lw * share
    return wgt


def alloc_paper_literal(b_c: float, beta: float, inf: np.ndarray, rounded: bool = True) -> np.ndarray:
    """Eq. 6 / Algorithm 2 in the paper's own parameters: C_ij = round-half-up(max(0, b_fixed + B_total * w_ij))
    with b_fixed = b_c (1 - 1/beta), B_total = (b_c / beta) L H and w_ij = head_weights.  The dynamic parts are
    not normalised: they sum to B_total (0.01 + sum_i L_i^2), not to B_total."""
    x = np.asarray(inf, dtype=np.float64)
    L, H = x.shape
    b_fixed, B_total = paper_fixed_and_pool(b_c, beta, L, H)
    b = b_fixed + B_total * np.array(head_weights(x), dtype=np.float64).reshape(L, H)
    if not rounded:
        return b
    return np.floor(np.maximum(0.0, b) + 0.5).astype(np.int64)


def alloc_budgets(inf: np.ndarray, fixed: int, total: int, within_layer: bool = False, cap: int = None,
                  paper_rounding: bool = False) -> np.ndarray:
    """Integer budgets C[i][j] from the INF_sc table (Sec. 3.3, Eq. 6, Algorithm 2), D = total - N * fixed the
    dynamic pool.

    Default: C >= fixed with sum exactly `total`: Algorithm 2's weights, normalised by their sum and rounded by
    largest remainder (ties: lower index).
    within_layer    the head normaliser of the prose under Eq. 6 instead of the algorithm's (see head_weights).
    cap             no head gets more than `cap` (say, the sequence length: rows beyond it could never be kept);
                    what a capped head cannot take goes to the others in proportion to their weights, again and
                    again until nobody is above the cap (water filling).  total <= N * cap, cap >= fixed.
    paper_rounding  Algorithm 2's own last line instead of the normalisation: C = floor(max(0, fixed + D * w) + 0.5)
                    per head, clipped at `cap` if given; the sum is whatever it comes to.

    Every floating-point operation is a separately rounded fp64 operation in the order written, sums run in index
    order: the CUDA kernel must reproduce the result bit for bit.
    """
    inf32 = np.asarray(inf, dtype=np.float32)
    if inf32.ndim != 2:
        raise OracleError("BAD_SHAPE", "inf must be [n_layers, n_heads]")
    L, H = inf32.shape
    N = L * H
    D = int(total) - N * int(fixed)
    if fixed < 0 or D < 0:
        raise OracleError("BUDGET_SUM", "total < n_heads_total * fixed")
    if cap is not None and (cap < fixed or (not paper_rounding and int(total) > N * int(cap))):
        raise OracleError("BUDGET_SUM", "cap below the fixed part, or total above n_heads_total * cap")
    x = inf32.astype(np.float64)
    if not np.all(np.isfinite(x)) or np.any(x < 0):
        raise OracleError("NEG_INF_SC", "INF_sc must be finite and >= 0")
    wgt = head_weights(inf32, within_layer)

    if paper_rounding:
        out = [0] * N
        no_scores = not np.any(x > 0)                        # all-zero INF_sc: the pool in equal parts
        for a in range(N):
            b = float(fixed) + float(D) * (1.0 / N if no_scores else wgt[a])
            c = int(math.floor(max(0.0, b) + 0.5))
            out[a] = c if cap is None else min(c, int(cap))
        return np.array(out, dtype=np.int64).reshape(L, H)

    active = [True] * N
    share = [0] * N                                          # dynamic part of every head
    d_rem = D
    room = None if cap is None else int(cap) - int(fixed)    # the most dynamic budget a head can take
    while True:
        W = 0.0
        n_active = 0
        for a in range(N):
            if active[a]:
                W = W + wgt[a]
                n_active += 1
        flat = not (W > 0.0)                                 # every weight left underflowed: share evenly
        if flat:
            W = float(n_active)
        if room is None or n_active == 0:
            break
        newly = [a for a in range(N) if active[a] and (float(d_rem) * (1.0 if flat else wgt[a])) / W >= float(room)]
        if not newly:
            break
        for a in newly:                                      # these heads are full; the rest share what is left
            active[a] = False
            share[a] = room
            d_rem -= room

    idx = [a for a in range(N) if active[a]]
    f = {}
    r = {}
    for a in idx:
        q = (float(d_rem) * (1.0 if flat else wgt[a])) / W
        fl = math.floor(q)
        f[a] = int(fl)
        r[a] = q - fl
    R = d_rem - sum(f.values())
    n_act = len(idx)
    if n_act and R >= n_act:                                 # cannot happen in exact arithmetic
        for a in idx:
            f[a] += R // n_act
        R = R % n_act
    if R > 0:
        order = sorted(idx, key=lambda a: (-r[a], a))        # largest remainder, ties -> lower index
        for a in order[:R]:
            f[a] += 1
    while R < 0:                                             # rounding pushed the floors above the pool
        cand = [a for a in idx if f[a] > 0]
        order = sorted(cand, key=lambda a: (r[a], -a))       # smallest remainder, ties -> higher index
        take = order[:min(-R, len(order))]
        for a in take:
            f[a] -= 1
        R += len(take)
    for a in idx:
        share[a] = f[a]
    return (np.array(share, dtype=np.int64) + int(fixed)).reshape(L, H)


# ----------------------------------------------------------------------------------------------
# Stage 1: Algorithm 1
# ----------------------------------------------------------------------------------------------
def behavior_scores(W: np.ndarray, needle_idx: Sequence[int], topk_idx: Sequence[int]) -> Tuple[float, float, float]:
    """Algorithm 1: (SF_sc, LG_sc, INF_sc) of one attention-weight row W; a 0/0 ratio counts as 0."""
    W = np.asarray(W, dtype=np.float64)
    Nset, Tset = set(int(i) for i in needle_idx), set(int(i) for i in topk_idx)
    WO = sum(float(W[i]) for i in sorted(Nset & Tset))
    WD = sum(float(W[i]) for i in sorted(Tset - Nset))
    TNW = sum(float(W[i]) for i in sorted(Nset))
    WS = max(0.0, TNW - WO)
    SF = WO / (WO + WD) if (WO + WD) > 0 else 0.0
    LG = WO / (WO + WS) if (WO + WS) > 0 else 0.0
    INF = 2.0 * SF * LG / (SF + LG) if (SF + LG) > 0 else 0.0
    return SF, LG, INF


# ----------------------------------------------------------------------------------------------
# Prefill: scores -> pool -> select -> gather
# ----------------------------------------------------------------------------------------------
def row_lse(q_win: np.ndarray, k: np.ndarray, cu_seqlens: Sequence[int], window: int,
            domain: str = "history") -> np.ndarray:
    """lse[s][h][i] = log sum_j exp(q_i . k_j / sqrt(d)) over row i's softmax domain (Eq. 3-4's denominator with
    Eq. 7's key set): the history keys, or with domain="all_causal" the history plus the window keys up to the
    row's own position.  fp64 [n_seqs, n_q_heads, window]; NaN for sequences without history."""
    q_win = np.asarray(q_win, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    B, w, Hq, d = q_win.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    out = np.full((B, Hq, w), np.nan)
    for s in range(B):
        t0, t1 = int(cu_seqlens[s]), int(cu_seqlens[s + 1])
        n_hist = max(t1 - t0 - w, 0)
        if n_hist == 0:
            continue
        for h in range(Hq):
            g = h // G
            for i in range(w):
                n_keys = n_hist if domain == "history" else n_hist + i + 1
                if domain not in ("history", "all_causal"):
                    raise ValueError(domain)
                x = (k[t0:t0 + n_keys, g, :] @ q_win[s, i, h, :]) / math.sqrt(d)
                m = x.max()
                out[s, h, i] = m + math.log(np.exp(x - m).sum())
    return out


def window_votes(q_win: np.ndarray, k: np.ndarray, cu_seqlens: Sequence[int], window: int,
                 domain: str = "history", lse: np.ndarray = None) -> List[np.ndarray]:
    """Per sequence: vote[g][j] = (1/G) sum_{h in group g} sum_{i in window} A^h_ij, fp64 [n_kv_heads, n_hist].

    q_win [n_seqs, window, n_q_heads, d] holds the queries of each sequence's last `window` tokens,
    k [total_tokens, n_kv_heads, d] the keys.  A^h = softmax_j(q_i . k_j / sqrt(d)) over the history keys
    j < n_hist = len - window (domain="history", Eq. 7 / Algorithm 3 line 6), or over all keys a window query
    may see causally (domain="all_causal": history plus window keys up to the query's own position), the
    window columns being dropped afterwards.  With `lse` ([n_seqs, n_q_heads, window], natural log) the rows'
    normalisers are taken from it as given: A^h_ij = exp(q_i . k_j / sqrt(d) - lse[s][h][i]).
    """
    q_win = np.asarray(q_win, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    B, w, Hq, d = q_win.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    assert w == window and Hq == G * Hkv
    out = []
    for s in range(B):
        t0, t1 = int(cu_seqlens[s]), int(cu_seqlens[s + 1])
        n_hist = max(t1 - t0 - w, 0)
        vote = np.zeros((Hkv, n_hist), dtype=np.float64)
        if n_hist > 0:
            for g in range(Hkv):
                Hist = k[t0:t0 + n_hist, g, :]                               # [n_hist, d]
                for h in range(g * G, (g + 1) * G):
                    Qw = q_win[s, :, h, :]                                   # [w, d]
                    S = (Qw @ Hist.T) / math.sqrt(d)                         # Eq. 3
                    if lse is not None:
                        A = np.exp(S - np.asarray(lse, dtype=np.float64)[s, h][:, None])
                    elif domain == "history":
                        m = S.max(axis=1, keepdims=True)
                        E = np.exp(S - m)
                        A = E / E.sum(axis=1, keepdims=True)                 # Eq. 4, keys = history
                    elif domain == "all_causal":
                        Kw = k[t0 + n_hist:t1, g, :]                         # [w, d] window keys
                        Sw = (Qw @ Kw.T) / math.sqrt(d)
                        Sw = np.where(np.tril(np.ones((w, w), dtype=bool)), Sw, -np.inf)
                        full = np.concatenate([S, Sw], axis=1)
                        m = full.max(axis=1, keepdims=True)
                        E = np.exp(full - m)
                        A = (E / E.sum(axis=1, keepdims=True))[:, :n_hist]
                    else:
                        raise ValueError(domain)
                    vote[g] += A.sum(axis=0)                                 # sum over the window rows
                vote[g] /= G                                                 # mean over the query group
        out.append(vote)
    return out


def pool(vote: np.ndarray, kernel: int, mode: str = "max") -> np.ndarray:
    """Stride-1 pooling along the last axis over [j - kernel//2, j + kernel//2] clipped to the array
    (max), or zero-padded mean (avg: sum over the clipped range divided by `kernel`)."""
    assert kernel >= 1 and kernel % 2 == 1
    vote = np.asarray(vote, dtype=np.float64)
    n = vote.shape[-1]
    r = kernel // 2
    out = np.empty_like(vote)
    for j in range(n):
        lo, hi = max(0, j - r), min(n - 1, j + r)
        seg = vote[..., lo:hi + 1]
        out[..., j] = seg.max(axis=-1) if mode == "max" else seg.sum(axis=-1) / kernel
    return out


def kept_counts(seq_len: int, budget: int, window: int) -> Tuple[int, int]:
    """(kept history rows, kept window rows) of one head: Algorithm 3 lines 1-4 and 7.

    Everything is kept when the length does not exceed the budget; the window is always kept (so a budget
    below the window acts as the window); otherwise C_H = C - window history rows survive.
    """
    kept = min(seq_len, max(int(budget), window))
    n_win = min(seq_len, window)
    return kept - n_win, n_win


def select_topk(scores: np.ndarray, k: int) -> np.ndarray:
    """Indices of the k largest scores, ties -> lower index, returned ascending (Eq. 8 / Alg. 3 line 8)."""
    scores = np.asarray(scores)
    order = np.argsort(-scores, kind="stable")                 # stable: equal scores keep index order
    return np.sort(order[:k]).astype(np.int64)


def compress(q_win, k, v, cu_seqlens, budgets, window: int, pool_kernel: int, pool_mode: str = "max",
             domain: str = "history"):
    """Algorithm 3 for every (sequence, KV head) segment.

    Returns dict: pooled (list per sequence of [n_kv_heads, n_hist] fp64), kept_idx (list per segment, positions
    within the sequence, selected history ascending then the window), offsets [n_seg+1], k_out / v_out (rows
    gathered from the inputs, same dtype as given).  Segment id = s * n_kv_heads + h.
    """
    k_arr, v_arr = np.asarray(k), np.asarray(v)
    Hkv = k_arr.shape[1]
    B = len(cu_seqlens) - 1
    votes = window_votes(q_win, k_arr, cu_seqlens, window, domain)
    pooled = [pool(vt, pool_kernel, pool_mode) for vt in votes]
    kept_idx, offsets, k_rows, v_rows = [], [0], [], []
    for s in range(B):
        t0, t1 = int(cu_seqlens[s]), int(cu_seqlens[s + 1])
        n = t1 - t0
        for h in range(Hkv):
            n_keep_hist, n_win = kept_counts(n, int(budgets[h]), window)
            hist = select_topk(pooled[s][h], n_keep_hist)
            idx = np.concatenate([hist, np.arange(n - n_win, n, dtype=np.int64)])
            kept_idx.append(idx)
            offsets.append(offsets[-1] + len(idx))
            k_rows.append(k_arr[t0 + idx, h, :])
            v_rows.append(v_arr[t0 + idx, h, :])
    d = k_arr.shape[2]
    k_out = np.concatenate(k_rows, axis=0) if k_rows else np.zeros((0, d), k_arr.dtype)
    v_out = np.concatenate(v_rows, axis=0) if v_rows else np.zeros((0, d), v_arr.dtype)
    return {"pooled": pooled, "kept_idx": kept_idx, "offsets": np.array(offsets, dtype=np.int64),
            "k_out": k_out, "v_out": v_out}
