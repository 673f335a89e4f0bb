"""Pins for the score / pool / select / compress oracle (Eq. 3-4, Eq. 7-8, Algorithm 3)."""
import math

import numpy as np
import pytest

from oracle import slkv_oracle as O


def brute_votes(q_win, k, n_hist, G):
    """Eq. 4 written as pure-Python loops: softmax over the history keys, summed over window rows,
    averaged over the G query heads of each KV head (independent of the oracle's matmul path)."""
    w, Hq, d = len(q_win), len(q_win[0]), len(q_win[0][0])
    Hkv = Hq // G
    vote = [[0.0] * n_hist for _ in range(Hkv)]
    for h in range(Hq):
        g = h // G
        for i in range(w):
            logits = []
            for j in range(n_hist):
                dot = 0.0
                for p in range(d):
                    dot += q_win[i][h][p] * k[j][g][p]
                logits.append(dot / math.sqrt(d))
            den = sum(math.exp(x) for x in logits)
            for j in range(n_hist):
                vote[g][j] += math.exp(logits[j]) / den / G
    return vote


@pytest.mark.parametrize("Hq,Hkv,d,L,w", [(2, 2, 4, 20, 3), (4, 2, 8, 40, 5), (4, 1, 6, 17, 4)])
def test_votes_match_brute_force(Hq, Hkv, d, L, w):
    rng = np.random.default_rng(Hq * 100 + L)
    q = rng.normal(size=(1, w, Hq, d))
    k = rng.normal(size=(L, Hkv, d))
    got = O.window_votes(q, k, [0, L], w)[0]
    ref = np.array(brute_votes(q[0].tolist(), k.tolist(), L - w, Hq // Hkv))
    assert got.shape == (Hkv, L - w)
    assert np.allclose(got, ref, rtol=1e-12, atol=0)


def test_votes_sum_to_window():
    rng = np.random.default_rng(1)
    q = rng.normal(size=(2, 8, 4, 16)) * 3
    k = rng.normal(size=(100 + 57, 2, 16)) * 3
    votes = O.window_votes(q, k, [0, 100, 157], 8)
    assert [v.shape for v in votes] == [(2, 92), (2, 49)]
    for v in votes:
        assert np.allclose(v.sum(axis=1), 8.0, rtol=1e-12)


def test_equal_keys_give_uniform_votes():
    rng = np.random.default_rng(2)
    q = rng.normal(size=(1, 4, 2, 8))
    k = np.tile(rng.normal(size=(1, 2, 8)), (36, 1, 1))
    v = O.window_votes(q, k, [0, 36], 4)[0]
    assert np.allclose(v, 4.0 / 32.0, rtol=1e-12)


def test_dominant_key_takes_all_votes():
    rng = np.random.default_rng(3)
    d = 8
    q = rng.normal(size=(1, 4, 1, d)) * 0.01
    u = np.zeros(d); u[2] = 1.0
    q[..., :] += 30.0 * u
    k = rng.normal(size=(50, 1, d)) * 0.01
    k[17, 0] = 30.0 * u                       # logit ~ 900/sqrt(8) at key 17
    v = O.window_votes(q, k, [0, 50], 4)[0][0]
    assert abs(v[17] - 4.0) < 1e-9 and np.all(np.delete(v, 17) < 1e-9)


def test_scale_is_one_over_sqrt_d():
    # two keys, one query: A = sigmoid((q.k0 - q.k1)/sqrt(d)); a wrong scale changes the value
    d = 16
    q = np.zeros((1, 1, 1, d)); q[..., 0] = 2.0
    k = np.zeros((3, 1, d)); k[0, 0, 0] = 3.0; k[1, 0, 0] = 1.0
    v = O.window_votes(q, k, [0, 3], 1)[0][0]
    expect = 1.0 / (1.0 + math.exp(-(6.0 - 2.0) / 4.0))
    assert abs(v[0] - expect) < 1e-15 and abs(v[1] - (1 - expect)) < 1e-15


def test_permuting_history_permutes_votes():
    rng = np.random.default_rng(4)
    q = rng.normal(size=(1, 4, 4, 8))
    k = rng.normal(size=(44, 2, 8))
    perm = rng.permutation(40)
    k2 = k.copy(); k2[:40] = k[perm]
    a = O.window_votes(q, k, [0, 44], 4)[0]
    b = O.window_votes(q, k2, [0, 44], 4)[0]
    assert np.allclose(b, a[:, perm], rtol=1e-12)


def test_window_keys_do_not_matter_in_history_domain_but_do_in_all_causal():
    rng = np.random.default_rng(5)
    q = rng.normal(size=(1, 4, 2, 8))
    k = rng.normal(size=(30, 2, 8))
    k2 = k.copy(); k2[26:] += 1.0
    a = O.window_votes(q, k, [0, 30], 4)[0]
    assert np.array_equal(a, O.window_votes(q, k2, [0, 30], 4)[0])
    c1 = O.window_votes(q, k, [0, 30], 4, domain="all_causal")[0]
    c2 = O.window_votes(q, k2, [0, 30], 4, domain="all_causal")[0]
    assert not np.allclose(c1, c2)
    # all-causal rows sum to less than 1 over the history (the rest sits on the window keys)
    assert np.all(c1.sum(axis=1) < 4.0) and np.all(c1 <= a * (1 + 1e-12))


def test_all_causal_matches_masked_full_attention():
    # brute force: full causal attention over the whole sequence, last w rows, history columns
    rng = np.random.default_rng(6)
    L, w, d = 12, 3, 4
    q_full = rng.normal(size=(L, d)); k = rng.normal(size=(L, 1, d))
    S = q_full @ k[:, 0].T / math.sqrt(d)
    S[np.triu_indices(L, 1)] = -np.inf
    A = np.exp(S) / np.exp(S).sum(axis=1, keepdims=True)
    ref = A[L - w:, :L - w].sum(axis=0)
    got = O.window_votes(q_full[None, L - w:, None, :], k, [0, L], w, domain="all_causal")[0][0]
    assert np.allclose(got, ref, rtol=1e-12)


def brute_lse(q_row, keys, d):
    """log of Eq. 4's denominator for one query row, pure Python."""
    tot = 0.0
    for kj in keys:
        tot += math.exp(sum(a * b for a, b in zip(q_row, kj)) / math.sqrt(d))
    return math.log(tot)


@pytest.mark.parametrize("domain", ["history", "all_causal"])
def test_row_lse_matches_brute_force(domain):
    rng = np.random.default_rng(41)
    w, Hq, Hkv, d = 3, 4, 2, 6
    q = rng.normal(size=(2, w, Hq, d))
    k = rng.normal(size=(11 + 2, Hkv, d))          # second sequence is shorter than the window: no rows
    got = O.row_lse(q, k, [0, 11, 13], w, domain)
    assert got.shape == (2, Hq, w) and np.all(np.isnan(got[1]))
    for h in range(Hq):
        for i in range(w):
            n_keys = 8 if domain == "history" else 8 + i + 1
            ref = brute_lse(q[0, i, h].tolist(), k[:n_keys, h // 2].tolist(), d)
            assert abs(got[0, h, i] - ref) < 1e-12


def test_row_lse_of_equal_keys_is_logit_plus_log_count():
    rng = np.random.default_rng(42)
    d = 8
    q = rng.normal(size=(1, 4, 2, d))
    k = np.tile(rng.normal(size=(1, 1, d)), (36, 1, 1))
    got = O.row_lse(q, k, [0, 36], 4)
    ref = (q[0] @ k[0, 0]) / math.sqrt(d) + math.log(32)         # [w, Hq]
    assert np.allclose(got[0], ref.T, rtol=0, atol=1e-12)
    got_c = O.row_lse(q, k, [0, 36], 4, "all_causal")
    ref_c = (q[0] @ k[0, 0]) / math.sqrt(d) + np.log(32 + 1 + np.arange(4))[:, None]
    assert np.allclose(got_c[0], ref_c.T, rtol=0, atol=1e-12)


@pytest.mark.parametrize("domain", ["history", "all_causal"])
def test_votes_from_supplied_lse(domain):
    rng = np.random.default_rng(43)
    q = rng.normal(size=(2, 4, 4, 8))
    k = rng.normal(size=(30 + 21, 2, 8))
    cu = [0, 30, 51]
    lse = O.row_lse(q, k, cu, 4, domain)
    a = O.window_votes(q, k, cu, 4, domain)
    b = O.window_votes(q, k, cu, 4, "history", lse=lse)          # the domain only matters for the normaliser
    for x, y in zip(a, b):
        assert np.allclose(x, y, rtol=1e-12, atol=0)
    # a normaliser one unit larger scales every vote of that row by 1/e: the array is used as given
    lse2 = lse.copy(); lse2[0, :, :] += 1.0
    c = O.window_votes(q, k, cu, 4, "history", lse=lse2)
    assert np.allclose(c[0], a[0] / math.e, rtol=1e-12) and np.allclose(c[1], a[1], rtol=1e-12)


def test_short_sequences_have_no_history():
    q = np.zeros((2, 4, 1, 2)); k = np.zeros((6, 1, 2))
    v = O.window_votes(q, k, [0, 4, 6], 4)
    assert v[0].shape == (1, 0) and v[1].shape == (1, 0)


# ---- pooling -----------------------------------------------------------------------------------
def test_max_pool_of_impulse_is_box():
    x = np.zeros((1, 20)); x[0, 9] = 1.0; x[0, 0] = 0.5
    y = O.pool(x, 5, "max")[0]
    expect = np.zeros(20); expect[7:12] = 1.0; expect[0:3] = 0.5
    assert np.array_equal(y, expect)
    assert np.array_equal(O.pool(x, 1, "max"), x)


def test_avg_pool_zero_padded():
    x = np.arange(1.0, 7.0)[None]
    y = O.pool(x, 3, "avg")[0]
    assert np.allclose(y, [(1 + 2) / 3, 2, 3, 4, 5, (5 + 6) / 3])
    ref = np.convolve(x[0], np.ones(3) / 3, mode="same")        # library routine: zero-padded moving mean
    assert np.allclose(y, ref)


def test_max_pool_matches_bruteforce():
    rng = np.random.default_rng(7)
    x = rng.random((3, 33))
    y = O.pool(x, 7, "max")
    for r in range(3):
        for j in range(33):
            assert y[r, j] == max(x[r, max(0, j - 3):j + 4])


# ---- selection ---------------------------------------------------------------------------------
def test_select_matches_python_sort_with_ties():
    rng = np.random.default_rng(8)
    for n in (1, 2, 7, 50):
        x = rng.integers(0, 5, size=n).astype(np.float64)        # many exact ties
        for k in range(0, n + 1):
            ref = sorted(sorted(range(n), key=lambda j: (-x[j], j))[:k])
            assert O.select_topk(x, k).tolist() == ref


def test_kept_counts():
    assert O.kept_counts(100, 40, 16) == (24, 16)         # C_H = C - window
    assert O.kept_counts(100, 10, 16) == (0, 16)          # budget below the window: window only
    assert O.kept_counts(30, 40, 16) == (14, 16)          # length <= budget: keep everything
    assert O.kept_counts(100, 100, 16) == (84, 16)
    assert O.kept_counts(10, 40, 16) == (0, 10)           # shorter than the window


def test_compress_invariants_and_needles():
    rng = np.random.default_rng(9)
    Hq, Hkv, d, w, p = 4, 2, 8, 4, 3
    lens = [60, 9, 3, 40]
    cu = np.concatenate([[0], np.cumsum(lens)])
    T = int(cu[-1])
    q = rng.normal(size=(len(lens), w, Hq, d))
    k = rng.normal(size=(T, Hkv, d)); v = rng.normal(size=(T, Hkv, d))
    u = np.ones(d) / math.sqrt(d)
    q += 4.0 * u
    needles = [10, 30, 50]
    for n in needles:
        k[n, :, :] = 6.0 * u                               # big logits at the needles of sequence 0
    budgets = [20, 5]
    out = O.compress(q, k, v, cu, budgets, w, p)
    assert out["offsets"][0] == 0 and len(out["offsets"]) == len(lens) * Hkv + 1
    for s, n in enumerate(lens):
        for h in range(Hkv):
            seg = s * Hkv + h
            idx = out["kept_idx"][seg]
            assert len(idx) == min(n, max(budgets[h], w))                 # kept == budget (clamped)
            assert out["offsets"][seg + 1] - out["offsets"][seg] == len(idx)
            assert np.all(np.diff(idx) > 0)
            nw = min(n, w)
            assert idx[len(idx) - nw:].tolist() == list(range(n - nw, n))   # window always kept, last
            rows = slice(out["offsets"][seg], out["offsets"][seg + 1])
            assert np.array_equal(out["k_out"][rows], k[cu[s] + idx, h])
            assert np.array_equal(out["v_out"][rows], v[cu[s] + idx, h])
    # head 0 of sequence 0 keeps 16 history rows >= 3 needles * pool 3: every needle and its neighbours
    kept0 = set(out["kept_idx"][0].tolist())
    for n in needles:
        assert {n - 1, n, n + 1} <= kept0
    # head 1: budget 5 -> one history row, which must be a needle neighbourhood
    assert out["kept_idx"][1][0] in {9, 10, 11, 29, 30, 31, 49, 50, 51}


def test_compress_full_keep_when_budget_covers_length():
    rng = np.random.default_rng(10)
    q = rng.normal(size=(1, 2, 1, 4)); k = rng.normal(size=(7, 1, 4))
    out = O.compress(q, k, k, [0, 7], [7], 2, 3)
    assert out["kept_idx"][0].tolist() == list(range(7))
    out = O.compress(q, k, k, [0, 7], [100], 2, 3)
    assert out["kept_idx"][0].tolist() == list(range(7))
