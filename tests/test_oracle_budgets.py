"""Pins for the budget oracle (Algorithm 2 / Eq. 6): closed forms, exact-rational apportionment, invariants."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import slkv_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _golden_rows(name):
    rows = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


def hamilton_exact(weights, D):
    """Textbook largest-remainder apportionment of D seats, exact rationals (independent of the oracle)."""
    tot = sum(Fraction(w) for w in weights)
    quota = [Fraction(w) * D / tot for w in weights]
    seats = [q.numerator // q.denominator for q in quota]
    rem = [q - s for q, s in zip(quota, seats)]
    left = D - sum(seats)
    for a in sorted(range(len(weights)), key=lambda a: (-rem[a], a))[:left]:
        seats[a] += 1
    return seats


def test_paper_hyperparameters_fixture():
    # beta = 1.351 and KV sizes 64..1024 (Table 1 caption / Fig. 6): fixed share = 1 - 1/beta of b_c
    for b_c, beta, fixed_expect, pool_per_head_expect in _golden_rows("paper_hyperparameters.txt"):
        b_c, beta = float(b_c), float(beta)
        fx, pool = O.paper_fixed_and_pool(b_c, beta, 32, 32)
        assert abs(fx - float(fixed_expect)) < 5e-3
        assert abs(pool / (32 * 32) - float(pool_per_head_expect)) < 5e-3
        assert abs(fx + pool / 1024 - b_c) < 1e-9            # the two parts add up to b_c per head


def test_mapping_fixed_total_to_bc_beta():
    # b_c = 128, fixed = 32  <=>  beta = 4/3, dynamic pool = 96 per head
    fx, pool = O.paper_fixed_and_pool(128.0, 4.0 / 3.0, 4, 8)
    assert abs(fx - 32.0) < 1e-12 and abs(pool - 96.0 * 32) < 1e-9


def test_literal_dynamic_sum_closed_form():
    # sum_ij (0.01 + L_i) S_ij = 0.01 + sum_i L_i^2   (from Algorithm 2 lines 3-6)
    rng = np.random.default_rng(0)
    inf = rng.lognormal(0.0, 1.5, size=(6, 5))
    b_c, beta = 128.0, 1.351
    b = O.alloc_paper_literal(b_c, beta, inf, rounded=False)
    fx, B_total = O.paper_fixed_and_pool(b_c, beta, 6, 5)
    Li = inf.sum(axis=1) / inf.sum()
    assert abs((b - fx).sum() - B_total * (0.01 + (Li ** 2).sum())) < 1e-9 * B_total
    # and it is NOT the pool: the printed formula is not normalised
    assert abs((b - fx).sum() - B_total) > 0.1 * B_total


def test_literal_hand_example():
    # 2 layers x 2 heads, worked by hand: inf = [[1,3],[2,2]], L_s = 8, L_i = [.5,.5], S = [[1/8,3/8],[2/8,2/8]]
    inf = np.array([[1.0, 3.0], [2.0, 2.0]])
    b_c, beta = 100.0, 2.0                  # fixed 50, B_total = 50*4 = 200
    b = O.alloc_paper_literal(b_c, beta, inf, rounded=False)
    expect = 50.0 + 200.0 * 0.51 * np.array([[1, 3], [2, 2]]) / 8.0
    assert np.allclose(b, expect, rtol=0, atol=1e-12)
    C = O.alloc_paper_literal(b_c, beta, inf)
    assert C.tolist() == [[63, 88], [76, 76]]          # 62.75->63, 88.25->88, 75.5->76 (round half up)


def test_literal_rounding_half_up_and_clamp():
    inf = np.array([[1.0, 1.0]])
    # b_c=1, beta=1 -> fixed 0, pool 2, each head gets 2*(1.01)*0.5 = 1.01 -> 1
    assert O.alloc_paper_literal(1.0, 1.0, inf).tolist() == [[1, 1]]
    # negative fixed part (beta < 1) is clamped at 0 by max(0, b)
    assert O.alloc_paper_literal(1.0, 0.25, np.array([[0.0, 1.0]])).tolist()[0][0] == 0


@pytest.mark.parametrize("seed", range(6))
def test_single_layer_is_hamilton(seed):
    # one layer => weights proportional to inf => textbook apportionment of D by inf
    rng = np.random.default_rng(seed)
    H = int(rng.integers(2, 12))
    inf = rng.integers(0, 50, size=(1, H)).astype(np.float64)
    if inf.sum() == 0:
        inf[0, 0] = 1
    fixed = int(rng.integers(0, 40))
    D = int(rng.integers(0, 500))
    C = O.alloc_budgets(inf, fixed, fixed * H + D)
    assert (C - fixed).ravel().tolist() == hamilton_exact([int(x) for x in inf[0]], D)


@pytest.mark.parametrize("seed", range(4))
def test_multi_layer_matches_exact_rational_weights(seed):
    # small-integer inf: the weights (0.01 + L_i) S_ij are exact rationals; apportion them exactly
    rng = np.random.default_rng(100 + seed)
    L, H = int(rng.integers(2, 5)), int(rng.integers(2, 6))
    inf = rng.integers(1, 20, size=(L, H))
    Ls = int(inf.sum())
    w = [(Fraction(1, 100) + Fraction(int(inf[i].sum()), Ls)) * Fraction(int(inf[i, j]), Ls)
         for i in range(L) for j in range(H)]
    D = int(rng.integers(50, 3000))
    fixed = 7
    C = O.alloc_budgets(inf.astype(np.float64), fixed, fixed * L * H + D)
    seats = hamilton_exact(w, D)
    got = (C - fixed).ravel().tolist()
    # fp64 quotas can differ from the exact ones only at exact-remainder ties; none for these draws
    assert got == seats


def test_uniform_inf():
    C = O.alloc_budgets(np.ones((3, 4)), 10, 10 * 12 + 24)
    assert np.all(C == 12)
    C = O.alloc_budgets(np.ones((1, 5)), 10, 10 * 5 + 7)          # 7 = 1*5 + 2: the first two heads get +1
    assert C.ravel().tolist() == [12, 12, 11, 11, 11]
    C = O.alloc_budgets(np.zeros((2, 3)), 4, 4 * 6 + 8)           # all-zero INF_sc: uniform
    assert C.ravel().tolist() == [6, 6, 5, 5, 5, 5]


def test_invariants_and_scaling():
    rng = np.random.default_rng(5)
    for _ in range(20):
        L, H = int(rng.integers(1, 8)), int(rng.integers(1, 9))
        inf = rng.lognormal(0.0, 1.5, size=(L, H)).astype(np.float32)
        fixed = int(rng.integers(0, 100))
        total = fixed * L * H + int(rng.integers(0, 100000))
        C = O.alloc_budgets(inf, fixed, total)
        assert C.dtype == np.int64 and C.min() >= fixed and int(C.sum()) == total
        for i in range(L):                                   # monotone in INF_sc within a layer
            order = np.argsort(inf[i], kind="stable")
            assert np.all(np.diff(C[i][order]) >= 0)
        for s in (0.25, 8.0, 2.0 ** -20):                    # power-of-two scaling is exact in fp64
            assert np.array_equal(O.alloc_budgets(inf * np.float32(s), fixed, total), C)


def test_layer_floor_matters():
    # a near-zero layer still gets a share through the 0.01 floor: more than it would get without it
    inf = np.array([[1.0, 1.0], [1e-3, 1e-3]])
    C = O.alloc_budgets(inf, 0, 1_000_000)
    Ls = inf.sum()
    no_floor = ((inf.sum(1, keepdims=True) / Ls) * inf / Ls)
    no_floor = no_floor / no_floor.sum() * 1_000_000
    assert C[1, 0] > 5 * no_floor[1, 0]


def test_errors():
    with pytest.raises(O.OracleError) as e:
        O.alloc_budgets(np.ones((2, 2)), 10, 39)
    assert e.value.code == "BUDGET_SUM"
    for bad in (-1.0, float("nan"), float("inf")):
        with pytest.raises(O.OracleError) as e:
            O.alloc_budgets(np.array([[1.0, bad]]), 1, 10)
        assert e.value.code == "NEG_INF_SC"


# ---- Algorithm 1 -------------------------------------------------------------------------------
def test_behavior_scores_hand_example():
    W = np.array([0.4, 0.1, 0.2, 0.05, 0.25])
    # needle = {0, 3}, top-k = {0, 4, 2}:  WO = .4, WD = .45, TNW = .45, WS = .05
    SF, LG, INF = O.behavior_scores(W, [0, 3], [0, 4, 2])
    assert abs(SF - 0.4 / 0.85) < 1e-15 and abs(LG - 0.4 / 0.45) < 1e-15
    assert abs(INF - 2 * SF * LG / (SF + LG)) < 1e-15
    assert abs(1.0 / INF - 0.5 * (1.0 / SF + 1.0 / LG)) < 1e-12       # harmonic mean
    assert O.behavior_scores(W, [1], [0]) == (0.0, 0.0, 0.0)          # nothing correct


def test_tables_6_8_consistent_with_harmonic_mean():
    # Tables 7 and 8 list SF_sc and INF_sc for the same heads; INF = 2 SF LG / (SF + LG) then gives
    # LG = INF SF / (2 SF - INF), which must be a valid score <= the 10th-largest LG_sc of Table 6
    # for every head that is absent from Table 6.
    sf = {r[0]: float(r[1]) for r in _golden_rows("table7_sf_top10.txt")}
    inf = {r[0]: float(r[1]) for r in _golden_rows("table8_inf_top10.txt")}
    lg = {r[0]: float(r[1]) for r in _golden_rows("table6_lg_top10.txt")}
    lg10 = min(lg.values())
    assert set(sf) == set(inf)
    for head in sf:
        LG = inf[head] * sf[head] / (2 * sf[head] - inf[head])
        assert 0.0 < LG <= 1.0 and sf[head] < inf[head] < LG        # harmonic mean lies between the two
        if head not in lg:
            assert LG < lg10
        # an attention row with exactly these SF and LG: one needle token inside the top-k set (weight WO), one
        # outside it (WS), one top-k token that is no needle (WD); Algorithm 1 on it must print the table's INF_sc
        WO = 0.3
        WD, WS = WO * (1 - sf[head]) / sf[head], WO * (1 - LG) / LG
        W = np.array([WO, WS, WD, 1.0 - WO - WS - WD])
        got_sf, got_lg, got_inf = O.behavior_scores(W, needle_idx=[0, 1], topk_idx=[0, 2])
        assert abs(got_sf - sf[head]) < 1e-12 and abs(got_lg - LG) < 1e-12
        assert abs(got_inf - inf[head]) < 1e-12


# ---- variants: head normaliser of the prose under Eq. 6, per-head cap, Algorithm 2's own rounding -----------------
def waterfill_exact(weights, D, room):
    """Apportion D seats by exact-rational weights with at most `room` seats per head: heads whose exact quota
    reaches `room` are filled and removed, the rest share what is left, until none does; then largest remainder
    (independent of the oracle: Fractions only)."""
    n = len(weights)
    active = list(range(n))
    seats = [0] * n
    left = D
    while active:
        tot = sum(Fraction(weights[a]) for a in active)
        full = [a for a in active if Fraction(weights[a]) * left / tot >= room]
        if not full:
            break
        for a in full:
            seats[a] = room
            left -= room
            active.remove(a)
    if active:
        tot = sum(Fraction(weights[a]) for a in active)
        quota = {a: Fraction(weights[a]) * left / tot for a in active}
        for a in active:
            seats[a] = quota[a].numerator // quota[a].denominator
        rest = left - sum(seats[a] for a in active)
        for a in sorted(active, key=lambda a: (-(quota[a] - seats[a]), a))[:rest]:
            seats[a] += 1
    return seats


def test_within_layer_equals_global_on_one_layer():
    rng = np.random.default_rng(5)
    for _ in range(5):
        inf = rng.lognormal(0, 1.5, size=(1, 9))
        a = O.alloc_budgets(inf, 16, 16 * 9 + 4000)
        b = O.alloc_budgets(inf, 16, 16 * 9 + 4000, within_layer=True)
        assert np.array_equal(a, b)


def test_within_layer_hand_example():
    # inf = [[1,1],[1,7]]: layer sums 2 and 8 of 10, so the layer factors are 0.21 and 0.81.
    # global head shares [[.1,.1],[.1,.7]]  -> weights [[.021,.021],[.081,.567]], sum .69
    # layer-wise shares  [[.5,.5],[.125,.875]] -> weights [[.105,.105],[.10125,.70875]], sum 1.02
    inf = np.array([[1.0, 1.0], [1.0, 7.0]])
    assert (O.alloc_budgets(inf, 0, 690) == np.array([[21, 21], [81, 567]])).all()
    # 1020 * w / 1.02 = [[105, 105], [101.25, 708.75]]: the odd seat goes to the larger remainder
    assert (O.alloc_budgets(inf, 0, 1020, within_layer=True) == np.array([[105, 105], [101, 709]])).all()
    # fixed parts ride on top
    assert (O.alloc_budgets(inf, 3, 1020 + 12, within_layer=True) == np.array([[108, 108], [104, 712]])).all()


def test_within_layer_makes_the_layer_floor_effective():
    # a layer with next to no influence keeps ~0.01 / (1 + 0.01 L) of the pool under the layer-wise normaliser
    # (what Sec. 3.3's "minimum layer budget" is for) and next to nothing under the global one
    rng = np.random.default_rng(6)
    L, H, D = 8, 6, 1_000_000
    inf = rng.lognormal(0, 1.0, size=(L, H))
    inf[3] = 1e-9
    g = O.alloc_budgets(inf, 0, D)
    w = O.alloc_budgets(inf, 0, D, within_layer=True)
    assert g[3].sum() <= 1
    assert abs(w[3].sum() - D * 0.01 / (1.0 + 0.01 * L)) <= H
    # every layer's total follows (0.01 + L_i) / (1 + 0.01 L)
    Li = inf.sum(axis=1) / inf.sum()
    assert np.all(np.abs(w.sum(axis=1) - D * (0.01 + Li) / (1.0 + 0.01 * L)) <= H)


@pytest.mark.parametrize("seed", range(8))
def test_cap_matches_exact_rational_water_filling(seed):
    rng = np.random.default_rng(300 + seed)
    while True:
        H = int(rng.integers(3, 10))
        inf = rng.integers(1, 40, size=(1, H))
        inf[0, rng.integers(0, H)] *= 25                   # one head would take most of the pool
        fixed = int(rng.integers(0, 10))
        room = int(rng.integers(20, 200))
        D = int(rng.integers(room, room * H))              # feasible, and at least one head hits the cap
        # fp64 quotas cannot reproduce exact ties between remainders: draw again when the exact remainders of the
        # heads that stay below the cap are not all different
        seats = waterfill_exact([int(v) for v in inf[0]], D, room)
        open_heads = [a for a in range(H) if seats[a] < room]
        left = D - room * (H - len(open_heads))
        tot = sum(int(inf[0, a]) for a in open_heads)
        rems = [Fraction(int(inf[0, a]) * left, tot) % 1 for a in open_heads]
        if len(set(rems)) == len(rems):
            break
    C = O.alloc_budgets(inf.astype(np.float64), fixed, fixed * H + D, cap=fixed + room)
    assert (C - fixed).ravel().tolist() == waterfill_exact([int(v) for v in inf[0]], D, room)
    assert int(C.sum()) == fixed * H + D and C.max() <= fixed + room and C.min() >= fixed


def test_cap_edges():
    inf = np.array([[100.0, 1.0, 1.0]])
    # no head reaches the cap: same as without
    assert np.array_equal(O.alloc_budgets(inf, 5, 15 + 30, cap=1000), O.alloc_budgets(inf, 5, 15 + 30))
    # total == N * cap: everybody is full
    assert O.alloc_budgets(inf, 5, 3 * 40, cap=40).ravel().tolist() == [40, 40, 40]
    # the heavy head is filled, the others split the rest evenly (equal weights): 5 + 35, then 20 over two heads
    assert O.alloc_budgets(inf, 5, 15 + 55, cap=40).ravel().tolist() == [40, 15, 15]
    # chain: filling one head pushes the next one over the cap as well
    assert O.alloc_budgets(np.array([[50.0, 30.0, 1.0, 1.0]]), 0, 100, cap=35).ravel().tolist() == [35, 35, 15, 15]
    for bad in (dict(cap=4), dict(cap=10)):                # cap below fixed; total above N * cap
        with pytest.raises(O.OracleError) as e:
            O.alloc_budgets(inf, 5, 15 + 30, **bad)
        assert e.value.code == "BUDGET_SUM"


def test_paper_rounding_agrees_with_the_papers_parameters():
    # (fixed, total) = (b_c (1 - 1/beta), b_c L H): the same numbers as Eq. 6 in (b_c, beta)
    rng = np.random.default_rng(7)
    inf = rng.lognormal(0, 1.5, size=(5, 4))
    b_c, beta = 128.0, 4.0 / 3.0                           # fixed 32, pool 96 per head
    a = O.alloc_paper_literal(b_c, beta, inf)
    b = O.alloc_budgets(inf, 32, 128 * 20, paper_rounding=True)
    assert np.array_equal(a, b)
    assert int(b.sum()) != 128 * 20                        # not normalised: the sum is not the total
    # the hand example of Eq. 6: fixed 50, pool 200
    assert O.alloc_budgets(np.array([[1.0, 3.0], [2.0, 2.0]]), 50, 400, paper_rounding=True).tolist() == [[63, 88], [76, 76]]
    # clipped at the cap, nothing handed on
    assert O.alloc_budgets(np.array([[1.0, 3.0], [2.0, 2.0]]), 50, 400, paper_rounding=True, cap=80).tolist() == [[63, 80], [76, 76]]
    # all-zero scores: the pool in equal parts
    assert O.alloc_budgets(np.zeros((2, 2)), 10, 40 + 10, paper_rounding=True).tolist() == [[13, 13], [13, 13]]
