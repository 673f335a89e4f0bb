"""GPU parity: slkv_alloc_budgets against the oracle, bit for bit (Algorithm 2 / Eq. 6)."""
import numpy as np
import pytest
import torch

from oracle import slkv_oracle as O
from paper_2508_15806_b200 import binding as B
from paper_2508_15806_b200 import synth

pytestmark = pytest.mark.gpu


def gpu_budgets(inf: torch.Tensor, fixed: int, total: int):
    dev = torch.device("cuda:0")
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    out = B.slkv_alloc_budgets(inf.to(dev).contiguous(), fixed, total, status=status)
    torch.cuda.synchronize()
    return out.cpu().numpy().astype(np.int64), int(status.item())


def test_all_configs_bit_exact():
    for wl in synth.workloads():
        inf = synth.inf_sc(wl)
        for total in wl.totals:
            got, st = gpu_budgets(inf, wl.fixed, total)
            ref = O.alloc_budgets(inf.numpy(), wl.fixed, total)
            assert st == 0 and np.array_equal(got, ref), wl.name
            assert int(got.sum()) == total and got.min() >= wl.fixed


@pytest.mark.parametrize("seed", range(8))
def test_random_tables_bit_exact(seed):
    rng = np.random.default_rng(seed)
    L, H = int(rng.integers(1, 40)), int(rng.integers(1, 40))
    inf = torch.from_numpy(rng.lognormal(0, 2.0, size=(L, H)).astype(np.float32))
    if seed % 3 == 0:
        inf[rng.integers(0, L), :] = 0.0
    fixed = int(rng.integers(0, 200))
    total = fixed * L * H + int(rng.integers(0, 5_000_000))
    got, st = gpu_budgets(inf, fixed, total)
    assert st == 0 and np.array_equal(got, O.alloc_budgets(inf.numpy(), fixed, total))


def test_edge_tables():
    cases = [(torch.ones(3, 5), 10, 150 + 7), (torch.zeros(2, 3), 4, 32), (torch.ones(1, 1), 0, 0),
             (torch.tensor([[1e-30, 1e30]]), 1, 1000), (torch.full((4, 4), 1e-45), 0, 99),
             (torch.rand(128, 128) , 64, 128 * 128 * 200)]
    for inf, fixed, total in cases:
        inf = inf.to(torch.float32)
        got, st = gpu_budgets(inf, fixed, total)
        assert st == 0 and np.array_equal(got, O.alloc_budgets(inf.numpy(), fixed, total))


def test_bad_inf_sets_status_word():
    for bad in (-1.0, float("nan"), float("inf")):
        inf = torch.ones(2, 4)
        inf[1, 2] = bad
        _, st = gpu_budgets(inf, 1, 100)
        assert st == B.ERR["NEG_INF_SC"]


# ---- the readings Sec. 3.3 leaves open: head normaliser, cap with water filling, Algorithm 2's own rounding --------
def gpu_budgets_ex(inf, fixed, total, within_layer=False, cap=0, paper_rounding=False):
    dev = torch.device("cuda:0")
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    opt = B.SlkvAllocOptions(head_normaliser=B.SLKV_NORM_WITHIN_LAYER if within_layer else B.SLKV_NORM_GLOBAL,
                             rounding=B.SLKV_ROUND_PAPER if paper_rounding else B.SLKV_ROUND_SUM_EXACT, cap=cap)
    out = B.slkv_alloc_budgets(inf.to(dev).contiguous(), fixed, total, status=status, options=opt)
    torch.cuda.synchronize()
    return out.cpu().numpy().astype(np.int64), int(status.item())


VARIANTS = [dict(within_layer=True), dict(paper_rounding=True), dict(within_layer=True, paper_rounding=True)]


@pytest.mark.parametrize("kw", VARIANTS)
def test_variants_on_all_configs_bit_exact(kw):
    for wl in synth.workloads():
        inf = synth.inf_sc(wl)
        for total in wl.totals:
            got, st = gpu_budgets_ex(inf, wl.fixed, total, **kw)
            ref = O.alloc_budgets(inf.numpy(), wl.fixed, total, **kw)
            assert st == 0 and np.array_equal(got, ref), (wl.name, kw)
            if not kw.get("paper_rounding"):
                assert int(got.sum()) == total and got.min() >= wl.fixed


def test_cap_at_the_sequence_length_on_all_configs():
    # the skewed table of the long-context workload hands six heads far more than a head can keep: capped at the
    # sequence length, the excess goes to the other heads and the total is still met
    for wl in synth.workloads():
        inf = synth.inf_sc(wl)
        cap = max(wl.seq_lens)
        for total in wl.totals:
            for within in (False, True):
                got, st = gpu_budgets_ex(inf, wl.fixed, total, within_layer=within, cap=cap)
                ref = O.alloc_budgets(inf.numpy(), wl.fixed, total, within_layer=within, cap=cap)
                assert st == 0 and np.array_equal(got, ref), wl.name
                assert int(got.sum()) == total and got.max() <= cap and got.min() >= wl.fixed
    wl = synth.workloads()[4]
    plain, _ = gpu_budgets(synth.inf_sc(wl), wl.fixed, wl.totals[0])
    capped, _ = gpu_budgets_ex(synth.inf_sc(wl), wl.fixed, wl.totals[0], cap=max(wl.seq_lens))
    assert plain.max() > max(wl.seq_lens) and (capped == max(wl.seq_lens)).sum() >= 1
    assert (capped >= np.minimum(plain, max(wl.seq_lens))).all()      # nobody loses by the cap


@pytest.mark.parametrize("seed", range(10))
def test_random_tables_with_options_bit_exact(seed):
    rng = np.random.default_rng(1000 + seed)
    L, H = int(rng.integers(1, 30)), int(rng.integers(1, 30))
    inf = torch.from_numpy(rng.lognormal(0, 2.5, size=(L, H)).astype(np.float32))
    if seed % 3 == 0:
        inf[rng.integers(0, L), :] = 0.0
    fixed = int(rng.integers(0, 100))
    room = int(rng.integers(1, 5000))
    total = fixed * L * H + int(rng.integers(0, room * L * H + 1))
    kw = dict(within_layer=bool(seed & 1), cap=fixed + room, paper_rounding=seed % 5 == 4)
    got, st = gpu_budgets_ex(inf, fixed, total, **kw)
    assert st == 0 and np.array_equal(got, O.alloc_budgets(inf.numpy(), fixed, total, **kw))


def test_option_edges():
    inf = torch.tensor([[100.0, 1.0, 1.0]])
    for kw, total in [(dict(cap=40), 3 * 40), (dict(cap=40), 15 + 55), (dict(cap=1000), 45),
                      (dict(cap=40, paper_rounding=True), 500)]:
        got, st = gpu_budgets_ex(inf, 5, total, **kw)
        assert st == 0 and np.array_equal(got, O.alloc_budgets(inf.numpy(), 5, total, **kw))
    z = torch.zeros(2, 2)
    for kw in (dict(paper_rounding=True), dict(within_layer=True), dict(cap=13)):
        got, st = gpu_budgets_ex(z, 10, 50, **kw)
        assert st == 0 and np.array_equal(got, O.alloc_budgets(z.numpy(), 10, 50, **kw))
    for kw in (dict(cap=4), dict(cap=10)):                       # cap below fixed; total above N * cap
        with pytest.raises(B.SlkvError) as e:
            gpu_budgets_ex(inf, 5, 45, **kw)
        assert e.value.code == B.ERR["BUDGET_SUM"]
