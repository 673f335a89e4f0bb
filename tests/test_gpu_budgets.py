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
