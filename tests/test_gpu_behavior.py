"""GPU parity of the Stage-1 attention behaviour analysis (Sec. 3.2, Algorithm 1) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import slkv_oracle as O
from paper_2508_15806_b200 import binding as B
from paper_2508_15806_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 2e-7      # the scores are ratios of fp64 sums of at most a few hundred fp32 weights, returned as fp32


def oracle_rows(attn, needle, topk):
    out = np.zeros((attn.shape[0], 3))
    for r in range(attn.shape[0]):
        n = needle[r] if needle.ndim == 2 else needle
        t = topk[r] if topk.ndim == 2 else topk
        n = [int(i) for i in n if 0 <= i < attn.shape[1]]
        t = [int(i) for i in t if 0 <= i < attn.shape[1]]
        out[r] = O.behavior_scores(attn[r], n, t)
    return out


def gpu_rows(attn, needle, topk):
    dev = torch.device("cuda:0")
    sf, lg, inf = B.slkv_behavior_scores(attn.to(dev), needle.to(dev), topk.to(dev))
    torch.cuda.synchronize()
    return np.stack([sf.cpu().numpy(), lg.cpu().numpy(), inf.cpu().numpy()], axis=1).astype(np.float64)


@pytest.mark.parametrize("n_rows,row_len,n_needle,top_k", [(1, 64, 4, 8), (300, 1024, 12, 16), (1000, 6144, 20, 50),
                                                            (77, 2000, 1, 1), (129, 4096, 40, 200)])
def test_matches_oracle_on_probe_shaped_rows(n_rows, row_len, n_needle, top_k):
    attn, needle, topk = synth.behavior_rows(n_rows, row_len, n_needle, top_k, seed=n_rows + top_k)
    got = gpu_rows(attn, needle, topk)
    ref = oracle_rows(attn.numpy(), needle.numpy(), topk.numpy())
    assert np.all(np.abs(got - ref) <= TOL * (1.0 + np.abs(ref)))
    assert np.all((got >= 0) & (got <= 1.0 + 1e-6))
    # the rows were built to cover the range: heads that ignore the needle and heads that retrieve it
    assert ref[:, 2].min() < 0.05 or n_rows < 50
    assert ref[:, 2].max() > 0.5 or n_rows < 50


def test_sets_padding_shared_lists_and_degenerate_rows():
    attn, needle, topk = synth.behavior_rows(40, 512, 6, 10, seed=3)
    # an index listed twice counts once; entries outside the row are padding
    needle2 = torch.cat([needle, needle[:, :3], torch.full((40, 2), -1, dtype=torch.int32)], dim=1).contiguous()
    topk2 = torch.cat([topk[:, :4], topk, torch.full((40, 3), 512, dtype=torch.int32)], dim=1).contiguous()
    ref = oracle_rows(attn.numpy(), needle.numpy(), topk.numpy())
    assert np.all(np.abs(gpu_rows(attn, needle2, topk2) - ref) <= TOL * (1.0 + np.abs(ref)))
    # one list for all rows
    shared_n, shared_t = needle[0].contiguous(), topk[0].contiguous()
    ref = oracle_rows(attn.numpy(), shared_n.numpy(), shared_t.numpy())
    assert np.all(np.abs(gpu_rows(attn, shared_n, shared_t) - ref) <= TOL * (1.0 + np.abs(ref)))
    # nothing correct -> all three scores 0; everything correct and complete -> all three 1
    W = torch.tensor([[0.5, 0.2, 0.2, 0.1]])
    assert gpu_rows(W, torch.tensor([[1]], dtype=torch.int32), torch.tensor([[0]], dtype=torch.int32)).tolist() == [[0.0, 0.0, 0.0]]
    assert gpu_rows(W, torch.tensor([[0, 1]], dtype=torch.int32), torch.tensor([[1, 0]], dtype=torch.int32)).tolist() == [[1.0, 1.0, 1.0]]
    # a row of zeros: every ratio is 0/0
    Z = torch.zeros(1, 4)
    assert gpu_rows(Z, torch.tensor([[0]], dtype=torch.int32), torch.tensor([[0]], dtype=torch.int32)).tolist() == [[0.0, 0.0, 0.0]]


def test_printed_table_values():
    # rows with the SF_sc / LG_sc of the paper's top-10 tables (LG from the harmonic-mean identity): INF_sc as printed
    import os
    gold = os.path.join(os.path.dirname(__file__), "golden")

    def rows(name):
        return {l.split()[0]: float(l.split()[1]) for l in open(os.path.join(gold, name)) if l.strip() and not l.startswith("#")}
    sf, inf = rows("table7_sf_top10.txt"), rows("table8_inf_top10.txt")
    heads = sorted(sf)
    W = []
    for h in heads:
        LG = inf[h] * sf[h] / (2 * sf[h] - inf[h])
        WO = 0.3
        WD, WS = WO * (1 - sf[h]) / sf[h], WO * (1 - LG) / LG
        W.append([WO, WS, WD, 1.0 - WO - WS - WD])
    got = gpu_rows(torch.tensor(W, dtype=torch.float32), torch.tensor([0, 1], dtype=torch.int32), torch.tensor([0, 2], dtype=torch.int32))
    for r, h in enumerate(heads):
        assert abs(got[r, 0] - sf[h]) < 1e-6 and abs(got[r, 2] - inf[h]) < 1e-6
