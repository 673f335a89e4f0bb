"""GPU parity of the all-causal softmax domain and of caller-supplied row log-sum-exps (Sec. 3.4, Eq. 7; Eq. 3-4),
and the bounded inter-CTA waits, through the C ABI."""
import numpy as np
import pytest
import torch

import parity as P
from oracle import slkv_oracle as O
from paper_2508_15806_b200 import binding as B
from paper_2508_15806_b200 import synth

pytestmark = pytest.mark.gpu

LSE_ABS_TOL = 2e-4        # a row normaliser off by this much moves every vote of the row by 2e-4 (bound: 1e-3)


def rand_case(Hq, Hkv, w, lens, seed, d=128, dtype=torch.bfloat16, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    T = sum(lens)
    q = (torch.randn(len(lens), w, Hq, d, generator=g) * scale).to(dtype)
    k = (torch.randn(T, Hkv, d, generator=g) * scale).to(dtype)
    v = torch.randn(T, Hkv, d, generator=g).to(dtype)
    return q, k, v, [0] + [int(x) for x in np.cumsum(lens)]


CASES = [
    # Hq, Hkv, w, lens, d, dtype, path
    (8, 8, 16, [300, 16, 17, 90], 64, torch.float32, B.SLKV_PATH_SIMT),       # fp32 FMA path, len == w and w + 1
    (8, 2, 32, [700, 160], 128, torch.bfloat16, B.SLKV_PATH_SIMT),
    (8, 2, 32, [700, 160, 33], 128, torch.bfloat16, B.SLKV_PATH_TENSOR),      # R = 128
    (8, 2, 64, [900, 333], 128, torch.bfloat16, B.SLKV_PATH_TENSOR),          # R = 256: two M tiles
    (4, 1, 16, [515], 128, torch.bfloat16, B.SLKV_PATH_TENSOR),               # R = 64
]


@pytest.mark.parametrize("Hq,Hkv,w,lens,d,dtype,path", CASES)
def test_all_causal_domain_matches_oracle(Hq, Hkv, w, lens, d, dtype, path):
    q, k, v, cu = rand_case(Hq, Hkv, w, lens, seed=Hq + w + len(lens), d=d, dtype=dtype, scale=1.5)
    bud = [w + 7 + 31 * h for h in range(Hkv)]
    gpu, stats = P.check_compress(q, k, v, cu, bud, w, 5, score_path=path, domain=B.SLKV_ALL_CAUSAL)
    assert stats["pooled_max_rel_err"] < 1e-3
    # the window keys take their share of every row: the history votes no longer sum to w
    hist = P.split_pooled(P.gpu_score(q, k, cu, w, 1, score_path=path, domain=B.SLKV_ALL_CAUSAL), cu, Hkv, w)
    assert all(h.sum(axis=1).max() < w for h in hist if h.size)


@pytest.mark.parametrize("Hq,Hkv,w,lens,d,dtype,path", CASES)
@pytest.mark.parametrize("domain", [B.SLKV_HISTORY, B.SLKV_ALL_CAUSAL])
def test_row_lse_matches_oracle(Hq, Hkv, w, lens, d, dtype, path, domain):
    q, k, v, cu = rand_case(Hq, Hkv, w, lens, seed=3 * Hq + w, d=d, dtype=dtype, scale=1.5)
    ref = O.row_lse(P.to_np64(q), P.to_np64(k), cu, w, "all_causal" if domain == B.SLKV_ALL_CAUSAL else "history")
    got = P.gpu_row_lse(q, k, cu, w, path, domain).cpu().numpy().astype(np.float64)
    has = ~np.isnan(ref)
    assert np.array_equal(np.isnan(got), ~has), "rows of sequences without history must stay untouched"
    assert np.max(np.abs(got[has] - ref[has])) < LSE_ABS_TOL
    got2 = P.gpu_row_lse(q, k, cu, w, path, domain, B.SLKV_LSE_LOG2).cpu().numpy().astype(np.float64)
    assert np.max(np.abs(got2[has] * np.log(2.0) - ref[has])) < LSE_ABS_TOL


@pytest.mark.parametrize("Hq,Hkv,w,lens,d,dtype,path", CASES)
@pytest.mark.parametrize("domain", [B.SLKV_HISTORY, B.SLKV_ALL_CAUSAL])
def test_supplied_lse_from_the_oracle(Hq, Hkv, w, lens, d, dtype, path, domain):
    q, k, v, cu = rand_case(Hq, Hkv, w, lens, seed=5 * Hq + w, d=d, dtype=dtype, scale=1.5)
    name = "all_causal" if domain == B.SLKV_ALL_CAUSAL else "history"
    lse = O.row_lse(P.to_np64(q), P.to_np64(k), cu, w, name)
    bud = [w + 5 + 40 * h for h in range(Hkv)]
    # the oracle with its own normalisers is the reference: fp64 -> fp32 of the lse costs ~1e-6
    ref = P.oracle_pooled(q, k, cu, w, 7, domain=domain)
    gpu = P.gpu_compress(q, k, v, cu, bud, w, 7, score_path=path, lse=lse)      # the domain flag plays no part now
    assert gpu["status"] == 0
    P.assert_pooled_close(gpu["pooled"], ref, cu, Hkv, w)
    P.assert_selection_valid(gpu, ref, cu, bud, w, k, v)
    # an lse that is not the rows' own is used as given: one unit more divides the votes by e
    lse_off = np.where(np.isnan(lse), lse, lse + 1.0)
    a = P.gpu_score(q, k, cu, w, 1, score_path=path, lse=lse)
    b = P.gpu_score(q, k, cu, w, 1, score_path=path, lse=lse_off)
    assert np.allclose(b * np.e, a, rtol=1e-5, atol=0)


@pytest.mark.parametrize("path,dtype,d", [(B.SLKV_PATH_TENSOR, torch.bfloat16, 128), (B.SLKV_PATH_SIMT, torch.float32, 64)])
@pytest.mark.parametrize("domain", [B.SLKV_HISTORY, B.SLKV_ALL_CAUSAL])
def test_feeding_back_the_librarys_lse_reproduces_the_call_bit_for_bit(path, dtype, d, domain):
    q, k, v, cu = rand_case(8, 2, 32, [2100, 40, 600], seed=17, d=d, dtype=dtype)
    own = P.gpu_score(q, k, cu, 32, 7, score_path=path, domain=domain)
    lse2 = P.gpu_row_lse(q, k, cu, 32, path, domain, B.SLKV_LSE_LOG2)
    lse2 = torch.nan_to_num(lse2, nan=0.0)
    fed = P.gpu_score(q, k, cu, 32, 7, score_path=path, domain=domain, lse=lse2, lse_units=B.SLKV_LSE_LOG2)
    assert np.array_equal(own.view(np.uint32), fed.view(np.uint32))
    # natural-log units round once on the way out and once on the way in
    lse_ln = torch.nan_to_num(P.gpu_row_lse(q, k, cu, 32, path, domain, B.SLKV_LSE_LN), nan=0.0)
    fed_ln = P.gpu_score(q, k, cu, 32, 7, score_path=path, domain=domain, lse=lse_ln)
    assert np.allclose(fed_ln, own, rtol=5e-6, atol=0)


def overlapped_layers(xs, cu, buds, w, p, domain=B.SLKV_HISTORY, lses=None, want_status=0):
    """The layers of `xs` through slkv_compress_overlapped + slkv_join; host results per layer."""
    dev = torch.device("cuda:0")
    cu = [int(c) for c in cu]
    cu_dev = torch.tensor(cu, dtype=torch.int32, device=dev)
    q0, k0, v0 = xs[0]
    params = B.make_params(q0.to(dev), k0.to(dev), v0.to(dev), w, p, B.SLKV_POOL_MAX, B.SLKV_PATH_TENSOR, domain)
    cap = B.slkv_packed_rows_upper_bound(params, cu)
    n_seg = (len(cu) - 1) * k0.shape[1]
    n_pool = B.slkv_pooled_elems(params, cu)
    ws = torch.empty(B.slkv_workspace_bytes_overlapped(params, cu), dtype=torch.uint8, device=dev)
    keep, outs = [], []
    for i, (q, k, v) in enumerate(xs):
        qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
        bud = torch.tensor(list(buds[i]), dtype=torch.int32, device=dev)
        lse = None if lses is None or lses[i] is None else P.lse_to_dev(lses[i])
        o = dict(k_out=torch.zeros(cap, 128, dtype=k.dtype, device=dev), v_out=torch.zeros(cap, 128, dtype=k.dtype, device=dev),
                 offsets=torch.full((n_seg + 1,), -1, dtype=torch.int32, device=dev),
                 kept=torch.full((cap,), -1, dtype=torch.int32, device=dev),
                 pooled=torch.full((n_pool,), float("nan"), dtype=torch.float32, device=dev),
                 status=torch.zeros(1, dtype=torch.int32, device=dev))
        B.slkv_compress_overlapped(params, qd, kd, vd, cu_dev, cu, bud, o["k_out"], o["v_out"], o["offsets"], o["kept"],
                                   ws, o["pooled"], o["status"], lse=lse)
        keep.append((qd, kd, vd, bud, lse))
        outs.append(o)
    B.slkv_join()
    torch.cuda.synchronize()
    res = []
    for o in outs:
        res.append({"offsets": o["offsets"].cpu().numpy().astype(np.int64), "kept_idx": o["kept"].cpu().numpy().astype(np.int64),
                    "k_out": o["k_out"].cpu(), "v_out": o["v_out"].cpu(), "pooled": o["pooled"].cpu().numpy(),
                    "status": int(o["status"].item())})
    return res


@pytest.mark.parametrize("n_layers", [1, 2, 5, 11, 43])
def test_overlapped_calls_with_supplied_lse(n_layers):
    # every layer comes with its row statistics: the list kernel runs the vote pass on both of its streams.  The
    # selections of a full list are held back until the next list is out; 43 layers take every workspace slot more
    # than twice while some are held back (inputs cycle through 6 cases, the budgets differ per layer).
    w, p, lens = 32, 7, [1500, 700]
    cases = []
    for c in range(min(n_layers, 6)):
        q, k, v, cu = rand_case(8, 2, w, lens, seed=100 + c, scale=1.2)
        dom = "all_causal" if c % 2 else "history"
        cases.append((q, k, v, O.row_lse(P.to_np64(q), P.to_np64(k), cu, w, dom),
                      P.oracle_pooled(q, k, cu, w, p, domain=B.SLKV_ALL_CAUSAL if c % 2 else B.SLKV_HISTORY)))
    xs = [cases[i % len(cases)][:3] for i in range(n_layers)]
    lses = [cases[i % len(cases)][3] for i in range(n_layers)]
    refs = [cases[i % len(cases)][4] for i in range(n_layers)]
    buds = [[w + 10 + 17 * i, 300 + i] for i in range(n_layers)]
    res = overlapped_layers(xs, cu, buds, w, p, lses=lses)
    for i, gpu in enumerate(res):
        assert gpu["status"] == 0
        P.assert_pooled_close(gpu["pooled"], refs[i], cu, 2, w)
        P.assert_selection_valid(gpu, refs[i], cu, buds[i], w, xs[i][1], xs[i][2])


def test_overlapped_calls_mixing_supplied_and_computed_lse_and_domains():
    w, p, lens = 32, 5, [900, 2300]
    xs, buds, lses, refs = [], [], [], []
    for i in range(7):
        q, k, v, cu = rand_case(8, 2, w, lens, seed=200 + i)
        xs.append((q, k, v))
        buds.append([w + 3 + 29 * i, 555])
        lses.append(O.row_lse(P.to_np64(q), P.to_np64(k), cu, w, "all_causal") if i in (2, 3, 6) else None)
        refs.append(P.oracle_pooled(q, k, cu, w, p, domain=B.SLKV_ALL_CAUSAL))
    res = overlapped_layers(xs, cu, buds, w, p, domain=B.SLKV_ALL_CAUSAL, lses=lses)
    for i, gpu in enumerate(res):
        assert gpu["status"] == 0
        P.assert_pooled_close(gpu["pooled"], refs[i], cu, 2, w)
        P.assert_selection_valid(gpu, refs[i], cu, buds[i], w, xs[i][1], xs[i][2])


def test_all_causal_on_a_full_cfg2_layer():
    wl = synth.workloads()[1]
    x = synth.layer_inputs(wl, 0)
    bud = O.alloc_budgets(synth.inf_sc(wl).numpy(), wl.fixed, wl.totals[0])[0].tolist()
    gpu, stats = P.check_compress(x.q_win, x.k, x.v, wl.cu_seqlens, bud, wl.window, wl.pool_kernel,
                                  domain=B.SLKV_ALL_CAUSAL)
    assert stats["pooled_max_rel_err"] < 1e-3


# ---- bounded waits -----------------------------------------------------------------------------------------------
def test_a_wait_that_runs_out_is_reported_and_leaves_the_next_call_intact():
    # The grid-wide barrier of the fused score kernel is told to expect one arrival more than there are CTAs: every
    # CTA gives up after its time limit, the status word says so, and the following call -- which may land on the same
    # barrier slot 64 launches later -- is correct.
    q, k, v, cu = rand_case(8, 2, 32, [6000], seed=31)
    bud = [100, 400]
    B.slkv_debug_expire_next_wait(True)
    broken = P.gpu_compress(q, k, v, cu, bud, 32, 7, score_path=B.SLKV_PATH_TENSOR)
    assert broken["status"] == B.ERR["DEVICE_TIMEOUT"]
    ref = P.oracle_pooled(q, k, cu, 32, 7)
    for _ in range(66):                                   # once around the table of barrier slots
        good = P.gpu_compress(q, k, v, cu, bud, 32, 7, score_path=B.SLKV_PATH_TENSOR, want_pooled=False)
        assert good["status"] == 0
    good = P.gpu_compress(q, k, v, cu, bud, 32, 7, score_path=B.SLKV_PATH_TENSOR)
    assert good["status"] == 0
    P.assert_pooled_close(good["pooled"], ref, cu, 2, 32)
    P.assert_selection_valid(good, ref, cu, bud, 32, k, v)


def test_a_wait_that_runs_out_in_the_list_kernel():
    w, p, lens = 32, 7, [3000]
    xs, buds = [], []
    for i in range(3):
        q, k, v, cu = rand_case(8, 2, w, lens, seed=300 + i)
        xs.append((q, k, v))
        buds.append([64, 200])
    B.slkv_debug_expire_next_wait(True)
    res = overlapped_layers(xs, cu, buds, w, p)
    assert any(r["status"] == B.ERR["DEVICE_TIMEOUT"] for r in res)
    B.slkv_debug_expire_next_wait(False)
    res = overlapped_layers(xs, cu, buds, w, p)
    for i, gpu in enumerate(res):
        assert gpu["status"] == 0
        ref = P.oracle_pooled(xs[i][0], xs[i][1], cu, w, p)
        P.assert_pooled_close(gpu["pooled"], ref, cu, 2, w)
        P.assert_selection_valid(gpu, ref, cu, buds[i], w, xs[i][1], xs[i][2])
