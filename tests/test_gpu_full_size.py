"""GPU parity at the full sizes of the five configurations (Eq. 7-8, Algorithm 3), through the C ABI.

Config 1 and 2 are covered in full by test_gpu_compress.py.  Here: whole layers of the 32k-context
configuration the benchmark times (same shapes, same budgets, same launch configuration), of the ragged
batch-of-8 configuration and of the 131072-token configuration, each against the oracle on the same bytes.
Inputs are drawn on the GPU by the shared generator and copied to the host for the oracle.
"""
import numpy as np
import pytest
import torch

import parity as P
from oracle import slkv_oracle as O
from paper_2508_15806_b200 import synth

pytestmark = pytest.mark.gpu


def full_layer(wl, layer, total):
    x = synth.layer_inputs(wl, layer, device="cuda")
    q, k, v = x.q_win.cpu(), x.k.cpu(), x.v.cpu()
    bud = O.alloc_budgets(synth.inf_sc(wl).numpy(), wl.fixed, total)[layer].tolist()
    gpu, stats = P.check_compress(q, k, v, wl.cu_seqlens, bud, wl.window, wl.pool_kernel)
    return x, bud, gpu, stats


@pytest.mark.parametrize("layer,total_index", [(0, 1), (1, 1), (17, 1), (31, 1), (17, 0), (17, 2)])
def test_config3_full_layers(layer, total_index):
    wl = synth.workloads()[2]
    x, bud, gpu, stats = full_layer(wl, layer, wl.totals[total_index])
    assert stats["segments"] == 8 and stats["pooled_max_rel_err"] < 1e-3
    assert int(gpu["offsets"][-1]) == sum(min(32768, max(b, wl.window)) for b in bud)
    for h in range(8):                      # needles survive wherever the head keeps enough history rows
        if bud[h] - wl.window >= 20 * wl.pool_kernel:
            a, b = gpu["offsets"][h], gpu["offsets"][h + 1]
            assert set(x.needles[0]) <= set(gpu["kept_idx"][a:b].tolist())


@pytest.mark.parametrize("layer", [0, 31])
def test_config4_ragged_batch_full_layer(layer):
    wl = synth.workloads()[3]
    _, bud, gpu, stats = full_layer(wl, layer, wl.totals[0])
    assert stats["segments"] == 8 * 8 and stats["pooled_max_rel_err"] < 1e-3


def test_config5_long_context_heavy_and_fixed_only_layers():
    wl = synth.workloads()[4]
    budgets = O.alloc_budgets(synth.inf_sc(wl).numpy(), wl.fixed, wl.totals[0])
    heavy = int(np.argmax((budgets > wl.total_tokens).sum(axis=1) * 10**9 + budgets.max(axis=1)))
    fixed_only = int(np.argmin(budgets.max(axis=1)))
    assert budgets[heavy].max() > 20000 and budgets[fixed_only].max() <= 2 * wl.fixed
    for layer in (heavy, fixed_only):
        _, bud, gpu, stats = full_layer(wl, layer, wl.totals[0])
        assert stats["segments"] == 8 and stats["pooled_max_rel_err"] < 1e-3


def test_config5_long_context_split_over_four_ranks():
    # the 131072-token sequence with its history keys split over 4 ranks (emulated on this GPU, one host thread and
    # stream per rank): the ranks' packed rows together against the oracle on the whole sequence
    from test_gpu_context_parallel import as_one_layer, run_ranks
    wl = synth.workloads()[4]
    budgets = O.alloc_budgets(synth.inf_sc(wl).numpy(), wl.fixed, wl.totals[0])
    layer = int(np.argmax((budgets > wl.total_tokens).sum(axis=1) * 10**9 + budgets.max(axis=1)))
    x = synth.layer_inputs(wl, layer, device="cuda")
    q, k, v = x.q_win.cpu(), x.k.cpu(), x.v.cpu()
    bud = budgets[layer].tolist()
    ref = P.oracle_pooled(q, k, wl.cu_seqlens, wl.window, wl.pool_kernel)
    outs = run_ranks(4, q, k, v, bud, wl.window, wl.pool_kernel)
    assert all(int(o["status"].item()) == 0 for o in outs)
    gpu = as_one_layer(outs, 4, wl.total_tokens, wl.window, wl.pool_kernel, wl.n_kv_heads)
    assert P.assert_pooled_close(gpu["pooled"], ref, wl.cu_seqlens, wl.n_kv_heads, wl.window) < 1e-3
    stats = P.assert_selection_valid(gpu, ref, wl.cu_seqlens, bud, wl.window, k, v)
    assert stats["segments"] == 8


def test_config3_full_layers_through_the_overlapped_entry_point():
    # the launch configuration bench.py times: layers queued by slkv_compress_overlapped, the score kernel taking
    # them a list at a time (here 10 layers: a full list of 8, then the rest at the join).  Pooled scores and the
    # selection of two of the layers against the oracle, every layer against slkv_compress bit for bit.
    from paper_2508_15806_b200 import binding as B
    wl = synth.workloads()[2]
    total = wl.totals[1]
    dev = torch.device("cuda:0")
    layers = [0, 1, 2, 3, 17, 18, 19, 20, 30, 31]
    budgets = O.alloc_budgets(synth.inf_sc(wl).numpy(), wl.fixed, total)
    xs = [synth.layer_inputs(wl, l, device=dev) for l in layers]
    cu = wl.cu_seqlens
    cu_dev = torch.tensor(cu, dtype=torch.int32, device=dev)
    params = B.make_params(xs[0].q_win, xs[0].k, xs[0].v, wl.window, wl.pool_kernel)
    ws = torch.empty(B.slkv_workspace_bytes_overlapped(params, cu), dtype=torch.uint8, device=dev)
    cap = B.slkv_packed_rows_upper_bound(params, cu)
    n_pool = B.slkv_pooled_elems(params, cu)
    buds = [torch.tensor(budgets[l].tolist(), dtype=torch.int32, device=dev) for l in layers]

    def outputs():
        return [dict(k_out=torch.zeros(cap, 128, dtype=torch.bfloat16, device=dev),
                     v_out=torch.zeros(cap, 128, dtype=torch.bfloat16, device=dev),
                     offsets=torch.zeros(9, dtype=torch.int32, device=dev),
                     kept=torch.full((cap,), -1, dtype=torch.int32, device=dev),
                     pooled=torch.full((n_pool,), float("nan"), dtype=torch.float32, device=dev),
                     status=torch.zeros(1, dtype=torch.int32, device=dev)) for _ in layers]

    def run(fn, outs, lses=None):
        for i, (x, bud, o) in enumerate(zip(xs, buds, outs)):
            fn(params, x.q_win, x.k, x.v, cu_dev, cu, bud, o["k_out"], o["v_out"], o["offsets"], o["kept"], ws,
               o["pooled"], o["status"], lse=None if lses is None else lses[i])
        B.slkv_join()
        torch.cuda.synchronize()

    a, b = outputs(), outputs()
    run(B.slkv_compress, a)
    run(B.slkv_compress_overlapped, b)
    # the same layers with their row log-sum-exps handed over (the vote pass alone on both streams of the list kernel,
    # three epilogue warpgroups per stream): with the library's own log-sum-exps the scores agree with the two-pass
    # results to rounding (another kernel computed the statistics, in another order) and the selections are valid
    lses = []
    for x in xs:
        lse = torch.empty(1, wl.n_q_heads, wl.window, dtype=torch.float32, device=dev)
        p2 = B.make_params(x.q_win, x.k, x.v, wl.window, wl.pool_kernel, lse_units=B.SLKV_LSE_LOG2)
        B.slkv_row_lse(p2, x.q_win, x.k, cu_dev, cu, lse, ws)
        lses.append(lse)
    torch.cuda.synchronize()
    c = outputs()
    params_log2 = B.make_params(xs[0].q_win, xs[0].k, xs[0].v, wl.window, wl.pool_kernel, lse_units=B.SLKV_LSE_LOG2)
    for i, (x, bud, o) in enumerate(zip(xs, buds, c)):
        B.slkv_compress_overlapped(params_log2, x.q_win, x.k, x.v, cu_dev, cu, bud, o["k_out"], o["v_out"], o["offsets"],
                                   o["kept"], ws, o["pooled"], o["status"], lse=lses[i])
    B.slkv_join()
    torch.cuda.synchronize()
    for i in range(len(layers)):
        assert int(c[i]["status"].item()) == 0
        n = int(a[i]["offsets"][-1].item())
        assert torch.equal(c[i]["offsets"], a[i]["offsets"])
        assert torch.allclose(c[i]["pooled"], a[i]["pooled"], rtol=2e-5, atol=0)
        off = a[i]["offsets"].tolist()
        swapped = sum(len(set(c[i]["kept"][s0:s1].tolist()) ^ set(a[i]["kept"][s0:s1].tolist())) // 2
                      for s0, s1 in zip(off, off[1:]))
        assert swapped <= 8                           # positions may swap only inside the rounding band at the threshold
    for i, l in enumerate(layers):
        assert int(b[i]["status"].item()) == 0
        n = int(a[i]["offsets"][-1].item())
        assert n == int(budgets[l].clip(wl.window, 32768).sum())
        assert torch.equal(a[i]["offsets"], b[i]["offsets"]) and torch.equal(a[i]["kept"][:n], b[i]["kept"][:n])
        assert torch.equal(a[i]["k_out"][:n], b[i]["k_out"][:n]) and torch.equal(a[i]["v_out"][:n], b[i]["v_out"][:n])
    for i in (1, 9):                                  # layer 1 (three near-zero heads) and layer 31
        x = xs[i]
        q, k, v = x.q_win.cpu(), x.k.cpu(), x.v.cpu()
        ref = P.oracle_pooled(q, k, cu, wl.window, wl.pool_kernel)
        for res in (b, c):                            # two passes, and the vote pass alone
            gpu = {"offsets": res[i]["offsets"].cpu().numpy().astype(np.int64),
                   "kept_idx": res[i]["kept"].cpu().numpy().astype(np.int64),
                   "k_out": res[i]["k_out"].cpu(), "v_out": res[i]["v_out"].cpu()}
            P.assert_pooled_close(res[i]["pooled"].cpu().numpy(), ref, cu, wl.n_kv_heads, wl.window)
            P.assert_selection_valid(gpu, ref, cu, budgets[layers[i]].tolist(), wl.window, k, v)
