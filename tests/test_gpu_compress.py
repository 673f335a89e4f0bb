"""GPU parity: slkv_score / slkv_compress against the oracle (Eq. 7-8, Algorithm 3), through the C ABI."""
import numpy as np
import pytest
import torch

import parity as P
from oracle import slkv_oracle as O
from paper_2508_15806_b200 import binding as B
from paper_2508_15806_b200 import synth

pytestmark = pytest.mark.gpu


def layer_budgets(wl, total, layer):
    """This layer's budget row, from the oracle's allocation (the GPU allocation is checked elsewhere)."""
    return O.alloc_budgets(synth.inf_sc(wl).numpy(), wl.fixed, total)[layer].tolist()


def run_workload_layer(wl, layer, total, score_path=B.SLKV_PATH_AUTO):
    x = synth.layer_inputs(wl, layer)
    bud = layer_budgets(wl, total, layer)
    gpu, stats = P.check_compress(x.q_win, x.k, x.v, wl.cu_seqlens, bud, wl.window, wl.pool_kernel,
                                  score_path=score_path)
    return x, bud, gpu, stats


def test_config1_fp32_full():
    wl = synth.workloads()[0]
    x, bud, gpu, stats = run_workload_layer(wl, 0, wl.totals[0])
    assert sum(bud) == 1024 and stats["segments"] == 8
    # every needle (and its pooling neighbourhood) survives in every head
    for h in range(8):
        a, b = gpu["offsets"][h], gpu["offsets"][h + 1]
        kept = set(gpu["kept_idx"][a:b].tolist())
        for n in x.needles[0]:
            assert {n - 2, n - 1, n, n + 1, n + 2} <= kept


def test_config2_bf16_gqa_full():
    wl = synth.workloads()[1]
    x, bud, gpu, stats = run_workload_layer(wl, 0, wl.totals[0])
    assert stats["segments"] == 8 and stats["pooled_max_rel_err"] < 1e-3
    for h in range(8):
        a, b = gpu["offsets"][h], gpu["offsets"][h + 1]
        kept = set(gpu["kept_idx"][a:b].tolist())
        if bud[h] - wl.window >= 16 * 7:
            for n in x.needles[0]:
                assert n in kept


@pytest.mark.parametrize("path", [B.SLKV_PATH_SIMT, B.SLKV_PATH_AUTO])
@pytest.mark.parametrize("cfg,lens,n_layers,layer", [
    (2, [3000], 4, 1),                 # cfg3 shape (sinks, layer-1 near-zero heads), ragged tail
    (3, [700, 64, 1500, 65, 3, 2049], 2, 1),   # cfg4 shape: ragged batch incl. len == w, len == w+1, len < w
    (4, [5000], 3, 2),                 # cfg5 shape: extreme skew, budgets above the length
])
def test_small_variants_of_big_configs(cfg, lens, n_layers, layer, path):
    base = synth.workloads()[cfg]
    n_heads_total = n_layers * base.n_kv_heads
    per_head = base.totals[0] // (32 * base.n_kv_heads)
    wl = synth.small_variant(base, lens, n_layers=n_layers, totals=[min(per_head, 512) * n_heads_total])
    _, bud, gpu, stats = run_workload_layer(wl, layer, wl.totals[0], score_path=path)
    assert stats["segments"] == len(lens) * base.n_kv_heads


@pytest.mark.parametrize("dtype,d,Hq,Hkv,w,p,lens", [
    (torch.float32, 64, 4, 4, 16, 5, [300]),
    (torch.float32, 128, 4, 2, 8, 3, [129, 1100]),
    (torch.bfloat16, 64, 8, 2, 32, 7, [1025, 40]),
    (torch.bfloat16, 128, 2, 1, 1, 1, [257]),
    (torch.bfloat16, 128, 16, 2, 24, 9, [2100]),
])
@pytest.mark.parametrize("mode", [B.SLKV_POOL_MAX, B.SLKV_POOL_AVG])
def test_shapes_and_pool_modes(dtype, d, Hq, Hkv, w, p, lens, mode):
    g = torch.Generator().manual_seed(d + Hq + w)
    T = sum(lens)
    cu = [0] + list(np.cumsum(lens))
    q = (torch.randn(len(lens), w, Hq, d, generator=g) * 1.5).to(dtype)
    k = torch.randn(T, Hkv, d, generator=g).to(dtype)
    v = torch.randn(T, Hkv, d, generator=g).to(dtype)
    bud = [w + 5 + 37 * h for h in range(Hkv)]
    P.check_compress(q, k, v, cu, bud, w, p, pool_mode=mode, score_path=B.SLKV_PATH_SIMT)


def test_score_entry_point_matches_oracle():
    wl = synth.small_variant(synth.workloads()[1], [1500, 900])
    x = synth.layer_inputs(wl, 0)
    got = P.gpu_score(x.q_win, x.k, wl.cu_seqlens, wl.window, wl.pool_kernel)
    ref = P.oracle_pooled(x.q_win, x.k, wl.cu_seqlens, wl.window, wl.pool_kernel)
    P.assert_pooled_close(got, ref, wl.cu_seqlens, wl.n_kv_heads, wl.window)


def test_budget_edge_cases():
    g = torch.Generator().manual_seed(5)
    w, p, Hkv = 8, 3, 4
    lens = [200, 8, 5, 9]
    cu = [0] + list(np.cumsum(lens))
    q = torch.randn(4, w, 4, 64, generator=g)
    k = torch.randn(sum(lens), Hkv, 64, generator=g)
    v = torch.randn(sum(lens), Hkv, 64, generator=g)
    # budget 0 / below the window / exactly the window / one more / exactly the length / above the length
    for bud in ([0, 3, 8, 9], [200, 199, 5000, 100]):
        P.check_compress(q, k, v, cu, bud, w, p, score_path=B.SLKV_PATH_SIMT)


def test_exact_ties_prefer_lower_index():
    # all keys equal -> all scores equal -> the k lowest positions are kept
    w, d = 4, 64
    q = torch.randn(1, w, 2, d)
    k = torch.ones(100, 2, d) * 0.25
    v = torch.randn(100, 2, d)
    gpu = P.gpu_compress(q, k, v, [0, 100], [10, 50], w, 1, score_path=B.SLKV_PATH_SIMT)
    assert gpu["kept_idx"][:10].tolist() == list(range(6)) + [96, 97, 98, 99]
    assert gpu["kept_idx"][10:60].tolist() == list(range(46)) + [96, 97, 98, 99]


def test_capacity_status_and_no_overrun():
    g = torch.Generator().manual_seed(6)
    q = torch.randn(1, 4, 2, 64, generator=g); k = torch.randn(80, 2, 64, generator=g)
    gpu = P.gpu_compress(q, k, k, [0, 80], [30, 30], 4, 3, capacity=40, score_path=B.SLKV_PATH_SIMT)
    assert gpu["status"] == B.ERR["CAPACITY"] and gpu["offsets"].tolist() == [0, 30, 60]
    assert len(gpu["kept_idx"]) == 40


def test_deterministic_and_pooled_optional():
    wl = synth.small_variant(synth.workloads()[1], [2000])
    x = synth.layer_inputs(wl, 0)
    bud = [100, 64, 300, 2000, 70, 90, 128, 65]
    a = P.gpu_compress(x.q_win, x.k, x.v, wl.cu_seqlens, bud, wl.window, wl.pool_kernel)
    b = P.gpu_compress(x.q_win, x.k, x.v, wl.cu_seqlens, bud, wl.window, wl.pool_kernel, want_pooled=False)
    assert np.array_equal(a["kept_idx"], b["kept_idx"]) and torch.equal(a["k_out"], b["k_out"])
    assert a["launches"] >= 3          # score (both passes in one launch where the device allows), select, gather


def test_strided_kv_layout():
    # K and V as slices of a fused [T, 2, Hkv, d] buffer (token stride 2*Hkv*d)
    g = torch.Generator().manual_seed(7)
    T, Hkv, d, w = 600, 2, 128, 16
    kv = torch.randn(T, 2, Hkv, d, generator=g).to(torch.bfloat16)
    q = torch.randn(1, w, 4, d, generator=g).to(torch.bfloat16)
    dev = torch.device("cuda:0")
    kvd = kv.to(dev)
    kd, vd, qd = kvd[:, 0], kvd[:, 1], q.to(dev)
    params = B.make_params(qd, kd, vd, w, 5, score_path=B.SLKV_PATH_SIMT)
    assert params.k_stride_tok == 2 * Hkv * d
    cu = [0, T]
    cap = B.slkv_packed_rows_upper_bound(params, cu)
    k_out = torch.zeros(cap, d, dtype=torch.bfloat16, device=dev); v_out = torch.zeros_like(k_out)
    offsets = torch.zeros(Hkv + 1, dtype=torch.int32, device=dev)
    kept = torch.zeros(cap, dtype=torch.int32, device=dev)
    bud = torch.tensor([100, 40], dtype=torch.int32, device=dev)
    ws = B.new_workspace(params, cu, dev)
    B.slkv_compress(params, qd, kd, vd, torch.tensor(cu, dtype=torch.int32, device=dev), cu, bud, k_out, v_out,
                    offsets, kept, ws)
    torch.cuda.synchronize()
    ref = P.gpu_compress(q, kv[:, 0].contiguous(), kv[:, 1].contiguous(), cu, [100, 40], w, 5,
                         score_path=B.SLKV_PATH_SIMT)
    assert np.array_equal(kept.cpu().numpy()[:140], ref["kept_idx"][:140])
    assert torch.equal(k_out.cpu()[:140], ref["k_out"][:140]) and torch.equal(v_out.cpu()[:140], ref["v_out"][:140])


def test_host_buffer_entry_point():
    wl = synth.small_variant(synth.workloads()[1], [1200, 500])
    x = synth.layer_inputs(wl, 0)
    cu = wl.cu_seqlens
    bud = [100, 64, 300, 2000, 70, 90, 128, 65]
    ref = P.gpu_compress(x.q_win, x.k, x.v, cu, bud, wl.window, wl.pool_kernel)
    dev = torch.device("cuda:0")
    params = B.make_params(x.q_win, x.k, x.v, wl.window, wl.pool_kernel)
    rows_expect = int(ref["offsets"][-1])
    cap = rows_expect + 3
    arena = torch.empty(B.slkv_compress_host_arena_bytes(params, cu, cap), dtype=torch.uint8, device=dev)
    pin = lambda t: t.pin_memory()
    k_out = pin(torch.zeros(cap, 128, dtype=torch.bfloat16)); v_out = pin(torch.zeros(cap, 128, dtype=torch.bfloat16))
    offsets = pin(torch.zeros(len(bud) * 2 + 1, dtype=torch.int32)); kept = pin(torch.zeros(cap, dtype=torch.int32))
    rows = B.slkv_compress_host(params, pin(x.q_win), pin(x.k), pin(x.v), cu, torch.tensor(bud, dtype=torch.int32),
                                k_out, v_out, offsets, kept, arena)
    assert rows == rows_expect
    assert np.array_equal(offsets.numpy().astype(np.int64), ref["offsets"])
    assert np.array_equal(kept.numpy()[:rows].astype(np.int64), ref["kept_idx"][:rows])
    assert torch.equal(k_out[:rows], ref["k_out"][:rows]) and torch.equal(v_out[:rows], ref["v_out"][:rows])
    with pytest.raises(B.SlkvError) as e:
        B.slkv_compress_host(params, x.q_win, x.k, x.v, cu, torch.tensor(bud, dtype=torch.int32),
                             k_out[:10], v_out[:10], offsets, kept[:10], arena)
    assert e.value.code == B.ERR["CAPACITY"]


def test_overlapped_calls_match_ordinary_calls():
    # four layers back to back through one workspace, then a join: bit-identical to one call at a time
    wl = synth.small_variant(synth.workloads()[2], [9000], n_layers=4, totals=[4 * 8 * 300])
    dev = torch.device("cuda:0")
    budgets = O.alloc_budgets(synth.inf_sc(wl).numpy(), wl.fixed, wl.totals[0])
    xs = [synth.layer_inputs(wl, l, device=dev) for l in range(4)]
    cu = wl.cu_seqlens
    cu_dev = torch.tensor(cu, dtype=torch.int32, device=dev)
    params = B.make_params(xs[0].q_win, xs[0].k, xs[0].v, wl.window, wl.pool_kernel)
    ws = torch.empty(B.slkv_workspace_bytes_overlapped(params, cu), dtype=torch.uint8, device=dev)
    assert ws.numel() > B.slkv_workspace_bytes(params, cu)
    cap = B.slkv_packed_rows_upper_bound(params, cu)
    # inputs of a call in flight must stay put: the budget rows live as long as the test
    buds = [torch.tensor(budgets[l].tolist(), dtype=torch.int32, device=dev) for l in range(4)]

    def outputs():
        return [dict(k_out=torch.zeros(cap, 128, dtype=torch.bfloat16, device=dev),
                     v_out=torch.zeros(cap, 128, dtype=torch.bfloat16, device=dev),
                     offsets=torch.zeros(9, dtype=torch.int32, device=dev),
                     kept=torch.full((cap,), -1, dtype=torch.int32, device=dev),
                     status=torch.zeros(1, dtype=torch.int32, device=dev)) for _ in range(4)]

    def run(fn, outs):
        for rep in range(3):                   # several rounds: both vote arrays get reused while in flight
            for l in range(4):
                o = outs[l]
                fn(params, xs[l].q_win, xs[l].k, xs[l].v, cu_dev, cu, buds[l], o["k_out"], o["v_out"],
                   o["offsets"], o["kept"], ws, None, o["status"])
        B.slkv_join()
        torch.cuda.synchronize()

    a, b = outputs(), outputs()
    run(B.slkv_compress, a)
    run(B.slkv_compress_overlapped, b)
    for l in range(4):
        assert int(b[l]["status"].item()) == 0
        n = int(a[l]["offsets"][-1].item())
        assert torch.equal(a[l]["offsets"], b[l]["offsets"]) and n == int(budgets[l].sum())
        assert torch.equal(a[l]["kept"][:n], b[l]["kept"][:n])
        assert torch.equal(a[l]["k_out"][:n], b[l]["k_out"][:n]) and torch.equal(a[l]["v_out"][:n], b[l]["v_out"][:n])
    # an ordinary call right after overlapped ones joins by itself
    o = outputs()[0]
    B.slkv_compress_overlapped(params, xs[0].q_win, xs[0].k, xs[0].v, cu_dev, cu, buds[0], b[0]["k_out"],
                               b[0]["v_out"], b[0]["offsets"], b[0]["kept"], ws, None, b[0]["status"])
    B.slkv_compress(params, xs[1].q_win, xs[1].k, xs[1].v, cu_dev, cu, buds[1], o["k_out"], o["v_out"],
                    o["offsets"], o["kept"], ws, None, o["status"])
    torch.cuda.synchronize()
    n = int(a[1]["offsets"][-1].item())
    assert torch.equal(o["kept"][:n], a[1]["kept"][:n]) and torch.equal(b[0]["kept"][:int(a[0]["offsets"][-1])], a[0]["kept"][:int(a[0]["offsets"][-1])])


def test_overlapped_calls_of_changing_shapes_and_streams():
    # layers of two different shapes through one workspace, queued in lists by the overlapped entry point: a change
    # of shape drains what is in flight before the workspace is carved up anew; results equal one call at a time
    dev = torch.device("cuda:0")
    base = synth.workloads()[2]
    shapes = [synth.small_variant(base, [5000], n_layers=3, totals=[3 * 8 * 200]),
              synth.small_variant(base, [2100, 900], n_layers=3, totals=[3 * 8 * 300])]
    cases = []
    for wl in shapes:
        budgets = O.alloc_budgets(synth.inf_sc(wl).numpy(), wl.fixed, wl.totals[0])
        for l in range(3):
            x = synth.layer_inputs(wl, l, device=dev)
            cases.append((wl, x, torch.tensor(budgets[l].tolist(), dtype=torch.int32, device=dev)))
    ws_bytes = 0
    prepared = []
    for wl, x, bud in cases:
        params = B.make_params(x.q_win, x.k, x.v, wl.window, wl.pool_kernel)
        cu = wl.cu_seqlens
        ws_bytes = max(ws_bytes, B.slkv_workspace_bytes_overlapped(params, cu))
        cap = B.slkv_packed_rows_upper_bound(params, cu)
        n_seg = (len(cu) - 1) * wl.n_kv_heads
        prepared.append((params, x, cu, torch.tensor(cu, dtype=torch.int32, device=dev), bud, cap, n_seg))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)

    def outputs():
        return [dict(k=torch.zeros(cap, 128, dtype=torch.bfloat16, device=dev), v=torch.zeros(cap, 128, dtype=torch.bfloat16, device=dev),
                     off=torch.zeros(n_seg + 1, dtype=torch.int32, device=dev), kept=torch.full((cap,), -1, dtype=torch.int32, device=dev),
                     status=torch.zeros(1, dtype=torch.int32, device=dev)) for (_, _, _, _, _, cap, n_seg) in prepared]

    side = torch.cuda.Stream()

    def run(fn, outs, order, streams):
        torch.cuda.synchronize()
        for n, i in enumerate(order):
            params, x, cu, cu_dev, bud, cap, n_seg = prepared[i]
            o = outs[i]
            fn(params, x.q_win, x.k, x.v, cu_dev, cu, bud, o["k"], o["v"], o["off"], o["kept"], ws, None, o["status"],
               streams[n % len(streams)])
        B.slkv_join()
        torch.cuda.synchronize()

    order = [0, 1, 3, 4, 2, 5, 0, 3]                  # shapes alternate in runs of different lengths
    a, b, c = outputs(), outputs(), outputs()
    run(B.slkv_compress, a, order, [None])
    run(B.slkv_compress_overlapped, b, order, [None])
    run(B.slkv_compress_overlapped, c, order, [None, None, side])     # every third call on another stream
    for i in range(len(prepared)):
        n = int(a[i]["off"][-1].item())
        assert int(c[i]["status"].item()) == 0 and torch.equal(a[i]["kept"][:n], c[i]["kept"][:n])
        assert torch.equal(a[i]["k"][:n], c[i]["k"][:n]) and torch.equal(a[i]["v"][:n], c[i]["v"][:n])
    for i in range(len(prepared)):
        assert int(b[i]["status"].item()) == 0
        n = int(a[i]["off"][-1].item())
        assert torch.equal(a[i]["off"], b[i]["off"]) and torch.equal(a[i]["kept"][:n], b[i]["kept"][:n])
        assert torch.equal(a[i]["k"][:n], b[i]["k"][:n]) and torch.equal(a[i]["v"][:n], b[i]["v"][:n])


def test_overlapped_calls_without_cooperative_launches():
    # where the device refuses cooperative launches the score kernel takes one layer's pass 1 per launch (beside
    # pass 2 of the layer before); SLKV_NO_COOPERATIVE=1 makes the library behave that way.  The switch is read
    # once per process, hence the child process.
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, SLKV_NO_COOPERATIVE="1")
    r = subprocess.run([sys.executable, "-m", "pytest", "-q", "-m", "gpu", "-x",
                        "tests/test_gpu_compress.py::test_overlapped_calls_match_ordinary_calls",
                        "tests/test_gpu_compress.py::test_overlapped_calls_of_changing_shapes_and_streams"],
                       cwd=root, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]
