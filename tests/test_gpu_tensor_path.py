"""GPU parity of the tensor-core (tcgen05 + TMA) score kernels against the oracle and the FMA kernels."""
import numpy as np
import pytest
import torch

import parity as P
from paper_2508_15806_b200 import binding as B
from paper_2508_15806_b200 import synth

pytestmark = pytest.mark.gpu


def rand_case(Hq, Hkv, w, lens, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    T = sum(lens)
    q = (torch.randn(len(lens), w, Hq, 128, generator=g) * scale).to(torch.bfloat16)
    k = (torch.randn(T, Hkv, 128, generator=g) * scale).to(torch.bfloat16)
    v = torch.randn(T, Hkv, 128, generator=g).to(torch.bfloat16)
    return q, k, v, [0] + list(np.cumsum(lens))


@pytest.mark.parametrize("Hq,Hkv,w,lens", [
    (4, 1, 32, [700]),                       # R = 128: one M tile, ragged last key tile
    (8, 2, 32, [128 + 32, 129 + 32, 31, 1000]),   # exact tile, one key over, shorter than the window
    (8, 2, 64, [900, 333]),                  # R = 256: two M tiles, two TMEM buffers
    (4, 1, 16, [515]),                       # R = 64: padded M tile
    (2, 2, 32, [260]),                       # R = 32, MHA
    (12, 2, 32, [2000]),                     # R = 192
    (32, 8, 32, [5000, 4100]),               # many segments per CTA boundary
])
def test_tensor_path_matches_oracle(Hq, Hkv, w, lens):
    q, k, v, cu = rand_case(Hq, Hkv, w, lens, seed=Hq * 7 + w)
    bud = [w + 11 + 53 * h for h in range(Hkv)]
    gpu, stats = P.check_compress(q, k, v, cu, bud, w, 7, score_path=B.SLKV_PATH_TENSOR)
    assert stats["pooled_max_rel_err"] < 1e-3


def test_tensor_and_fma_paths_agree_closely():
    q, k, v, cu = rand_case(8, 2, 32, [3000], seed=3, scale=1.3)
    a = P.gpu_score(q, k, cu, 32, 1, score_path=B.SLKV_PATH_TENSOR)
    b = P.gpu_score(q, k, cu, 32, 1, score_path=B.SLKV_PATH_SIMT)
    assert np.max(np.abs(a - b) / (np.abs(b) + 1e-30)) < 2e-4


def test_large_logits_and_needles():
    # planted keys 30+ logits above the bulk: the running maximum must move and rescale correctly
    wl = synth.small_variant(synth.workloads()[1], [4000])
    wl.needle_logit = 40.0
    x = synth.layer_inputs(wl, 0)
    bud = [64, 100, 200, 400, 800, 1600, 3200, 4000]
    P.check_compress(x.q_win, x.k, x.v, wl.cu_seqlens, bud, wl.window, wl.pool_kernel, score_path=B.SLKV_PATH_TENSOR)


def test_strided_views_on_tensor_path():
    # K as a slice of a fused [T, 2, Hkv, d] buffer and Q stored head-major [B, Hq, w, d]
    g = torch.Generator().manual_seed(11)
    T, Hkv, Hq, w = 1500, 2, 8, 32
    kv = torch.randn(T, 2, Hkv, 128, generator=g).to(torch.bfloat16)
    q_hm = torch.randn(1, Hq, w, 128, generator=g).to(torch.bfloat16)
    dev = torch.device("cuda:0")
    kvd, qd = kv.to(dev), q_hm.to(dev).permute(0, 2, 1, 3)          # logical [B, w, Hq, d], head stride > row stride
    kd = kvd[:, 0]
    params = B.make_params(qd, kd, None, w, 7, score_path=B.SLKV_PATH_TENSOR)
    assert params.q_stride_head > params.q_stride_row and params.k_stride_tok == 2 * Hkv * 128
    cu = [0, T]
    ws = B.new_workspace(params, cu, dev)
    n = B.slkv_pooled_elems(params, cu)
    pooled = torch.zeros(n, dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    B.slkv_score(params, qd, kd, torch.tensor(cu, dtype=torch.int32, device=dev), cu, pooled, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = P.oracle_pooled(q_hm.permute(0, 2, 1, 3).contiguous(), kv[:, 0].contiguous(), cu, w, 7)
    P.assert_pooled_close(pooled.cpu().numpy(), ref, cu, Hkv, w)


def overlapped_result(q, k, v, cu, bud, w, p, repeats=2):
    """The layer `repeats` times through slkv_compress_overlapped + slkv_join; host results of the last call."""
    dev = torch.device("cuda:0")
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    cu = [int(x) for x in cu]
    params = B.make_params(qd, kd, vd, w, p, B.SLKV_POOL_MAX, B.SLKV_PATH_TENSOR)
    cap = B.slkv_packed_rows_upper_bound(params, cu)
    n_seg = (len(cu) - 1) * k.shape[1]
    cu_dev = torch.tensor(cu, dtype=torch.int32, device=dev)
    budd = torch.tensor(list(bud), dtype=torch.int32, device=dev)
    ws = torch.empty(B.slkv_workspace_bytes_overlapped(params, cu), dtype=torch.uint8, device=dev)
    n_pool = B.slkv_pooled_elems(params, cu)
    outs = []
    for _ in range(repeats):
        o = dict(k_out=torch.zeros(cap, 128, dtype=k.dtype, device=dev), v_out=torch.zeros(cap, 128, dtype=k.dtype, device=dev),
                 offsets=torch.full((n_seg + 1,), -1, dtype=torch.int32, device=dev),
                 kept=torch.full((cap,), -1, dtype=torch.int32, device=dev),
                 pooled=torch.full((n_pool,), float("nan"), dtype=torch.float32, device=dev),
                 status=torch.zeros(1, dtype=torch.int32, device=dev))
        B.slkv_compress_overlapped(params, qd, kd, vd, cu_dev, cu, budd, o["k_out"], o["v_out"], o["offsets"], o["kept"], ws,
                                   o["pooled"], o["status"])
        outs.append(o)
    B.slkv_join()
    torch.cuda.synchronize()
    o = outs[-1]
    assert int(o["status"].item()) == 0
    return {"offsets": o["offsets"].cpu().numpy().astype(np.int64), "kept_idx": o["kept"].cpu().numpy().astype(np.int64),
            "k_out": o["k_out"].cpu(), "v_out": o["v_out"].cpu(), "pooled": o["pooled"].cpu().numpy()}


@pytest.mark.parametrize("kind", ["overflow", "underflow"])
def test_extreme_logits_on_both_entry_points(kind):
    # overflow: a few keys 120 logits above the bulk (2^x overflows fp32 under a fixed reference of 0);
    # underflow: every logit of every row near -150 (every 2^x underflows under that reference).
    # Both must leave the fixed-reference fast path for the exact one, in the single-layer kernel (slkv_compress)
    # and in the two-stream kernel (slkv_compress_overlapped).
    q, k, v, cu = rand_case(8, 2, 16, [1500, 700], seed=21)
    qf, kf = q.float(), k.float()
    qf[..., 0] += 41.0
    if kind == "underflow":
        kf[..., 0] -= 41.0                       # adds -41 * 41 / sqrt(128) = -148.6 to every logit
    else:
        for t in (5, 333, 1499, 1500 + 77):
            kf[t, :, 0] += 33.0                  # +119.6 on these keys
    q, k = qf.to(torch.bfloat16), kf.to(torch.bfloat16)
    bud = [200, 64]
    w, p = 16, 5
    ref = P.oracle_pooled(q, k, cu, w, p)
    ordinary = P.gpu_compress(q, k, v, cu, bud, w, p, score_path=B.SLKV_PATH_TENSOR)
    assert ordinary["status"] == 0
    overlapped = overlapped_result(q, k, v, cu, bud, w, p)
    for gpu in (ordinary, overlapped):
        P.assert_pooled_close(gpu["pooled"], ref, cu, k.shape[1], w)
        if kind == "underflow":
            P.assert_selection_valid(gpu, ref, cu, bud, w, k, v)
        else:
            # next to keys 120 logits up every other probability is below fp32's range (exp(-120)), so the order of
            # the rest cannot be compared; the planted keys and their pooling neighbourhoods must be kept
            for h in range(2):
                a, b = gpu["offsets"][h], gpu["offsets"][h + 1]
                kept = set(gpu["kept_idx"][a:b].tolist())
                assert {3, 4, 5, 6, 7, 331, 332, 333, 334, 335} <= kept


@pytest.mark.parametrize("lens", [
    [5, 16, 9],                                  # no sequence longer than the window: nothing to score
    [40 + 3 * i for i in range(70)],             # more sequences than the per-sequence tables in kernel parameters hold
    [16 + 128 * 4, 17, 16 + 128],                # histories of whole key tiles beside a one-key history
])
def test_overlapped_entry_point_on_degenerate_batches(lens):
    w, p = 16, 3
    q, k, v, cu = rand_case(8, 2, w, lens, seed=len(lens))
    bud = [w + 9, 3 * w]
    ordinary = P.gpu_compress(q, k, v, cu, bud, w, p, score_path=B.SLKV_PATH_TENSOR)
    assert ordinary["status"] == 0
    ref = P.oracle_pooled(q, k, cu, w, p)
    P.assert_selection_valid(ordinary, ref, cu, bud, w, k, v)
    overlapped = overlapped_result(q, k, v, cu, bud, w, p, repeats=3)
    n = int(ordinary["offsets"][-1])
    assert np.array_equal(overlapped["offsets"], ordinary["offsets"])
    assert np.array_equal(overlapped["kept_idx"][:n], ordinary["kept_idx"][:n])
    assert torch.equal(overlapped["k_out"][:n], ordinary["k_out"][:n]) and torch.equal(overlapped["v_out"][:n], ordinary["v_out"][:n])
