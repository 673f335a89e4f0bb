"""KV-head sharding shown on one GPU: a layer compressed as several calls, each on its own heads through strided
views, gives -- stitched with the host logic the multi-GPU path uses -- the packed cache of the whole-layer call
(Algorithm 3 runs per head; Sec. 3.4)."""
import numpy as np
import pytest
import torch

import parity as P
from paper_2508_15806_b200 import binding as B
from paper_2508_15806_b200 import sharding as S
from paper_2508_15806_b200 import synth

pytestmark = pytest.mark.gpu


def compress_views(qd, kd, vd, cu, bud, w, p):
    """slkv_compress on device views; returns device results."""
    dev = qd.device
    params = B.make_params(qd, kd, vd, w, p)
    cap = B.slkv_packed_rows_upper_bound(params, cu)
    n_seg = (len(cu) - 1) * kd.shape[1]
    out = dict(k=torch.zeros(cap, kd.shape[2], dtype=kd.dtype, device=dev), v=torch.zeros(cap, kd.shape[2], dtype=kd.dtype, device=dev),
               off=torch.full((n_seg + 1,), -1, dtype=torch.int32, device=dev), idx=torch.full((cap,), -1, dtype=torch.int32, device=dev),
               pooled=torch.full((max(B.slkv_pooled_elems(params, cu), 1),), float("nan"), dtype=torch.float32, device=dev),
               status=torch.zeros(1, dtype=torch.int32, device=dev))
    B.slkv_compress(params, qd, kd, vd, torch.tensor(cu, dtype=torch.int32, device=dev), cu, bud, out["k"], out["v"],
                    out["off"], out["idx"], B.new_workspace(params, cu, dev), out["pooled"], out["status"])
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    return out


@pytest.mark.parametrize("world,lens,fused_kv", [(2, [3000], False), (4, [1500, 40, 700], False), (3, [2100, 900], True)])
def test_head_sharded_calls_stitch_to_the_whole_layer(world, lens, fused_kv):
    wl = synth.small_variant(synth.workloads()[1], lens)          # 32 query / 8 KV heads, bf16, w 32, pool 7
    x = synth.layer_inputs(wl, 0)
    cu = [int(c) for c in wl.cu_seqlens]
    dev = torch.device("cuda:0")
    q, k, v = x.q_win.to(dev), x.k.to(dev), x.v.to(dev)
    if fused_kv:                                                  # K and V as slices of one [T, 2, Hkv, d] buffer
        kv = torch.stack([k, v], dim=1).contiguous()
        k, v = kv[:, 0], kv[:, 1]
    n_kv, n_seqs, w, p = k.shape[1], len(lens), wl.window, wl.pool_kernel
    bud = torch.tensor([40, 64, 100, 900, 33, 250, 5000, 512], dtype=torch.int32, device=dev)
    whole = compress_views(q, k, v, cu, bud, w, p)
    ref = P.oracle_pooled(x.q_win, x.k, cu, w, p)

    shards, kept = [], []
    for r in range(world):
        h0, h1 = S.head_range(n_kv, r, world)
        qs, ks, vs, bs = S.shard_inputs(q, k, v, bud, h0, h1)
        assert not ks.is_contiguous() or h1 - h0 == n_kv           # views, not copies
        o = compress_views(qs, ks, vs, cu, bs, w, p)
        shards.append((h0, h1, o))
        kept.append(S.local_kept(o["off"].cpu(), n_seqs, h1 - h0))
    offsets, bases = S.stitch(kept)
    # offsets are a function of budgets and lengths only: bit-exact
    assert offsets.tolist() == whole["off"].cpu().to(torch.int64).tolist()

    # every shard is valid against the oracle by the rules of every other parity test ...
    for h0, h1, o in shards:
        gpu = {"offsets": o["off"].cpu().numpy().astype(np.int64), "kept_idx": o["idx"].cpu().numpy().astype(np.int64),
               "k_out": o["k"].cpu(), "v_out": o["v"].cpu()}
        ref_s = [r_[h0:h1] for r_ in ref]
        n_pool = sum(r_.size for r_ in ref_s)
        P.assert_pooled_close(o["pooled"][:n_pool].cpu().numpy(), ref_s, cu, h1 - h0, w)
        P.assert_selection_valid(gpu, ref_s, cu, bud[h0:h1].tolist(), w, x.k[:, h0:h1], x.v[:, h0:h1])
    # ... and the stitched cache is the whole-layer call's, segment by segment (a head's result can differ from the
    # whole-layer call only inside the tolerance band of its k-th score, where the two calls merge the row statistics
    # of differently cut key ranges; on these inputs no segment does)
    whole_off = whole["off"].cpu().numpy()
    whole_idx, whole_k, whole_v = whole["idx"].cpu(), whole["k"].cpu(), whole["v"].cpu()
    for r, (h0, h1, o) in enumerate(shards):
        so, si, sk, sv = o["off"].cpu().numpy(), o["idx"].cpu(), o["k"].cpu(), o["v"].cpu()
        for s in range(n_seqs):
            for hl in range(h1 - h0):
                a, b = so[s * (h1 - h0) + hl], so[s * (h1 - h0) + hl + 1]
                g0 = int(bases[r][s, hl])
                assert g0 == whole_off[s * n_kv + h0 + hl]
                assert torch.equal(si[a:b], whole_idx[g0:g0 + (b - a)])
                assert torch.equal(sk[a:b], whole_k[g0:g0 + (b - a)]) and torch.equal(sv[a:b], whole_v[g0:g0 + (b - a)])
