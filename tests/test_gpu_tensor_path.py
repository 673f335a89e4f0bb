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
