"""slkv_score_noalloc: the score step for callers that have no way to allocate device scratch.

An application that has given all free GPU memory to its own pool (or a plug-in without access to the
host's allocator) cannot supply slkv_score's workspace; this entry point uses a fixed array inside the
library instead.  It must give what slkv_score gives, call after call, whatever the array held before.
This file sorts last on purpose: a run that stops at the first failure has then run every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2508_15806_b200 import binding as B
from paper_2508_15806_b200 import build as builder

import parity as P      # the parity rules of the other GPU tests: pooled scores within 1e-3 of the oracle


def _case(seed, lens, Hq=8, Hkv=2, w=32, dtype=torch.bfloat16, d=128):
    g = torch.Generator().manual_seed(seed)
    T = sum(lens)
    q = torch.randn(len(lens), w, Hq, d, generator=g).to(dtype)
    k = torch.randn(T, Hkv, d, generator=g).to(dtype)
    return q, k, [0] + list(np.cumsum(lens))


def _both(q, k, cu, w, p):
    dev = torch.device("cuda:0")
    qd, kd = q.to(dev), k.to(dev)
    params = B.make_params(qd, kd, None, w, p)
    cu = [int(x) for x in cu]
    cu_dev = torch.tensor(cu, dtype=torch.int32, device=dev)
    n = B.slkv_pooled_elems(params, cu)
    ref = torch.full((n,), float("nan"), dtype=torch.float32, device=dev)
    B.slkv_score(params, qd, kd, cu_dev, cu, ref, B.new_workspace(params, cu, dev))
    got = torch.full((n,), float("nan"), dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    B.slkv_score_noalloc(params, qd, kd, cu_dev, cu, got, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return got.cpu().numpy(), ref.cpu().numpy()


@pytest.mark.gpu
def test_matches_slkv_score_on_two_calls_in_a_row():
    # second call: other shapes and values, so whatever the first left in the shared scratch is stale
    for seed, lens, w, p in [(1, [3000, 700], 32, 7), (2, [513, 40, 2100], 32, 5)]:
        q, k, cu = _case(seed, lens, w=w)
        got, ref = _both(q, k, cu, w, p)
        assert np.all(np.isfinite(got))
        # the same kernels on the same inputs: the two entry points agree bit for bit ...
        assert np.array_equal(got.view(np.uint32), ref.view(np.uint32))
        # ... and with the oracle within the tolerance of every other parity test
        P.assert_pooled_close(got, P.oracle_pooled(q, k, cu, w, p), cu, k.shape[1], w)


@pytest.mark.gpu
def test_fp32_path_too():
    q, k, cu = _case(3, [900], Hq=4, Hkv=4, w=16, dtype=torch.float32, d=64)
    got, ref = _both(q, k, cu, 16, 5)
    assert np.array_equal(got.view(np.uint32), ref.view(np.uint32))
    P.assert_pooled_close(got, P.oracle_pooled(q, k, cu, 16, 5), cu, k.shape[1], 16)


def test_oversized_shapes_are_rejected_on_the_host():
    # decided before any CUDA call, so this runs without a GPU
    builder.build()
    L = B.lib()
    assert B.slkv_noalloc_scratch_bytes() == 8 << 20
    p = B.SlkvParams(n_seqs=1, n_q_heads=32, n_kv_heads=8, head_dim=128, window=32, pool_kernel=7, dtype=B.SLKV_BF16,
                     pool_mode=B.SLKV_POOL_MAX, softmax_domain=B.SLKV_HISTORY, score_path=B.SLKV_PATH_AUTO,
                     lse_units=B.SLKV_LSE_LN, history_only=0, k_stride_tok=1024, k_stride_head=128, v_stride_tok=1024, v_stride_head=128,
                     q_stride_seq=32 * 32 * 128, q_stride_row=32 * 128, q_stride_head=128)
    cu = (C.c_int32 * 2)(0, 131072)
    assert B.slkv_workspace_bytes(p, [0, 131072]) > B.slkv_noalloc_scratch_bytes()
    fake = C.c_void_p(4096)
    assert L.slkv_score_noalloc(C.byref(p), fake, fake, fake, cu, None, fake, None, None) == B.ERR["WORKSPACE"]
    # argument errors keep the codes slkv_score gives them, and come first
    assert L.slkv_score_noalloc(C.byref(p), None, fake, fake, cu, None, fake, None, None) == B.ERR["NULL_PTR"]
    p.head_dim = 96
    assert L.slkv_score_noalloc(C.byref(p), fake, fake, fake, cu, None, fake, None, None) == B.ERR["BAD_SHAPE"]
