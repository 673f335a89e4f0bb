"""No-GPU checks of the C-ABI library: it loads, exports every declared symbol, validates arguments on the host."""
import ctypes as C
import os
import re

import pytest

from paper_2508_15806_b200 import binding as B
from paper_2508_15806_b200 import build as builder

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    builder.build()
    return B.lib()


def declared_functions():
    src = open(os.path.join(ROOT, "include", "slkv.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(slkv_[a-z_0-9]+)\s*\(", src)))


def test_exports_every_declared_symbol(L):
    names = declared_functions()
    assert {"slkv_alloc_budgets", "slkv_score", "slkv_compress", "slkv_compress_host"} <= set(names)
    for n in names:
        assert hasattr(L, n), f"libslkv.so does not export {n}"
    assert L.slkv_version() >= 100
    assert B.lib().slkv_strerror(0) == b"SLKV_OK" and b"CAPACITY" in L.slkv_strerror(-7)


def params(**kw):
    d = dict(n_seqs=1, n_q_heads=8, n_kv_heads=2, head_dim=128, window=16, pool_kernel=5, dtype=B.SLKV_BF16,
             pool_mode=B.SLKV_POOL_MAX, softmax_domain=B.SLKV_HISTORY, score_path=B.SLKV_PATH_AUTO,
             lse_units=B.SLKV_LSE_LN, history_only=0,
             k_stride_tok=256, k_stride_head=128, v_stride_tok=256, v_stride_head=128,
             q_stride_seq=16 * 8 * 128, q_stride_row=8 * 128, q_stride_head=128)
    d.update(kw)
    return B.SlkvParams(**d)


def test_size_queries(L):
    p = params(n_seqs=3)
    cu = [0, 100, 110, 400]
    assert B.slkv_pooled_elems(p, cu) == 2 * (84 + 0 + 274)
    assert B.slkv_packed_rows_upper_bound(p, cu) == 2 * 400
    assert B.slkv_workspace_bytes(p, cu) > 2 * 2 * 358 * 4
    assert B.slkv_compress_host_arena_bytes(p, cu, 800) > B.slkv_workspace_bytes(p, cu)


@pytest.mark.parametrize("kw", [dict(head_dim=96), dict(n_q_heads=7), dict(window=0), dict(pool_kernel=4),
                                dict(n_seqs=0), dict(k_stride_head=64), dict(window=1000)])
def test_bad_shapes_rejected(L, kw):
    p = params(**kw)
    assert B.slkv_workspace_bytes(p, [0, 100]) == 0
    assert B.slkv_pooled_elems(p, [0, 100]) == -1


def test_bad_enums_and_alignment(L):
    cu = (C.c_int32 * 2)(0, 100)
    fake = C.c_void_p(4096)          # never dereferenced: validation fails first
    for kw, code in [(dict(dtype=7), "BAD_DTYPE"), (dict(pool_mode=3), "BAD_DTYPE"),
                     (dict(softmax_domain=2), "BAD_DTYPE"), (dict(score_path=9), "BAD_DTYPE"),
                     (dict(lse_units=2), "BAD_DTYPE"), (dict(history_only=2), "BAD_DTYPE"),
                     (dict(k_stride_tok=257), "BAD_ALIGN")]:
        p = params(**kw)
        rc = L.slkv_score(C.byref(p), fake, fake, fake, cu, None, fake, None, fake, 1 << 30, None)
        assert rc == B.ERR[code], (kw, rc)
    p = params()
    assert L.slkv_score(C.byref(p), None, fake, fake, cu, None, fake, None, fake, 1 << 30, None) == B.ERR["NULL_PTR"]
    assert L.slkv_score(C.byref(p), fake, fake, fake, cu, None, fake, None, None, 0, None) == B.ERR["WORKSPACE"]
    assert L.slkv_score(C.byref(p), fake, fake, fake, cu, None, fake, None, fake, 16, None) == B.ERR["WORKSPACE"]
    assert L.slkv_score(C.byref(p), C.c_void_p(4100), fake, fake, cu, None, fake, None, fake, 1 << 30, None) == B.ERR["BAD_ALIGN"]
    bad_cu = (C.c_int32 * 2)(0, -5)
    assert L.slkv_score(C.byref(p), fake, fake, fake, bad_cu, None, fake, None, fake, 1 << 30, None) == B.ERR["BAD_SHAPE"]


def test_alloc_argument_errors(L):
    fake = C.c_void_p(4096)
    f = L.slkv_alloc_budgets
    assert f(None, 1, 8, 32, 1024, fake, None, None) == B.ERR["NULL_PTR"]
    assert f(fake, 1, 8, 32, 255, fake, None, None) == B.ERR["BUDGET_SUM"]
    assert f(fake, 1, 8, -1, 255, fake, None, None) == B.ERR["BUDGET_SUM"]
    assert f(fake, 0, 8, 1, 255, fake, None, None) == B.ERR["BAD_SHAPE"]
    assert f(fake, 2048, 32, 0, 255, fake, None, None) == B.ERR["BAD_SHAPE"]


def test_alloc_ex_argument_errors(L):
    fake = C.c_void_p(4096)
    f = L.slkv_alloc_budgets_ex
    opt = B.SlkvAllocOptions(head_normaliser=0, rounding=0, cap=0)
    assert f(None, 1, 8, 32, 1024, C.byref(opt), fake, None, None) == B.ERR["NULL_PTR"]
    assert f(fake, 1, 8, 32, 255, None, fake, None, None) == B.ERR["BUDGET_SUM"]
    for kw, code in [(dict(head_normaliser=2), "BAD_DTYPE"), (dict(rounding=5), "BAD_DTYPE"), (dict(cap=-1), "BAD_SHAPE"),
                     (dict(cap=31), "BUDGET_SUM"), (dict(cap=100), "BUDGET_SUM")]:
        o = B.SlkvAllocOptions(head_normaliser=0, rounding=0, cap=0)
        for k, v in kw.items():
            setattr(o, k, v)
        assert f(fake, 1, 8, 32, 1024, C.byref(o), fake, None, None) == B.ERR[code], kw
    # Algorithm 2's own rounding does not meet a total, so a cap that the total does not fit under is accepted
    # (the launch itself needs a device, so only the rejections are checked here)


def test_compress_argument_errors(L):
    fake = C.c_void_p(4096)
    cu = (C.c_int32 * 2)(0, 100)
    p = params()
    args = [C.byref(p), fake, fake, fake, fake, cu, fake, None, fake, fake, 10, fake, fake, None, None, fake, 1 << 30,
            None]
    bad = list(args); bad[6] = None
    assert L.slkv_compress(*bad) == B.ERR["NULL_PTR"]
    bad = list(args); bad[10] = -1
    assert L.slkv_compress(*bad) == B.ERR["CAPACITY"]
    pt = params(score_path=B.SLKV_PATH_TENSOR, dtype=B.SLKV_F32, k_stride_tok=256, head_dim=64, k_stride_head=64,
                v_stride_head=64, q_stride_head=64)
    bad = list(args); bad[0] = C.byref(pt)
    assert L.slkv_compress(*bad) == B.ERR["BAD_DTYPE"]      # the tensor path takes bf16 only


def test_history_only_and_context_parallel_argument_errors(L):
    fake = C.c_void_p(4096)
    cu = (C.c_int32 * 2)(0, 100)
    ph = params(history_only=1)
    assert B.slkv_pooled_elems(ph, [0, 100]) == 2 * 100          # every row given is a history row
    assert B.slkv_pooled_elems(params(), [0, 100]) == 2 * 84
    assert B.slkv_workspace_bytes(params(history_only=1, n_seqs=2), [0, 50, 100]) == 0      # one sequence only
    args = [C.byref(ph), fake, fake, fake, fake, cu, fake, None, fake, fake, 10, fake, fake, None, None, fake, 1 << 30,
            None]
    assert L.slkv_compress(*args) == B.ERR["BAD_SHAPE"]          # nothing to append behind the selected rows
    assert L.slkv_compress_overlapped(*args) == B.ERR["BAD_SHAPE"]
    p = params()
    assert L.slkv_cp_merge_lse(C.byref(p), None, 2, fake, None) == B.ERR["NULL_PTR"]
    assert L.slkv_cp_merge_lse(C.byref(p), fake, 0, fake, None) == B.ERR["BAD_SHAPE"]
    assert L.slkv_cp_select_init(fake, 0, 16, 100, fake, fake, None) == B.ERR["BAD_SHAPE"]
    assert L.slkv_cp_select_init(fake, 2, 16, 1 << 31, fake, fake, None) == B.ERR["BAD_SHAPE"]
    assert L.slkv_cp_histogram(fake, 2, 100, 90, 20, 0, fake, fake, None) == B.ERR["BAD_SHAPE"]      # past the row
    assert L.slkv_cp_histogram(fake, 2, 100, 0, 20, 3, fake, fake, None) == B.ERR["BAD_SHAPE"]
    assert L.slkv_cp_descend(fake, 2, -1, fake, fake, None) == B.ERR["BAD_SHAPE"]
    assert L.slkv_cp_local_ties(fake, None, 2, fake, None) == B.ERR["NULL_PTR"]
    assert L.slkv_cp_workspace_bytes(2, 500, 1000) >= 4000 and L.slkv_cp_workspace_bytes(0, 5, 10) == 0
    emit = [C.byref(p), fake, fake, 100, fake, 100, 0, 84, 0, fake, fake, fake, 2, 1, 16, 84, fake, fake, 200, fake, fake,
            None, fake, 1 << 20, None]
    bad = list(emit); bad[7] = 90                                 # owned rows run into the window rows
    assert L.slkv_cp_emit(*bad) == B.ERR["BAD_SHAPE"]
    bad = list(emit); bad[13] = 2                                 # part >= n_parts
    assert L.slkv_cp_emit(*bad) == B.ERR["BAD_SHAPE"]
    bad = list(emit); bad[18] = -1
    assert L.slkv_cp_emit(*bad) == B.ERR["CAPACITY"]
    bad = list(emit); bad[23] = 16
    assert L.slkv_cp_emit(*bad) == B.ERR["WORKSPACE"]
    bad = list(emit); bad[1] = None
    assert L.slkv_cp_emit(*bad) == B.ERR["NULL_PTR"]
