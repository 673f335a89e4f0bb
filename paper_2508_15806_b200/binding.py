"""ctypes binding of libslkv.so: the same entry points as include/slkv.h, argument marshalling only.

Tensors are torch tensors (device memory and streams come from torch); every step of the method runs in
the library's kernels.  There is no fallback: if the shared library is missing, lib() raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libslkv.so")

SLKV_OK = 0
ERR = {"NULL_PTR": -1, "BAD_SHAPE": -2, "BAD_DTYPE": -3, "BAD_ALIGN": -4, "BUDGET_SUM": -5, "NEG_INF_SC": -6,
       "CAPACITY": -7, "WORKSPACE": -8, "CUDA": -9, "DEVICE_TIMEOUT": -10}
SLKV_F32, SLKV_BF16 = 0, 1
SLKV_POOL_MAX, SLKV_POOL_AVG = 0, 1
SLKV_HISTORY, SLKV_ALL_CAUSAL = 0, 1
SLKV_LSE_LN, SLKV_LSE_LOG2 = 0, 1
SLKV_PATH_AUTO, SLKV_PATH_SIMT, SLKV_PATH_TENSOR = 0, 1, 2


class SlkvParams(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_seqs", "n_q_heads", "n_kv_heads", "head_dim", "window", "pool_kernel",
                                         "dtype", "pool_mode", "softmax_domain", "score_path", "lse_units",
                                         "history_only")] + \
               [(n, C.c_int64) for n in ("k_stride_tok", "k_stride_head", "v_stride_tok", "v_stride_head",
                                         "q_stride_seq", "q_stride_row", "q_stride_head")]


class SlkvAllocOptions(C.Structure):
    _fields_ = [("head_normaliser", C.c_int32), ("rounding", C.c_int32), ("cap", C.c_int64)]


SLKV_NORM_GLOBAL, SLKV_NORM_WITHIN_LAYER = 0, 1
SLKV_ROUND_SUM_EXACT, SLKV_ROUND_PAPER = 0, 1


class SlkvError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().slkv_strerror(code).decode()
        if code == ERR["CUDA"]:
            msg += f" (cudaError {lib().slkv_last_cuda_error()})"
        super().__init__(f"{where}: {msg}")


_lib = None


def lib() -> C.CDLL:
    """The loaded shared library (loads it on first use; raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2508_15806_b200.build` "
                               "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        vp, i32p, i64, i32, sz = C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_size_t
        pp = C.POINTER(SlkvParams)
        L.slkv_strerror.restype = C.c_char_p
        L.slkv_strerror.argtypes = [C.c_int]
        L.slkv_last_cuda_error.restype = C.c_int
        L.slkv_last_launch_count.restype = C.c_int
        L.slkv_version.restype = C.c_int
        L.slkv_alloc_budgets.restype = C.c_int
        L.slkv_alloc_budgets.argtypes = [vp, i32, i32, i32, i64, vp, vp, vp]
        L.slkv_alloc_budgets_ex.restype = C.c_int
        L.slkv_alloc_budgets_ex.argtypes = [vp, i32, i32, i32, i64, C.POINTER(SlkvAllocOptions), vp, vp, vp]
        L.slkv_behavior_scores.restype = C.c_int
        L.slkv_behavior_scores.argtypes = [vp, i64, i32, i64, vp, i32, i64, vp, i32, i64, vp, vp, vp, vp]
        L.slkv_workspace_bytes.restype = sz
        L.slkv_workspace_bytes.argtypes = [pp, i32p]
        L.slkv_pooled_elems.restype = i64
        L.slkv_pooled_elems.argtypes = [pp, i32p]
        L.slkv_packed_rows_upper_bound.restype = i64
        L.slkv_packed_rows_upper_bound.argtypes = [pp, i32p]
        L.slkv_score.restype = C.c_int
        L.slkv_score.argtypes = [pp, vp, vp, vp, i32p, vp, vp, vp, vp, sz, vp]
        L.slkv_row_lse.restype = C.c_int
        L.slkv_row_lse.argtypes = [pp, vp, vp, vp, i32p, vp, vp, vp, sz, vp]
        L.slkv_debug_expire_next_wait.restype = C.c_int
        L.slkv_debug_expire_next_wait.argtypes = [C.c_int]
        L.slkv_compress.restype = C.c_int
        L.slkv_compress.argtypes = [pp, vp, vp, vp, vp, i32p, vp, vp, vp, vp, i64, vp, vp, vp, vp, vp, sz, vp]
        L.slkv_compress_overlapped.restype = C.c_int
        L.slkv_compress_overlapped.argtypes = L.slkv_compress.argtypes
        L.slkv_workspace_bytes_overlapped.restype = sz
        L.slkv_workspace_bytes_overlapped.argtypes = [pp, i32p]
        L.slkv_join.restype = C.c_int
        L.slkv_join.argtypes = [vp]
        L.slkv_compress_host_arena_bytes.restype = sz
        L.slkv_compress_host_arena_bytes.argtypes = [pp, i32p, i64]
        L.slkv_compress_host.restype = C.c_int
        L.slkv_compress_host.argtypes = [pp, vp, vp, vp, i32p, vp, vp, vp, i64, vp, vp, C.POINTER(C.c_int64),
                                         vp, sz, vp]
        L.slkv_score_noalloc.restype = C.c_int
        L.slkv_score_noalloc.argtypes = [pp, vp, vp, vp, i32p, vp, vp, vp, vp]
        L.slkv_noalloc_scratch_bytes.restype = sz
        L.slkv_noalloc_last_cuda_error.restype = C.c_int
        L.slkv_profile_enable.restype = C.c_int
        L.slkv_profile_enable.argtypes = [C.c_int]
        L.slkv_profile_collect.restype = C.c_int
        L.slkv_profile_collect.argtypes = [C.POINTER(C.c_float), C.POINTER(C.c_int32), C.c_int32]
        L.slkv_kernel_name.restype = C.c_char_p
        L.slkv_kernel_name.argtypes = [C.c_int]
        L.slkv_kernel_count.restype = C.c_int
        L.slkv_trace_set_buffer.restype = C.c_int
        L.slkv_trace_set_buffer.argtypes = [C.c_void_p, C.c_size_t]
        i32 = C.c_int32
        L.slkv_cp_merge_lse.restype = C.c_int
        L.slkv_cp_merge_lse.argtypes = [pp, vp, i32, vp, vp]
        L.slkv_cp_select_init.restype = C.c_int
        L.slkv_cp_select_init.argtypes = [vp, i32, i32, i64, vp, vp, vp]
        L.slkv_cp_histogram.restype = C.c_int
        L.slkv_cp_histogram.argtypes = [vp, i32, i64, i32, i32, i32, vp, vp, vp]
        L.slkv_cp_descend.restype = C.c_int
        L.slkv_cp_descend.argtypes = [vp, i32, i32, vp, vp, vp]
        L.slkv_cp_local_ties.restype = C.c_int
        L.slkv_cp_local_ties.argtypes = [vp, vp, i32, vp, vp]
        L.slkv_cp_workspace_bytes.restype = sz
        L.slkv_cp_workspace_bytes.argtypes = [i32, i32, i64]
        L.slkv_cp_emit.restype = C.c_int
        L.slkv_cp_emit.argtypes = [pp, vp, vp, i64, vp, i64, i32, i32, i64, vp, vp, vp, i32, i32, i32, i64, vp, vp, i64,
                                   vp, vp, vp, vp, sz, vp]
        _lib = L
    return _lib


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def _cu_host(cu_seqlens: Sequence[int]):
    arr = (C.c_int32 * len(cu_seqlens))(*[int(x) for x in cu_seqlens])
    return arr


def make_params(q_win: torch.Tensor, k: torch.Tensor, v: Optional[torch.Tensor], window: int, pool_kernel: int,
                pool_mode: int = SLKV_POOL_MAX, score_path: int = SLKV_PATH_AUTO,
                softmax_domain: int = SLKV_HISTORY, lse_units: int = SLKV_LSE_LN) -> SlkvParams:
    """Shapes and strides from the tensors: q_win [n_seqs, w, Hq, d], k / v [T, Hkv, d] (last dim contiguous)."""
    assert q_win.dim() == 4 and k.dim() == 3 and q_win.stride(3) == 1 and k.stride(2) == 1
    if v is None:
        v = k
    dt = {torch.float32: SLKV_F32, torch.bfloat16: SLKV_BF16}[k.dtype]
    assert q_win.dtype == k.dtype == v.dtype
    return SlkvParams(n_seqs=q_win.shape[0], n_q_heads=q_win.shape[2], n_kv_heads=k.shape[1], head_dim=k.shape[2],
                      window=window, pool_kernel=pool_kernel, dtype=dt, pool_mode=pool_mode,
                      softmax_domain=softmax_domain, score_path=score_path, lse_units=lse_units, history_only=0,
                      k_stride_tok=k.stride(0), k_stride_head=k.stride(1),
                      v_stride_tok=v.stride(0), v_stride_head=v.stride(1),
                      q_stride_seq=q_win.stride(0), q_stride_row=q_win.stride(1), q_stride_head=q_win.stride(2))


def slkv_version() -> int:
    return lib().slkv_version()


def slkv_last_launch_count() -> int:
    return lib().slkv_last_launch_count()


def slkv_alloc_budgets(inf_sc: torch.Tensor, fixed: int, total: int, budgets: Optional[torch.Tensor] = None,
                       status: Optional[torch.Tensor] = None, stream=None,
                       options: Optional[SlkvAllocOptions] = None) -> torch.Tensor:
    """inf_sc: CUDA float32 [n_layers, n_heads] -> CUDA int32 budgets of the same shape (slkv_alloc_budgets, or
    slkv_alloc_budgets_ex when `options` is given)."""
    assert inf_sc.is_cuda and inf_sc.dtype == torch.float32 and inf_sc.dim() == 2 and inf_sc.is_contiguous()
    if budgets is None:
        budgets = torch.empty(inf_sc.shape, dtype=torch.int32, device=inf_sc.device)
    if options is not None:
        rc = lib().slkv_alloc_budgets_ex(inf_sc.data_ptr(), inf_sc.shape[0], inf_sc.shape[1], int(fixed), int(total),
                                         C.byref(options), budgets.data_ptr(), _ptr(status), _stream(stream))
        if rc != SLKV_OK:
            raise SlkvError(rc, "slkv_alloc_budgets_ex")
        return budgets
    rc = lib().slkv_alloc_budgets(inf_sc.data_ptr(), inf_sc.shape[0], inf_sc.shape[1], int(fixed), int(total),
                                  budgets.data_ptr(), _ptr(status), _stream(stream))
    if rc != SLKV_OK:
        raise SlkvError(rc, "slkv_alloc_budgets")
    return budgets


def slkv_behavior_scores(attn: torch.Tensor, needle_idx: torch.Tensor, topk_idx: torch.Tensor, stream=None):
    """Algorithm 1 for a batch: attn CUDA float32 [n_rows, row_len]; needle_idx / topk_idx CUDA int32 [n_rows, n] or
    [n] (one list for all rows), entries < 0 are padding.  Returns (SF_sc, LG_sc, INF_sc), CUDA float32 [n_rows]."""
    assert attn.is_cuda and attn.dtype == torch.float32 and attn.dim() == 2 and attn.stride(1) == 1
    n_rows, row_len = attn.shape
    outs = [torch.empty(n_rows, dtype=torch.float32, device=attn.device) for _ in range(3)]

    def lst(t):
        assert t.is_cuda and t.dtype == torch.int32 and t.is_contiguous() and t.dim() in (1, 2)
        return t.data_ptr(), t.shape[-1], (t.shape[-1] if t.dim() == 2 else 0)
    (np_, nn, ns), (tp, tn, ts) = lst(needle_idx), lst(topk_idx)
    rc = lib().slkv_behavior_scores(attn.data_ptr(), n_rows, row_len, attn.stride(0), np_, nn, ns, tp, tn, ts,
                                    outs[0].data_ptr(), outs[1].data_ptr(), outs[2].data_ptr(), _stream(stream))
    if rc != SLKV_OK:
        raise SlkvError(rc, "slkv_behavior_scores")
    return tuple(outs)


def slkv_workspace_bytes(params: SlkvParams, cu_seqlens: Sequence[int]) -> int:
    return int(lib().slkv_workspace_bytes(C.byref(params), _cu_host(cu_seqlens)))


def slkv_pooled_elems(params: SlkvParams, cu_seqlens: Sequence[int]) -> int:
    return int(lib().slkv_pooled_elems(C.byref(params), _cu_host(cu_seqlens)))


def slkv_packed_rows_upper_bound(params: SlkvParams, cu_seqlens: Sequence[int]) -> int:
    return int(lib().slkv_packed_rows_upper_bound(C.byref(params), _cu_host(cu_seqlens)))


def new_workspace(params: SlkvParams, cu_seqlens: Sequence[int], device) -> torch.Tensor:
    n = slkv_workspace_bytes(params, cu_seqlens)
    if n == 0:
        raise SlkvError(ERR["BAD_SHAPE"], "slkv_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=device)


def _lse(lse: Optional[torch.Tensor], params: SlkvParams) -> Optional[int]:
    if lse is None:
        return None
    assert lse.is_cuda and lse.dtype == torch.float32 and lse.is_contiguous()
    assert lse.numel() == params.n_seqs * params.n_q_heads * params.window, "lse is [n_seqs, n_q_heads, window]"
    return lse.data_ptr()


def slkv_score(params: SlkvParams, q_win: torch.Tensor, k: torch.Tensor, cu_dev: torch.Tensor,
               cu_seqlens: Sequence[int], pooled: torch.Tensor, workspace: torch.Tensor,
               status: Optional[torch.Tensor] = None, stream=None, lse: Optional[torch.Tensor] = None) -> torch.Tensor:
    rc = lib().slkv_score(C.byref(params), q_win.data_ptr(), k.data_ptr(), cu_dev.data_ptr(), _cu_host(cu_seqlens),
                          _lse(lse, params), pooled.data_ptr(), _ptr(status), workspace.data_ptr(), workspace.numel(),
                          _stream(stream))
    if rc != SLKV_OK:
        raise SlkvError(rc, "slkv_score")
    return pooled


def slkv_row_lse(params: SlkvParams, q_win: torch.Tensor, k: torch.Tensor, cu_dev: torch.Tensor,
                 cu_seqlens: Sequence[int], lse_out: torch.Tensor, workspace: torch.Tensor,
                 status: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """lse_out: CUDA float32 [n_seqs, n_q_heads, window], the window rows' log-sum-exp in params.lse_units."""
    _lse(lse_out, params)
    rc = lib().slkv_row_lse(C.byref(params), q_win.data_ptr(), k.data_ptr(), cu_dev.data_ptr(), _cu_host(cu_seqlens),
                            lse_out.data_ptr(), _ptr(status), workspace.data_ptr(), workspace.numel(), _stream(stream))
    if rc != SLKV_OK:
        raise SlkvError(rc, "slkv_row_lse")
    return lse_out


def slkv_debug_expire_next_wait(on: bool = True) -> None:
    lib().slkv_debug_expire_next_wait(1 if on else 0)


def slkv_score_noalloc(params: SlkvParams, q_win: torch.Tensor, k: torch.Tensor, cu_dev: torch.Tensor,
                       cu_seqlens: Sequence[int], pooled: torch.Tensor, status: Optional[torch.Tensor] = None,
                       stream=None, lse: Optional[torch.Tensor] = None) -> torch.Tensor:
    """slkv_score for callers that cannot allocate: the scratch is a fixed array inside the library
    (slkv_noalloc_scratch_bytes() bytes); larger shapes raise SLKV_ERR_WORKSPACE."""
    rc = lib().slkv_score_noalloc(C.byref(params), q_win.data_ptr(), k.data_ptr(), cu_dev.data_ptr(),
                                  _cu_host(cu_seqlens), _lse(lse, params), pooled.data_ptr(), _ptr(status),
                                  _stream(stream))
    if rc != SLKV_OK:
        raise SlkvError(rc, "slkv_score_noalloc")
    return pooled


def slkv_noalloc_scratch_bytes() -> int:
    return int(lib().slkv_noalloc_scratch_bytes())


def slkv_compress(params: SlkvParams, q_win, k, v, cu_dev, cu_seqlens: Sequence[int], budgets, k_out, v_out,
                  offsets, kept_idx, workspace, pooled: Optional[torch.Tensor] = None,
                  status: Optional[torch.Tensor] = None, stream=None, lse: Optional[torch.Tensor] = None) -> None:
    rc = lib().slkv_compress(C.byref(params), q_win.data_ptr(), k.data_ptr(), v.data_ptr(), cu_dev.data_ptr(),
                             _cu_host(cu_seqlens), budgets.data_ptr(), _lse(lse, params), k_out.data_ptr(),
                             v_out.data_ptr(),
                             k_out.shape[0], offsets.data_ptr(), kept_idx.data_ptr(), _ptr(pooled), _ptr(status),
                             workspace.data_ptr(), workspace.numel(), _stream(stream))
    if rc != SLKV_OK:
        raise SlkvError(rc, "slkv_compress")


def slkv_compress_overlapped(params: SlkvParams, q_win, k, v, cu_dev, cu_seqlens: Sequence[int], budgets, k_out,
                             v_out, offsets, kept_idx, workspace, pooled: Optional[torch.Tensor] = None,
                             status: Optional[torch.Tensor] = None, stream=None,
                             lse: Optional[torch.Tensor] = None) -> None:
    """slkv_compress with successive calls overlapped on the GPU; outputs are valid behind slkv_join()."""
    rc = lib().slkv_compress_overlapped(C.byref(params), q_win.data_ptr(), k.data_ptr(), v.data_ptr(),
                                        cu_dev.data_ptr(), _cu_host(cu_seqlens), budgets.data_ptr(),
                                        _lse(lse, params), k_out.data_ptr(), v_out.data_ptr(), k_out.shape[0], offsets.data_ptr(),
                                        kept_idx.data_ptr(), _ptr(pooled), _ptr(status), workspace.data_ptr(),
                                        workspace.numel(), _stream(stream))
    if rc != SLKV_OK:
        raise SlkvError(rc, "slkv_compress_overlapped")


def slkv_workspace_bytes_overlapped(params: SlkvParams, cu_seqlens: Sequence[int]) -> int:
    return int(lib().slkv_workspace_bytes_overlapped(C.byref(params), _cu_host(cu_seqlens)))


def slkv_join(stream=None) -> None:
    rc = lib().slkv_join(_stream(stream))
    if rc != SLKV_OK:
        raise SlkvError(rc, "slkv_join")


def slkv_compress_host_arena_bytes(params: SlkvParams, cu_seqlens: Sequence[int], capacity_rows: int) -> int:
    return int(lib().slkv_compress_host_arena_bytes(C.byref(params), _cu_host(cu_seqlens), int(capacity_rows)))


def slkv_compress_host(params: SlkvParams, q_win, k, v, cu_seqlens: Sequence[int], budgets, k_out, v_out, offsets,
                       kept_idx, arena: torch.Tensor, stream=None) -> int:
    """All tensors except `arena` are HOST tensors (pinned for speed); returns the number of packed rows."""
    for t in (q_win, k, v, budgets, k_out, v_out, offsets, kept_idx):
        assert not t.is_cuda and t.is_contiguous()
    assert arena.is_cuda
    rows = C.c_int64(0)
    rc = lib().slkv_compress_host(C.byref(params), q_win.data_ptr(), k.data_ptr(), v.data_ptr(), _cu_host(cu_seqlens),
                                  budgets.data_ptr(), k_out.data_ptr(), v_out.data_ptr(), k_out.shape[0],
                                  offsets.data_ptr(), kept_idx.data_ptr(), C.byref(rows), arena.data_ptr(),
                                  arena.numel(), _stream(stream))
    if rc != SLKV_OK:
        raise SlkvError(rc, "slkv_compress_host")
    return int(rows.value)


def slkv_profile_enable(on) -> None:
    """False / 0: off; True / 1: every kernel (one stream); 2: the score kernels only, side streams kept."""
    lib().slkv_profile_enable(int(on))


def slkv_profile_collect() -> dict:
    """{kernel name: (total milliseconds, launches)} since the last collect, for kernels that ran."""
    n = lib().slkv_kernel_count()
    ms = (C.c_float * n)()
    cnt = (C.c_int32 * n)()
    rc = lib().slkv_profile_collect(ms, cnt, n)
    if rc != SLKV_OK:
        raise SlkvError(rc, "slkv_profile_collect")
    return {lib().slkv_kernel_name(i).decode(): (float(ms[i]), int(cnt[i])) for i in range(n) if cnt[i] > 0}


def slkv_trace_set_buffer(buf: Optional[torch.Tensor]) -> None:
    """buf: CUDA int64 tensor that receives the score kernels' timeline stamps, or None to switch tracing off."""
    if buf is None:
        lib().slkv_trace_set_buffer(None, 0)
    else:
        lib().slkv_trace_set_buffer(buf.data_ptr(), buf.numel() * buf.element_size())


# ---- context-parallel selection (one sequence's keys split over ranks): thin wrappers, see include/slkv.h ------------
def _check(rc: int, what: str) -> None:
    if rc != SLKV_OK:
        raise SlkvError(rc, what)


def slkv_cp_merge_lse(params: SlkvParams, lse_parts: torch.Tensor, lse_out: torch.Tensor, stream=None) -> torch.Tensor:
    """lse_parts: CUDA float32 [n_parts, n_q_heads, window] (contiguous); lse_out: [1, n_q_heads, window]."""
    _check(lib().slkv_cp_merge_lse(C.byref(params), lse_parts.data_ptr(), int(lse_parts.shape[0]), lse_out.data_ptr(),
                                   _stream(stream)), "slkv_cp_merge_lse")
    return lse_out


def slkv_cp_select_init(budgets: torch.Tensor, window: int, seq_len: int, prefix: torch.Tensor, need: torch.Tensor,
                        stream=None) -> None:
    _check(lib().slkv_cp_select_init(budgets.data_ptr(), int(budgets.numel()), int(window), int(seq_len),
                                     prefix.data_ptr(), need.data_ptr(), _stream(stream)), "slkv_cp_select_init")


def slkv_cp_histogram(pooled: torch.Tensor, n_kv_heads: int, row_stride: int, own_begin: int, own_count: int, level: int,
                      prefix: torch.Tensor, hist: torch.Tensor, stream=None) -> torch.Tensor:
    _check(lib().slkv_cp_histogram(pooled.data_ptr(), int(n_kv_heads), int(row_stride), int(own_begin), int(own_count),
                                   int(level), prefix.data_ptr(), hist.data_ptr(), _stream(stream)), "slkv_cp_histogram")
    return hist


def slkv_cp_descend(hist: torch.Tensor, level: int, prefix: torch.Tensor, need: torch.Tensor, stream=None) -> None:
    _check(lib().slkv_cp_descend(hist.data_ptr(), int(prefix.numel()), int(level), prefix.data_ptr(), need.data_ptr(),
                                 _stream(stream)), "slkv_cp_descend")


def slkv_cp_local_ties(hist_local: torch.Tensor, prefix: torch.Tensor, ties: torch.Tensor, stream=None) -> torch.Tensor:
    _check(lib().slkv_cp_local_ties(hist_local.data_ptr(), prefix.data_ptr(), int(prefix.numel()), ties.data_ptr(),
                                    _stream(stream)), "slkv_cp_local_ties")
    return ties


def slkv_cp_workspace_bytes(n_kv_heads: int, own_count: int, capacity_rows: int) -> int:
    return int(lib().slkv_cp_workspace_bytes(int(n_kv_heads), int(own_count), int(capacity_rows)))


def slkv_cp_emit(params: SlkvParams, k: torch.Tensor, v: torch.Tensor, rows: int, pooled: torch.Tensor, row_stride: int,
                 own_begin: int, own_count: int, pos0: int, threshold: torch.Tensor, need: torch.Tensor,
                 ties_all: torch.Tensor, part: int, window_rows: int, window_pos0: int, k_out: torch.Tensor,
                 v_out: torch.Tensor, offsets: torch.Tensor, kept_idx: torch.Tensor, workspace: torch.Tensor,
                 status: Optional[torch.Tensor] = None, stream=None) -> None:
    _check(lib().slkv_cp_emit(C.byref(params), k.data_ptr(), v.data_ptr(), int(rows), pooled.data_ptr(), int(row_stride),
                              int(own_begin), int(own_count), int(pos0), threshold.data_ptr(), need.data_ptr(),
                              ties_all.data_ptr(), int(ties_all.shape[0]), int(part), int(window_rows), int(window_pos0),
                              k_out.data_ptr(), v_out.data_ptr(), int(k_out.shape[0]), offsets.data_ptr(),
                              kept_idx.data_ptr(), _ptr(status), workspace.data_ptr(), workspace.numel(),
                              _stream(stream)), "slkv_cp_emit")
