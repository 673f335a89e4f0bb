"""Seeded synthetic inputs for the KV-compression path (shapes of the paper's workloads).

This module only *draws inputs*: a counter-based random generator, Gaussian Q/K/V with planted
"needle" keys and optional attention-sink keys, ragged sequence lengths and INF_sc tables.  It holds
none of the method's arithmetic (no scoring, pooling, budgeting or selection) and is the one module
that both the CPU oracle's tests and the CUDA path's tests/bench may import.

Every value is a pure function of (seed, tensor id, layer, flat element index):

    key  = mix(seed ^ tensor_id << 56 ^ layer << 40)
    z_c  = mix(key + (2*index + c) * GOLDEN)          c in {0, 1}
    u_c  = ((z_c >> 11) + 0.5) * 2^-53                in (0, 1)
    n    = sqrt(-2 ln u_0) * cos(2 pi u_1)            (Box-Muller, fp64)

with mix() the splitmix64 finaliser.  All tensor math is torch, so the same code runs on the CPU
(parity tests: the bytes handed to the oracle and to the GPU are the same host bytes) and on a CUDA
device (bench: fills device buffers directly; the bytes the oracle sees are copied back from them).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import torch

_GOLDEN = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB
_MASK = (1 << 64) - 1

# tensor ids (the "stream" a value belongs to)
TID_Q, TID_K, TID_V, TID_DIR, TID_INF, TID_LEN, TID_NEEDLE, TID_MISC = 1, 2, 3, 4, 5, 6, 7, 8


def _s64(x: int) -> int:
    """Python int (mod 2^64) -> the signed value holding the same 64 bits."""
    x &= _MASK
    return x - (1 << 64) if x >= (1 << 63) else x


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of an int64 tensor seen as uint64."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix_t(z: torch.Tensor) -> torch.Tensor:
    z = (z ^ _lsr(z, 30)) * _s64(_M1)
    z = (z ^ _lsr(z, 27)) * _s64(_M2)
    return z ^ _lsr(z, 31)


def mix_int(z: int) -> int:
    """splitmix64 finaliser on a Python int (reference for the tensor version)."""
    z &= _MASK
    z = ((z ^ (z >> 30)) * _M1) & _MASK
    z = ((z ^ (z >> 27)) * _M2) & _MASK
    return z ^ (z >> 31)


def stream_key(seed: int, tensor_id: int, layer: int = 0) -> int:
    return mix_int((seed & _MASK) ^ ((tensor_id & 0xFF) << 56) ^ ((layer & 0xFFFF) << 40))


def _bits(key: int, idx: torch.Tensor, c: int) -> torch.Tensor:
    # (2*idx + c) * GOLDEN + key, all mod 2^64 (int64 arithmetic wraps)
    return _mix_t((idx * 2 + c) * _s64(_GOLDEN) + _s64(key))


def uniform(key: int, n: int, device="cpu", start: int = 0, c: int = 0) -> torch.Tensor:
    """n uniforms in (0,1), fp64, for element indices start..start+n-1 of stream `key`."""
    idx = torch.arange(start, start + n, dtype=torch.int64, device=device)
    z = _bits(key, idx, c)
    return (_lsr(z, 11).to(torch.float64) + 0.5) * (2.0 ** -53)


def normal(key: int, n: int, device="cpu", start: int = 0, chunk: int = 1 << 22) -> torch.Tensor:
    """n standard normals, fp64 (Box-Muller on two uniforms per element)."""
    out = torch.empty(n, dtype=torch.float64, device=device)
    for a in range(0, n, chunk):
        m = min(chunk, n - a)
        u0 = uniform(key, m, device, start + a, 0)
        u1 = uniform(key, m, device, start + a, 1)
        out[a:a + m] = torch.sqrt(-2.0 * torch.log(u0)) * torch.cos((2.0 * math.pi) * u1)
    return out


def randint(key: int, n: int, lo: int, hi: int) -> List[int]:
    """n integers uniform in [lo, hi] (host, small n)."""
    u = uniform(key, n).tolist()
    return [min(hi, lo + int(x * (hi - lo + 1))) for x in u]


# ----------------------------------------------------------------------------------------------
# workload description
# ----------------------------------------------------------------------------------------------
@dataclass
class Workload:
    """One of the benchmark/parity configurations (shapes and input structure only)."""
    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    window: int
    pool_kernel: int
    dtype: str                      # "f32" | "bf16"
    seq_lens: List[int]
    fixed: int
    totals: List[int]               # one or more total budgets (summed over n_layers*n_kv_heads heads)
    seed: int
    value_scale: float = 1.0        # Q, K, V components ~ N(0,1) * value_scale
    n_needles: int = 0
    needle_logit: float = 8.0       # q.k/sqrt(d) added at a needle key
    n_sinks: int = 0                # first n_sinks keys pushed along the mean window-query direction
    sink_gain: float = 6.0
    inf_recipe: str = "lognormal"   # see inf_sc()
    parity_layers: List[int] = field(default_factory=lambda: [0])

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def elem_size(self) -> int:
        return 4 if self.dtype == "f32" else 2

    @property
    def total_tokens(self) -> int:
        return sum(self.seq_lens)

    @property
    def cu_seqlens(self) -> List[int]:
        cu = [0]
        for n in self.seq_lens:
            cu.append(cu[-1] + n)
        return cu


def ragged_lengths(seed: int, n_seqs: int, lo: int, hi: int) -> List[int]:
    return randint(stream_key(seed, TID_LEN), n_seqs, lo, hi)


def workloads() -> List[Workload]:
    """The five configurations (index = config number - 1)."""
    c1 = Workload("cfg1_f32_mha8_d64_L1024", 1, 8, 8, 64, 16, 5, "f32", [1024], 32, [8 * 128], seed=1,
                  value_scale=0.125, n_needles=4, inf_recipe="lognormal_one_x10")
    c2 = Workload("cfg2_llama8b_1layer_L8192", 1, 32, 8, 128, 32, 7, "bf16", [8192], 64, [8 * 512], seed=2,
                  n_needles=16, inf_recipe="two_percent_high")
    c3 = Workload("cfg3_llama8b_32layers_L32768", 32, 32, 8, 128, 32, 7, "bf16", [32768], 64,
                  [256 * 128, 256 * 512, 256 * 2048], seed=3, n_needles=16, n_sinks=4,
                  inf_recipe="lognormal15_layer1_low", parity_layers=[0, 1, 17, 31])
    c4 = Workload("cfg4_mistral7b_32layers_B8_ragged", 32, 32, 8, 128, 64, 7, "bf16",
                  ragged_lengths(4, 8, 4096, 32768), 64, [256 * 1024], seed=4, n_needles=16,
                  inf_recipe="lognormal15", parity_layers=[0, 31])
    c5 = Workload("cfg5_long_32layers_L131072", 32, 32, 8, 128, 64, 7, "bf16", [131072], 64, [256 * 4096],
                  seed=5, n_needles=16, n_sinks=4, inf_recipe="extreme_skew", parity_layers=[])
    return [c1, c2, c3, c4, c5]


def small_variant(wl: Workload, seq_lens: Sequence[int], n_layers: Optional[int] = None,
                  totals: Optional[Sequence[int]] = None) -> Workload:
    """Same structure, shorter sequences (for cases the oracle finishes in seconds)."""
    import copy
    v = copy.deepcopy(wl)
    v.name = wl.name + "_small"
    v.seq_lens = list(seq_lens)
    if n_layers is not None:
        v.n_layers = n_layers
        v.parity_layers = [l for l in wl.parity_layers if l < n_layers] or [0]
    if totals is not None:
        v.totals = list(totals)
    return v


# ----------------------------------------------------------------------------------------------
# INF_sc tables
# ----------------------------------------------------------------------------------------------
def inf_sc(wl: Workload) -> torch.Tensor:
    """INF_sc per (layer, KV head), float32 [n_layers, n_kv_heads] on the CPU.

    Recipes follow the shape the paper reports for these scores (heavily skewed, a few percent of the
    heads high, three near-zero heads in layer 1); the real table is not published.
    """
    nl, hq, hkv = wl.n_layers, wl.n_q_heads, wl.n_kv_heads
    g = hq // hkv
    key = stream_key(wl.seed, TID_INF)
    r = wl.inf_recipe
    if r == "lognormal_one_x10":
        t = torch.exp(normal(key, nl * hkv)).reshape(nl, hkv)
        t[:, 3 % hkv] *= 10.0
    elif r == "two_percent_high":
        # per query head: low heads 0.02*lognormal(0,0.5); one head per layer uniform in (0.5,0.9);
        # a KV head's score is the mean over its query group
        t = 0.02 * torch.exp(0.5 * normal(key, nl * hq)).reshape(nl, hq)
        hi = uniform(stream_key(wl.seed, TID_INF, 1), nl) * 0.4 + 0.5
        pos = randint(stream_key(wl.seed, TID_INF, 2), nl, 0, hq - 1)
        for i in range(nl):
            t[i, pos[i]] = hi[i]
        t = t.reshape(nl, hkv, g).mean(dim=2)
    elif r in ("lognormal15", "lognormal15_layer1_low"):
        t = torch.exp(1.5 * normal(key, nl * hkv)).reshape(nl, hkv)
        if r.endswith("layer1_low") and nl > 1:
            t[1, 0:3] = 1e-6
    elif r == "extreme_skew":
        t = 1e-4 * torch.exp(0.5 * normal(key, nl * hkv)).reshape(nl, hkv)
        n_heavy = min(6, nl * hkv)
        flat = randint(stream_key(wl.seed, TID_INF, 1), n_heavy, 0, nl * hkv - 1)
        for f in flat:
            t.view(-1)[f] = 1.0
    elif r == "lognormal":
        t = torch.exp(normal(key, nl * hkv)).reshape(nl, hkv)
    else:
        raise ValueError(f"unknown INF_sc recipe {r}")
    return t.to(torch.float32).contiguous()


# ----------------------------------------------------------------------------------------------
# Q / K / V of one layer
# ----------------------------------------------------------------------------------------------
@dataclass
class LayerInputs:
    q_win: torch.Tensor      # [n_seqs, window, n_q_heads, head_dim]
    k: torch.Tensor          # [total_tokens, n_kv_heads, head_dim]
    v: torch.Tensor          # [total_tokens, n_kv_heads, head_dim]
    needles: List[List[int]]  # per sequence: needle positions (within the sequence's history)


def needle_positions(wl: Workload, layer: int, s: int, n_hist: int) -> List[int]:
    """Needle positions in [n_sinks, n_hist), pairwise more than pool_kernel apart (one per stratum)."""
    n = wl.n_needles
    if n == 0 or n_hist <= 0:
        return []
    lo = min(wl.n_sinks, n_hist)
    span = n_hist - lo
    n = min(n, span // (2 * wl.pool_kernel + 2))
    if n <= 0:
        return []
    stratum = span // n
    u = uniform(stream_key(wl.seed, TID_NEEDLE, layer), n, start=s * 4096).tolist()
    free = stratum - (wl.pool_kernel + 1)
    return [lo + i * stratum + int(u[i] * free) for i in range(n)]


def layer_inputs(wl: Workload, layer: int, device="cpu") -> LayerInputs:
    """Q_win, K, V of one layer in the workload's dtype, on `device`."""
    hq, hkv, d, w = wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window
    g = hq // hkv
    T, B = wl.total_tokens, len(wl.seq_lens)
    cu = wl.cu_seqlens
    sc = wl.value_scale

    k = (normal(stream_key(wl.seed, TID_K, layer), T * hkv * d, device) * sc).reshape(T, hkv, d)
    v = (normal(stream_key(wl.seed, TID_V, layer), T * hkv * d, device) * sc).reshape(T, hkv, d)
    q = (normal(stream_key(wl.seed, TID_Q, layer), B * w * hq * d, device) * sc).reshape(B, w, hq, d)

    # one unit direction per (sequence, KV head); the group's query heads share it
    u = normal(stream_key(wl.seed, TID_DIR, layer), B * hkv * d, device).reshape(B, hkv, d)
    u = u / u.norm(dim=2, keepdim=True)
    amp = math.sqrt(wl.needle_logit * math.sqrt(d))     # c = s, c*s/sqrt(d) = needle_logit
    needles: List[List[int]] = []
    for s in range(B):
        n_hist = max(wl.seq_lens[s] - w, 0)
        pos = needle_positions(wl, layer, s, n_hist)
        needles.append(pos)
        if pos:
            q[s] += amp * u[s].repeat_interleave(g, dim=0).unsqueeze(0)          # [1, hq, d]
            pidx = torch.tensor(pos, dtype=torch.int64, device=device) + cu[s]
            k[pidx] = (amp * u[s]).unsqueeze(0).expand(len(pos), hkv, d)
        if wl.n_sinks > 0 and n_hist > wl.n_sinks:
            qm = q[s].reshape(w, hkv, g, d).mean(dim=(0, 2))                       # [hkv, d]
            qm = qm / qm.norm(dim=1, keepdim=True)
            k[cu[s]:cu[s] + wl.n_sinks] += wl.sink_gain * qm.unsqueeze(0)
    dt = wl.torch_dtype
    return LayerInputs(q.to(dt).contiguous(), k.to(dt).contiguous(), v.to(dt).contiguous(), needles)


# ---------------------------------------------------------------------------------------------------
# attention rows for the Stage-1 behaviour analysis (shapes of the paper's needle-in-a-haystack probes)
# ---------------------------------------------------------------------------------------------------
TID_ATTN = 9


def behavior_rows(n_rows: int, row_len: int, n_needle: int = 12, top_k: int = 16, seed: int = 11, device="cpu"):
    """Attention-weight rows as a needle-in-a-haystack probe produces them, with their index sets.

    Every row is a probability vector over `row_len` context positions: a heavy first position (attention sink),
    a contiguous needle span of `n_needle` tokens at a seeded depth that receives a seeded share of the mass
    (near 0 for heads that ignore the needle, most of it for retrieval heads), a few seeded distractor spikes
    elsewhere, and a lognormal background.  Returns (attn float32 [n_rows, row_len], needle_idx int32
    [n_rows, n_needle], topk_idx int32 [n_rows, top_k]); topk_idx are the positions of the row's top_k largest
    weights (equal weights: lower position first), the input Algorithm 1 calls T.
    """
    assert row_len > n_needle + 8 and top_k <= row_len
    key = stream_key(seed, TID_ATTN)
    bg = torch.exp(0.7 * normal(key, n_rows * row_len, device)).reshape(n_rows, row_len)
    u = uniform(stream_key(seed, TID_ATTN, 1), n_rows * 8, device).reshape(n_rows, 8)
    start = 1 + (u[:, 0] * (row_len - n_needle - 1)).to(torch.int64)                  # needle depth
    needle = start[:, None] + torch.arange(n_needle, device=device)[None, :]
    share = u[:, 1] ** 3                                                               # most heads: little mass on it
    bg = bg / bg.sum(dim=1, keepdim=True) * (1.0 - share)[:, None] * 0.7
    rows = bg.clone()
    rows[:, 0] += 0.3 * (1.0 - share)                                                  # the sink
    w_needle = torch.exp(1.2 * normal(stream_key(seed, TID_ATTN, 2), n_rows * n_needle, device)).reshape(n_rows, n_needle)
    rows.scatter_add_(1, needle, w_needle / w_needle.sum(dim=1, keepdim=True) * share[:, None])
    for d in range(3):                                                                 # distractor spikes
        pos = 1 + (u[:, 2 + d] * (row_len - 1)).to(torch.int64)
        rows.scatter_add_(1, pos[:, None], (0.05 * u[:, 5 + d] * (1.0 - share))[:, None])
    rows = (rows / rows.sum(dim=1, keepdim=True)).to(torch.float32)
    order = torch.sort(rows.to(torch.float64), dim=1, descending=True, stable=True).indices[:, :top_k]
    return rows.contiguous(), needle.to(torch.int32).contiguous(), order.to(torch.int32).contiguous()
