"""GPU parity on seeded random problem shapes: head counts, group sizes, windows, pooling kernels, ragged batches
and budgets drawn at random, every case checked against the oracle (Eq. 7-8, Algorithm 3) through the C ABI,
and the overlapped entry point checked bit for bit against the ordinary one on the same inputs."""
import numpy as np
import pytest
import torch

import parity as P
from paper_2508_15806_b200 import binding as B

pytestmark = pytest.mark.gpu


def draw_case(seed, tensor_path=False):
    """tensor_path: only shapes the tensor-core score kernel takes (bf16, d = 128, G * w a multiple of 32)."""
    rng = np.random.default_rng((5000 if tensor_path else 1000) + seed)
    dtype = torch.bfloat16 if tensor_path else [torch.bfloat16, torch.float32][int(rng.integers(0, 2))]
    d = 128 if tensor_path else int(rng.choice([64, 128]))
    Hkv = int(rng.choice([1, 2, 4, 8]))
    G = int(rng.choice([1, 2, 4, 8]))
    w = int(rng.choice([w for w in (4, 8, 16, 32, 64) if G * w <= 256 and (not tensor_path or (G * w) % 32 == 0)]))
    p = int(rng.choice([1, 3, 5, 7]))
    n_seqs = int(rng.integers(1, 5))
    lens = []
    for _ in range(n_seqs):
        kind = int(rng.integers(0, 6))
        if kind == 0:
            lens.append(int(rng.integers(1, w + 2)))                  # shorter than, equal to, one more than the window
        elif kind == 1:
            lens.append(w + 128 * int(rng.integers(1, 6)))            # history a whole number of key tiles
        else:
            lens.append(int(rng.integers(w + 2, 2600)))
    budgets = []
    for s in range(n_seqs):
        for h in range(Hkv):
            kind = int(rng.integers(0, 5))
            if kind == 0:
                budgets.append(int(rng.integers(0, w + 1)))           # at most the window
            elif kind == 1:
                budgets.append(lens[s] + int(rng.integers(0, 20)))    # everything is kept
            else:
                budgets.append(int(rng.integers(w, max(w + 1, lens[s]))))
    mode = [B.SLKV_POOL_MAX, B.SLKV_POOL_AVG][int(rng.integers(0, 2))]
    return dtype, d, Hkv, G, w, p, lens, budgets, mode


def make_inputs(seed, dtype, d, Hkv, G, w, lens):
    g = torch.Generator().manual_seed(77 + seed)
    T = sum(lens)
    q = (torch.randn(len(lens), w, Hkv * G, d, generator=g) * 1.25).to(dtype)
    k = torch.randn(T, Hkv, d, generator=g).to(dtype)
    v = torch.randn(T, Hkv, d, generator=g).to(dtype)
    # a few keys aligned with the window queries, so that the scores are not all alike
    for s in range(len(lens)):
        a = int(np.cumsum([0] + lens)[s])
        if lens[s] > w + 8:
            for j in (3, lens[s] // 2):
                k[a + j] = (q[s, -1].reshape(Hkv, G, d).float().mean(dim=1) * 0.6).to(dtype)
    return q, k, v


@pytest.mark.parametrize("tensor_path", [False, True])
@pytest.mark.parametrize("seed", range(20))
def test_random_shape_matches_oracle(seed, tensor_path):
    dtype, d, Hkv, G, w, p, lens, budgets, mode = draw_case(seed, tensor_path)
    q, k, v = make_inputs(seed, dtype, d, Hkv, G, w, lens)
    cu = [0] + [int(x) for x in np.cumsum(lens)]
    gpu, stats = P.check_compress(q, k, v, cu, budgets, w, p, pool_mode=mode)
    assert stats["segments"] == len(lens) * Hkv

    # the same layer three times through the overlapped entry point (both halves of its workspace get reused), then a join
    dev = torch.device("cuda:0")
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    params = B.make_params(qd, kd, vd, w, p, mode, B.SLKV_PATH_AUTO)
    cap = B.slkv_packed_rows_upper_bound(params, cu)
    cu_dev = torch.tensor(cu, dtype=torch.int32, device=dev)
    bud = torch.tensor(budgets, dtype=torch.int32, device=dev)
    ws = torch.empty(max(B.slkv_workspace_bytes_overlapped(params, cu), 1), dtype=torch.uint8, device=dev)
    outs = [dict(k=torch.zeros(max(cap, 1), d, dtype=dtype, device=dev), v=torch.zeros(max(cap, 1), d, dtype=dtype, device=dev),
                 off=torch.full((len(lens) * Hkv + 1,), -1, dtype=torch.int32, device=dev),
                 kept=torch.full((max(cap, 1),), -1, dtype=torch.int32, device=dev),
                 status=torch.zeros(1, dtype=torch.int32, device=dev)) for _ in range(3)]
    for o in outs:
        B.slkv_compress_overlapped(params, qd, kd, vd, cu_dev, cu, bud, o["k"], o["v"], o["off"], o["kept"], ws, None,
                                   o["status"])
    B.slkv_join()
    torch.cuda.synchronize()
    n = int(gpu["offsets"][-1])
    for o in outs:
        assert int(o["status"].item()) == 0
        assert np.array_equal(o["off"].cpu().numpy().astype(np.int64), gpu["offsets"])
        assert np.array_equal(o["kept"][:n].cpu().numpy().astype(np.int64), gpu["kept_idx"][:n])
        assert torch.equal(o["k"][:n].cpu(), gpu["k_out"][:n]) and torch.equal(o["v"][:n].cpu(), gpu["v_out"][:n])
