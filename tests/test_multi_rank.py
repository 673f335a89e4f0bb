"""The N > 1 host logic of bench.py on CPU: two gloo ranks (no GPU, no data-path collective)."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import bench
    from paper_2508_15806_b200 import synth
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = bench.rank_workload(synth.small_variant(synth.workloads()[1], [300]), rank, world)
    x = synth.layer_inputs(wl, 0)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))       # slowest rank decides
    dist.barrier()
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"seed": wl.seed, "ms": ms, "k0": float(x.k.float().sum()),
                   "value": bench.whole_job_value(world, wl.total_tokens, wl.n_layers, ms)}, f)
    dist.destroy_process_group()


def test_two_ranks_shard_by_sequence_batch_and_time_by_the_slowest(tmp_path):
    world, port = 2, 29000 + os.getpid() % 2000
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r = [json.load(open(tmp_path / f"r{i}.json")) for i in range(world)]
    assert r[0]["seed"] != r[1]["seed"] and r[0]["k0"] != r[1]["k0"]          # each rank has its own inputs
    assert r[0]["ms"] == r[1]["ms"] == 15.0                                   # max over ranks, on every rank
    assert abs(r[0]["value"] - 2 * 300 / 15e-3) < 1e-6                        # whole-job tokens/s/layer


def _head_shard_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import numpy as np
    from oracle import slkv_oracle as O
    from paper_2508_15806_b200 import sharding as S
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # a layer of 5 KV heads over 2 ranks (3 + 2), 3 sequences; the kept counts a rank's compression would report for
    # its heads come from the oracle's rule here (no GPU in this test): what is checked is the exchange and stitching
    n_kv, window, lens, budgets = 5, 4, [30, 3, 9], [6, 40, 2, 9, 12]
    h0, h1 = S.head_range(n_kv, rank, world)
    kept = torch.tensor([[sum(O.kept_counts(n, budgets[h], window)) for h in range(h0, h1)] for n in lens], dtype=torch.int32)
    local_offsets = torch.zeros(kept.numel() + 1, dtype=torch.int32)
    local_offsets[1:] = torch.cumsum(kept.reshape(-1), 0)
    assert torch.equal(S.local_kept(local_offsets, len(lens), h1 - h0), kept)
    offsets, bases = S.stitch(S.all_gather_kept(kept))
    with open(os.path.join(out_dir, f"h{rank}.json"), "w") as f:
        json.dump({"range": [h0, h1], "offsets": offsets.tolist(), "base": bases[rank].tolist()}, f)
    dist.destroy_process_group()


def test_two_ranks_shard_by_kv_head_and_stitch_offsets(tmp_path):
    from oracle import slkv_oracle as O
    world, port = 2, 31000 + os.getpid() % 2000
    mp.spawn(_head_shard_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r = [json.load(open(tmp_path / f"h{i}.json")) for i in range(world)]
    assert r[0]["range"] == [0, 3] and r[1]["range"] == [3, 5]
    n_kv, window, lens, budgets = 5, 4, [30, 3, 9], [6, 40, 2, 9, 12]
    expect = [0]
    for n in lens:
        for h in range(n_kv):
            expect.append(expect[-1] + sum(O.kept_counts(n, budgets[h], window)))
    assert r[0]["offsets"] == expect and r[1]["offsets"] == expect            # every rank ends with the same offsets
    for rank in range(world):
        h0, h1 = r[rank]["range"]
        for s in range(len(lens)):
            assert r[rank]["base"][s] == [expect[s * n_kv + h] for h in range(h0, h1)]


def test_head_ranges_cover_all_heads():
    from paper_2508_15806_b200 import sharding as S
    for n_kv in (1, 5, 8, 9):
        for world in (1, 2, 3, 4, 8):
            rs = [S.head_range(n_kv, r, world) for r in range(world)]
            assert rs[0][0] == 0 and rs[-1][1] == n_kv and all(a[1] == b[0] for a, b in zip(rs, rs[1:]))
            assert max(b - a for a, b in rs) - min(b - a for a, b in rs) <= 1


def test_reference_arm_only_rank0_works():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert p.returncode == 0 and p.stdout.strip() == ""


def _cp_select_main(rank, world, port, out_dir):
    """The distributed selection of the context-parallel path, restated with numpy on every rank and run over gloo:
    the histograms and tie counts travel through the package's communicator, the arithmetic is the test's own."""
    sys.path.insert(0, ROOT)
    import numpy as np
    from paper_2508_15806_b200 import context_parallel as CP
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    comm = CP.DistComm()
    assert (comm.rank, comm.world) == (rank, world)
    rng = np.random.default_rng(11)                       # the same scores on every rank; each uses its own range
    n_kv, w, L = 3, 8, 8 + 1237
    scores = rng.choice(np.array([0.0, 0.5, 1.0, 2.5, 1e-20], dtype=np.float32), size=(n_kv, L - w))
    scores[2] = rng.random(L - w).astype(np.float32)
    budgets = [w + 400, w + 1, L]
    b, e = CP.key_ranges(L, w, world)[rank]
    bits = scores[:, b:e].view(np.uint32).astype(np.int64)
    need = np.array([min(L, max(c, w)) - w for c in budgets], dtype=np.int64)
    prefix = np.zeros(n_kv, dtype=np.int64)
    own_last = None
    for level, (shift, nbits) in enumerate(((21, 11), (10, 11), (0, 10))):
        hist = np.zeros((n_kv, 2048), dtype=np.int32)
        for h in range(n_kv):
            sel = bits[h] if level == 0 else bits[h][(bits[h] >> (shift + nbits)) == (prefix[h] >> (shift + nbits))]
            np.add.at(hist[h], (sel >> shift) & ((1 << nbits) - 1), 1)
        own_last = hist.copy()
        total = comm.all_reduce_sum(torch.from_numpy(hist)).numpy()
        for h in range(n_kv):
            if need[h] <= 0:
                prefix[h], need[h] = 0xFFFFFFFF, 0
                continue
            above, d = 0, (1 << nbits) - 1
            while d > 0 and above + total[h, d] < need[h]:
                above += total[h, d]
                d -= 1
            prefix[h] |= d << shift
            need[h] -= above
    ties = np.array([0 if prefix[h] == 0xFFFFFFFF else own_last[h, prefix[h] & 1023] for h in range(n_kv)], dtype=np.int32)
    ties_all = comm.all_gather(torch.from_numpy(ties)).numpy()
    kept = []
    for h in range(n_kv):
        take = int(np.clip(need[h] - ties_all[:rank, h].sum(), 0, ties[h]))
        gt = np.nonzero(bits[h] > prefix[h])[0]
        eq = np.nonzero(bits[h] == prefix[h])[0][:take]
        kept.append((np.sort(np.concatenate([gt, eq])) + b).tolist())
    with open(os.path.join(out_dir, f"c{rank}.json"), "w") as f:
        json.dump({"kept": kept}, f)
    dist.destroy_process_group()


def test_ranks_select_one_top_k_over_split_scores(tmp_path):
    import numpy as np
    from oracle import slkv_oracle as O
    for world in (2, 3):
        port = 33000 + (os.getpid() + world) % 2000
        mp.spawn(_cp_select_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
        rng = np.random.default_rng(11)
        n_kv, w, L = 3, 8, 8 + 1237
        scores = rng.choice(np.array([0.0, 0.5, 1.0, 2.5, 1e-20], dtype=np.float32), size=(n_kv, L - w))
        scores[2] = rng.random(L - w).astype(np.float32)
        budgets = [w + 400, w + 1, L]
        for h in range(n_kv):
            got = sum((json.load(open(tmp_path / f"c{r}.json"))["kept"][h] for r in range(world)), [])
            kh, _ = O.kept_counts(L, budgets[h], w)
            assert got == O.select_topk(scores[h].astype(np.float64), kh).tolist(), (world, h)


def test_key_ranges_cover_the_history_in_order():
    from paper_2508_15806_b200 import context_parallel as CP
    for L, w, world in ((1000, 32, 3), (40, 32, 5), (32, 32, 2), (131072, 64, 8)):
        r = CP.key_ranges(L, w, world)
        assert r[0][0] == 0 and r[-1][1] == L - w and all(a[1] == b[0] for a, b in zip(r, r[1:]))
        assert max(e - b for b, e in r) - min(e - b for b, e in r) <= 1
