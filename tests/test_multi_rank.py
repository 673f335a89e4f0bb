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


def test_reference_arm_only_rank0_works():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert p.returncode == 0 and p.stdout.strip() == ""
