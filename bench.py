#!/usr/bin/env python
"""Benchmark of the prefill KV-compression step:  python bench.py [--gpus N] [--steps K] [--warmup W]

One step = the whole hot path (window scores -> pooling -> per-head top-k -> packed K/V gather) for every
layer of the workload, budgets precomputed once by slkv_alloc_budgets (they are per model, not per step).
Workload at N=1: the 32k-context Llama-3-8B-shaped configuration (32 layers, 32 query / 8 KV heads,
head_dim 128, window 32, pool 7, average budget 512 per KV head), synthetic seeded inputs resident in HBM.
Every layer has its own Q/K/V (4.3 GB in total, far larger than L2), so K is really streamed from HBM.

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2508_15806_b200 import synth  # noqa: E402

METRIC = "context tokens compressed per second per layer"
UNIT = "tokens/s/layer"
WORKLOAD_INDEX = 2          # the 32k-context, 32-layer configuration (third of the five workloads)
TOTAL_INDEX = 1             # average budget 512 per KV head
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic_per_key_row.txt")
KERNEL_SOURCES = {"k_score_pipe": ["slkv_score_pipe.cu", "slkv_tc_device.cuh"],
                  "k_score_fused": ["slkv_score_tc.cu", "slkv_tc_device.cuh"]}


def source_sha16(kernel: str):
    """First 16 hex digits of the SHA-256 of the kernel's source files (to tell whether a capture is still current)."""
    import hashlib
    h = hashlib.sha256()
    for f in KERNEL_SOURCES.get(kernel, []):
        with open(os.path.join(ROOT, "paper_2508_15806_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def dram_traffic_per_key_row(kernel: str, mode: str):
    """DRAM bytes per key row (256 B of K) of one launch from the tracked ncu summary, or None when there is no
    capture of this kernel and mode, or the kernel's sources have changed since the capture was taken."""
    try:
        with open(TRAFFIC_FILE) as f:
            for line in f:
                t = line.split()
                if len(t) >= 4 and not line.startswith("#") and t[0] == kernel and t[1] == mode:
                    if t[3] != source_sha16(kernel):
                        return None
                    return {"bytes": float(t[2]), "source": "profiles/" + " ".join(t[4:])}
    except OSError:
        pass
    return None


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    except Exception:
        return {"hbm_gbs": 6650.0, "bf16_tflops": 1400.0, "source": "fallback"}


# ---------------------------------------------------------------------------------------------------
# clocks during the timed region
# ---------------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples SM clock and throttle reasons of the bench's GPU through NVML while the timed loops run."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, device_index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            props = torch.cuda.get_device_properties(device_index)
            try:
                bus = "%08x:%02x:%02x.0" % (props.pci_domain_id, props.pci_bus_id, props.pci_device_id)
                self.h = pynvml.nvmlDeviceGetHandleByPciBusId(bus.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.nv = pynvml
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in self.REASONS.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.02)

    def start(self):
        if self.nv is not None:
            self._stop.clear()
            self._thr = threading.Thread(target=self._run, daemon=True)
            self._thr.start()

    def stop(self):
        if self._thr is not None:
            self._stop.set()
            self._thr.join()
            self._thr = None

    def summary(self):
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ---------------------------------------------------------------------------------------------------
# the CUDA arm
# ---------------------------------------------------------------------------------------------------
def rows_of_layer(lens, budgets_row, window):
    return sum(min(n, max(int(c), window)) for n in lens for c in budgets_row)


def rank_workload(wl, rank: int, world: int):
    """Weak scaling: every rank compresses its own sequence batch (same shapes, its own seed)."""
    if world > 1:
        wl.seed = wl.seed + 1000 * rank
    return wl


def max_over_ranks(ms: float, dist, device) -> float:
    """The step time of the job is the slowest rank's (dist = torch.distributed or None)."""
    if dist is None:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world: int, tokens_per_rank: int, n_layers: int, ms_per_step: float) -> float:
    """Tokens per second per layer summed over all ranks (= world * T / t_layer)."""
    return world * tokens_per_rank * n_layers / (ms_per_step * 1e-3)


def run_cuda(args):
    from paper_2508_15806_b200 import binding as B

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    B.lib()

    wl = synth.workloads()[(args.workload - 1) if args.workload else WORKLOAD_INDEX]
    if args.layers:
        wl = synth.small_variant(wl, wl.seq_lens, n_layers=args.layers,
                                 totals=[t // wl.n_layers * args.layers for t in wl.totals])
    wl = rank_workload(wl, rank, world)
    total = wl.totals[TOTAL_INDEX if len(wl.totals) > TOTAL_INDEX else 0]
    cu = wl.cu_seqlens
    T, nl, hkv, d, w = wl.total_tokens, wl.n_layers, wl.n_kv_heads, wl.head_dim, wl.window
    e = wl.elem_size

    # budgets: once per model, on the GPU
    inf = synth.inf_sc(wl).to(dev)
    budgets = B.slkv_alloc_budgets(inf, wl.fixed, total)
    torch.cuda.synchronize()
    budgets_host = budgets.cpu()
    assert int(budgets_host.sum()) == total

    layers = []
    cu_dev = torch.tensor(cu, dtype=torch.int32, device=dev)
    params = None
    for l in range(nl):
        x = synth.layer_inputs(wl, l, device=dev)
        if args.kv_head_major:
            # the same values, stored [n_kv_heads, tokens, head_dim]: the library takes the layout through the strides
            x.k = x.k.permute(1, 0, 2).contiguous().permute(1, 0, 2)
            x.v = x.v.permute(1, 0, 2).contiguous().permute(1, 0, 2)
        if params is None:
            params = B.make_params(x.q_win, x.k, x.v, w, wl.pool_kernel)
        rows = rows_of_layer(wl.seq_lens, budgets_host[l].tolist(), w)
        layers.append({"q": x.q_win, "k": x.k, "v": x.v, "rows": rows, "bud": budgets[l].contiguous(),
                       "k_out": torch.empty(rows, d, dtype=wl.torch_dtype, device=dev),
                       "v_out": torch.empty(rows, d, dtype=wl.torch_dtype, device=dev),
                       "offsets": torch.empty(len(wl.seq_lens) * hkv + 1, dtype=torch.int32, device=dev),
                       "kept": torch.empty(rows, dtype=torch.int32, device=dev)})
    overlap = not args.no_overlap
    ws = torch.empty(B.slkv_workspace_bytes_overlapped(params, cu), dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    # the rows' log-sum-exps, as a prefill attention kernel that keeps its softmax statistics would hand them over
    # (computed once, outside every timed region; used by the "with_lse" figures only)
    for L in layers:
        L["lse"] = torch.zeros(len(wl.seq_lens), wl.n_q_heads, w, dtype=torch.float32, device=dev)
        B.slkv_row_lse(params, L["q"], L["k"], cu_dev, cu, L["lse"], ws, status)
    torch.cuda.synchronize()
    use_lse = [bool(args.with_lse)]

    launches_per_step = 0

    def step():
        nonlocal launches_per_step
        n = 0
        # the layers of a step are independent: their calls may overlap on the GPU (selection and gather of one
        # layer beside the score kernels of the next); the join orders the stream after all of them
        call = B.slkv_compress_overlapped if overlap else B.slkv_compress
        for L in layers:
            call(params, L["q"], L["k"], L["v"], cu_dev, cu, L["bud"], L["k_out"], L["v_out"],
                 L["offsets"], L["kept"], ws, None, status, stream, L["lse"] if use_lse[0] else None)
            n += B.slkv_last_launch_count()
        B.slkv_join(stream)
        launches_per_step = n + B.slkv_last_launch_count()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    def timed(n_steps, fn):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        a.record(stream)
        for _ in range(n_steps):
            fn()
        b.record(stream)
        barrier()
        return max_over_ranks(a.elapsed_time(b), dist, dev)

    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "device status word set during warm-up"
    eager_step = step
    eager_us_per_layer = None
    use_graph = overlap and not args.no_graph

    def captured(fn):
        """fn's calls captured once in a CUDA graph (they are stream-ordered and allocate nothing; the side streams
        of the overlapped calls fork from and rejoin the captured stream); returns the replaying step."""
        nonlocal stream
        cap = torch.cuda.Stream()
        stream = cap
        try:
            with torch.cuda.stream(cap):
                fn()
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=cap):
                fn()
        finally:
            stream = torch.cuda.current_stream()
        for _ in range(2):
            graph.replay()
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        return graph.replay

    def lse_eager_step():
        use_lse[0] = True
        try:
            eager_step()
        finally:
            use_lse[0] = bool(args.with_lse)

    lse_step = lse_eager_step
    if use_graph:
        try:
            step = captured(eager_step)
            lse_step = captured(lse_eager_step)
        except Exception as exc:                       # no capture on this driver: issue the calls every step
            print(f"bench: CUDA graph capture failed ({exc}); timing the calls themselves", file=sys.stderr)
            torch.cuda.synchronize()
            B.slkv_join()
            stream = torch.cuda.current_stream()
            step, lse_step = eager_step, lse_eager_step
            use_graph = False
    steps = args.steps
    if steps is None:                                   # aim at ~3 s of timed work
        one = timed(1, step)
        steps = int(min(2000, max(10, 3000.0 / max(one, 1e-3))))

    sampler = ClockSampler(local)
    sampler.start()
    ms_total = timed(steps, step)
    sampler.stop()
    clocks = sampler.summary()
    ms_per_step = ms_total / steps

    if use_graph:
        # the same calls issued every step, right behind the timed run (same clocks and temperature)
        n_eager = max(10, min(steps, 300))
        eager_us_per_layer = timed(n_eager, eager_step) / n_eager * 1e3 / nl
    # ---- attribution, (1): the score kernels alone bracketed by event pairs, everything else where it normally runs
    # (selections and gathers on their side streams): the dominant kernel's time in the regime of the timed step,
    # taken right behind it
    prof_steps = min(max(steps, 10), 50)
    B.slkv_profile_enable(2)
    barrier()
    for _ in range(3):
        eager_step()
    torch.cuda.synchronize()
    B.slkv_profile_collect()
    regime_ms = timed(prof_steps, eager_step) / prof_steps
    score_kernels = B.slkv_profile_collect()
    B.slkv_profile_enable(0)

    # ---- the same step with every layer's row log-sum-exps handed over by the caller (vote pass only); not the headline
    with_lse = None
    if overlap and not args.with_lse:
        torch.cuda.synchronize()
        time.sleep(1.5)                                             # idle, as before the headline's timed steps
        for _ in range(warmup):
            lse_step()
        first = timed(steps, lse_step) / steps                      # as many steps as the headline
        with_lse = {"us_per_layer": first * 1e3 / nl, "value": whole_job_value(world, T, nl, first),
                    "what": "lse_opt of slkv_compress_overlapped = the rows' log-sum-exps (from slkv_row_lse, outside "
                            "the timed region), as a prefill attention kernel that keeps its softmax statistics hands "
                            "them over: the score kernel runs the vote pass alone"}

    # ---- the same steps for at least two more seconds: the figures the part holds once its power limit has engaged
    sustained = None
    if not args.no_sustained:
        n_sus = max(steps, int(math.ceil(2200.0 / max(ms_per_step, 1e-3))))
        sus_sampler = ClockSampler(local)
        sus_sampler.start()
        sus_ms = timed(n_sus, step) / n_sus
        sus_sampler.stop()
        sustained = {"steps": n_sus, "ms_per_step": sus_ms, "us_per_layer": sus_ms * 1e3 / nl,
                     "value": whole_job_value(world, T, nl, sus_ms), "clocks": sus_sampler.summary()}
        if with_lse:
            n_lse = int(math.ceil(1500.0 / max(with_lse["us_per_layer"] * nl * 1e-3, 1e-3)))
            lse_sampler = ClockSampler(local)
            lse_sampler.start()
            held = timed(n_lse, lse_step) / n_lse
            lse_sampler.stop()
            with_lse["sustained_us_per_layer"] = held * 1e3 / nl
            with_lse["sustained_clocks"] = lse_sampler.summary()

    # ---- attribution, (2): every kernel bracketed, on one stream: the other kernels' own times (that step is slower
    # than the timed one); the score kernels' figures stay those of (1)
    B.slkv_profile_enable(1)
    barrier()
    for _ in range(prof_steps):
        eager_step()
    torch.cuda.synchronize()
    per_kernel = B.slkv_profile_collect()
    B.slkv_profile_enable(0)
    for name, v in score_kernels.items():
        per_kernel[name] = v
    assert int(status.item()) == 0

    t_layer_us = ms_per_step * 1e3 / nl
    value = whole_job_value(world, T, nl, ms_per_step)

    # ---- end to end through the host-buffer entry point (pinned host memory, copies in the timed region)
    e2e = None
    if not args.no_e2e:
        cap = max(L["rows"] for L in layers)
        arena = torch.empty(B.slkv_compress_host_arena_bytes(params, cu, cap), dtype=torch.uint8, device=dev)
        n_host = min(nl, args.e2e_layers)
        host = []
        for L in layers[:n_host]:
            host.append({"q": L["q"].cpu().pin_memory(), "k": L["k"].cpu().pin_memory(), "v": L["v"].cpu().pin_memory(),
                         "bud": L["bud"].cpu(), "rows": L["rows"]})
        k_out_h = torch.empty(cap, d, dtype=wl.torch_dtype).pin_memory()
        v_out_h = torch.empty(cap, d, dtype=wl.torch_dtype).pin_memory()
        off_h = torch.empty(len(wl.seq_lens) * hkv + 1, dtype=torch.int32).pin_memory()
        kept_h = torch.empty(cap, dtype=torch.int32).pin_memory()

        def e2e_step():
            for l in range(nl):
                Hh = host[l % n_host]
                B.slkv_compress_host(params, Hh["q"], Hh["k"], Hh["v"], cu, Hh["bud"], k_out_h, v_out_h, off_h,
                                     kept_h, arena, stream)

        e2e_step()
        e2e_steps = max(1, min(steps, args.e2e_steps))
        barrier()
        t0 = time.perf_counter()
        ev_ms = timed(e2e_steps, e2e_step)
        wall_ms = (time.perf_counter() - t0) * 1e3
        e2e_ms = max(ev_ms, 0.0)
        h2d = sum((Hh["q"].numel() + Hh["k"].numel() + Hh["v"].numel()) * e + (len(cu) + hkv) * 4
                  for Hh in (host[l % n_host] for l in range(nl)))
        d2h = sum(host[l % n_host]["rows"] * (2 * d * e + 4) + (len(wl.seq_lens) * hkv + 1) * 4 for l in range(nl))
        e2e = {"value": whole_job_value(world, T, nl, e2e_ms / e2e_steps), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / e2e_steps, "steps": e2e_steps,
               "host_layers_cycled": n_host, "wall_ms": wall_ms,
               "api": "slkv_compress_host (pinned host buffers in, packed rows + offsets + indices out)"}
        del arena

    # ---- roofline of the dominant kernel and of the whole layer
    peaks = measured_peaks()
    n_hist = sum(max(n - w, 0) for n in wl.seq_lens)
    q_bytes = len(wl.seq_lens) * w * wl.n_q_heads * d * e
    k_scan = hkv * n_hist * d * e
    rows_avg = sum(L["rows"] for L in layers) / nl
    alg = {"k_score_fused": k_scan + q_bytes + 4 * hkv * n_hist, "k_score_pipe": k_scan + q_bytes + 4 * hkv * n_hist, "k_score_lse": k_scan + q_bytes, "k_score_vote": k_scan + q_bytes + 4 * hkv * n_hist,
           "k_pool": 8 * hkv * n_hist, "k_select": 4 * hkv * n_hist + 4 * rows_avg,
           "k_gather": 4 * rows_avg * d * e + 4 * rows_avg, "k_setup": 0}
    kern = {}
    prof_total = sum(ms for ms, _ in per_kernel.values()) or 1.0
    for name, (ms, cnt) in per_kernel.items():
        kern[name] = {"launches_per_step": cnt / prof_steps, "avg_us": ms * 1e3 / cnt, "share": ms / prof_total}
    top = max(per_kernel, key=lambda n: per_kernel[n][0])
    top_us = kern[top]["avg_us"]
    # the two-layer score kernel takes a list of layers per launch: a launch's units are those of all its layers
    layers_per_launch = nl / kern[top]["launches_per_step"] if top == "k_score_pipe" else 1.0
    alg_top = alg[top] * layers_per_launch
    achieved = alg_top / (top_us * 1e-6) / 1e9
    layer_bytes = k_scan + q_bytes + 4 * rows_avg * d * e
    passes = 1 if args.with_lse else 2                              # row statistics + votes, or votes alone
    flops_layer = passes * 2.0 * wl.n_q_heads * w * n_hist * d
    exps_layer = float(passes) * wl.n_q_heads * w * n_hist
    f_sm = (clocks["sm_mhz"] or 1965.0) * 1e6
    ceilings = {"t_hbm_us": layer_bytes / (peaks["hbm_gbs"] * 1e9) * 1e6,
                "t_tensor_us": flops_layer / (peaks["bf16_tflops"] * 1e12) * 1e6,
                "t_ex2_us": exps_layer / (148 * 16 * f_sm) * 1e6}
    roofline = {"bound": "hbm", "kernel": top, "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "traffic": None, "peak_source": peaks["source"],
                "alg_bytes_per_launch": alg_top, "layers_per_launch": layers_per_launch, "avg_launch_us": top_us,
                "layer": {"alg_bytes": layer_bytes, "us": t_layer_us,
                          "achieved": layer_bytes / (t_layer_us * 1e-6) / 1e9,
                          "frac": layer_bytes / (t_layer_us * 1e-6) / 1e9 / peaks["hbm_gbs"],
                          "frac_of_8TBs_nominal": layer_bytes / (t_layer_us * 1e-6) / 8e12},
                "ceilings": ceilings}
    # The score kernel's own ceiling is the special-function unit, not HBM: two exponentials per (query row, key)
    # at 16 ex2.approx per clock per SM need longer than streaming K once.  Reported beside the HBM figures.
    if top.startswith("k_score"):
        n_exp = (exps_layer if top in ("k_score_fused", "k_score_pipe") else exps_layer / 2) * layers_per_launch
        peak_gexp = 148 * 16 * 1965e6 / 1e9
        roofline["alu"] = {"bound": "alu", "unit": "Gexp/s", "achieved": n_exp / (top_us * 1e-6) / 1e9, "peak": peak_gexp,
                           "frac": n_exp / (top_us * 1e-6) / 1e9 / peak_gexp, "exps_per_launch": n_exp,
                           "peak_source": "148 SMs x 16 ex2.approx per clock x 1965 MHz (nominal unit count and maximum clock)"}
    tr = dram_traffic_per_key_row(top, "lse" if args.with_lse else "two_pass")
    if tr:
        roofline["traffic"] = tr["bytes"] * hkv * n_hist * layers_per_launch
        roofline["traffic_source"] = tr["source"]
    # the dominant kernel's launches of one step, timed in the step's own regime, must fit inside that step
    roofline["kernel_us_per_step"] = top_us * kern[top]["launches_per_step"]
    roofline["step_us_in_that_regime"] = regime_ms * 1e3
    if top in score_kernels:
        assert roofline["kernel_us_per_step"] <= regime_ms * 1e3 * 1.02, "per-kernel timing exceeds the step it is a share of"
    if sustained:
        sustained["layer_frac_of_hbm"] = layer_bytes / (sustained["us_per_layer"] * 1e-6) / 1e9 / peaks["hbm_gbs"]
    if with_lse:
        lb = layer_bytes + 4 * len(wl.seq_lens) * wl.n_q_heads * w          # + the log-sum-exps read
        with_lse["layer_frac_of_hbm"] = lb / (with_lse["us_per_layer"] * 1e-6) / 1e9 / peaks["hbm_gbs"]
        if "sustained_us_per_layer" in with_lse:
            with_lse["sustained_layer_frac_of_hbm"] = lb / (with_lse["sustained_us_per_layer"] * 1e-6) / 1e9 / peaks["hbm_gbs"]

    # ---- the oracle on the host cores (rank 0, N=1 only): a reported baseline, not a target
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = time_oracle(wl, [(L["q"], L["k"], L["v"], budgets_host[i].tolist()) for i, L in enumerate(layers)],
                                   budget_s=args.cpu_budget_s)

    if rank == 0:
        out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
               "ms_per_step": ms_per_step, "us_per_layer": t_layer_us, "us_per_layer_without_graph": eager_us_per_layer,
               "us_per_layer_with_lse": with_lse["us_per_layer"] if with_lse else None,
               "sustained": sustained, "with_lse": with_lse,
               "higher_is_better": True, "scaling": "weak",
               "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
               "config": {"workload": wl.name, "n_layers": nl, "n_q_heads": wl.n_q_heads, "n_kv_heads": hkv,
                          "head_dim": d, "seq_lens": wl.seq_lens, "window": w, "pool_kernel": wl.pool_kernel,
                          "avg_budget_per_kv_head": total // (nl * hkv), "fixed": wl.fixed,
                          "row_lse": "supplied by the caller (--with-lse)" if args.with_lse else "computed (two passes over K)",
                          "parallelism":
                          f"dp{world} (one sequence batch per GPU, no collective)",
                          "api": ("slkv_compress_overlapped + slkv_join per step" +
                                  (", captured once in a CUDA graph and replayed" if use_graph else ""))
                          if overlap else "slkv_compress",
                          "l2": "inputs larger than L2: every layer has its own Q/K/V (%.1f GB per step)" %
                                (nl * (2 * T * hkv * d * e) / 1e9)},
               "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * steps,
               "gpu_launches_per_step": launches_per_step, "kernels": kern, "roofline": roofline,
               "cpu_baseline": cpu_baseline}
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


# ---------------------------------------------------------------------------------------------------
# the oracle arm
# ---------------------------------------------------------------------------------------------------
def oracle_layer(wl, q, k, v, budgets_row):
    import numpy as np
    from oracle import slkv_oracle as O
    f64 = lambda t: t.cpu().to(torch.float32).numpy().astype(np.float64)
    f32 = lambda t: t.cpu().to(torch.float32).numpy()
    return O.compress(f64(q), f32(k), f32(v), wl.cu_seqlens, budgets_row, wl.window, wl.pool_kernel)


def time_oracle(wl, layer_inputs, budget_s=20.0):
    """Times the oracle, as it stands, on a bounded sample of layers; returns the cpu_baseline object."""
    times = []
    t_begin = time.perf_counter()
    for (q, k, v, bud) in layer_inputs:
        qh, kh, vh = q.cpu(), k.cpu(), v.cpu()
        t0 = time.perf_counter()
        oracle_layer(wl, qh, kh, vh, bud)
        times.append(time.perf_counter() - t0)
        if time.perf_counter() - t_begin > budget_s:
            break
    t_layer = sum(times) / len(times)
    return {"value": wl.total_tokens / t_layer, "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle",
            "host_cores": os.cpu_count(), "s_per_layer": t_layer,
            "sample": f"layers 0..{len(times) - 1} of {wl.name} ({len(times)} of {wl.n_layers} layers, full length, "
                      f"all heads; numpy fp64, BLAS threads = cores)"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    from oracle import slkv_oracle as O
    wl = synth.workloads()[WORKLOAD_INDEX]
    total = wl.totals[TOTAL_INDEX]
    budgets = O.alloc_budgets(synth.inf_sc(wl).numpy(), wl.fixed, total)
    gen_dev = "cuda" if torch.cuda.is_available() else "cpu"
    n_samples = 2
    inputs = []
    for l in range(n_samples):
        x = synth.layer_inputs(wl, l, device=gen_dev)
        inputs.append((x.q_win.cpu(), x.k.cpu(), x.v.cpu(), budgets[l].tolist()))
    warmup, steps = max(args.warmup, 1), (args.steps or 10)
    # one step = the oracle on one layer (a 1/32 sample of the 32-layer step); bounded to a few minutes
    t0 = time.perf_counter()
    oracle_layer(wl, *inputs[0])
    one = time.perf_counter() - t0
    steps = max(1, min(steps, int(150.0 / max(one, 1e-3))))
    warmup = max(1, min(warmup, int(30.0 / max(one, 1e-3))))
    for i in range(warmup):
        oracle_layer(wl, *inputs[i % n_samples])
    t0 = time.perf_counter()
    for i in range(steps):
        oracle_layer(wl, *inputs[i % n_samples])
    t_layer = (time.perf_counter() - t0) / steps
    value = wl.total_tokens / t_layer
    sample = f"one step = one layer of {wl.name} (layers 0,1 alternating; 1/32 of the 32-layer step), full length"
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
           "steps": steps, "warmup": warmup, "ms_per_step": t_layer * 1e3, "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": wl.name, "n_layers": wl.n_layers, "n_q_heads": wl.n_q_heads,
                      "n_kv_heads": wl.n_kv_heads, "head_dim": wl.head_dim, "seq_lens": wl.seq_lens,
                      "window": wl.window, "pool_kernel": wl.pool_kernel,
                      "avg_budget_per_kv_head": total // (wl.n_layers * wl.n_kv_heads), "fixed": wl.fixed},
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle",
                            "sample": sample},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out))


def run_context_parallel(args):
    """`--context-parallel`: ONE long sequence (the 131072-token workload unless --workload says otherwise) with its
    history keys split over the ranks; strong scaling.  The per-rank call sequence and its collectives (NCCL) are
    paper_2508_15806_b200/context_parallel.py's; a step = every layer of the model once.  Not the headline: the
    headline is the default run (independent sequence batches per rank, no collective)."""
    import torch.distributed as dist
    from paper_2508_15806_b200 import binding as B
    from paper_2508_15806_b200 import context_parallel as CP

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29517")
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    comm = CP.DistComm()
    wl = synth.workloads()[(args.workload - 1) if args.workload else 4]
    assert len(wl.seq_lens) == 1, "context parallel splits one sequence"
    total = wl.totals[0]
    budgets = B.slkv_alloc_budgets(synth.inf_sc(wl).to(dev), wl.fixed, total)
    n_distinct = min(args.layers or 4, wl.n_layers)       # distinct layers held; a step cycles through them n_layers times
    shards = []
    for l in range(n_distinct):
        x = synth.layer_inputs(wl, l, device=dev)         # every rank draws the same layer and keeps its own rows
        sh = CP.shard_of(x.q_win, x.k, x.v, wl.window, wl.pool_kernel, rank, world)
        sh.k, sh.v = sh.k.clone(), sh.v.clone()
        shards.append(sh)
        del x
    torch.cuda.empty_cache()

    def step():
        outs = None
        for l in range(wl.n_layers):
            outs = CP.compress_rank(shards[l % n_distinct], budgets[l].contiguous(), wl.pool_kernel, comm)
        return outs

    def barrier():
        torch.cuda.synchronize()
        dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        outs = step()
    torch.cuda.synchronize()
    assert int(outs["status"].item()) == 0
    steps = args.steps or 5
    sampler = ClockSampler(local)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.start()
    a.record()
    for _ in range(steps):
        step()
    b.record()
    barrier()
    sampler.stop()
    ms = max_over_ranks(a.elapsed_time(b), dist, dev) / steps
    if rank == 0:
        print(json.dumps({
            "metric": "context tokens compressed per second per layer", "unit": "tokens/s/layer",
            "value": wl.total_tokens * wl.n_layers / (ms * 1e-3), "n_gpus": world, "steps": steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms, "us_per_layer": ms * 1e3 / wl.n_layers,
            "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": wl.name, "n_layers": wl.n_layers, "seq_lens": wl.seq_lens, "window": wl.window,
                       "parallelism": f"cp{world}: one sequence's history keys split over the ranks; per layer one "
                                      "all-gather of row statistics, three all-reduces of radix histograms, one "
                                      "all-gather of tie counts (NCCL)",
                       "api": "context_parallel.compress_rank (slkv_row_lse, slkv_score, slkv_cp_*)",
                       "l2": f"{n_distinct} distinct layers cycled; a rank's K and V are larger than L2 together"},
            "clocks": sampler.summary(), "e2e": None, "gpu_launches": None, "roofline": None, "cpu_baseline": None}))
    dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--layers", type=int, default=0, help="use fewer layers (profiling captures only)")
    ap.add_argument("--workload", type=int, default=0, choices=[0, 1, 2, 3, 4, 5],
                    help="time another of the five workloads (default: the 32k-context one); the others are parity cases")
    ap.add_argument("--no-graph", action="store_true",
                    help="issue the calls of every step (default: capture a step's calls in a CUDA graph once and replay it)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--kv-head-major", action="store_true",
                    help="store K and V head-major ([n_kv_heads, tokens, head_dim]) instead of token-major; not the headline")
    ap.add_argument("--with-lse", action="store_true",
                    help="hand every layer's row log-sum-exps to the calls (vote pass only); not the headline")
    ap.add_argument("--no-overlap", action="store_true", help="one layer at a time (slkv_compress) instead of overlapped calls")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sustained", action="store_true", help="skip the two extra seconds of the same step")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--e2e-layers", type=int, default=8, help="distinct layers kept in pinned host memory")
    ap.add_argument("--cpu-budget-s", type=float, default=20.0)
    ap.add_argument("--context-parallel", action="store_true",
                    help="split ONE long sequence's keys over the ranks (strong scaling, NCCL collectives); not the headline")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.context_parallel:
        run_context_parallel(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
