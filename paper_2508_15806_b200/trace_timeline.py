"""Timeline of one step of overlapped calls, from the library's tracing hook (slkv_trace_set_buffer).

    python -m paper_2508_15806_b200.trace_timeline [--layers 32] [--replays 300]

Builds the 32k-context workload, captures one step (a call per layer + a join) in a CUDA graph with a trace buffer
per score launch, replays it until the clocks have settled and prints, per launch of the two-stream score kernel:
when its CTAs started, when the first accumulator of pass 1 was ready, when the two streams and the CTAs finished
(nanoseconds from the first CTA's start), and the SM clock the launch ran at (SM cycle counter / nanosecond timer).
"""
from __future__ import annotations

import argparse

import numpy as np
import torch

from . import binding as B
from . import synth

SLOTS = 64          # trace words per CTA (see kTraceSlots in csrc/slkv_tc_device.cuh)
LIST = 8            # layers per launch of the score kernel (kPipeMaxLayers)


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--replays", type=int, default=300)
    args = ap.parse_args()
    dev = torch.device("cuda:0")
    nl = args.layers
    wl = synth.workloads()[2]
    wl = synth.small_variant(wl, wl.seq_lens, n_layers=nl, totals=[t // wl.n_layers * nl for t in wl.totals])
    budgets = B.slkv_alloc_budgets(synth.inf_sc(wl).to(dev), wl.fixed, wl.totals[1])
    buds = [budgets[l].contiguous() for l in range(nl)]
    cu = wl.cu_seqlens
    cu_dev = torch.tensor(cu, dtype=torch.int32, device=dev)
    xs = [synth.layer_inputs(wl, l, device=dev) for l in range(nl)]
    params = B.make_params(xs[0].q_win, xs[0].k, xs[0].v, wl.window, wl.pool_kernel)
    ws = torch.empty(B.slkv_workspace_bytes_overlapped(params, cu), dtype=torch.uint8, device=dev)
    rows = B.slkv_packed_rows_upper_bound(params, cu)
    n_seg = len(wl.seq_lens) * wl.n_kv_heads
    outs = [dict(k=torch.empty(rows, wl.head_dim, dtype=xs[0].k.dtype, device=dev),
                 v=torch.empty(rows, wl.head_dim, dtype=xs[0].k.dtype, device=dev),
                 o=torch.empty(n_seg + 1, dtype=torch.int32, device=dev),
                 i=torch.empty(rows, dtype=torch.int32, device=dev)) for _ in range(nl)]
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    n_sm = torch.cuda.get_device_properties(0).multi_processor_count
    n_launches = (nl + LIST - 1) // LIST
    traces = [torch.zeros(2 * n_sm * SLOTS, dtype=torch.int64, device=dev) for _ in range(n_launches)]

    def step(stream):
        for l in range(nl):
            # launch k goes out during call LIST * (k + 1) (the list is full and one more layer has come), the last
            # one at the join; the launcher takes the trace buffer that is set at that moment
            if l == 0 or (l > 1 and l % LIST == 1):
                B.slkv_trace_set_buffer(traces[(l - 1) // LIST if l else 0])
            B.slkv_compress_overlapped(params, xs[l].q_win, xs[l].k, xs[l].v, cu_dev, cu, buds[l], outs[l]["k"],
                                       outs[l]["v"], outs[l]["o"], outs[l]["i"], ws, None, status, stream)
        B.slkv_join(stream)

    cap = torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(cap):
        step(cap)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=cap):
        step(cap)
    B.slkv_trace_set_buffer(None)
    for _ in range(args.replays):
        graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(100):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    print(f"{wl.name}: {nl} layers per step, {e0.elapsed_time(e1) * 10:.1f} us per step (graph replay)")

    t_first = None
    for i, tr in enumerate(traces):
        f = tr.cpu().numpy()
        n_cta = int((f[0:n_sm * SLOTS:SLOTS] > 0).sum())
        if n_cta == 0:
            continue
        t = f[:n_cta * SLOTS].reshape(n_cta, SLOTS).astype(np.int64)
        if t_first is None:
            t_first = t[:, 0].min()
        rel = lambda col: t[:, col] - t_first
        clock = np.median((t[:, 61] - t[:, 60]) / np.maximum(t[:, 4] - t[:, 0], 1))
        print(f"launch {i}: {n_cta} CTAs start {rel(0).min()}..{rel(0).max()}  first accumulator (pass 1) "
              f"{np.median(rel(2)):.0f}  pass 1 done {np.median(rel(5)):.0f}  pass 2 done {np.median(rel(6)):.0f}  "
              f"CTA end median {np.median(rel(4)):.0f} max {rel(4).max()}  SM clock {clock:.3f} GHz")
    assert int(status.item()) == 0


if __name__ == "__main__":
    main()
