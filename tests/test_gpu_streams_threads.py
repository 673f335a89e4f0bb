"""GPU: slkv_compress_overlapped from two host threads and on several streams (Algorithm 3, same results).

Calls made on different streams keep separate queues, slots and events inside the library; a join orders its stream
behind every call made so far and forgets only the calls of its own stream.  Every case is compared bit for bit with
slkv_compress, one call at a time.
"""
import threading

import pytest
import torch

from oracle import slkv_oracle as O
from paper_2508_15806_b200 import binding as B
from paper_2508_15806_b200 import synth

pytestmark = pytest.mark.gpu

DEV = torch.device("cuda:0")


class Job:
    """One stream's share of the work: its own layers, outputs and workspace."""

    def __init__(self, seq_lens, n_layers, avg_budget, seed_shift, with_lse=False):
        base = synth.workloads()[2]
        wl = synth.small_variant(base, seq_lens, n_layers=n_layers, totals=[n_layers * 8 * avg_budget])
        self.wl, self.cu = wl, wl.cu_seqlens
        budgets = O.alloc_budgets(synth.inf_sc(wl).numpy(), wl.fixed, wl.totals[0])
        self.xs = [synth.layer_inputs(wl, (l + seed_shift) % base.n_layers, device=DEV) for l in range(n_layers)]
        self.buds = [torch.tensor(budgets[l].tolist(), dtype=torch.int32, device=DEV) for l in range(n_layers)]
        self.params = B.make_params(self.xs[0].q_win, self.xs[0].k, self.xs[0].v, wl.window, wl.pool_kernel)
        self.cu_dev = torch.tensor(self.cu, dtype=torch.int32, device=DEV)
        self.cap = B.slkv_packed_rows_upper_bound(self.params, self.cu)
        self.n_seg = (len(self.cu) - 1) * wl.n_kv_heads
        self.ws = torch.empty(B.slkv_workspace_bytes_overlapped(self.params, self.cu), dtype=torch.uint8, device=DEV)
        self.lses = None
        if with_lse:
            self.lses = []
            for x in self.xs:
                o = torch.empty(len(seq_lens), wl.n_q_heads, wl.window, dtype=torch.float32, device=DEV)
                B.slkv_row_lse(self.params, x.q_win, x.k, self.cu_dev, self.cu, o, self.ws)
                self.lses.append(o)
            torch.cuda.synchronize()

    def outputs(self):
        return [dict(k=torch.zeros(self.cap, 128, dtype=torch.bfloat16, device=DEV),
                     v=torch.zeros(self.cap, 128, dtype=torch.bfloat16, device=DEV),
                     off=torch.full((self.n_seg + 1,), -1, dtype=torch.int32, device=DEV),
                     kept=torch.full((self.cap,), -1, dtype=torch.int32, device=DEV),
                     status=torch.zeros(1, dtype=torch.int32, device=DEV)) for _ in self.xs]

    def call(self, fn, l, o, stream):
        x = self.xs[l]
        fn(self.params, x.q_win, x.k, x.v, self.cu_dev, self.cu, self.buds[l], o["k"], o["v"], o["off"], o["kept"],
           self.ws, None, o["status"], stream, lse=None if self.lses is None else self.lses[l])

    def reference(self):
        outs = self.outputs()
        for l in range(len(self.xs)):
            self.call(B.slkv_compress, l, outs[l], None)
        torch.cuda.synchronize()
        return outs

    def assert_equal(self, got, ref):
        for g, r in zip(got, ref):
            n = int(r["off"][-1].item())
            assert int(g["status"].item()) == 0 and torch.equal(g["off"], r["off"])
            assert torch.equal(g["kept"][:n], r["kept"][:n])
            assert torch.equal(g["k"][:n], r["k"][:n]) and torch.equal(g["v"][:n], r["v"][:n])


def test_two_host_threads_each_on_its_own_stream():
    # 21 and 13 layers of different shapes (more than a list, more than the slots of a workspace), three times each,
    # the two threads free-running against each other; one of them hands its layers' log-sum-exps over
    jobs = [Job([6000], 21, 300, 0), Job([2500, 1200], 13, 200, 5, with_lse=True)]
    refs = [j.reference() for j in jobs]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    results = [[], []]
    errors = []

    def worker(t):
        try:
            torch.cuda.set_device(0)
            job, st = jobs[t], streams[t]
            for _ in range(3):
                with torch.cuda.stream(st):
                    outs = job.outputs()               # allocated and cleared on this thread's stream
                    for l in range(len(job.xs)):
                        job.call(B.slkv_compress_overlapped, l, outs[l], st)
                    B.slkv_join(st)
                st.synchronize()                       # this thread's own stream only
                results[t].append(outs)
        except Exception as e:                          # noqa: BLE001 - reported below, in the main thread
            errors.append(e)

    torch.cuda.synchronize()
    threads = [threading.Thread(target=worker, args=(t,)) for t in range(2)]
    for th in threads:
        th.start()
    for th in threads:
        th.join(timeout=300)
    assert not errors, errors
    assert all(not th.is_alive() for th in threads)
    torch.cuda.synchronize()
    for t in range(2):
        assert len(results[t]) == 3
        for outs in results[t]:
            jobs[t].assert_equal(outs, refs[t])


def test_one_thread_interleaving_two_streams():
    # calls alternate between two streams with a workspace each; either stream's join orders only what the test
    # then reads on that stream
    jobs = [Job([4000], 11, 256, 1), Job([1800, 700, 300], 10, 128, 3)]
    refs = [j.reference() for j in jobs]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    outs = [j.outputs() for j in jobs]
    torch.cuda.synchronize()
    for l in range(11):
        for t in range(2):
            if l < len(jobs[t].xs):
                jobs[t].call(B.slkv_compress_overlapped, l, outs[t][l], streams[t])
    B.slkv_join(streams[1])
    streams[1].synchronize()
    jobs[1].assert_equal(outs[1], refs[1])             # stream 1's results are complete behind its join
    B.slkv_join(streams[0])                            # ... and stream 0's join still covers stream 0's calls
    streams[0].synchronize()
    jobs[0].assert_equal(outs[0], refs[0])


def test_join_on_another_stream_and_a_shared_workspace():
    # (1) a join on a third stream orders that stream behind calls made elsewhere; (2) two streams that share one
    # workspace are serialised by the library (the later call waits for what the other stream has in flight)
    job = Job([3000, 1000], 12, 200, 2)
    ref = job.reference()
    s1, s2, s3 = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    outs = job.outputs()
    torch.cuda.synchronize()
    for l in range(12):
        job.call(B.slkv_compress_overlapped, l, outs[l], s1)
    B.slkv_join(s3)
    s3.synchronize()
    job.assert_equal(outs, ref)
    B.slkv_join(s1)
    outs = job.outputs()
    torch.cuda.synchronize()
    for l in range(12):
        job.call(B.slkv_compress_overlapped, l, outs[l], s1 if l % 3 else s2)       # one workspace, two streams
    B.slkv_join(s1)
    B.slkv_join(s2)
    torch.cuda.synchronize()
    job.assert_equal(outs, ref)


def test_more_streams_than_the_library_keeps_states_for():
    # ten streams in turn: the library keeps eight per device and hands the one used longest ago to a new stream
    job = Job([2000], 3, 150, 4)
    ref = job.reference()
    streams = [torch.cuda.Stream() for _ in range(10)]
    for st in streams:                                 # first sweep over the streams: every stream joins for itself
        outs = job.outputs()
        torch.cuda.synchronize()
        for l in range(3):
            job.call(B.slkv_compress_overlapped, l, outs[l], st)
        B.slkv_join(st)
        torch.cuda.synchronize()
        job.assert_equal(outs, ref)
    alive = []
    for st in streams:                                 # second sweep: left in flight; the library drains the state it
        outs = job.outputs()                           # hands on, and the last join covers the rest
        torch.cuda.synchronize()
        for l in range(3):
            job.call(B.slkv_compress_overlapped, l, outs[l], st)
        alive.append(outs)
    B.slkv_join(None)
    torch.cuda.synchronize()
    for outs in alive:
        job.assert_equal(outs, ref)
