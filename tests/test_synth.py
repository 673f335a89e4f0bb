"""The seeded input generators: reproducible, device-independent definition, right shapes and structure."""
import math

import torch

from paper_2508_15806_b200 import synth


def test_mix_matches_python_reference():
    key = synth.stream_key(7, synth.TID_K, 3)
    idx = torch.arange(0, 64, dtype=torch.int64)
    got = synth._bits(key, idx, 1).tolist()
    for i, g in enumerate(got):
        ref = synth.mix_int(((2 * i + 1) * 0x9E3779B97F4A7C15 + key) & ((1 << 64) - 1))
        assert (g & ((1 << 64) - 1)) == ref


def test_uniform_and_normal_moments_and_chunking():
    key = synth.stream_key(1, synth.TID_Q)
    u = synth.uniform(key, 200000)
    assert 0.0 < float(u.min()) and float(u.max()) < 1.0 and abs(float(u.mean()) - 0.5) < 5e-3
    n = synth.normal(key, 200000)
    assert abs(float(n.mean())) < 1e-2 and abs(float(n.std()) - 1.0) < 1e-2
    assert torch.equal(synth.normal(key, 1000, chunk=64), n[:1000])
    assert torch.equal(synth.normal(key, 10, start=500), n[500:510])


def test_workloads_shapes():
    wls = synth.workloads()
    assert [w.total_tokens for w in wls[:3]] == [1024, 8192, 32768] and wls[4].total_tokens == 131072
    c4 = wls[3]
    assert len(c4.seq_lens) == 8 and all(4096 <= n <= 32768 for n in c4.seq_lens)
    assert c4.seq_lens == synth.workloads()[3].seq_lens
    for w in wls:
        inf = synth.inf_sc(w)
        assert inf.shape == (w.n_layers, w.n_kv_heads) and inf.dtype == torch.float32
        assert bool((inf >= 0).all()) and bool(torch.isfinite(inf).all())
    inf3 = synth.inf_sc(wls[2])
    assert float(inf3[1, :3].max()) <= 1e-6
    inf5 = synth.inf_sc(wls[4])
    assert int((inf5 == 1.0).sum()) >= 5


def test_layer_inputs_structure():
    wl = synth.small_variant(synth.workloads()[1], [600, 300])
    x = synth.layer_inputs(wl, 0)
    T = 900
    assert x.k.shape == (T, 8, 128) and x.v.shape == (T, 8, 128) and x.q_win.shape == (2, 32, 32, 128)
    assert x.k.dtype == torch.bfloat16
    y = synth.layer_inputs(wl, 0)
    assert torch.equal(x.k, y.k) and torch.equal(x.q_win, y.q_win)
    assert not torch.equal(x.k, synth.layer_inputs(wl, 1).k)
    # needles: > pool_kernel apart, inside the history, logit boost ~ needle_logit
    for s, pos in enumerate(x.needles):
        n_hist = wl.seq_lens[s] - wl.window
        assert len(pos) > 0 and all(0 <= p < n_hist for p in pos)
        assert all(b - a > wl.pool_kernel for a, b in zip(pos, pos[1:]))
        p = pos[0] + wl.cu_seqlens[s]
        logit = (x.q_win[s, 0, 0].double() @ x.k[p, 0].double()) / math.sqrt(128)
        assert 4.0 < float(logit) < 14.0
