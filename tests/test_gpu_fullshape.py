"""Parity at the benchmark's full layer shape and launch configuration (``-m gpu``).

32 query / 8 KV heads, d = 128, B = 2048, batch 32, several layers in one context, decode steps
replayed from a CUDA graph with the side streams on - exactly how bench.py drives the library.  The
CPU oracle follows two sampled (layer, sequence) units through the same inputs (it cannot afford all
64); for the other units properties that hold at any size are checked: entry count, sinks, distinct
positions, evicted count, finite outputs.
"""
import numpy as np
import pytest
import torch

from oracle import indexmem_oracle as orc
from paper_2605_25475_b200 import synth

pytestmark = pytest.mark.gpu


def test_stack_shape_sampled_units_under_graph_replay():
    from paper_2605_25475_b200 import binding as im
    from tests.parity import bf16_ulp
    wl = synth.CONFIGS["llama8b_stack"].replace(name="stack_sampled", n_layers=2, ctx=4096)
    dev = torch.device("cuda:0")
    g = im.IndexMem(im.Config(n_layers=wl.n_layers, max_seqs=wl.n_seq, n_q_heads=wl.H, n_kv_heads=wl.Hkv,
                              head_dim=wl.d, budget=wl.B, max_chunk=wl.chunk, n_sink=wl.n_sink), dev)
    ids = list(range(wl.n_seq))
    sampled = [(0, 5), (1, 29)]
    oracles = {}
    for layer in range(wl.n_layers):
        w = synth.make_weights(wl, layer)
        g.set_weights(layer, w)
        for (l, s) in sampled:
            if l == layer:
                o = orc.OracleLayer(orc.OracleConfig(H=wl.H, Hkv=wl.Hkv, d=wl.d, B=wl.B, n_sink=wl.n_sink), 1)
                o.set_weights({k: synth.f32(v) for k, v in w.items()})
                oracles[(l, s)] = o
    for c in range(wl.ctx // wl.chunk):
        for layer in range(wl.n_layers):
            X, Q, K, V = synth.prefill_inputs(wl, layer, c)
            g.prefill_chunk(layer, ids, X.to(dev), Q.to(dev), K.to(dev), V.to(dev))
            for (l, s), o in oracles.items():
                if l == layer:
                    o.prefill_chunk(0, synth.f32(X[s]), synth.f32(Q[s]), synth.f32(K[s]), synth.f32(V[s]))
    assert g.status() == 0
    for (l, s), o in oracles.items():
        assert sorted(g.export(l, s, im.IM_S_POS).tolist()) == o.positions(0).tolist()

    # decode: static input buffers, one captured step, replayed (bench.py's launch configuration)
    n_steps = 4
    ins = [[synth.decode_inputs(wl, layer, st) for layer in range(wl.n_layers)] for st in range(n_steps)]
    sx = torch.empty((wl.n_layers, wl.n_seq, wl.D), dtype=torch.bfloat16, device=dev)
    sq = torch.empty((wl.n_layers, wl.n_seq, wl.H, wl.d), dtype=torch.bfloat16, device=dev)
    sk = torch.empty((wl.n_layers, wl.n_seq, wl.Hkv, wl.d), dtype=torch.bfloat16, device=dev)
    sv = torch.empty_like(sk)
    out = torch.empty((wl.n_layers, wl.n_seq, wl.H, wl.d), dtype=torch.bfloat16, device=dev)

    def load(st):
        for layer in range(wl.n_layers):
            x, q, k, v = ins[st][layer]
            sx[layer].copy_(x); sq[layer].copy_(q); sk[layer].copy_(k); sv[layer].copy_(v)

    def one_step():
        for layer in range(wl.n_layers):
            g.decode_step(layer, ids, sx[layer], sq[layer], sq[layer], sk[layer], sv[layer], out[layer])

    stream = torch.cuda.Stream(dev)
    with torch.cuda.stream(stream):
        load(0)
        one_step()                      # eager first step: reaches n = B
        stream.synchronize()
        results = [out.float().cpu().numpy().copy()]
        graph = torch.cuda.CUDAGraph()
        load(1)
        with torch.cuda.graph(graph, stream=stream):
            one_step()
        for st in range(1, n_steps):
            load(st)
            graph.replay()
            stream.synchronize()
            results.append(out.float().cpu().numpy().copy())
    assert g.status() == 0

    # oracle on the sampled units
    for (l, s), o in oracles.items():
        for st in range(n_steps):
            x, q, k, v = ins[st][l]
            ob, od = o.decode_step(0, synth.f32(x[s]), synth.f32(q[s]), synth.f32(q[s]), synth.f32(k[s]), synth.f32(v[s]))
            got = results[st][l, s].astype(np.float64)
            scale = np.abs(od).max()
            half_ulp = 0.5 * bf16_ulp(np.maximum(np.abs(od), np.abs(got)))
            assert np.all(np.abs(got - od) <= 2e-3 * scale + half_ulp), f"unit {(l, s)} step {st}"
        assert sorted(g.export(l, s, im.IM_S_POS).tolist()) == o.positions(0).tolist()
        Mo, bo = o.memory_kv(0)
        Mg = g.export(l, s, im.IM_S_M).astype(np.float64)
        assert np.abs(Mg - Mo).max() <= 2e-3 * np.abs(Mo).max()
        assert np.abs(g.export(l, s, im.IM_S_B) - bo).max() <= 2e-3 * np.abs(bo).max()

    # properties for every unit
    for layer in range(wl.n_layers):
        for s in range(0, wl.n_seq, 7):
            cnt = g.counts(layer, s)
            assert cnt["n"] == wl.B and cnt["T"] == wl.ctx + n_steps and cnt["n_evicted"] == 1
            pos = g.export(layer, s, im.IM_S_POS)
            assert len(set(pos.tolist())) == wl.B and set(range(wl.n_sink)) <= set(pos.tolist())
            assert pos.max() < wl.ctx + n_steps
    assert np.isfinite(results[-1]).all()


def test_stack_shape_long_interval_one_graph_per_phase():
    """The benchmark's layer shape with a compression interval of 32 (`bench.py --tau`): one CUDA graph per phase of
    the interval, captured in order and replayed in order with the inputs in place.  31 phases append and attend
    over B + p entries; the last one selects 32 entries per sequence (more than the fused front kernel or the
    pending list hold), writes Phi^T V of all 32 sequences with one batched tensor-core launch and compacts.  Two
    sampled units follow the oracle through a whole eager interval and 34 replayed steps."""
    from paper_2605_25475_b200 import binding as im
    from tests.parity import bf16_ulp
    tau = 32
    wl = synth.CONFIGS["llama8b_stack"].replace(name="stack_tau", n_layers=2, ctx=4096, tau=tau)
    dev = torch.device("cuda:0")
    g = im.IndexMem(im.Config(n_layers=wl.n_layers, max_seqs=wl.n_seq, n_q_heads=wl.H, n_kv_heads=wl.Hkv,
                              head_dim=wl.d, budget=wl.B, compress_interval=tau, max_chunk=wl.chunk,
                              n_sink=wl.n_sink), dev)
    ids = list(range(wl.n_seq))
    sampled = [(0, 11), (1, 30)]
    oracles = {}
    for layer in range(wl.n_layers):
        w = synth.make_weights(wl, layer)
        g.set_weights(layer, w)
        for (l, s) in sampled:
            if l == layer:
                o = orc.OracleLayer(orc.OracleConfig(H=wl.H, Hkv=wl.Hkv, d=wl.d, B=wl.B, tau=tau, n_sink=wl.n_sink), 1)
                o.set_weights({k: synth.f32(v) for k, v in w.items()})
                oracles[(l, s)] = o
    for c in range(wl.ctx // wl.chunk):
        for layer in range(wl.n_layers):
            X, Q, K, V = synth.prefill_inputs(wl, layer, c)
            g.prefill_chunk(layer, ids, X.to(dev), Q.to(dev), K.to(dev), V.to(dev))
            for (l, s), o in oracles.items():
                if l == layer:
                    o.prefill_chunk(0, synth.f32(X[s]), synth.f32(Q[s]), synth.f32(K[s]), synth.f32(V[s]))
    assert g.status() == 0

    n_eager, n_replay = tau, tau + 2
    n_steps = n_eager + n_replay
    n_in = 4                                                     # input sets, cycled (tau is a multiple)
    ins = [[synth.decode_inputs(wl, layer, st) for layer in range(wl.n_layers)] for st in range(n_in)]
    dins = [[tuple(t.to(dev) for t in ins[k][layer]) for layer in range(wl.n_layers)] for k in range(n_in)]
    out = torch.empty((wl.n_layers, wl.n_seq, wl.H, wl.d), dtype=torch.bfloat16, device=dev)

    def one_step(k):
        for layer in range(wl.n_layers):
            x, q, kk, v = dins[k % n_in][layer]
            g.decode_step(layer, ids, x, q, q, kk, v, out[layer])

    results = []
    stream = torch.cuda.Stream(dev)
    with torch.cuda.stream(stream):
        for st in range(n_eager):                                # a whole interval eagerly: phase 0 again
            one_step(st)
            stream.synchronize()
            results.append(out.float().cpu().numpy().copy())
        graphs = []
        for ph in range(tau):                                    # tau is a multiple of n_in: graph ph reads set ph % n_in
            gk = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gk, stream=stream):
                one_step(ph)
            graphs.append(gk)
        for st in range(n_replay):
            graphs[st % tau].replay()
            stream.synchronize()
            results.append(out.float().cpu().numpy().copy())
    assert g.status() == 0

    for (l, s), o in oracles.items():
        for st in range(n_steps):
            x, q, k, v = ins[(st if st < n_eager else st - n_eager) % n_in][l]
            ob, od = o.decode_step(0, synth.f32(x[s]), synth.f32(q[s]), synth.f32(q[s]), synth.f32(k[s]), synth.f32(v[s]))
            got = results[st][l, s].astype(np.float64)
            scale = np.abs(od).max()
            half_ulp = 0.5 * bf16_ulp(np.maximum(np.abs(od), np.abs(got)))
            assert np.all(np.abs(got - od) <= 2e-3 * scale + half_ulp), f"unit {(l, s)} step {st}"
        assert o.evict_steps(0) == 1 + 2                         # the second prefill chunk, two full intervals
        assert sorted(g.export(l, s, im.IM_S_POS).tolist()) == o.positions(0).tolist()
        Mo, bo = o.memory_kv(0)
        Mg = g.export(l, s, im.IM_S_M).astype(np.float64)
        assert np.abs(Mg - Mo).max() <= 2e-3 * np.abs(Mo).max()
        assert np.abs(g.export(l, s, im.IM_S_B) - bo).max() <= 2e-3 * np.abs(bo).max()
    for layer in range(wl.n_layers):
        for s in range(0, wl.n_seq, 7):
            cnt = g.counts(layer, s)
            assert cnt["n"] == wl.B + 2 and cnt["T"] == wl.ctx + n_steps
            pos = g.export(layer, s, im.IM_S_POS)
            assert len(set(pos.tolist())) == wl.B + 2 and set(range(wl.n_sink)) <= set(pos.tolist())


def test_llama8b_b1_configuration_at_full_size():
    """The Llama-3-8B-shaped single-sequence configuration as stated: 32 q / 8 KV heads, d 128, a 4096-token
    context ingested in one chunk (3584 evictions in one evict step: the tensor-core scoring, selection,
    phi and Phi^T V kernels at their full sizes), budget 512, lognormal key norms, 256 decode steps; every
    state and every output checked against the oracle."""
    from tests.parity import Pair
    wl = synth.CONFIGS["llama8b_b1"]
    p = Pair(wl)
    p.prefill(0)
    for s in range(wl.steps):
        p.decode(s)
    st = p.stats
    assert st["steps"] == 256 and st["kidx_flips"] == 0
    assert st["max_out_err"] <= 2e-3 and st["max_M_err"] <= 2e-3 and st["max_score_err"] <= 1e-5
    assert st["cut_divergences"] <= 4


def test_mistral_prefill_chunks_at_full_chunk_size():
    """The Mistral-shaped chunked prefill at its stated chunk size and budget (2048 / 2048), prompt cut to three
    chunks so that the oracle finishes in half a minute: the second and third chunk score 4096 cached keys
    against 2048 queries (tcgen05 scoring GEMM at its benchmark size), evict 2048 entries each and write
    them to the memory through the tensor-core GEMMs; selection, cached keys and memory against the oracle."""
    from tests.parity import Pair
    wl = synth.CONFIGS["mistral7b_prefill"].replace(name="mistral_full_chunk", ctx=3 * 2048, steps=2)
    p = Pair(wl)
    for c in range(3):
        p.prefill(c)
    assert p.o.evict_steps(0) == 2 and p.g.counts(0, 0)["n"] == 2048
    for s in range(wl.steps):
        p.decode(s)
    st = p.stats
    assert st["kidx_flips"] == 0 and st["max_M_err"] <= 2e-3 and st["max_score_err"] <= 1e-5 and st["max_out_err"] <= 2e-3


def test_qwen_shape_one_shot_compression_of_a_long_context():
    """Qwen2.5-7B shape (28 q / 4 KV heads, 7 indexer heads, d_M 448) with the one-shot compression of the
    stated configuration at half its context (8192 tokens -> B = 1024 in a single evict step of 7168 entries,
    two of the eight sequences, 64 needles each; the oracle needs about a minute for the full 16384), then
    decode steps."""
    from tests.parity import Pair
    wl = synth.CONFIGS["qwen7b_b8"].replace(name="qwen_oneshot", n_seq=2, ctx=8192, chunk=8192, steps=8)
    p = Pair(wl)
    p.prefill(0)
    assert p.g.counts(0, 1)["n"] == 1024 and p.g.counts(0, 1)["n_evicted"] == 7168
    for s in range(wl.steps):
        p.decode(s)
    st = p.stats
    assert st["kidx_flips"] == 0 and st["max_M_err"] <= 2e-3 and st["max_score_err"] <= 1e-5 and st["max_out_err"] <= 2e-3
