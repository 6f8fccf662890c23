"""im_decode_stack (one decode token for several layers in one call, layers overlapping) against the oracle and
against im_decode_step (``-m gpu``).

The call promises the results of layer-by-layer im_decode_step calls.  Its pipelined schedule keeps three layers
in flight on scratch sets and streams of their own, with the streaming kernels' blocks claiming their work by SM
id; a hazard between layers (a scratch buffer reused too early, a worker id claimed twice or never) would show as
a difference from the layer-by-layer run, which uses neither.  So besides the oracle comparison of sampled units
the outputs and the exported state of EVERY unit are compared bit for bit with a twin context driven by
im_decode_step on the same inputs.
"""
import numpy as np
import pytest
import torch

from paper_2605_25475_b200 import synth
from tests.test_gpu_fullshape import SampledUnits, _decode_under_graph_replay

pytestmark = pytest.mark.gpu


def _stack(**kw):
    base = dict(n_layers=7, n_seq=6, ctx=1024, chunk=512, B=512, steps=12)
    base.update(kw)
    return synth.CONFIGS["llama8b_stack"].replace(name="stack_small", **base)


def _twin(wl, **over):
    """Two contexts with the same weights and the same ingested context."""
    from paper_2605_25475_b200 import binding as im
    dev = torch.device("cuda:0")
    cfg = dict(n_layers=wl.n_layers, max_seqs=wl.n_seq, n_q_heads=wl.H, n_kv_heads=wl.Hkv, head_dim=wl.d, budget=wl.B,
               compress_interval=wl.tau, max_chunk=wl.chunk, n_sink=wl.n_sink)
    bulk = over.pop("bulk_readout", False)
    cfg.update(over)
    gs = [im.IndexMem(im.Config(**cfg), dev) for _ in range(2)]
    # (one run per warp: the attention kernel then cuts its tiles exactly as im_decode_step's does, and every sum is
    # formed in the same order)
    im.im_set_option(gs[1].ctx, im.IM_OPT_STACK_CHUNKS, 1)
    # (and phi(q)^T Mhat by the plain-load kernel in both: the bulk-copy kernel a stack call would take cuts the rows
    # into per-block partial vectors, as many as there are blocks)
    for g in gs:
        im.im_set_option(g.ctx, im.IM_OPT_READOUT_STAGES, 2 if bulk else 0)
    ids = list(range(wl.n_seq))
    for layer in range(wl.n_layers):
        w = synth.make_weights(wl, layer)
        for g in gs:
            g.set_weights(layer, w)
    for c in range(wl.ctx // wl.chunk):
        for layer in range(wl.n_layers):
            X, Qp, _, K, V = synth.prefill_inputs(wl, layer, c, dev)
            for g in gs:
                g.prefill_chunk(layer, ids, X, Qp, K, V)
    return im, gs, ids, dev


def _step_inputs(wl, st, dev):
    parts = [synth.decode_inputs(wl, layer, st, dev) for layer in range(wl.n_layers)]
    return tuple(torch.stack([p[i] for p in parts]).contiguous() for i in range(5))


def _same_state(im, a, b, wl, what):
    for layer in range(wl.n_layers):
        for s in range(wl.n_seq):
            assert a.counts(layer, s) == b.counts(layer, s), f"{what}: counters of unit {(layer, s)}"
            for piece in (im.IM_S_POS, im.IM_S_IMP, im.IM_S_KIDX, im.IM_S_K, im.IM_S_V, im.IM_S_M, im.IM_S_B):
                assert np.array_equal(a.export(layer, s, piece), b.export(layer, s, piece)), \
                    f"{what}: piece {piece} of unit {(layer, s)} differs"


@pytest.mark.parametrize("tau", [1, 5])
def test_stack_call_equals_layer_calls_bit_for_bit(tau):
    """Eager calls: all layers in one call (and a call over a subset of the layers in another order) leave the outputs
    and the whole state of every unit exactly as im_decode_step does, through evict steps, plain steps (tau = 5) and
    folds of the pending list (four entries)."""
    wl = _stack(tau=tau, steps=14)
    im, (ga, gb), ids, dev = _twin(wl, pending_slots=4)
    L = wl.n_layers
    layers = list(range(L))
    for st in range(wl.steps):
        x, qp, q, k, v = _step_inputs(wl, st, dev)
        ref = torch.stack([ga.decode_step(l, ids, x[l], qp[l], q[l], k[l], v[l]) for l in layers])
        if st % 3 == 2:      # two calls over disjoint subsets, the first in descending order
            order = layers[::-1][: L // 2]
            rest = [l for l in layers if l not in order]
            got = torch.empty_like(ref)
            for sub in (order, rest):
                o = gb.decode_stack(sub, ids, [x[l] for l in sub], [qp[l] for l in sub], [q[l] for l in sub],
                                    [k[l] for l in sub], [v[l] for l in sub])
                for j, l in enumerate(sub):
                    got[l] = o[j]
        else:
            got = gb.decode_stack(layers, ids, x, qp, q, k, v)
        torch.cuda.synchronize()
        assert ga.status() == 0 and gb.status() == 0
        assert torch.equal(ref, got), f"step {st}: outputs differ in {int((ref != got).sum())} elements"
        if st % 4 == 3 or st == wl.steps - 1:
            _same_state(im, ga, gb, wl, f"step {st}")
    ga.close(); gb.close()


def test_stack_call_with_events_takes_inputs_and_hands_out_outputs_layer_by_layer():
    """im_decode_stack_events: every layer's inputs are copied from pinned host memory on a copy stream of the test's
    while the call is being made and runs, one event per layer telling the call when they are complete, and every
    layer's output is copied back on a third stream behind the call's event for that layer.  Outputs on the host and
    the state of every unit equal those of im_decode_step calls on resident inputs, bit for bit, through evict steps
    (the device buffers are overwritten with a poison value before every step: a kernel that read its inputs before
    their event would see it)."""
    wl = _stack(n_layers=7, n_seq=6, steps=10)
    im, (ga, gb), ids, dev = _twin(wl, pending_slots=4)
    layers = list(range(wl.n_layers))
    L = wl.n_layers
    cur = torch.cuda.current_stream(dev)
    cs, ds = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    ready = [torch.cuda.Event() for _ in range(L)]
    done = [torch.cuda.Event() for _ in range(L)]
    for e in ready + done:
        e.record(cur)              # (an event has a handle once it has been recorded)
    fork, join = torch.cuda.Event(), torch.cuda.Event()
    x0 = _step_inputs(wl, 0, dev)
    dbuf = [torch.empty_like(t) for t in x0]
    hbuf = [torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in x0]
    dout = torch.empty((L, wl.n_seq, wl.H, wl.d), dtype=torch.bfloat16, device=dev)
    hout = torch.empty((L, wl.n_seq, wl.H, wl.d), dtype=torch.bfloat16).pin_memory()
    for st in range(wl.steps):
        inp = _step_inputs(wl, st, dev)
        for h, t in zip(hbuf, inp):
            h.copy_(t.cpu())
        for d in dbuf:
            d.fill_(float("nan"))
        dout.fill_(float("nan"))
        hout.fill_(float("nan"))
        torch.cuda.synchronize(dev)
        fork.record(cur)
        cs.wait_event(fork)
        ds.wait_event(fork)
        with torch.cuda.stream(cs):
            for layer in range(L):
                for d, h in zip(dbuf, hbuf):
                    d[layer].copy_(h[layer], non_blocking=True)
                ready[layer].record(cs)
        oa = gb.decode_stack(layers, ids, *dbuf, out=dout, ready_events=ready, done_events=done)
        assert oa.data_ptr() == dout.data_ptr()
        with torch.cuda.stream(ds):
            for layer in range(L):
                ds.wait_event(done[layer])
                hout[layer].copy_(dout[layer], non_blocking=True)
            join.record(ds)
        cur.wait_event(join)
        x, qp, q, k, v = inp
        ob = torch.stack([ga.decode_step(layer, ids, x[layer], qp[layer], q[layer], k[layer], v[layer]) for layer in layers])
        torch.cuda.synchronize(dev)
        assert ga.status() == 0 and gb.status() == 0
        assert torch.equal(hout.view(torch.int16), ob.cpu().view(torch.int16)), f"step {st}: outputs on the host differ"
        if st % 3 == 2 or st == wl.steps - 1:
            _same_state(im, ga, gb, wl, f"step {st}")
    # without the pipeline the same call runs layer by layer and honours the events in stream order
    im.im_set_option(gb.ctx, im.IM_OPT_STACK_PIPELINE, 0)
    inp = _step_inputs(wl, wl.steps, dev)
    for r in ready:
        r.record(cur)
    oa = gb.decode_stack(layers, ids, *inp, ready_events=ready, done_events=done)
    x, qp, q, k, v = inp
    ob = torch.stack([ga.decode_step(layer, ids, x[layer], qp[layer], q[layer], k[layer], v[layer]) for layer in layers])
    done[-1].synchronize()
    torch.cuda.synchronize(dev)
    assert torch.equal(oa.view(torch.int16), ob.view(torch.int16))
    ga.close(); gb.close()


def test_stack_call_with_the_bulk_copy_readout_equals_layer_calls():
    """One sequence per call: the bulk-copy readout kernel then cuts a sequence's rows into the same runs in a stack
    call and in a layer call (fewer chunks than blocks in both), so the two agree bit for bit with that kernel too."""
    wl = _stack(n_layers=5, n_seq=1, steps=8)
    im, (ga, gb), ids, dev = _twin(wl, bulk_readout=True)
    layers = list(range(wl.n_layers))
    for st in range(wl.steps):
        x, qp, q, k, v = _step_inputs(wl, st, dev)
        ref = torch.stack([ga.decode_step(l, ids, x[l], qp[l], q[l], k[l], v[l]) for l in layers])
        got = gb.decode_stack(layers, ids, x, qp, q, k, v)
        torch.cuda.synchronize()
        assert torch.equal(ref, got), f"step {st}: outputs differ in {int((ref != got).sum())} elements"
    assert ga.status() == 0 and gb.status() == 0
    _same_state(im, ga, gb, wl, "with the bulk-copy readout")
    ga.close(); gb.close()


def test_stack_call_replayed_from_a_graph_equals_layer_calls():
    """The call captured once into a CUDA graph and replayed (tau = 1: every step alike), against eager
    im_decode_step calls on the twin."""
    wl = _stack(n_layers=9, n_seq=5, steps=10)
    im, (ga, gb), ids, dev = _twin(wl)
    L = wl.n_layers
    layers = list(range(L))
    sx, sqp, sq, sk, sv = [t.clone() for t in _step_inputs(wl, 0, dev)]
    out = torch.empty((L, wl.n_seq, wl.H, wl.d), dtype=torch.bfloat16, device=dev)
    stream = torch.cuda.Stream(dev)
    graph = None
    with torch.cuda.stream(stream):
        for st in range(wl.steps):
            ins = _step_inputs(wl, st, dev)
            for dst, src in zip((sx, sqp, sq, sk, sv), ins):
                dst.copy_(src)
            ref = torch.stack([ga.decode_step(l, ids, sx[l], sqp[l], sq[l], sk[l], sv[l]) for l in layers])
            if st == 0:
                gb.decode_stack(layers, ids, sx, sqp, sq, sk, sv, out)
            else:
                if graph is None:
                    graph = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(graph, stream=stream):
                        gb.decode_stack(layers, ids, sx, sqp, sq, sk, sv, out)
                graph.replay()
            stream.synchronize()
            assert torch.equal(ref, out), f"step {st}: outputs differ in {int((ref != out).sum())} elements"
    assert ga.status() == 0 and gb.status() == 0
    _same_state(im, ga, gb, wl, "after the replays")
    del graph
    ga.close(); gb.close()


def test_stack_call_against_the_oracle():
    """Sampled units of a reduced stack follow the oracle through the ingestion and through decode steps made by
    im_decode_stack under graph replay: every parity rule after every step.  Three SMs instead of eight are set
    aside for the small kernels here, which changes how the attention kernel cuts its tiles into runs."""
    wl = _stack(n_layers=6, n_seq=8, steps=20)
    su = SampledUnits(wl, [(0, 1), (2, 7), (3, 0), (5, 4)], pending_slots=8)
    su.im.im_set_option(su.g.ctx, su.im.IM_OPT_STACK_RESERVED, 3)
    for c in range(wl.ctx // wl.chunk):
        su.prefill(c)
    _decode_under_graph_replay(su, wl.steps, full_check_every=5, stack_call=True)
    su.check_properties(wl.B, wl.ctx + wl.steps, n_evicted=1, stride=3)
    assert su.stats["kidx_flips"] == 0 and su.stats["cut_divergences"] <= 2


@pytest.mark.parametrize("shape", ["qwen7b_b8", "tiny"])
def test_stack_call_other_head_shapes_against_the_oracle(shape):
    """The stack call at the Qwen head shape (7 query heads per KV head, 4 KV heads, memory width 448: eight column
    slices per readout item row) and at head_dim 64 with one KV head (the other instance of the attention kernel),
    three layers, sampled units against the oracle under graph replay."""
    base = synth.CONFIGS[shape]
    wl = base.replace(name="stack_" + shape, n_layers=3, n_seq=4, ctx=600, chunk=300, B=256, steps=10,
                      n_needles=min(base.n_needles, 4))
    su = SampledUnits(wl, [(0, 3), (1, 0), (2, 2)])
    for c in range(wl.ctx // wl.chunk):
        su.prefill(c)
    _decode_under_graph_replay(su, wl.steps, full_check_every=5, stack_call=True)
    su.check_properties(wl.B, wl.ctx + wl.steps, n_evicted=1, stride=2)
    assert su.stats["kidx_flips"] == 0 and su.stats["cut_divergences"] <= 2


def test_stack_call_falls_back_and_refuses_bad_arguments():
    """Calls that do not qualify for the pipelined schedule (it is switched off; one layer only) run layer by layer
    with the same results; a repeated layer and a layer out of range are refused."""
    wl = _stack(n_layers=3, n_seq=2, steps=4)
    im, (ga, gb), ids, dev = _twin(wl)
    layers = list(range(wl.n_layers))
    for st in range(wl.steps):
        x, qp, q, k, v = _step_inputs(wl, st, dev)
        ref = torch.stack([ga.decode_step(l, ids, x[l], qp[l], q[l], k[l], v[l]) for l in layers])
        if st == 1:
            im.im_set_option(gb.ctx, im.IM_OPT_STACK_PIPELINE, 0)
        if st == 2:
            im.im_set_option(gb.ctx, im.IM_OPT_STACK_PIPELINE, 1)
            got = torch.stack([gb.decode_stack([l], ids, x[l:l + 1], qp[l:l + 1], q[l:l + 1], k[l:l + 1], v[l:l + 1])[0] for l in layers])
        else:
            got = gb.decode_stack(layers, ids, x, qp, q, k, v)
        torch.cuda.synchronize()
        assert torch.equal(ref, got), f"step {st}"
    x, qp, q, k, v = _step_inputs(wl, wl.steps, dev)
    with pytest.raises(im.IndexMemError):
        gb.decode_stack([0, 1, 1], ids, x, qp, q, k, v)
    with pytest.raises(im.IndexMemError):
        gb.decode_stack([0, 1, 7], ids, x, qp, q, k, v)
    _same_state(im, ga, gb, wl, "after the refused calls")
    ga.close(); gb.close()


def test_stack_call_with_a_wait_that_runs_out_leaves_its_counters_clean():
    """The give-up path of the attention kernel inside a stack call (IM_OPT_WAIT_LIMIT = 1: a consumer gets no attempt
    to wait for its tile copies, nothing is broken or left to hang).  Every block, with or without a worker id, must
    still hand the claim counters back: the status reads IM_ERR_TIMEOUT, and after the limit is restored and both
    contexts are reset and fed the same context again, stack calls on the context that saw the time-out agree with
    im_decode_step on its twin bit for bit."""
    wl = _stack(n_layers=4, n_seq=3, ctx=512, chunk=256, B=256, steps=5)
    im, (ga, gb), ids, dev = _twin(wl)
    layers = list(range(wl.n_layers))
    x, qp, q, k, v = _step_inputs(wl, 0, dev)
    gb.decode_stack(layers, ids, x, qp, q, k, v)             # a good step first
    torch.cuda.synchronize()
    assert gb.status() == 0
    im.im_set_option(gb.ctx, im.IM_OPT_WAIT_LIMIT, 1)
    x, qp, q, k, v = _step_inputs(wl, 1, dev)
    gb.decode_stack(layers, ids, x, qp, q, k, v)
    torch.cuda.synchronize()
    with pytest.raises(im.IndexMemError) as e:
        gb.status()
    assert e.value.code == im.IM_ERR_TIMEOUT, str(e.value)
    im.im_set_option(gb.ctx, im.IM_OPT_WAIT_LIMIT, 0)
    for g in (ga, gb):
        g.reset()
        assert g.status() == 0
        for c in range(wl.ctx // wl.chunk):
            for layer in layers:
                X, Qp, _, K, V = synth.prefill_inputs(wl, layer, c, dev)
                g.prefill_chunk(layer, ids, X, Qp, K, V)
    for st in range(wl.steps):
        x, qp, q, k, v = _step_inputs(wl, st, dev)
        ref = torch.stack([ga.decode_step(l, ids, x[l], qp[l], q[l], k[l], v[l]) for l in layers])
        got = gb.decode_stack(layers, ids, x, qp, q, k, v)
        torch.cuda.synchronize()
        assert torch.equal(ref, got), f"step {st}: outputs differ in {int((ref != got).sum())} elements"
    assert ga.status() == 0 and gb.status() == 0
    _same_state(im, ga, gb, wl, "after the time-out and the reset")
    ga.close(); gb.close()
