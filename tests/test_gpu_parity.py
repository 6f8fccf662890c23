"""GPU-vs-oracle parity of the hot path, through the C ABI (``-m gpu``).

Every test drives the CUDA library and the CPU oracle with the same seeded inputs (tests/parity.py)
at sizes the oracle finishes in seconds, spanning several tiles and ragged tails, plus the edge
cases of the method (ties, sinks, empty eviction, decay, interval pooling, disabled memory,
non-power-of-two head shapes).
"""
import numpy as np
import pytest
import torch

from oracle import indexmem_oracle as orc
from paper_2605_25475_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def im():
    from paper_2605_25475_b200 import binding
    return binding


def _pair(*a, **k):
    from tests.parity import Pair
    return Pair(*a, **k)


TINY = synth.CONFIGS["tiny"]


# ------------------------------------------------------------------ K2 alone: bit-exact selection
@pytest.mark.parametrize("n,B,n_sink", [(1, 1, 0), (7, 3, 2), (300, 300, 4), (300, 400, 4), (2049, 2048, 4),
                                         (4096, 2048, 4), (5000, 1, 0), (16384, 1024, 4), (777, 0, 0)])
def test_topb_select_bit_exact(im, n, B, n_sink):
    rng = np.random.default_rng(n * 131 + B)
    rows = 5
    # heavy ties: half of the ReLU scores are exactly zero, both signs of zero, unscored (-inf) entries
    sc = rng.standard_normal((rows, n)).astype(np.float32)
    sc[rng.random((rows, n)) < 0.4] = 0.0
    sc[rng.random((rows, n)) < 0.1] = -0.0
    sc[rng.random((rows, n)) < 0.05] = -np.inf
    sc[1] = 0.0                                           # one row of pure ties
    sc[2] = np.round(sc[2] * 2) / 2                       # few distinct values
    pos = np.stack([rng.permutation(n * 3)[:n] for _ in range(rows)]).astype(np.int32)
    keep, nev = im.im_topb_select(torch.tensor(sc).cuda(), torch.tensor(pos).cuda(), B, n_sink)
    torch.cuda.synchronize()
    keep, nev = keep.cpu().numpy(), nev.cpu().numpy()
    for r in range(rows):
        want = orc.select_top_b(sc[r], pos[r], B, n_sink)
        assert np.array_equal(keep[r], want), f"row {r}"
        assert nev[r] == n - min(n, B)


# ------------------------------------------------------------------ the small benchmark configuration
def test_tiny_config_end_to_end():
    """1 layer, 4 q heads / 1 KV head, d 64, 1024-token context in one chunk -> B 256, 64 decode steps."""
    p = _pair(TINY)
    p.prefill(0)
    for s in range(TINY.steps):
        p.decode(s)
    st = p.stats
    assert st["kidx_flips"] == 0
    assert st["cut_divergences"] <= 2
    assert st["max_out_err"] <= 2e-3 and st["max_M_err"] <= 2e-3 and st["max_score_err"] <= 1e-5


def test_tiny_config_float32_output():
    wl = TINY.replace(name="tiny_f32", ctx=512, chunk=512, B=128, steps=12)
    p = _pair(wl, out_f32=1)
    p.prefill(0)
    for s in range(wl.steps):
        out, ob, od = p.decode(s)
        assert out.dtype == torch.float32
    assert p.stats["max_out_err"] <= 1e-4


# ------------------------------------------------------------------ reduced copies of the larger configurations
def test_llama_shape_reduced():
    """32 q / 8 KV heads, d 128 (widths 8 x 16, d_M 512), lognormal key norms; ragged sizes."""
    wl = synth.CONFIGS["llama8b_b1"].replace(name="llama_red", ctx=700, chunk=700, B=300, steps=20)
    p = _pair(wl)
    p.prefill(0)
    for s in range(wl.steps):
        p.decode(s)
    assert p.stats["max_out_err"] <= 2e-3 and p.stats["max_M_err"] <= 2e-3


def test_qwen_shape_reduced_batch():
    """28 q / 4 KV heads (G_q 7, H_I 7, d_M 448): nothing is a power of two; 3 sequences, needles."""
    wl = synth.CONFIGS["qwen7b_b8"].replace(name="qwen_red", n_seq=3, ctx=600, chunk=600, B=200, steps=10, n_needles=8)
    p = _pair(wl)
    p.prefill(0)
    for s in range(wl.steps):
        p.decode(s)
    assert p.stats["max_out_err"] <= 2e-3 and p.stats["max_M_err"] <= 2e-3


def test_chunked_prefill_reduced():
    """Mistral-shaped chunked prefill: several chunks, eviction to the budget after each."""
    wl = synth.CONFIGS["mistral7b_prefill"].replace(name="mistral_red", ctx=4 * 160, chunk=160, B=192, steps=4)
    p = _pair(wl)
    for c in range(4):
        p.prefill(c)
    for s in range(wl.steps):
        p.decode(s)
    assert p.o.evict_steps(0) == 3 + wl.steps
    assert p.stats["max_M_err"] <= 2e-3


def test_prefill_chunks_and_decode_steps_enqueued_back_to_back():
    """Nothing waits for the device between the calls: a prefill call leaves the state update of its memory write
    running on a stream of the library's own, and whatever call comes next has to order itself behind it.  Six chunks
    whose evicted sets exceed the pending list, then decode steps, all enqueued at once; the final state and the outputs
    against the oracle."""
    wl = synth.CONFIGS["mistral7b_prefill"].replace(name="mistral_b2b", ctx=6 * 256, chunk=256, B=320, steps=3)
    p = _pair(wl)
    dev = p.device
    ins = [tuple(t.to(dev) for t in synth.prefill_inputs(wl, 0, c)) for c in range(6)]
    dec = [tuple(t.to(dev) for t in synth.decode_inputs(wl, 0, s)) for s in range(wl.steps)]
    torch.cuda.synchronize()
    outs = []
    for X, Qp, _, K, V in ins:
        p.g.prefill_chunk(0, p.seq_ids, X, Qp, K, V)
    for x, qp, q, k, v in dec[:-1]:
        outs.append(p.g.decode_step(0, p.seq_ids, x, qp, q, k, v))
    torch.cuda.synchronize()
    assert p.g.status() == 0
    for c in range(6):
        X, Qp, _, K, V = synth.prefill_inputs(wl, 0, c)
        p.o.prefill_batch(p.seq_ids, synth.f32(X), synth.f32(Qp), synth.f32(K), synth.f32(V))
    for s in range(wl.steps - 1):
        x, qp, q, k, v = synth.decode_inputs(wl, 0, s)
        ob, od = p.o.decode_batch(p.seq_ids, synth.f32(x), synth.f32(qp), synth.f32(q), synth.f32(k), synth.f32(v))
        p.check_out(outs[s], ob, od)
    assert p.check_state()
    p.decode(wl.steps - 1)                       # and one more step, checked in full
    assert p.stats["max_M_err"] <= 2e-3 and p.stats["cut_divergences"] == 0


# ------------------------------------------------------------------ edge cases of the method
def test_budget_never_reached_is_exact_attention(im):
    wl = TINY.replace(name="nobudget", ctx=100, chunk=100, B=4096, steps=5, n_needles=2)
    p = _pair(wl, max_chunk=100)
    p.prefill(0)
    for s in range(wl.steps):
        p.decode(s)
    assert p.o.evict_steps(0) == 0 and p.g.counts(0, 0)["n"] == 105
    assert not p.g.export(0, 0, im.IM_S_M).any()


def test_memory_disabled():
    wl = TINY.replace(name="nomem", ctx=300, chunk=300, B=64, steps=8, n_needles=2)
    p = _pair(wl, enable_memory=0)
    p.prefill(0)
    for s in range(wl.steps):
        p.decode(s)
    assert p.stats["max_out_err"] <= 2e-3


def test_decay_and_write_strength():
    wl = TINY.replace(name="decay", ctx=300, chunk=300, B=64, steps=40, n_needles=2)
    p = _pair(wl, lambda_=0.9, eta=0.5, pending_slots=4)
    p.prefill(0)
    for s in range(wl.steps):
        p.decode(s)
    assert p.stats["max_M_err"] <= 2e-3


def test_long_pending_list_folds_in_several_passes():
    """A pending list of 40 entries (the fold kernels take 32 listed entries per pass over a stripe of M) with decay and a
    write strength, at the Llama head shape with a memory matrix of several stripes and column tiles: M, b and the
    outputs against the oracle through two folds."""
    wl = synth.CONFIGS["llama8b_b1"].replace(name="pend40", n_seq=2, ctx=400, chunk=200, B=128, steps=90, n_needles=0)
    p = _pair(wl, lambda_=0.97, eta=0.7, pending_slots=40)
    p.prefill(0)
    p.prefill(1)
    for s in range(wl.steps):
        p.decode(s, check=(s % 9 == 8 or s == wl.steps - 1))
    assert p.stats["max_M_err"] <= 2e-3 and p.stats["max_out_err"] <= 2e-3


def test_fold_on_the_tensor_cores_differs_from_the_ffma_fold_by_rounding_only(im):
    """The pending list of the default length (32 entries, one pass over M) folded by the tensor-core kernel and, on a
    second context fed the same inputs, by the float32 multiply-add kernel (IM_OPT_FOLD_TENSOR 0), with decay and a write
    strength, at the Llama and the Qwen head shape (d_M = 512 and 448, D_kv = 1024 and 512): M of both after every fold
    agrees to a few float32 roundings relative to its largest entry, both follow the oracle, and the caches are
    identical (no selection depends on M)."""
    for shape in ("llama8b_b1", "qwen7b_b8"):
        wl = synth.CONFIGS[shape].replace(name="foldtc_" + shape, n_seq=2, ctx=400, chunk=200, B=128, steps=70, n_needles=0)
        pt = _pair(wl, lambda_=0.97, eta=0.7)
        pf = _pair(wl, lambda_=0.97, eta=0.7)
        im.im_set_option(pf.g.ctx, im.IM_OPT_FOLD_TENSOR, 0)
        for p in (pt, pf):
            p.prefill(0)
            p.prefill(1)
        worst = 0.0
        for s in range(wl.steps):
            chk = s % 8 == 7 or s == wl.steps - 1
            pt.decode(s, check=chk)
            pf.decode(s, check=chk)
            if chk:
                for q in range(wl.n_seq):
                    Mt = pt.g.export(0, q, im.IM_S_M).astype(np.float64)
                    Mf = pf.g.export(0, q, im.IM_S_M).astype(np.float64)
                    worst = max(worst, float(np.abs(Mt - Mf).max() / np.abs(Mf).max()))
                    assert np.array_equal(pt.g.export(0, q, im.IM_S_K), pf.g.export(0, q, im.IM_S_K))
        assert pt.g.counts(0, 0)["n_pending"] < 32 and wl.steps > 64, "the list has been folded at least twice"
        assert worst <= 2e-6, (shape, worst)
        assert pt.stats["max_M_err"] <= 2e-3 and pf.stats["max_M_err"] <= 2e-3


def test_prefill_calls_that_leave_their_tail_running_equal_calls_that_do_not(im):
    """IM_OPT_PREFILL_PIPELINE: chunk calls that return with scoring, selection, gather and memory write still running
    on the library's own streams (the next chunk's projections run next to them) leave every piece of the state, bit
    for bit, as calls that leave only the state update running, chunk after chunk (each export joins the streams), for
    two layers called in turn, and the decode steps that follow give the same outputs; both follow the oracle."""
    wl = synth.CONFIGS["llama8b_b1"].replace(name="pftail", n_seq=2, ctx=6 * 256, chunk=256, B=128, steps=3, n_needles=0)
    dev = torch.device("cuda:0")
    cfg = dict(n_layers=2, max_seqs=wl.n_seq, n_q_heads=wl.H, n_kv_heads=wl.Hkv, head_dim=wl.d, budget=wl.B,
               compress_interval=1, max_chunk=wl.chunk, n_sink=wl.n_sink, lambda_=0.98, eta=0.8)
    gs = [im.IndexMem(im.Config(**cfg), dev) for _ in range(2)]
    im.im_set_option(gs[1].ctx, im.IM_OPT_PREFILL_PIPELINE, 0)
    ids = list(range(wl.n_seq))
    for layer in range(2):
        w = synth.make_weights(wl, layer)
        for g in gs:
            g.set_weights(layer, w)
    pieces = (im.IM_S_POS, im.IM_S_IMP, im.IM_S_KIDX, im.IM_S_K, im.IM_S_V, im.IM_S_M, im.IM_S_B)
    for c in range(wl.ctx // wl.chunk):
        ins = [synth.prefill_inputs(wl, layer, c, dev) for layer in range(2)]
        for g in gs:
            for layer in range(2):
                X, Qp, _, K, V = ins[layer]
                g.prefill_chunk(layer, ids, X, Qp, K, V)
        if c % 2 == 1 or c == wl.ctx // wl.chunk - 1:
            for layer in range(2):
                for q in ids:
                    assert gs[0].counts(layer, q) == gs[1].counts(layer, q)
                    for piece in pieces:
                        assert np.array_equal(gs[0].export(layer, q, piece), gs[1].export(layer, q, piece)), (c, layer, q, piece)
    for st in range(wl.steps):
        for layer in range(2):
            x, qp, q, k, v = synth.decode_inputs(wl, layer, st, dev)
            oa = gs[0].decode_step(layer, ids, x, qp, q, k, v)
            ob = gs[1].decode_step(layer, ids, x, qp, q, k, v)
            assert torch.equal(oa, ob)
    assert gs[0].status() == 0 and gs[1].status() == 0
    for g in gs:
        g.close()
    # and against the oracle, through the usual pair (pipelined by default)
    p = _pair(wl, lambda_=0.98, eta=0.8)
    for c in range(wl.ctx // wl.chunk):
        p.prefill(c)
    for s_ in range(wl.steps):
        p.decode(s_)
    assert p.stats["max_M_err"] <= 2e-3 and p.stats["max_out_err"] <= 2e-3


def test_interval_pooling_tau():
    """tau = 8: scores pooled by max over the interval's queries, 8 entries evicted at once."""
    wl = TINY.replace(name="tau8", ctx=200, chunk=200, B=96, steps=24, tau=8, n_needles=2)
    p = _pair(wl, pending_slots=16)
    p.prefill(0)
    for s in range(wl.steps):
        p.decode(s)
        assert p.g.counts(0, 0)["n"] == 96 + (s + 1) % 8
    assert p.o.evict_steps(0) == 1 + 3


def test_identity_activation_and_all_ties():
    wl = TINY.replace(name="ident", ctx=150, chunk=150, B=40, steps=4, n_needles=0)
    p = _pair(wl, act=1)
    p.prefill(0)
    for s in range(wl.steps):
        p.decode(s)
    # G = 0: alpha = 0, every score ties at zero, the lowest positions stay
    p2 = _pair(wl.replace(name="ties"))
    w = dict(p2.weights)
    w["G"] = torch.zeros_like(w["G"])
    p2.o.set_weights({k: synth.f32(v) for k, v in w.items()})
    p2.g.set_weights(0, w)
    p2.prefill(0)
    assert p2.o.positions(0).tolist() == list(range(40))
    for s in range(3):
        p2.decode(s)


def test_single_token_chunks_and_subset_of_sequences(im):
    """Chunks of one token; calls that address a subset of the sequences in arbitrary order."""
    wl = TINY.replace(name="subset", n_seq=3, ctx=24, chunk=1, B=10, steps=0, n_needles=0)
    p = _pair(wl, max_chunk=8)
    for c in range(12):
        p.prefill(c)
    dev = p.device
    # sequences 2 and 0 only, in that order
    x, qp, q, k, v = synth.decode_inputs(wl, 0, 0)
    ids = [2, 0]
    ob, od = p.o.decode_batch(ids, synth.f32(x[ids]), synth.f32(qp[ids]), synth.f32(q[ids]), synth.f32(k[ids]), synth.f32(v[ids]))
    out = p.g.decode_step(0, ids, x[ids].to(dev).contiguous(), qp[ids].to(dev).contiguous(), q[ids].to(dev).contiguous(),
                          k[ids].to(dev).contiguous(), v[ids].to(dev).contiguous())
    assert p.g.status() == 0
    p.check_out(out, ob, od)
    assert p.g.counts(0, 1)["T"] == 12 and p.g.counts(0, 0)["T"] == 13


def test_errors_are_reported_not_fatal(im):
    wl = TINY.replace(name="errs", ctx=32, chunk=32, B=16, steps=0, n_needles=0)
    p = _pair(wl)
    dev = p.device
    X, Q, _, K, V = [t.to(dev) for t in synth.prefill_inputs(wl, 0, 0)]
    with pytest.raises(im.IndexMemError) as e:
        im.im_prefill_chunk(p.g.ctx, 0, [5], 32, X, Q, K, V)
    assert e.value.code == im.IM_ERR_ARG
    with pytest.raises(im.IndexMemError) as e:
        im.im_prefill_chunk(p.g.ctx, 0, [0], 33, X, Q, K, V)
    assert e.value.code == im.IM_ERR_ARG
    with pytest.raises(im.IndexMemError) as e:
        im.im_prefill_chunk(p.g.ctx, 1, [0], 32, X, Q, K, V)
    assert e.value.code == im.IM_ERR_ARG
    # the context is still usable
    p.prefill(0)
    assert p.g.status() == 0


def test_seeded_weight_init_statistics(im):
    g = im.IndexMem(im.Config(n_layers=2, max_seqs=1, n_q_heads=8, n_kv_heads=2, head_dim=64, budget=32, seed=7))
    g2 = im.IndexMem(im.Config(n_layers=2, max_seqs=1, n_q_heads=8, n_kv_heads=2, head_dim=64, budget=32, seed=7))
    w0, w1, v0 = g.get_weights(0), g.get_weights(1), g2.get_weights(0)
    for name in ("U_q", "U_k", "G", "W_theta", "w_g"):
        a = w0[name].float()
        assert torch.equal(w0[name], v0[name])               # same seed, same weights
        assert not torch.equal(w0[name], w1[name])           # layers differ
        if a.numel() > 2000:
            assert abs(a.mean().item()) < 3 * 0.02 / a.numel() ** 0.5 + 1e-4
            assert abs(a.std().item() - 0.02) < 0.002
    assert w0["b_g"].item() == 0.0


def test_generic_attention_path_small_head_dim():
    """d = 32 has no TMA/mma fast path: the generic split kernels serve it."""
    wl = synth.Workload("d32", 1, 2, 4, 2, 32, 200, 200, 72, 6, n_needles=2)
    p = _pair(wl, dI=8, dM=24)
    p.prefill(0)
    for s in range(wl.steps):
        p.decode(s)
    assert p.stats["max_out_err"] <= 2e-3 and p.stats["max_M_err"] <= 2e-3


def test_long_interval_unfused_select_and_large_evicted_set():
    """tau = 24: more evicted entries per compression than the fused decode kernel or the pending
    list take, so the stand-alone select / gather / move kernels and the direct accumulation run."""
    wl = TINY.replace(name="tau24", ctx=180, chunk=180, B=100, steps=48, tau=24, n_needles=2)
    p = _pair(wl, lambda_=0.95)
    p.prefill(0)
    for s in range(wl.steps):
        p.decode(s)
    assert p.o.evict_steps(0) == 1 + 2
    assert p.stats["max_M_err"] <= 2e-3


# ------------------------------------------------------------------ prefill scoring: tensor-core and CUDA-core kernels
@pytest.mark.parametrize("tensor", [1, 0])
def test_prefill_scoring_both_kernels_several_key_tiles_ragged_chunks(im, tensor):
    """Llama-shaped widths (8 x 16); 5 chunks of 333 tokens (not a multiple of the 32-query tile) into a
    budget of 700, so that a call scores 1033 keys = 8 full key tiles and a ragged ninth, old keys that every
    query sees next to chunk keys under the causal mask, for three sequences at once."""
    wl = synth.CONFIGS["mistral7b_prefill"].replace(name="score_both", n_seq=3, ctx=5 * 333, chunk=333, B=700, steps=2)
    p = _pair(wl)
    im.im_set_option(p.g.ctx, im.IM_OPT_PREFILL_TENSOR, tensor)
    for c in range(5):
        p.prefill(c)
    for s in range(wl.steps):
        p.decode(s)
    assert p.stats["max_score_err"] <= 1e-5 and p.stats["max_M_err"] <= 2e-3
    assert p.stats["cut_divergences"] <= 2


def test_prefill_scoring_tensor_identity_activation_and_narrow_widths(im):
    """act = identity (scores of both signs: the pooled maximum goes through negative values) at the tiny
    widths (one indexer head of 8 features: zero-padded head slots and K group), two chunks."""
    wl = TINY.replace(name="score_ident", ctx=2 * 190, chunk=190, B=120, steps=2, n_needles=0)
    p = _pair(wl, act=1)
    for c in range(2):
        p.prefill(c)
    for s in range(wl.steps):
        p.decode(s)
    assert p.stats["max_score_err"] <= 1e-5


def test_prefill_scoring_tensor_unsupported_shape_is_refused(im):
    """More than eight indexer heads: the tensor-core kernel is not used, asking for it is an error."""
    wl = TINY.replace(name="score_wide", H=48, Hkv=4, ctx=100, chunk=100, B=60, steps=1, n_needles=0)
    p = _pair(wl)                                   # H_I = 12
    with pytest.raises(im.IndexMemError):
        im.im_set_option(p.g.ctx, im.IM_OPT_PREFILL_TENSOR, 1)
    p.prefill(0)
    p.decode(0)


# ------------------------------------------------------------------ decode with the attention kernel started before the selection
def test_peaked_attention_evicted_entry_dominates_softmax(im):
    """softmax_scale = 6: every head's attention is close to one-hot, so the entry evicted in a step often
    carries nearly all of a head's softmax mass.  The merge must then recompute the head over the retained
    entries (removing the term from the sums would cancel catastrophically); the counter shows that it did."""
    wl = TINY.replace(name="peaked", ctx=64, chunk=64, B=32, steps=60, n_needles=0)
    p = _pair(wl, scale=6.0)
    p.prefill(0)
    for s in range(wl.steps):
        p.decode(s)
    assert p.stats["max_out_err"] <= 2e-3
    assert im.im_event_count(p.g.ctx, im.IM_COUNT_MERGE_RECOMPUTE) > 0


@pytest.mark.parametrize("conc,tensor", [(0, 1), (1, 1), (0, 0), (1, 0)])
def test_decode_schedules_agree_with_the_oracle(im, conc, tensor):
    """The in-order schedule and the concurrent one (attention first, evicted terms removed in the merge), each with
    the tensor-core attention kernel and with the mma.sync one, against the oracle on the same inputs: several
    sequences, evictions every step, needles, then steps on a cache that is not full yet (nothing evicted, the new
    token only added)."""
    wl = synth.CONFIGS["llama8b_b1"].replace(name="sched", n_seq=3, ctx=333, chunk=333, B=300, steps=12, n_needles=4)
    p = _pair(wl)
    im.im_set_option(p.g.ctx, im.IM_OPT_CONCURRENCY, conc)
    im.im_set_option(p.g.ctx, im.IM_OPT_DECODE_TENSOR, tensor)
    p.prefill(0)
    for s in range(wl.steps):
        p.decode(s)
    assert p.stats["max_out_err"] <= 2e-3 and p.stats["max_M_err"] <= 2e-3
    wl2 = wl.replace(name="sched_notfull", ctx=40, chunk=40, B=64, steps=30)   # fills up at step 24
    p2 = _pair(wl2)
    im.im_set_option(p2.g.ctx, im.IM_OPT_CONCURRENCY, conc)
    im.im_set_option(p2.g.ctx, im.IM_OPT_DECODE_TENSOR, tensor)
    p2.prefill(0)
    for s in range(wl2.steps):
        p2.decode(s)
    assert p2.stats["max_out_err"] <= 2e-3


def test_decode_many_sequences_without_sm_partition(im):
    """More sequences than a quarter of the SMs: the concurrent schedule then sets no SMs aside for the front
    kernel (attention waits for the projections, the readout runs in its light variant next to the front kernel).
    40 and 64 sequences of a small shape (16 query / 4 KV heads of 64, 4 indexer heads, d_M = 128: readout rows
    that do not fill a batch), evictions every step.  (With the tiny shape's single indexer head a sequence whose
    alpha nearly cancels shows that float32 dot product's rounding in all its scores; more heads average it out.)"""
    for n_seq in (40, 64):
        wl = TINY.replace(name=f"many{n_seq}", n_seq=n_seq, H=16, Hkv=4, ctx=96, chunk=96, B=80, steps=6, n_needles=2)
        p = _pair(wl)
        p.prefill(0)
        for s in range(wl.steps):
            p.decode(s)
        assert p.stats["max_out_err"] <= 2e-3 and p.stats["max_M_err"] <= 2e-3


def test_decode_long_interval_several_sequences_batched_memory_write(im):
    """tau = 40 at Llama widths with three sequences: every 40th step evicts 40 entries per sequence, more than the
    pending list or the fused front kernel hold, so the step runs in order and writes Phi^T V of all sequences
    with one batched tensor-core launch; the 39 steps between attend to a growing cache without selecting."""
    wl = synth.CONFIGS["llama8b_b1"].replace(name="tau40", n_seq=3, ctx=150, chunk=150, B=100, steps=85, tau=40, n_needles=2)
    p = _pair(wl)
    p.prefill(0)
    for s in range(wl.steps):
        p.decode(s)
    assert p.stats["max_out_err"] <= 2e-3 and p.stats["max_M_err"] <= 2e-3
    assert p.o.evict_steps(0) == 1 + 2


def test_decode_from_an_empty_cache(im):
    """No prefill at all: the first decode step attends to the new token alone."""
    wl = TINY.replace(name="empty_start", ctx=0, chunk=8, B=16, steps=24, n_needles=0)
    p = _pair(wl)
    for s in range(wl.steps):
        p.decode(s)
    assert p.stats["max_out_err"] <= 2e-3


# ------------------------------------------------------------------ layer outputs of a prefill chunk's own queries
@pytest.mark.parametrize("tensor", [1, 0])
def test_chunk_outputs_llama_shape_several_chunks(im, tensor):
    """32 q / 8 KV heads, d 128: four ragged chunks of 200 tokens into a budget of 256, two sequences; from the
    second chunk on the queries see a retained prefix (holes filled in arbitrary slot order) plus the causal
    chunk and read a non-empty memory; then decode steps continue from the same state."""
    wl = synth.CONFIGS["llama8b_b1"].replace(name="chunk_out", n_seq=2, ctx=4 * 200, chunk=200, B=256, steps=3, n_needles=4)
    p = _pair(wl, chunk_outputs=1)
    im.im_set_option(p.g.ctx, im.IM_OPT_PREFILL_TENSOR, tensor)   # tcgen05 / mma.sync attention (and scoring)
    for c in range(4):
        p.prefill_attend(c)
    for s in range(wl.steps):
        p.decode(s)
    assert p.stats["max_out_err"] <= 2e-3 and p.stats["max_M_err"] <= 2e-3


def test_chunk_outputs_qwen_shape_and_pending_list(im):
    """28 q / 4 KV heads (7 heads per KV head: 18 queries x 7 heads = 126 of a block's 128 rows), d_M 448;
    decode steps in between leave rank-one writes pending, which the call folds before it reads the memory;
    float32 outputs."""
    wl = synth.CONFIGS["qwen7b_b8"].replace(name="chunk_out_q", n_seq=2, ctx=3 * 150, chunk=150, B=180, steps=5, n_needles=0)
    p = _pair(wl, chunk_outputs=1, out_f32=1)
    p.prefill_attend(0)
    p.prefill_attend(1)
    for s in range(wl.steps):
        p.decode(s)
    assert p.g.counts(0, 0)["n_pending"] > 0
    p.prefill_attend(2)
    assert p.stats["max_out_err"] <= 1e-4


def test_chunk_outputs_tiny_shape_no_memory_and_single_token_chunks(im):
    wl = TINY.replace(name="chunk_out_t", ctx=3 * 70, chunk=70, B=90, steps=2, n_needles=0)
    p = _pair(wl, chunk_outputs=1, enable_memory=0)
    for c in range(3):
        p.prefill_attend(c)
    wl1 = TINY.replace(name="chunk_out_1", ctx=40, chunk=1, B=24, steps=1, n_needles=0)
    p1 = _pair(wl1, chunk_outputs=1)
    for c in range(40):
        p1.prefill_attend(c)
    assert p1.stats["max_out_err"] <= 2e-3


def test_chunk_outputs_head_dim_128_other_group_sizes_and_short_chunks(im):
    """The tcgen05 chunk attention lays 2 x 128 rows = queries x heads of a KV head over two Q tiles: 8 heads per KV
    head (16 queries per tile), 1 head per KV head (128 queries per tile, so a chunk of 100 leaves the second Q tile
    without a valid row), and chunks of 1 and 3 tokens (one block, one key tile at first, the retained prefix
    growing past a tile), all at head_dim 128."""
    base = synth.CONFIGS["llama8b_b1"]
    wl8 = base.replace(name="chunk_out_g8", H=8, Hkv=1, n_seq=2, ctx=3 * 90, chunk=90, B=120, steps=2, n_needles=0)
    p8 = _pair(wl8, chunk_outputs=1)
    for c in range(3):
        p8.prefill_attend(c)
    for s in range(wl8.steps):
        p8.decode(s)
    assert p8.stats["max_out_err"] <= 2e-3 and p8.stats["max_M_err"] <= 2e-3
    wl1 = base.replace(name="chunk_out_g1", H=4, Hkv=4, n_seq=1, ctx=3 * 100, chunk=100, B=130, steps=2, n_needles=0)
    p1 = _pair(wl1, chunk_outputs=1, out_f32=1)
    for c in range(3):
        p1.prefill_attend(c)
    assert p1.stats["max_out_err"] <= 1e-4
    for chunk, n in ((1, 70), (3, 30)):
        wls = base.replace(name=f"chunk_out_c{chunk}", H=8, Hkv=2, n_seq=1, ctx=chunk * n, chunk=chunk, B=48, steps=1, n_needles=0)
        ps = _pair(wls, chunk_outputs=1)
        for c in range(n):
            ps.prefill_attend(c)
        assert ps.stats["max_out_err"] <= 2e-3 and ps.stats["max_M_err"] <= 2e-3


def test_chunk_outputs_call_captured_into_a_cuda_graph(im):
    """im_prefill_chunk_attend forks onto the side streams (projections, the output kernels next to the compression
    chain) and joins back with events only: the second chunk's call is captured into a CUDA graph, replayed once,
    and outputs and state are compared with the oracle as for an eager call."""
    wl = synth.CONFIGS["llama8b_b1"].replace(name="chunk_out_graph", n_seq=2, ctx=2 * 160, chunk=160, B=200, steps=1, n_needles=2)
    p = _pair(wl, chunk_outputs=1)
    p.prefill_attend(0)
    X, Qp, Q, K, V = synth.prefill_inputs(wl, p.layer, 1)
    ob, od = p.o.prefill_batch_out(p.seq_ids, synth.f32(X), synth.f32(Qp), synth.f32(Q), synth.f32(K), synth.f32(V))
    dev = p.device
    Xd, Qpd, Qd, Kd, Vd = X.to(dev), Qp.to(dev), Q.to(dev), K.to(dev), V.to(dev)
    stream = torch.cuda.Stream(dev)
    with torch.cuda.stream(stream):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            out = p.g.prefill_chunk_attend(0, p.seq_ids, Xd, Qpd, Qd, Kd, Vd)
        graph.replay()
        stream.synchronize()
    assert p.g.status() == 0
    p.check_selection()
    p.check_state()
    n, Cn = od.shape[0], od.shape[1]
    p.check_out(out.reshape(n * Cn, wl.H, wl.d), ob.reshape(n * Cn, wl.H, wl.d), od.reshape(n * Cn, wl.H, wl.d))
    assert p.stats["max_out_err"] <= 2e-3 and p.stats["max_M_err"] <= 2e-3


def test_chunk_outputs_need_their_workspace(im):
    wl = TINY.replace(name="chunk_out_e", ctx=32, chunk=32, B=64, steps=1)
    p = _pair(wl)
    X, Qp, Q, K, V = synth.prefill_inputs(wl, 0, 0)
    with pytest.raises(im.IndexMemError):
        p.g.prefill_chunk_attend(0, [0], X.cuda(), Qp.cuda(), Q.cuda(), K.cuda(), V.cuda())


def test_one_tensor_as_both_queries(im):
    """The header allows q_pre to alias q: one device tensor passed for both (every other test passes two tensors
    with different values, the pre-RoPE query for the indexer and the rotated one for attention, Linear_theta and
    the gate)."""
    wl = TINY.replace(name="alias", H=8, Hkv=2, ctx=200, chunk=100, B=64, steps=6, n_needles=4)
    p = _pair(wl, alias_q=True, chunk_outputs=1)
    p.prefill_attend(0)
    p.prefill_attend(1)
    for s in range(wl.steps):
        p.decode(s)
    assert p.stats["max_out_err"] <= 2e-3 and p.stats["max_score_err"] <= 1e-5


@pytest.mark.parametrize("tensor", [1, 0])
@pytest.mark.parametrize("shape", ["llama8b_b1", "qwen7b_b8"])
def test_decode_attention_float32_ragged_rows_and_rising_maxima(im, tensor, shape):
    """The streaming attention kernels with the float32 result exposed (bound 1e-4 of the tensor's max-abs) at
    head_dim 128, G_q = 4 and 7: five sequences whose rows hold several 128-key tiles with ragged tails, a softmax
    scale four times the usual one, so that a row's running maximum rises by more than 2^8 several times along the
    row (the tensor-core kernel then rescales its accumulators in tensor memory) and the entry evicted in a step
    often carries most of a head's mass (the merge then recomputes the head)."""
    wl = synth.CONFIGS[shape].replace(name="attn_f32_" + shape, n_seq=5, ctx=700, chunk=700, B=645, steps=10, n_needles=6)
    p = _pair(wl, out_f32=1, scale=4.0 / np.sqrt(wl.d))
    im.im_set_option(p.g.ctx, im.IM_OPT_DECODE_TENSOR, tensor)
    p.prefill(0)
    for s in range(wl.steps):
        p.decode(s)
    assert p.stats["max_out_err"] <= 1e-4 and p.stats["max_M_err"] <= 2e-3
    # rows of different lengths in one call, none of them full: 37, 131 and 257 entries (no eviction yet)
    for k, ctx in enumerate((36, 130, 256)):
        wl2 = wl.replace(name=f"attn_f32_short{k}", n_seq=2, ctx=ctx, chunk=ctx, B=400, steps=3, n_needles=0)
        p2 = _pair(wl2, out_f32=1)
        im.im_set_option(p2.g.ctx, im.IM_OPT_DECODE_TENSOR, tensor)
        p2.prefill(0)
        for s in range(wl2.steps):
            p2.decode(s)
        assert p2.stats["max_out_err"] <= 1e-4


def test_decode_tensor_option_is_refused_for_other_head_dims(im):
    p = _pair(TINY.replace(name="opt", ctx=32, chunk=32, B=16, steps=0))
    with pytest.raises(im.IndexMemError) as e:
        im.im_set_option(p.g.ctx, im.IM_OPT_DECODE_TENSOR, 1)
    assert e.value.code == im.IM_ERR_ARG
    im.im_set_option(p.g.ctx, im.IM_OPT_DECODE_TENSOR, 0)


@pytest.mark.parametrize("tensor,stages", [(0, 0), (0, 1), (0, 3), (1, 2), (1, 6)])
def test_decode_readout_through_bulk_copy_ring(im, tensor, stages):
    """phi(q)^T Mhat formed by the persistent bulk-copy kernel (a ring of 32 KB stages per CTA next to the attention
    kernel, partial vectors per CTA added by the merge) instead of the kernel on plain loads: Llama widths (D_kv 1024,
    8 rows per chunk) and Qwen widths (D_kv 512, d_M 448: 16 rows per chunk, two row groups per column), several
    sequences, evictions every step with decay, float32 outputs held to 1e-4, the memory to 2e-3."""
    for shape, n_seq in (("llama8b_b1", 3), ("qwen7b_b8", 5)):
        wl = synth.CONFIGS[shape].replace(name=f"ro_ring_{shape}", n_seq=n_seq, ctx=300, chunk=300, B=200, steps=24, n_needles=3)
        p = _pair(wl, out_f32=1, lambda_=0.95, eta=0.5)
        im.im_set_option(p.g.ctx, im.IM_OPT_DECODE_TENSOR, tensor)
        im.im_set_option(p.g.ctx, im.IM_OPT_READOUT_STAGES, stages)
        p.prefill(0)
        for s in range(wl.steps):
            p.decode(s)
        assert p.stats["max_out_err"] <= 1e-4 and p.stats["max_M_err"] <= 2e-3
    # shapes the ring kernel does not take are refused
    p = _pair(TINY.replace(name="ro_ring_refused", H=12, Hkv=3, ctx=32, chunk=32, B=16, steps=0))   # D_kv = 192
    with pytest.raises(im.IndexMemError) as e:
        im.im_set_option(p.g.ctx, im.IM_OPT_READOUT_STAGES, 2)
    assert e.value.code == im.IM_ERR_ARG
