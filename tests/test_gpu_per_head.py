"""A retained set per KV head (configuration scorer = 1 Knorm, 2 scores from the caller), ``-m gpu``.

Every KV head of a sequence keeps its own B positions; the evict step's memory write assembles the slices a token
loses into one model-space pair.  The library runs next to the oracle's per-head mode on the same seeded inputs;
after every call, per head: retained positions, scores, K / V copies and what the selection saw, and per sequence
the memory (M, b) and the outputs.  Knorm scores are float32 square roots on both sides; a selection decided inside
the 1e-5 gap at a head's cut re-synchronises the sequence from the oracle.
"""
import numpy as np
import pytest
import torch

from oracle import indexmem_oracle as orc
from paper_2605_25475_b200 import synth

pytestmark = pytest.mark.gpu


class PerHeadPair:
    def __init__(self, wl, scorer, **over):
        from paper_2605_25475_b200 import binding as im
        self.im, self.wl, self.scorer = im, wl, scorer
        self.dev = torch.device("cuda:0")
        cfg = dict(n_layers=1, max_seqs=wl.n_seq, n_q_heads=wl.H, n_kv_heads=wl.Hkv, head_dim=wl.d, budget=wl.B,
                   compress_interval=wl.tau, max_chunk=wl.chunk, n_sink=wl.n_sink, scorer=scorer)
        ocfg = dict(H=wl.H, Hkv=wl.Hkv, d=wl.d, B=wl.B, tau=wl.tau, n_sink=wl.n_sink, scorer=scorer)
        for k, v in over.items():
            cfg[k] = v
            if k in ("lambda_", "eta", "enable_memory"):
                ocfg[k] = v
        self.out_f32 = bool(over.get("out_f32", 0))
        self.g = im.IndexMem(im.Config(**cfg), self.dev)
        self.o = orc.OracleLayer(orc.OracleConfig(**ocfg), wl.n_seq)
        w = synth.make_weights(wl, 0)
        self.g.set_weights(0, w)
        self.o.set_weights({k: synth.f32(v) for k, v in w.items()})
        self.ids = list(range(wl.n_seq))
        self.rng = np.random.default_rng(1234)
        self.T = 0
        self.stats = {"cut_divergences": 0, "max_out_err": 0.0, "max_M_err": 0.0, "max_score_err": 0.0, "distinct_sets": 0}

    def _ext(self, n_pos):
        """Scores from the caller: random per (sequence, head, position), a few exact ties."""
        if self.scorer != 2:
            return None, None
        ext = self.rng.standard_normal((self.wl.n_seq, self.wl.Hkv, n_pos)).astype(np.float32)
        ext[:, :, ::7] = np.round(ext[:, :, ::7])
        return ext, torch.tensor(ext).to(self.dev)

    def prefill(self, c):
        wl, dev = self.wl, self.dev
        _, _, _, K, V = synth.prefill_inputs(wl, 0, c)
        self.T += wl.chunk
        ext, ext_d = self._ext(self.T)
        if ext_d is not None:
            self.g.set_scores(0, ext_d)
        self.g.prefill_chunk(0, self.ids, None, None, K.to(dev), V.to(dev))
        for s in self.ids:
            self.o.ph_prefill_chunk(s, synth.f32(K[s]), synth.f32(V[s]), ext=None if ext is None else ext[s])
        assert self.g.status() == 0
        self.check_state(True)

    def decode(self, step):
        wl, dev = self.wl, self.dev
        _, _, q, k, v = synth.decode_inputs(wl, 0, step)
        self.T += 1
        due = (self.g.counts(0, 0)["since"] + 1 == wl.tau)
        ext, ext_d = self._ext(self.T) if due else (None, None)
        if ext_d is not None:
            self.g.set_scores(0, ext_d)
        out = self.g.decode_step(0, self.ids, None, None, q.to(dev), k.to(dev), v.to(dev))
        refs = [self.o.ph_decode_step(s, synth.f32(q[s]), synth.f32(k[s]), synth.f32(v[s]), ext=None if ext is None else ext[s])[1]
                for s in self.ids]
        assert self.g.status() == 0
        clean = self.check_state(due)
        from tests.parity import check_unit_out
        for s in self.ids:
            if clean[s]:
                got = out[s].float().cpu().numpy().astype(np.float64)
                check_unit_out(got, refs[s], not self.out_f32, f"step {step} seq {s}", self.stats, 1e-4 if self.out_f32 else 2e-3)

    def check_state(self, compressed):
        from tests.parity import check_scores, TOL_SCORE, TOL_OUT
        im, g, o, wl = self.im, self.g, self.o, self.wl
        clean = {}
        for s in self.ids:
            cnt = g.counts(0, s)
            resync = False
            sets = []
            for h in range(wl.Hkv):
                e = o.ph_entries(s, h)
                assert cnt["n"] == len(e["pos"]), f"seq {s} head {h}: {cnt['n']} entries vs oracle {len(e['pos'])}"
                gpos = g.export_head(0, s, h, im.IM_S_POS)
                order = np.argsort(gpos, kind="stable")
                sets.append(tuple(sorted(gpos.tolist())))
                if compressed:
                    opos, osc = o.ph_last_selection(s, h)
                    spos = g.export_head(0, s, h, im.IM_S_SEL_POS)
                    so = np.argsort(spos, kind="stable")
                    assert np.array_equal(spos[so], opos), f"seq {s} head {h}: candidate positions differ"
                    check_scores(g.export_head(0, s, h, im.IM_S_SEL_IMP)[so], osc, f"seq {s} head {h}", self.stats)
                    assert len(g.export_head(0, s, h, im.IM_S_EVICTED)) == len(o.ph_last_evicted(s, h))
                if not np.array_equal(gpos[order], e["pos"]):
                    # allowed only inside the 1e-5 gap at this head's cut
                    opos, osc = o.ph_last_selection(s, h)
                    key = np.where(opos < wl.n_sink, np.inf, osc.astype(np.float64) + 0.0)
                    s_cut = np.sort(key)[::-1][wl.B - 1]
                    for ps in set(gpos.tolist()) ^ set(e["pos"].tolist()):
                        kk = key[np.nonzero(opos == ps)[0][0]]
                        assert abs(kk - s_cut) <= TOL_SCORE * max(1.0, abs(s_cut)), f"seq {s} head {h}: position {ps} (score {kk}), cut {s_cut}"
                    self.stats["cut_divergences"] += 1
                    resync = True
                    continue
                assert np.array_equal(g.export_head(0, s, h, im.IM_S_K)[order], e["K"]), f"seq {s} head {h}: K slab differs"
                assert np.array_equal(g.export_head(0, s, h, im.IM_S_V)[order], e["V"]), f"seq {s} head {h}: V slab differs"
                if self.scorer == 1:
                    check_scores(g.export_head(0, s, h, im.IM_S_IMP)[order], e["score"], f"seq {s} head {h} Knorm", self.stats)
            assert cnt["T"] == o.tokens_seen(s) and cnt["since"] == o.since(s) and cnt["evict_steps"] == o.evict_steps(s)
            self.stats["distinct_sets"] += len(set(sets)) > 1
            if not resync:
                Mo, bo = o.memory_kv(s)
                Mg = g.export(0, s, im.IM_S_M).astype(np.float64)
                bg = g.export(0, s, im.IM_S_B).astype(np.float64)
                if np.abs(Mo).max() > 0:
                    errM = np.abs(Mg - Mo).max() / np.abs(Mo).max()
                    self.stats["max_M_err"] = max(self.stats["max_M_err"], float(errM))
                    assert errM <= TOL_OUT, f"seq {s}: M error {errM:.3e}"
                    assert np.abs(bg - bo).max() / np.abs(bo).max() <= TOL_OUT, f"seq {s}: b error"
                else:
                    assert not Mg.any() and not bg.any()
            else:
                Mo, bo = o.memory_kv(s)
                heads = [o.ph_entries(s, h) for h in range(wl.Hkv)]
                g.import_head_state(0, s, heads=heads, M_kv=Mo.astype(np.float32), b=bo.astype(np.float32), T=o.tokens_seen(s),
                                    since=o.since(s), evict_steps=o.evict_steps(s))
            clean[s] = not resync
        return clean


@pytest.mark.parametrize("shape,scorer", [("llama8b_b1", 1), ("llama8b_b1", 2), ("qwen7b_b8", 1), ("qwen7b_b8", 2)])
def test_per_head_sets_against_the_oracle(shape, scorer):
    """G_q = 4 (Llama widths, 8 KV heads) and G_q = 7 (Qwen widths, 4 KV heads, d_M 448), three sequences, lognormal key
    norms so that Knorm separates the heads: two prefill chunks (the second evicts more entries per head than the first
    holds), then decode steps with an eviction every token, decay, float32 outputs held to 1e-4."""
    wl = synth.CONFIGS[shape].replace(name=f"ph_{shape}_{scorer}", n_seq=3, ctx=400, chunk=200, B=150, steps=14, tau=1,
                                     key_norm_sigma=0.5, n_needles=0)
    p = PerHeadPair(wl, scorer, out_f32=1, lambda_=0.9, eta=0.5)
    for c in range(wl.ctx // wl.chunk):
        p.prefill(c)
    for s in range(wl.steps):
        p.decode(s)
    st = p.stats
    assert st["max_out_err"] <= 1e-4 and st["max_M_err"] <= 2e-3 and st["max_score_err"] <= 1e-5 and st["cut_divergences"] <= 3
    assert st["distinct_sets"] > 0                      # the heads really keep different positions


def test_per_head_sets_long_interval_tiny_shape_and_no_memory():
    """head_dim 64 (the generic attention kernels), 2 KV heads, an eviction of 5 entries per head every 5 tokens, bf16
    outputs; then the same with the memory disabled (attention over each head's own set alone)."""
    for mem in (1, 0):
        wl = synth.CONFIGS["tiny"].replace(name=f"ph_tiny{mem}", H=8, Hkv=2, n_seq=2, ctx=90, chunk=90, B=40, steps=17, tau=5,
                                          key_norm_sigma=0.5, n_needles=0)
        p = PerHeadPair(wl, 1, enable_memory=mem)
        p.prefill(0)
        for s in range(wl.steps):
            p.decode(s)
        assert p.stats["max_out_err"] <= 2e-3 and p.stats["max_M_err"] <= 2e-3
        assert p.o.evict_steps(0) == 1 + 3


def test_per_head_with_one_row_for_all_heads_is_the_shared_row_path():
    """Handed, as every head's row, the scores the indexer path itself selected with (exported from a second context
    in the ordinary mode), the per-head context keeps the same positions in every head and produces the ordinary
    context's memory and outputs."""
    from paper_2605_25475_b200 import binding as im
    wl = synth.CONFIGS["llama8b_b1"].replace(name="ph_same_rows", n_seq=2, ctx=220, chunk=220, B=128, steps=6, n_needles=2)
    dev = torch.device("cuda:0")
    base = dict(n_layers=1, max_seqs=wl.n_seq, n_q_heads=wl.H, n_kv_heads=wl.Hkv, head_dim=wl.d, budget=wl.B, max_chunk=wl.chunk,
                n_sink=wl.n_sink, out_f32=1)
    a = im.IndexMem(im.Config(**base), dev)
    b = im.IndexMem(im.Config(scorer=2, **base), dev)
    w = synth.make_weights(wl, 0)
    a.set_weights(0, w)
    b.set_weights(0, w)
    ids = list(range(wl.n_seq))

    def rows_from(a, T):
        ext = np.full((wl.n_seq, wl.Hkv, T), -np.inf, np.float32)
        for s in ids:
            pos = a.export(0, s, im.IM_S_SEL_POS)
            ext[s, :, pos] = a.export(0, s, im.IM_S_SEL_IMP)[:, None]
        return torch.tensor(ext).to(dev)

    X, Qp, Q, K, V = [t.to(dev) for t in synth.prefill_inputs(wl, 0, 0)]
    a.prefill_chunk(0, ids, X, Qp, K, V)
    ext = rows_from(a, wl.ctx)
    b.set_scores(0, ext)
    b.prefill_chunk(0, ids, None, None, K, V)
    for step in range(wl.steps):
        x, qp, q, k, v = [t.to(dev) for t in synth.decode_inputs(wl, 0, step)]
        oa = a.decode_step(0, ids, x, qp, q, k, v).float().cpu().numpy()
        ext = rows_from(a, wl.ctx + step + 1)
        b.set_scores(0, ext)
        ob = b.decode_step(0, ids, None, None, q, k, v).float().cpu().numpy()
        assert a.status() == 0 and b.status() == 0
        assert np.abs(oa - ob).max() <= 1e-4 * np.abs(oa).max()
        for s in ids:
            want = sorted(a.export(0, s, im.IM_S_POS).tolist())
            for h in range(wl.Hkv):
                assert sorted(b.export_head(0, s, h, im.IM_S_POS).tolist()) == want
            Ma, Mb = a.export(0, s, im.IM_S_M), b.export(0, s, im.IM_S_M)
            assert np.abs(Ma - Mb).max() <= 1e-4 * np.abs(Ma).max()


def test_per_head_errors():
    from paper_2605_25475_b200 import binding as im
    wl = synth.CONFIGS["tiny"].replace(name="ph_err", H=8, Hkv=2, ctx=40, chunk=40, B=16, steps=1)
    dev = torch.device("cuda:0")
    g = im.IndexMem(im.Config(n_layers=1, max_seqs=1, n_q_heads=wl.H, n_kv_heads=wl.Hkv, head_dim=wl.d, budget=wl.B,
                              max_chunk=wl.chunk, scorer=2), dev)
    _, _, _, K, V = [t.to(dev) for t in synth.prefill_inputs(wl, 0, 0)]
    with pytest.raises(im.IndexMemError) as e:           # no scores yet
        g.prefill_chunk(0, [0], None, None, K, V)
    assert e.value.code == im.IM_ERR_STATE
    g.set_scores(0, torch.zeros((1, wl.Hkv, 39), device=dev))
    with pytest.raises(im.IndexMemError) as e:           # position 39 not covered
        g.prefill_chunk(0, [0], None, None, K, V)
    assert e.value.code == im.IM_ERR_ARG
    with pytest.raises(im.IndexMemError) as e:           # shared-row pieces are refused in this mode
        g.export(0, 0, im.IM_S_POS)
    assert e.value.code == im.IM_ERR_ARG
    # configurations that combine per-head sets with score reuse or chunk outputs are invalid
    for kw in (dict(score_share=2, n_layers=2), dict(chunk_outputs=1)):
        base = dict(n_layers=1, max_seqs=1, n_q_heads=8, n_kv_heads=2, head_dim=64, budget=16, scorer=1)
        base.update(kw)
        assert im.im_workspace_bytes(im.Config(**base).to_c()) == 0
