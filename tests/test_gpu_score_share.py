"""Reuse of one layer's indexer scores by the following layers of its group (``-m gpu``).

Configuration field ``score_share = g``: layers l with l % g != 0 make the selection of layer l - l % g (they
compute no indexer features and cache no indexer keys) and everything else - memory write from their own evicted
pairs, attention over their own retained entries, readout of their own memory - themselves.  Every layer of the
library context is followed by an oracle layer; the followers' oracles adopt their leader's pooled importances
(``decode_step_follow`` / ``prefill_chunk_follow``).  Retained positions, K / V copies, memory and outputs of every
layer are compared after every call; a selection decided inside the 1e-5 cut gap re-synchronises the whole group.
"""
import numpy as np
import pytest
import torch

from oracle import indexmem_oracle as orc
from paper_2605_25475_b200 import synth

pytestmark = pytest.mark.gpu


class Group:
    def __init__(self, wl, share, **over):
        from paper_2605_25475_b200 import binding as im
        self.im, self.wl, self.share = im, wl, share
        self.dev = torch.device("cuda:0")
        cfg = dict(n_layers=wl.n_layers, max_seqs=wl.n_seq, n_q_heads=wl.H, n_kv_heads=wl.Hkv, head_dim=wl.d, budget=wl.B,
                   compress_interval=wl.tau, max_chunk=wl.chunk, n_sink=wl.n_sink, score_share=share)
        ocfg = dict(H=wl.H, Hkv=wl.Hkv, d=wl.d, B=wl.B, tau=wl.tau, n_sink=wl.n_sink)
        for k, v in over.items():
            cfg[k] = v
            if k in ("lambda_", "eta"):
                ocfg[k] = v
        self.out_f32 = bool(over.get("out_f32", 0))
        self.g = im.IndexMem(im.Config(**cfg), self.dev)
        self.o = []
        for layer in range(wl.n_layers):
            w = synth.make_weights(wl, layer)
            self.g.set_weights(layer, w)
            o = orc.OracleLayer(orc.OracleConfig(**ocfg), wl.n_seq)
            o.set_weights({k: synth.f32(v) for k, v in w.items()})
            self.o.append(o)
        self.ids = list(range(wl.n_seq))
        self.stats = {"cut_divergences": 0, "kidx_flips": 0, "max_out_err": 0.0, "max_M_err": 0.0, "max_score_err": 0.0}

    def lead_of(self, layer):
        return layer - layer % self.share if self.share >= 2 else layer

    def _check(self, outs, refs, what):
        from tests.parity import check_unit_state, check_unit_out, resync_unit
        wl = self.wl
        for l0 in range(0, wl.n_layers, max(self.share, 1)):
            group = list(range(l0, min(l0 + max(self.share, 1), wl.n_layers)))
            for s in self.ids:
                clean = all([check_unit_state(self.g, l, s, self.o[l], s, self.stats, indexer=(l == self.lead_of(l))) for l in group])
                if not clean:
                    for l in group:       # one layer was re-synchronised (sorted slot order): keep the group's layouts alike
                        resync_unit(self.g, l, s, self.o[l], s)
                    continue
                if outs is None:
                    continue
                for l in group:
                    got = outs[l][s].float().cpu().numpy().astype(np.float64).reshape(refs[l][s].shape)
                    check_unit_out(got, refs[l][s], not self.out_f32, f"{what} unit {(l, s)}", self.stats, 1e-4 if self.out_f32 else 2e-3)
        assert self.g.status() == 0

    def prefill(self, c, attend=False):
        wl, dev = self.wl, self.dev
        outs, refs = {}, {}
        for layer in range(wl.n_layers):
            X, Qp, Q, K, V = synth.prefill_inputs(wl, layer, c)
            lead = self.lead_of(layer)
            if attend:
                outs[layer] = self.g.prefill_chunk_attend(layer, self.ids, X.to(dev), Qp.to(dev), Q.to(dev), K.to(dev), V.to(dev))
            else:
                self.g.prefill_chunk(layer, self.ids, X.to(dev), Qp.to(dev), K.to(dev), V.to(dev))
            ref = []
            for s in self.ids:
                if lead == layer:
                    _, od = self.o[layer].prefill_chunk_out(s, synth.f32(X[s]), synth.f32(Qp[s]), synth.f32(Q[s]), synth.f32(K[s]), synth.f32(V[s]))
                else:
                    _, od = self.o[layer].prefill_chunk_follow(s, self.o[lead], s, synth.f32(K[s]), synth.f32(V[s]), Q=synth.f32(Q[s]))
                ref.append(od)
            refs[layer] = ref
        self._check(outs if attend else None, refs, f"chunk {c}")

    def decode(self, step):
        wl, dev = self.wl, self.dev
        outs, refs = {}, {}
        for layer in range(wl.n_layers):
            x, qp, q, k, v = synth.decode_inputs(wl, layer, step)
            lead = self.lead_of(layer)
            outs[layer] = self.g.decode_step(layer, self.ids, x.to(dev), qp.to(dev), q.to(dev), k.to(dev), v.to(dev))
            ref = []
            for s in self.ids:
                if lead == layer:
                    _, od = self.o[layer].decode_step(s, synth.f32(x[s]), synth.f32(qp[s]), synth.f32(q[s]), synth.f32(k[s]), synth.f32(v[s]))
                else:
                    _, od = self.o[layer].decode_step_follow(s, self.o[lead], s, synth.f32(q[s]), synth.f32(k[s]), synth.f32(v[s]))
                ref.append(od)
            refs[layer] = ref
        self._check(outs, refs, f"step {step}")


@pytest.mark.parametrize("tau", [1, 5])
def test_groups_of_layers_share_one_score_row(tau):
    """Seven Llama-shaped layers in groups of three (the last group has one layer), two sequences, chunked prefill with
    the layer outputs of the chunks, then decode steps with an eviction every `tau` tokens, decay and float32 outputs."""
    wl = synth.CONFIGS["llama8b_b1"].replace(name=f"share_tau{tau}", n_layers=7, n_seq=2, ctx=360, chunk=120, B=150, steps=16,
                                            tau=tau, n_needles=3)
    grp = Group(wl, 3, out_f32=1, lambda_=0.95, eta=0.5, chunk_outputs=1)
    for c in range(wl.ctx // wl.chunk):
        grp.prefill(c, attend=True)
    for s in range(wl.steps):
        grp.decode(s)
    st = grp.stats
    assert st["max_out_err"] <= 1e-4 and st["max_M_err"] <= 2e-3 and st["max_score_err"] <= 1e-5 and st["cut_divergences"] <= 2
    # the followers of a group hold their leader's positions
    for l in range(wl.n_layers):
        for s in range(wl.n_seq):
            assert sorted(grp.g.export(l, s, grp.im.IM_S_POS).tolist()) == sorted(grp.g.export(grp.lead_of(l), s, grp.im.IM_S_POS).tolist())


def test_group_of_four_tiny_shape_and_period_one_is_todays_path():
    """The paper's period (four consecutive layers) at the tiny shape (head_dim 64: the generic kernels), and
    score_share = 1, which is every layer for itself."""
    wl = synth.CONFIGS["tiny"].replace(name="share4", n_layers=4, H=8, Hkv=2, n_seq=2, ctx=96, chunk=96, B=40, steps=10, n_needles=2)
    grp = Group(wl, 4)
    grp.prefill(0)
    for s in range(wl.steps):
        grp.decode(s)
    assert grp.stats["max_out_err"] <= 2e-3 and grp.stats["max_M_err"] <= 2e-3
    one = Group(wl.replace(name="share1", n_layers=2), 1)
    one.prefill(0)
    for s in range(4):
        one.decode(s)
    assert one.stats["max_out_err"] <= 2e-3


def test_a_follower_called_before_its_leader_is_refused():
    from paper_2605_25475_b200 import binding as im
    wl = synth.CONFIGS["tiny"].replace(name="share_order", n_layers=2, ctx=32, chunk=32, B=16, steps=1)
    grp = Group(wl, 2)
    dev = grp.dev
    X, Qp, Q, K, V = [t.to(dev) for t in synth.prefill_inputs(wl, 1, 0)]
    with pytest.raises(im.IndexMemError) as e:
        grp.g.prefill_chunk(1, grp.ids, X, Qp, K, V)
    assert e.value.code == im.IM_ERR_STATE
    grp.prefill(0)
    x, qp, q, k, v = [t.to(dev) for t in synth.decode_inputs(wl, 1, 0)]
    with pytest.raises(im.IndexMemError) as e:
        grp.g.decode_step(1, grp.ids, x, qp, q, k, v)
    assert e.value.code == im.IM_ERR_STATE
