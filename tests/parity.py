"""Drives the CUDA library and the CPU oracle side by side on the same seeded inputs and applies the
parity rules:

* retained position sets and evicted counts: bit-exact, except where the oracle's own float32
  scores leave a gap under 1e-5 * max(1, |s_cut|) at the cut (then the GPU state is re-synchronised
  from the oracle and the divergence is counted);
* cached indexer keys: bit-exact except isolated one-ulp bf16 flips (counted, re-synchronised);
* pooled scores: |gpu - oracle| <= 1e-5 * max(|s|, rms(row));
* outputs, M, b: max-abs error <= 2e-3 * max-abs of the oracle tensor; the bf16 output may in addition
  sit one bf16 ulp away from the oracle's rounded value (storage rounding of two values that agree
  to 1e-5 can still fall on different sides of a rounding boundary).

The oracle never receives anything computed by the CUDA path; re-synchronisation copies oracle
state into the library.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import indexmem_oracle as orc
from paper_2605_25475_b200 import binding as im
from paper_2605_25475_b200 import synth

TOL_SCORE = 1e-5
TOL_OUT = 2e-3


def bf16_ulp(x: np.ndarray) -> np.ndarray:
    """Spacing of bf16 numbers around x (float64 array)."""
    ax = np.maximum(np.abs(x), 2.0 ** -126)
    e = np.floor(np.log2(ax))
    return 2.0 ** (e - 7)


class Pair:
    def __init__(self, wl: synth.Workload, layer: int = 0, device="cuda:0", alias_q: bool = False, **over):
        # alias_q: pass ONE tensor as both the pre-RoPE query and the attention query (the header allows it);
        # otherwise the two are distinct tensors with different values, as in a backbone with rotary embeddings
        self.wl, self.layer, self.device, self.alias_q = wl, layer, device, alias_q
        ocfg = dict(H=wl.H, Hkv=wl.Hkv, d=wl.d, B=wl.B, tau=wl.tau, n_sink=wl.n_sink)
        gcfg = dict(n_layers=1, max_seqs=wl.n_seq, n_q_heads=wl.H, n_kv_heads=wl.Hkv, head_dim=wl.d, budget=wl.B,
                    compress_interval=wl.tau, max_chunk=wl.chunk, n_sink=wl.n_sink)
        names = {"HI": "n_index_heads", "dI": "index_dim", "dM": "mem_dim", "act": "act",
                 "enable_memory": "enable_memory", "lambda_": "lambda_", "eta": "eta", "eps": "eps",
                 "norm_eps": "norm_eps", "scale": "softmax_scale"}
        for k, v in over.items():
            if k in names:
                ocfg[k] = v
                gcfg[names[k]] = v
            else:
                gcfg[k] = v            # library-only knobs (out_f32, pending_slots, max_chunk)
        self.o = orc.OracleLayer(orc.OracleConfig(**ocfg), wl.n_seq)
        self.g = im.IndexMem(im.Config(**gcfg), device)
        # widths may have been overridden: draw the weights at the oracle's shapes, seeded like
        # synth.make_weights (identical to it when the widths are the paper's defaults)
        w = {}
        for name, shape in self.o.weight_shapes().items():
            if name == "b_g":
                w[name] = torch.zeros(1)
            else:
                w[name] = (synth._randn(shape, "cpu", wl.name, "w", layer, name) * wl.init_std).to(torch.bfloat16)
        self.weights = w
        self.o.set_weights({k: synth.f32(v) for k, v in w.items()})
        self.g.set_weights(0, w)
        self.stats = {"kidx_flips": 0, "cut_divergences": 0, "max_out_err": 0.0, "max_score_err": 0.0,
                      "max_M_err": 0.0, "steps": 0}
        self.seq_ids = list(range(wl.n_seq))

    # ------------------------------------------------------------------ drive both sides
    def prefill(self, chunk_idx: int, check=True):
        wl = self.wl
        X, Qp, _, K, V = synth.prefill_inputs(wl, self.layer, chunk_idx)
        self.o.prefill_batch(self.seq_ids, synth.f32(X), synth.f32(Qp), synth.f32(K), synth.f32(V))
        dev = self.device
        self.g.prefill_chunk(0, self.seq_ids, X.to(dev), Qp.to(dev), K.to(dev), V.to(dev))
        assert self.g.status() == 0
        if check:
            self.check_selection()
            self.check_state()

    def prefill_attend(self, chunk_idx: int, check=True):
        """The chunk through im_prefill_chunk_attend: state checks as for prefill(), plus the layer outputs of
        the chunk's own queries against the oracle (same bound as the decode outputs, row by row)."""
        wl = self.wl
        X, Qp, Q, K, V = synth.prefill_inputs(wl, self.layer, chunk_idx)
        if self.alias_q:
            Qp = Q
        ob, od = self.o.prefill_batch_out(self.seq_ids, synth.f32(X), synth.f32(Qp), synth.f32(Q), synth.f32(K), synth.f32(V))
        dev = self.device
        Qd = Q.to(dev)
        out = self.g.prefill_chunk_attend(0, self.seq_ids, X.to(dev), Qd if self.alias_q else Qp.to(dev), Qd, K.to(dev), V.to(dev))
        assert self.g.status() == 0
        if check:
            self.check_selection()
            self.check_state()
            n, Cn = od.shape[0], od.shape[1]
            self.check_out(out.reshape(n * Cn, wl.H, wl.d), ob.reshape(n * Cn, wl.H, wl.d), od.reshape(n * Cn, wl.H, wl.d))
        return out, ob, od

    def decode(self, step: int, check=True):
        wl = self.wl
        x, qp, q, k, v = synth.decode_inputs(wl, self.layer, step)
        if self.alias_q:
            qp = q
        ob, od = self.o.decode_batch(self.seq_ids, synth.f32(x), synth.f32(qp), synth.f32(q), synth.f32(k), synth.f32(v))
        dev = self.device
        qd = q.to(dev)
        out = self.g.decode_step(0, self.seq_ids, x.to(dev), qd if self.alias_q else qp.to(dev), qd, k.to(dev), v.to(dev))
        assert self.g.status() == 0
        self.stats["steps"] += 1
        if check:
            due = all(self.o.since(s) == 0 for s in self.seq_ids)
            if due:
                self.check_selection()
            ok = self.check_state()
            if ok:
                self.check_out(out, ob, od)
        return out, ob, od

    # ------------------------------------------------------------------ checks
    def check_out(self, out: torch.Tensor, ob: np.ndarray, od: np.ndarray):
        got = out.detach().to("cpu", torch.float32).numpy().astype(np.float64).reshape(od.shape)
        for s in range(od.shape[0]):
            ref = od[s]
            scale = np.abs(ref).max()
            err = np.abs(got[s] - ref)
            if out.dtype == torch.bfloat16:
                # storage rounding: half a bf16 ulp of the stored value (the larger binade if the two differ)
                half_ulp = 0.5 * bf16_ulp(np.maximum(np.abs(ref), np.abs(got[s])))
                assert np.all(err <= TOL_OUT * scale + half_ulp), \
                    f"seq {s}: out error {err.max():.3e} vs max-abs {scale:.3e}"
                # the pre-rounding error is what the 2e-3 bound is about: estimate it without the storage term
                self.stats["max_out_err"] = max(self.stats["max_out_err"],
                                                float(np.maximum(err - half_ulp, 0).max() / scale))
                # stored values that differ from the oracle's stored values are rounding flips; they are
                # counted, not bounded: planted needles make outputs exact bf16 ties (the mean of two
                # bf16 values), where a 1e-8 difference decides the rounding
                flips = got[s] != ob[s].astype(np.float64)
                self.stats["out_flips"] = self.stats.get("out_flips", 0) + int(flips.sum())
            else:
                assert err.max() <= TOL_OUT * scale, f"seq {s}: out error {err.max():.3e} vs max-abs {scale:.3e}"
                self.stats["max_out_err"] = max(self.stats["max_out_err"], float(err.max() / scale))

    def check_selection(self):
        """Compare what the last compression saw (scores) and decided (evicted set)."""
        for s in self.seq_ids:
            opos, oacc = self.o.last_selection(s)
            gpos = self.g.export(0, s, im.IM_S_SEL_POS)
            gimp = self.g.export(0, s, im.IM_S_SEL_IMP)
            assert len(gpos) == len(opos), f"seq {s}: selection saw {len(gpos)} entries, oracle {len(opos)}"
            order = np.argsort(gpos, kind="stable")
            assert np.array_equal(gpos[order], opos), f"seq {s}: candidate positions differ"
            self._check_scores(gimp[order], oacc, s)
            gev = self.g.export(0, s, im.IM_S_EVICTED)
            oev = self.o.last_evicted(s)
            assert len(gev) == len(oev), f"seq {s}: evicted {len(gev)} vs oracle {len(oev)}"

    def _check_scores(self, got: np.ndarray, ref: np.ndarray, s: int):
        check_scores(got, ref, f"seq {s}", self.stats)

    def check_state(self) -> bool:
        """Retained sets, cached indexer keys, memory.  Returns False if a benign divergence was
        found and the library was re-synchronised from the oracle (outputs of this step are then
        not comparable)."""
        clean = True
        for s in self.seq_ids:
            clean &= check_unit_state(self.g, 0, s, self.o, s, self.stats)
        return clean

    def resync(self, s):
        resync_unit(self.g, 0, s, self.o, s)


# ---------------------------------------------------------------------- one (layer, sequence) unit against its oracle
def check_unit_state(g, layer: int, seq: int, o, oseq: int, stats: dict, indexer: bool = True) -> bool:
    """State of library unit (layer, seq) against sequence ``oseq`` of oracle ``o``: counters, retained
    positions, cached indexer keys, pooled scores, K/V copies, M and b.  A divergence the parity rules
    allow (a selection decided inside the 1e-5 cut gap, an isolated one-ulp flip of a cached indexer key) is
    counted in ``stats`` and the unit re-synchronised from the oracle; the function then returns False (the
    outputs of the step just made are not comparable).  Anything else fails.  indexer = False: the unit belongs to a
    layer that reuses another layer's scores and keeps no indexer keys or pooled scores of its own."""
    e = o.entries(oseq)
    cnt = g.counts(layer, seq)
    assert cnt["n"] == len(e["pos"]), f"unit {(layer, seq)}: {cnt['n']} entries vs oracle {len(e['pos'])}"
    assert cnt["T"] == o.tokens_seen(oseq) and cnt["since"] == o.since(oseq)
    assert cnt["evict_steps"] == o.evict_steps(oseq)
    gpos = g.export(layer, seq, im.IM_S_POS)
    order = np.argsort(gpos, kind="stable")
    resync = False
    if not np.array_equal(gpos[order], e["pos"]):
        assert_cut_gap(o, oseq, set(gpos.tolist()), set(e["pos"].tolist()))
        stats["cut_divergences"] = stats.get("cut_divergences", 0) + 1
        resync = True
    else:
        gk = g.export(layer, seq, im.IM_S_KIDX)[order] if indexer else e["kidx"]
        diff = gk != e["kidx"]
        if diff.any():
            ulp = bf16_ulp(e["kidx"].astype(np.float64))
            assert np.all(np.abs(gk - e["kidx"])[diff] <= ulp[diff] * 1.0001), f"unit {(layer, seq)}: kidx off by more than one ulp"
            assert diff.sum() <= max(2, diff.size // 1000), f"unit {(layer, seq)}: {diff.sum()} kidx flips"
            stats["kidx_flips"] = stats.get("kidx_flips", 0) + int(diff.sum())
            resync = True
        if not resync and indexer:
            gimp = g.export(layer, seq, im.IM_S_IMP)[order]
            check_scores(gimp, e["acc"], f"unit {(layer, seq)}", stats)
        # K / V are copies: bit-exact
        assert np.array_equal(g.export(layer, seq, im.IM_S_K)[order], e["K"]), f"unit {(layer, seq)}: K cache differs"
        assert np.array_equal(g.export(layer, seq, im.IM_S_V)[order], e["V"]), f"unit {(layer, seq)}: V cache differs"
    if not resync:
        Mo, bo = o.memory_kv(oseq)
        Mg = g.export(layer, seq, im.IM_S_M).astype(np.float64)
        bg = g.export(layer, seq, im.IM_S_B).astype(np.float64)
        sm, sb = np.abs(Mo).max(), np.abs(bo).max()
        if sm > 0:
            errM = np.abs(Mg - Mo).max() / sm
            stats["max_M_err"] = max(stats.get("max_M_err", 0.0), float(errM))
            assert errM <= TOL_OUT, f"unit {(layer, seq)}: M error {errM:.3e}"
            assert np.abs(bg - bo).max() / sb <= TOL_OUT, f"unit {(layer, seq)}: b error"
        else:
            assert not Mg.any() and not bg.any()
    if resync:
        resync_unit(g, layer, seq, o, oseq)
    return not resync


def check_scores(got: np.ndarray, ref: np.ndarray, what: str, stats: dict):
    inf_ref = np.isneginf(ref)
    assert np.array_equal(np.isneginf(got), inf_ref), f"{what}: unscored entries differ"
    fin = ~inf_ref
    if fin.any():
        r = ref[fin].astype(np.float64)
        gg = got[fin].astype(np.float64)
        rms = np.sqrt(np.mean(r ** 2))
        rel = np.abs(gg - r) / np.maximum(np.abs(r), rms + 1e-300)
        stats["max_score_err"] = max(stats.get("max_score_err", 0.0), float(rel.max()))
        assert rel.max() <= TOL_SCORE, f"{what}: score error {rel.max():.3e}"


def check_unit_out(got: np.ndarray, od: np.ndarray, is_bf16: bool, what: str, stats: dict, tol: float = TOL_OUT):
    """One sequence's output rows ``got`` (float64 view of what the library stored) against the oracle's unrounded
    float64 rows ``od``: max-abs error within ``tol`` of the tensor's max-abs; a bf16 output gets half an ulp of
    storage rounding on top."""
    scale = np.abs(od).max()
    err = np.abs(got - od)
    if is_bf16:
        half_ulp = 0.5 * bf16_ulp(np.maximum(np.abs(od), np.abs(got)))
        assert np.all(err <= tol * scale + half_ulp), f"{what}: out error {err.max():.3e} vs max-abs {scale:.3e}"
        stats["max_out_err"] = max(stats.get("max_out_err", 0.0), float(np.maximum(err - half_ulp, 0).max() / scale))
    else:
        assert err.max() <= tol * scale, f"{what}: out error {err.max():.3e} vs max-abs {scale:.3e}"
        stats["max_out_err"] = max(stats.get("max_out_err", 0.0), float(err.max() / scale))


def assert_cut_gap(o, oseq: int, gset: set, oset: set):
    """Positions on which the two retained sets differ must all sit within 1e-5 * max(1, |s_cut|) of the
    oracle's own cut score."""
    opos, oacc = o.last_selection(oseq)
    key = np.where(opos < o.cfg.n_sink, np.inf, oacc.astype(np.float64) + 0.0)
    srt = np.sort(key)[::-1]
    s_cut = srt[o.cfg.B - 1]
    tol = TOL_SCORE * max(1.0, abs(s_cut))
    for p in (gset ^ oset):
        k = key[np.nonzero(opos == p)[0][0]]
        assert abs(k - s_cut) <= tol, f"position {p} (score {k}) differs from the oracle's set, cut {s_cut}"


def resync_unit(g, layer: int, seq: int, o, oseq: int):
    """Copies the oracle's state of one unit INTO the library (never the other way)."""
    e = o.entries(oseq)
    Mo, bo = o.memory_kv(oseq)
    g.import_state(layer, seq, pos=e["pos"], imp=e["acc"], kidx=e["kidx"], K=e["K"], V=e["V"],
                   M_kv=Mo.astype(np.float32), b=bo.astype(np.float32), T=o.tokens_seen(oseq),
                   since=o.since(oseq), evict_steps=o.evict_steps(oseq))
