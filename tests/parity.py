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
    def __init__(self, wl: synth.Workload, layer: int = 0, device="cuda:0", **over):
        self.wl, self.layer, self.device = wl, layer, device
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
        X, Q, K, V = synth.prefill_inputs(wl, self.layer, chunk_idx)
        self.o.prefill_batch(self.seq_ids, synth.f32(X), synth.f32(Q), synth.f32(K), synth.f32(V))
        dev = self.device
        self.g.prefill_chunk(0, self.seq_ids, X.to(dev), Q.to(dev), K.to(dev), V.to(dev))
        assert self.g.status() == 0
        if check:
            self.check_selection()
            self.check_state()

    def prefill_attend(self, chunk_idx: int, check=True):
        """The chunk through im_prefill_chunk_attend: state checks as for prefill(), plus the layer outputs of
        the chunk's own queries against the oracle (same bound as the decode outputs, row by row)."""
        wl = self.wl
        X, Q, K, V = synth.prefill_inputs(wl, self.layer, chunk_idx)
        ob, od = self.o.prefill_batch_out(self.seq_ids, synth.f32(X), synth.f32(Q), synth.f32(Q), synth.f32(K), synth.f32(V))
        dev = self.device
        out = self.g.prefill_chunk_attend(0, self.seq_ids, X.to(dev), Q.to(dev), Q.to(dev), K.to(dev), V.to(dev))
        assert self.g.status() == 0
        if check:
            self.check_selection()
            self.check_state()
            n, Cn = od.shape[0], od.shape[1]
            self.check_out(out.reshape(n * Cn, wl.H, wl.d), ob.reshape(n * Cn, wl.H, wl.d), od.reshape(n * Cn, wl.H, wl.d))
        return out, ob, od

    def decode(self, step: int, check=True):
        wl = self.wl
        x, q, k, v = synth.decode_inputs(wl, self.layer, step)
        ob, od = self.o.decode_batch(self.seq_ids, synth.f32(x), synth.f32(q), synth.f32(q), synth.f32(k), synth.f32(v))
        dev = self.device
        out = self.g.decode_step(0, self.seq_ids, x.to(dev), q.to(dev), q.to(dev), k.to(dev), v.to(dev))
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
        inf_ref = np.isneginf(ref)
        assert np.array_equal(np.isneginf(got), inf_ref), f"seq {s}: unscored entries differ"
        fin = ~inf_ref
        if fin.any():
            r = ref[fin].astype(np.float64)
            g = got[fin].astype(np.float64)
            rms = np.sqrt(np.mean(r ** 2))
            rel = np.abs(g - r) / np.maximum(np.abs(r), rms + 1e-300)
            self.stats["max_score_err"] = max(self.stats["max_score_err"], float(rel.max()))
            assert rel.max() <= TOL_SCORE, f"seq {s}: score error {rel.max():.3e}"

    def check_state(self) -> bool:
        """Retained sets, cached indexer keys, memory.  Returns False if a benign divergence was
        found and the library was re-synchronised from the oracle (outputs of this step are then
        not comparable)."""
        clean = True
        for s in self.seq_ids:
            e = self.o.entries(s)
            cnt = self.g.counts(0, s)
            assert cnt["n"] == len(e["pos"]), f"seq {s}: {cnt['n']} entries vs oracle {len(e['pos'])}"
            assert cnt["T"] == self.o.tokens_seen(s) and cnt["since"] == self.o.since(s)
            assert cnt["evict_steps"] == self.o.evict_steps(s)
            gpos = self.g.export(0, s, im.IM_S_POS)
            order = np.argsort(gpos, kind="stable")
            resync = False
            if not np.array_equal(gpos[order], e["pos"]):
                self._assert_cut_gap(s, set(gpos.tolist()), set(e["pos"].tolist()))
                self.stats["cut_divergences"] += 1
                resync = True
            else:
                gk = self.g.export(0, s, im.IM_S_KIDX)[order]
                diff = gk != e["kidx"]
                if diff.any():
                    ulp = bf16_ulp(e["kidx"].astype(np.float64))
                    assert np.all(np.abs(gk - e["kidx"])[diff] <= ulp[diff] * 1.0001), f"seq {s}: kidx off by more than one ulp"
                    assert diff.sum() <= max(2, diff.size // 1000), f"seq {s}: {diff.sum()} kidx flips"
                    self.stats["kidx_flips"] += int(diff.sum())
                    resync = True
                gimp = self.g.export(0, s, im.IM_S_IMP)[order]
                if not resync:
                    self._check_scores(gimp, e["acc"], s)
                # K / V are copies: bit-exact
                assert np.array_equal(self.g.export(0, s, im.IM_S_K)[order], e["K"]), f"seq {s}: K cache differs"
                assert np.array_equal(self.g.export(0, s, im.IM_S_V)[order], e["V"]), f"seq {s}: V cache differs"
            if not resync:
                Mo, bo = self.o.memory_kv(s)
                Mg = self.g.export(0, s, im.IM_S_M).astype(np.float64)
                bg = self.g.export(0, s, im.IM_S_B).astype(np.float64)
                sm, sb = np.abs(Mo).max(), np.abs(bo).max()
                if sm > 0:
                    errM = np.abs(Mg - Mo).max() / sm
                    self.stats["max_M_err"] = max(self.stats["max_M_err"], float(errM))
                    assert errM <= TOL_OUT, f"seq {s}: M error {errM:.3e}"
                    assert np.abs(bg - bo).max() / sb <= TOL_OUT, f"seq {s}: b error"
                else:
                    assert not Mg.any() and not bg.any()
            if resync:
                self.resync(s)
                clean = False
        return clean

    def _assert_cut_gap(self, s, gset, oset):
        opos, oacc = self.o.last_selection(s)
        wl = self.wl
        key = np.where(opos < wl.n_sink, np.inf, oacc.astype(np.float64) + 0.0)
        srt = np.sort(key)[::-1]
        B = self.o.cfg.B
        s_cut = srt[B - 1]
        tol = TOL_SCORE * max(1.0, abs(s_cut))
        for p in (gset ^ oset):
            k = key[np.nonzero(opos == p)[0][0]]
            assert abs(k - s_cut) <= tol, f"seq {s}: position {p} (score {k}) differs from the oracle's set, cut {s_cut}"

    def resync(self, s):
        e = self.o.entries(s)
        Mo, bo = self.o.memory_kv(s)
        self.g.import_state(0, s, pos=e["pos"], imp=e["acc"], kidx=e["kidx"], K=e["K"], V=e["V"],
                            M_kv=Mo.astype(np.float32), b=bo.astype(np.float32), T=self.o.tokens_seen(s),
                            since=self.o.since(s), evict_steps=self.o.evict_steps(s))
