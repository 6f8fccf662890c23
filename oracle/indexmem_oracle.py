"""ctypes front end of the IndexMem CPU oracle (TEST INFRASTRUCTURE, not product code).

Only the tests, the smoke check and the CPU-baseline leg of the benchmark may import this
module.  It loads ``libindexmem_oracle.so`` built from ``indexmem_oracle.cpp`` (plain C++17,
double accumulation) and never touches the CUDA library.

All arrays crossing this boundary are float32 numpy arrays holding bf16-representable values
(inputs, weights, caches) or float64 arrays (scores, state, unrounded outputs).
"""
from __future__ import annotations

import ctypes as C
import math
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "indexmem_oracle.cpp")
_LIB = os.path.join(_HERE, "libindexmem_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (-O2 -fopenmp).  Building the checker is not using it."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-std=c++17", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


class _Cfg(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("H", "Hkv", "d", "HI", "dI", "dM", "B", "tau", "n_sink", "act", "enable_memory", "scorer")] + \
               [(n, C.c_double) for n in ("scale", "lambda_", "eta", "eps", "norm_eps")]


@dataclass
class OracleConfig:
    """Hyper-parameters of one IndexMem layer, in the paper's notation.

    Widths default to the paper's training set-up: H_index = H/4, d_index = d_head/8,
    d_mem = d_model/8.
    """
    H: int
    Hkv: int
    d: int
    B: int
    HI: int = 0
    dI: int = 0
    dM: int = 0
    tau: int = 1
    n_sink: int = 4
    act: int = 0
    enable_memory: int = 1
    scorer: int = 0          # 0 the learnable indexer; retained sets per KV head: 1 Knorm (Sec. 2.2), 2 scores from the caller
    scale: float = 0.0
    lambda_: float = 1.0
    eta: float = 1.0
    eps: float = 1e-6
    norm_eps: float = 1e-6

    def resolved(self) -> "OracleConfig":
        c = OracleConfig(**self.__dict__)
        if c.HI == 0:
            c.HI = max(1, c.H // 4)
        if c.dI == 0:
            c.dI = max(1, c.d // 8)
        if c.dM == 0:
            c.dM = max(1, (c.H * c.d) // 8)
        if c.scale == 0.0:
            c.scale = 1.0 / math.sqrt(c.d)
        return c


_lib = None


def _load():
    global _lib
    if _lib is not None:
        return _lib
    build()
    L = C.CDLL(_LIB)
    vp, i32, i64, f64 = C.c_void_p, C.c_int32, C.c_int64, C.c_double
    L.orc_create.restype = vp
    L.orc_create.argtypes = [C.POINTER(_Cfg), C.c_int]
    L.orc_destroy.argtypes = [vp]
    L.orc_set_weights.argtypes = [vp, C.c_int, vp, i64]
    L.orc_prefill_chunk.argtypes = [vp, C.c_int, C.c_int, vp, vp, vp, vp]
    L.orc_decode_step.argtypes = [vp, C.c_int, vp, vp, vp, vp, vp, vp, vp]
    L.orc_decode_batch.argtypes = [vp, C.c_int, vp, vp, vp, vp, vp, vp, vp, vp]
    L.orc_prefill_batch.argtypes = [vp, C.c_int, vp, C.c_int, vp, vp, vp, vp]
    L.orc_prefill_chunk_out.argtypes = [vp, C.c_int, C.c_int, vp, vp, vp, vp, vp, vp, vp]
    L.orc_prefill_batch_out.argtypes = [vp, C.c_int, vp, C.c_int, vp, vp, vp, vp, vp, vp, vp]
    L.orc_decode_step_follow.argtypes = [vp, C.c_int, vp, C.c_int, vp, vp, vp, vp, vp]
    L.orc_prefill_chunk_follow.argtypes = [vp, C.c_int, vp, C.c_int, C.c_int, vp, vp, vp, vp, vp]
    L.orc_ph_decode_step.argtypes = [vp, C.c_int, vp, vp, vp, vp, i64, vp, vp]
    L.orc_ph_prefill_chunk.argtypes = [vp, C.c_int, C.c_int, vp, vp, vp, vp, i64, vp, vp]
    L.orc_ph_count.argtypes = [vp, C.c_int, C.c_int]
    L.orc_ph_export.argtypes = [vp, C.c_int, C.c_int, vp, vp, vp, vp]
    L.orc_ph_last_evicted.argtypes = [vp, C.c_int, C.c_int, vp, C.c_int]
    L.orc_ph_last_selection.argtypes = [vp, C.c_int, C.c_int, vp, vp, C.c_int]
    L.orc_count.argtypes = [vp, C.c_int]
    L.orc_tokens_seen.argtypes = [vp, C.c_int]
    L.orc_tokens_seen.restype = i64
    L.orc_since.argtypes = [vp, C.c_int]
    L.orc_evict_steps.argtypes = [vp, C.c_int]
    L.orc_evict_steps.restype = i64
    L.orc_export_entries.argtypes = [vp, C.c_int, vp, vp, vp, vp, vp]
    L.orc_export_memory.argtypes = [vp, C.c_int, vp, vp]
    L.orc_last_evicted.argtypes = [vp, C.c_int, vp, C.c_int]
    L.orc_last_selection.argtypes = [vp, C.c_int, vp, vp, C.c_int]
    L.orc_index_key.argtypes = [vp, vp, vp]
    L.orc_index_query.argtypes = [vp, vp, vp, vp, vp]
    L.orc_index_scores.argtypes = [vp, vp, vp, vp, C.c_int, vp]
    L.orc_select_top_b.argtypes = [vp, vp, C.c_int, C.c_int, C.c_int, vp]
    L.orc_phi.argtypes = [vp, vp, vp]
    L.orc_phi_kv.argtypes = [vp, vp, vp]
    L.orc_mem_read.argtypes = [vp, C.c_int, vp, vp, vp]
    L.orc_attention.argtypes = [vp, C.c_int, vp, vp]
    L.orc_bf16_round.argtypes = [f64]
    L.orc_bf16_round.restype = f64
    _lib = L
    return L


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float32))


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


WEIGHT_NAMES = ("U_q", "U_k", "G", "W_theta", "w_g", "b_g")


class OracleLayer:
    """One IndexMem layer with ``n_seq`` independent sequence states."""

    def __init__(self, cfg: OracleConfig, n_seq: int = 1):
        self.lib = _load()
        self.cfg = cfg.resolved()
        c = self.cfg
        assert c.H % c.Hkv == 0
        self.D, self.Dkv, self.Gq = c.H * c.d, c.Hkv * c.d, c.H // c.Hkv
        raw = _Cfg(c.H, c.Hkv, c.d, c.HI, c.dI, c.dM, c.B, c.tau, c.n_sink, c.act, c.enable_memory, c.scorer,
                   c.scale, c.lambda_, c.eta, c.eps, c.norm_eps)
        self.n_seq = n_seq
        self.h = self.lib.orc_create(C.byref(raw), n_seq)

    def __del__(self):
        if getattr(self, "h", None):
            self.lib.orc_destroy(self.h)
            self.h = None

    # ---- weights
    def weight_shapes(self):
        c = self.cfg
        return {"U_q": (c.HI * c.dI, self.D), "U_k": (c.dI, self.D), "G": (c.HI, self.D),
                "W_theta": (c.dM, self.D), "w_g": (self.D,), "b_g": (1,)}

    def set_weights(self, weights: dict):
        for i, name in enumerate(WEIGHT_NAMES):
            if name in weights:
                a = _f32(weights[name]).reshape(-1)
                rc = self.lib.orc_set_weights(self.h, i, _p(a), a.size)
                assert rc == 0, f"bad weight {name}: {a.size}"

    # ---- the two calls
    def prefill_chunk(self, seq: int, X, Qpre, K, V):
        X, Qpre, K, V = _f32(X), _f32(Qpre), _f32(K), _f32(V)
        Cn = X.shape[0]
        assert X.shape == (Cn, self.D) and Qpre.size == Cn * self.D and K.size == Cn * self.Dkv and V.size == K.size
        self.lib.orc_prefill_chunk(self.h, seq, Cn, _p(X), _p(Qpre), _p(K), _p(V))

    def prefill_batch(self, seq_ids, X, Qpre, K, V):
        X, Qpre, K, V = _f32(X), _f32(Qpre), _f32(K), _f32(V)
        ids = np.ascontiguousarray(np.asarray(seq_ids, dtype=np.int32))
        n, Cn = X.shape[0], X.shape[1]
        assert n == ids.size and X.shape == (n, Cn, self.D)
        self.lib.orc_prefill_batch(self.h, n, _p(ids), Cn, _p(X), _p(Qpre), _p(K), _p(V))

    def prefill_chunk_out(self, seq: int, X, Qpre, Q, K, V):
        """prefill_chunk that also returns the layer outputs of the chunk's own queries:
        (out_bf16 [C,H,d] float32 holding bf16 values, out_f64 [C,H,d])."""
        X, Qpre, Q, K, V = _f32(X), _f32(Qpre), _f32(Q), _f32(K), _f32(V)
        Cn = X.shape[0]
        assert X.shape == (Cn, self.D) and Qpre.size == Cn * self.D and Q.size == Cn * self.D
        assert K.size == Cn * self.Dkv and V.size == K.size
        ob = np.empty((Cn, self.cfg.H, self.cfg.d), dtype=np.float32)
        od = np.empty((Cn, self.cfg.H, self.cfg.d), dtype=np.float64)
        self.lib.orc_prefill_chunk_out(self.h, seq, Cn, _p(X), _p(Qpre), _p(Q), _p(K), _p(V), _p(ob), _p(od))
        return ob, od

    def prefill_batch_out(self, seq_ids, X, Qpre, Q, K, V):
        X, Qpre, Q, K, V = _f32(X), _f32(Qpre), _f32(Q), _f32(K), _f32(V)
        ids = np.ascontiguousarray(np.asarray(seq_ids, dtype=np.int32))
        n, Cn = X.shape[0], X.shape[1]
        assert n == ids.size and X.shape == (n, Cn, self.D) and Q.size == X.size
        ob = np.empty((n, Cn, self.cfg.H, self.cfg.d), dtype=np.float32)
        od = np.empty((n, Cn, self.cfg.H, self.cfg.d), dtype=np.float64)
        self.lib.orc_prefill_batch_out(self.h, n, _p(ids), Cn, _p(X), _p(Qpre), _p(Q), _p(K), _p(V), _p(ob), _p(od))
        return ob, od

    def decode_step(self, seq: int, x, q_pre, q, k_new, v_new):
        """Returns (out_bf16 [H,d] float32 holding bf16 values, out_f64 [H,d])."""
        x, q_pre, q, k_new, v_new = _f32(x), _f32(q_pre), _f32(q), _f32(k_new), _f32(v_new)
        assert x.size == self.D and q_pre.size == self.D and q.size == self.D
        assert k_new.size == self.Dkv and v_new.size == self.Dkv
        ob = np.empty((self.cfg.H, self.cfg.d), np.float32)
        od = np.empty((self.cfg.H, self.cfg.d), np.float64)
        self.lib.orc_decode_step(self.h, seq, _p(x), _p(q_pre), _p(q), _p(k_new), _p(v_new), _p(ob), _p(od))
        return ob, od

    def decode_batch(self, seq_ids, x, q_pre, q, k_new, v_new):
        x, q_pre, q, k_new, v_new = _f32(x), _f32(q_pre), _f32(q), _f32(k_new), _f32(v_new)
        ids = np.ascontiguousarray(np.asarray(seq_ids, dtype=np.int32))
        n = ids.size
        assert x.size == n * self.D and k_new.size == n * self.Dkv
        ob = np.empty((n, self.cfg.H, self.cfg.d), np.float32)
        od = np.empty((n, self.cfg.H, self.cfg.d), np.float64)
        self.lib.orc_decode_batch(self.h, n, _p(ids), _p(x), _p(q_pre), _p(q), _p(k_new), _p(v_new), _p(ob), _p(od))
        return ob, od

    # ---- a layer that reuses the indexer scores of the leading layer of its group (App. B, IndexCache-style reuse)
    def decode_step_follow(self, seq: int, lead: "OracleLayer", lead_seq: int, q, k_new, v_new):
        """decode_step for a layer that adopts `lead`'s pooled importances (matched by token position) instead of
        scoring with an indexer of its own; `lead` must already have made the call for the same token."""
        q, k_new, v_new = _f32(q), _f32(k_new), _f32(v_new)
        assert q.size == self.D and k_new.size == self.Dkv and v_new.size == self.Dkv
        ob = np.empty((self.cfg.H, self.cfg.d), np.float32)
        od = np.empty((self.cfg.H, self.cfg.d), np.float64)
        rc = self.lib.orc_decode_step_follow(self.h, seq, lead.h, lead_seq, _p(q), _p(k_new), _p(v_new), _p(ob), _p(od))
        assert rc == 0, "the leading layer's scores do not cover this layer's entries"
        return ob, od

    def prefill_chunk_follow(self, seq: int, lead: "OracleLayer", lead_seq: int, K, V, Q=None):
        """prefill_chunk for such a layer; with Q [C,H,d] also returns the layer outputs of the chunk's own queries."""
        K, V = _f32(K), _f32(V)
        Cn = K.size // self.Dkv
        assert K.size == Cn * self.Dkv and V.size == K.size
        ob = od = None
        if Q is not None:
            Q = _f32(Q)
            assert Q.size == Cn * self.D
            ob = np.empty((Cn, self.cfg.H, self.cfg.d), dtype=np.float32)
            od = np.empty((Cn, self.cfg.H, self.cfg.d), dtype=np.float64)
        rc = self.lib.orc_prefill_chunk_follow(self.h, seq, lead.h, lead_seq, Cn, _p(Q) if Q is not None else None, _p(K), _p(V),
                                               _p(ob) if ob is not None else None, _p(od) if od is not None else None)
        assert rc == 0, "the leading layer's scores do not cover this layer's entries"
        return ob, od

    # ---- a retained set per KV head (Sec. 2.2 framework; configuration scorer = 1 Knorm, 2 scores from the caller)
    def _ext(self, ext):
        if ext is None:
            return None, 0
        ext = np.ascontiguousarray(np.asarray(ext, dtype=np.float32))
        assert ext.ndim == 2 and ext.shape[0] == self.cfg.Hkv, "scores are [Hkv, positions]"
        return ext, ext.shape[1]

    def ph_decode_step(self, seq: int, q, k_new, v_new, ext=None):
        """One decode token; ext: float32 [Hkv, positions] scores by token position (scorer 2), used if the call compresses."""
        q, k_new, v_new = _f32(q), _f32(k_new), _f32(v_new)
        assert q.size == self.D and k_new.size == self.Dkv and v_new.size == self.Dkv
        ext, n_pos = self._ext(ext)
        ob = np.empty((self.cfg.H, self.cfg.d), np.float32)
        od = np.empty((self.cfg.H, self.cfg.d), np.float64)
        rc = self.lib.orc_ph_decode_step(self.h, seq, _p(q), _p(k_new), _p(v_new), _p(ext) if ext is not None else None, n_pos, _p(ob), _p(od))
        assert rc == 0, "scores from the caller are missing or do not cover the cached positions"
        return ob, od

    def ph_prefill_chunk(self, seq: int, K, V, Q=None, ext=None):
        K, V = _f32(K), _f32(V)
        Cn = K.size // self.Dkv
        assert K.size == Cn * self.Dkv and V.size == K.size
        ext, n_pos = self._ext(ext)
        ob = od = None
        if Q is not None:
            Q = _f32(Q)
            assert Q.size == Cn * self.D
            ob = np.empty((Cn, self.cfg.H, self.cfg.d), dtype=np.float32)
            od = np.empty((Cn, self.cfg.H, self.cfg.d), dtype=np.float64)
        rc = self.lib.orc_ph_prefill_chunk(self.h, seq, Cn, _p(Q) if Q is not None else None, _p(K), _p(V),
                                           _p(ext) if ext is not None else None, n_pos,
                                           _p(ob) if ob is not None else None, _p(od) if od is not None else None)
        assert rc == 0, "scores from the caller are missing or do not cover the cached positions"
        return ob, od

    def ph_entries(self, seq: int, head: int):
        """dict(pos int32[n], score f32[n], K f32[n,d], V f32[n,d]) of one KV head's retained set; ascending pos."""
        n, c = self.lib.orc_ph_count(self.h, seq, head), self.cfg
        pos = np.empty(n, np.int32)
        score = np.empty(n, np.float32)
        K = np.empty((n, c.d), np.float32)
        V = np.empty((n, c.d), np.float32)
        self.lib.orc_ph_export(self.h, seq, head, _p(pos), _p(score), _p(K), _p(V))
        return {"pos": pos, "score": score, "K": K, "V": V}

    def ph_last_evicted(self, seq: int, head: int) -> np.ndarray:
        cap = max(1, self.lib.orc_ph_last_evicted(self.h, seq, head, None, 0))
        buf = np.empty(cap, np.int32)
        n = self.lib.orc_ph_last_evicted(self.h, seq, head, _p(buf), cap)
        return buf[:n]

    def ph_last_selection(self, seq: int, head: int):
        n = self.lib.orc_ph_last_selection(self.h, seq, head, None, None, 0)
        pos = np.empty(max(n, 1), np.int32)
        score = np.empty(max(n, 1), np.float32)
        self.lib.orc_ph_last_selection(self.h, seq, head, _p(pos), _p(score), n)
        return pos[:n], score[:n]

    # ---- state
    def count(self, seq=0) -> int:
        return self.lib.orc_count(self.h, seq)

    def tokens_seen(self, seq=0) -> int:
        return self.lib.orc_tokens_seen(self.h, seq)

    def since(self, seq=0) -> int:
        return self.lib.orc_since(self.h, seq)

    def evict_steps(self, seq=0) -> int:
        return self.lib.orc_evict_steps(self.h, seq)

    def entries(self, seq=0):
        """dict(pos int32[n], acc f32[n], kidx f32[n,dI], K f32[n,Hkv,d], V f32[n,Hkv,d]); ascending pos."""
        n, c = self.count(seq), self.cfg
        pos = np.empty(n, np.int32)
        acc = np.empty(n, np.float32)
        kidx = np.empty((n, c.dI), np.float32)
        K = np.empty((n, c.Hkv, c.d), np.float32)
        V = np.empty((n, c.Hkv, c.d), np.float32)
        self.lib.orc_export_entries(self.h, seq, _p(pos), _p(acc), _p(kidx), _p(K), _p(V))
        return {"pos": pos, "acc": acc, "kidx": kidx, "K": K, "V": V}

    def positions(self, seq=0) -> np.ndarray:
        n = self.count(seq)
        pos = np.empty(n, np.int32)
        self.lib.orc_export_entries(self.h, seq, _p(pos), None, None, None, None)
        return pos

    def memory(self, seq=0):
        """(M [dM, D] model space, b [dM]) as float64."""
        c = self.cfg
        M = np.empty((c.dM, self.D), np.float64)
        b = np.empty(c.dM, np.float64)
        self.lib.orc_export_memory(self.h, seq, _p(M), _p(b))
        return M, b

    def memory_kv(self, seq=0):
        """The latent state in KV space: M_kv[m, g*d + c] = M[m, j*d + c] for any query head j of group g."""
        c = self.cfg
        M, b = self.memory(seq)
        Mv = M.reshape(c.dM, c.H, c.d)[:, ::self.Gq, :].reshape(c.dM, self.Dkv)
        return np.ascontiguousarray(Mv), b

    def last_evicted(self, seq=0) -> np.ndarray:
        cap = max(1, self.lib.orc_last_evicted(self.h, seq, None, 0))
        buf = np.empty(cap, np.int32)
        n = self.lib.orc_last_evicted(self.h, seq, _p(buf), cap)
        return buf[:n]

    def last_selection(self, seq=0):
        """(pos int32[n], acc float32[n]) of the entries the latest compression chose among."""
        n = self.lib.orc_last_selection(self.h, seq, None, None, 0)
        pos = np.empty(max(n, 1), np.int32)
        acc = np.empty(max(n, 1), np.float32)
        self.lib.orc_last_selection(self.h, seq, _p(pos), _p(acc), n)
        return pos[:n], acc[:n]

    # ---- stage functions
    def index_key(self, x) -> np.ndarray:
        x = _f32(x)
        out = np.empty(self.cfg.dI, np.float32)
        self.lib.orc_index_key(self.h, _p(x), _p(out))
        return out

    def index_query(self, x, q_pre):
        x, q_pre = _f32(x), _f32(q_pre)
        qf = np.empty((self.cfg.HI, self.cfg.dI), np.float64)
        al = np.empty(self.cfg.HI, np.float64)
        self.lib.orc_index_query(self.h, _p(x), _p(q_pre), _p(qf), _p(al))
        return qf, al

    def index_scores(self, qf, alpha, kidx) -> np.ndarray:
        qf = np.ascontiguousarray(qf, np.float64)
        alpha = np.ascontiguousarray(alpha, np.float64)
        kidx = _f32(kidx)
        n = kidx.shape[0]
        A = np.empty(n, np.float64)
        self.lib.orc_index_scores(self.h, _p(qf), _p(alpha), _p(kidx), n, _p(A))
        return A

    def phi(self, u_model) -> np.ndarray:
        u = _f32(u_model)
        out = np.empty(self.cfg.dM, np.float64)
        self.lib.orc_phi(self.h, _p(u), _p(out))
        return out

    def phi_kv(self, kv) -> np.ndarray:
        kv = _f32(kv)
        out = np.empty(self.cfg.dM, np.float64)
        self.lib.orc_phi_kv(self.h, _p(kv), _p(out))
        return out

    def mem_read(self, seq, q):
        q = _f32(q)
        m = np.empty(self.D, np.float64)
        g = C.c_double(0.0)
        self.lib.orc_mem_read(self.h, seq, _p(q), _p(m), C.byref(g))
        return m, g.value

    def attention(self, seq, q) -> np.ndarray:
        q = _f32(q)
        o = np.empty((self.cfg.H, self.cfg.d), np.float64)
        self.lib.orc_attention(self.h, seq, _p(q), _p(o))
        return o


def select_top_b(score, pos, B: int, n_sink: int) -> np.ndarray:
    """keep mask (uint8[n]) of the budgeted selection: (key desc, position asc), sinks first."""
    L = _load()
    score = _f32(score)
    pos = np.ascontiguousarray(pos, np.int32)
    keep = np.empty(score.size, np.uint8)
    L.orc_select_top_b(_p(score), _p(pos), score.size, B, n_sink, _p(keep))
    return keep


def bf16_round(x: float) -> float:
    return _load().orc_bf16_round(float(x))
