"""Thin ctypes binding of ``libindexmem.so`` (see ``include/indexmem.h``).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.  PyTorch
supplies device memory (tensors), the current CUDA stream and nothing else.  There is no CPU
fallback: if the shared library is missing, importing this module raises.

Module-level functions carry the names of the C entry points (``im_create`` ... ``im_destroy``);
``IndexMem`` is a small object wrapper around them.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass, fields

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "lib", "libindexmem.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2605_25475_b200.buildlib` "
        "(there is no CPU fallback)")
_lib = C.CDLL(LIB_PATH)

IM_OK, IM_ERR_ARG, IM_ERR_CAPACITY, IM_ERR_STATE, IM_ERR_CUDA, IM_ERR_TIMEOUT = 0, -1, -2, -3, -4, -5
IM_W_UQ, IM_W_UK, IM_W_G, IM_W_THETA, IM_W_WG, IM_W_BG = range(6)
IM_S_COUNTS, IM_S_POS, IM_S_IMP, IM_S_KIDX, IM_S_K, IM_S_V, IM_S_M, IM_S_B, IM_S_EVICTED, IM_S_SEL_POS, IM_S_SEL_IMP = range(11)
WEIGHT_IDS = {"U_q": IM_W_UQ, "U_k": IM_W_UK, "G": IM_W_G, "W_theta": IM_W_THETA, "w_g": IM_W_WG, "b_g": IM_W_BG}


class im_config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "n_layers", "max_seqs", "n_q_heads", "n_kv_heads", "head_dim", "n_index_heads", "index_dim", "mem_dim",
        "budget", "compress_interval", "max_chunk", "n_sink", "act", "enable_memory", "out_f32", "pending_slots", "chunk_outputs", "score_share", "scorer")] + \
        [(n, C.c_float) for n in ("softmax_scale", "lambda_", "eta", "eps", "norm_eps", "init_std")] + \
        [("seed", C.c_uint64)]


class IndexMemError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"indexmem error {code}: {msg}")
        self.code = code


_vp, _i32, _sz = C.c_void_p, C.c_int, C.c_size_t
_lib.im_workspace_bytes.restype = _sz
_lib.im_workspace_bytes.argtypes = [C.POINTER(im_config)]
_lib.im_create.argtypes = [C.POINTER(im_config), _vp, _sz, C.POINTER(_vp)]
_lib.im_destroy.argtypes = [_vp]
_lib.im_reset.argtypes = [_vp, _i32, _i32, _vp]
_lib.im_prefill_chunk.argtypes = [_vp, _i32, _i32, _vp, _i32, _vp, _vp, _vp, _vp, _vp]
_lib.im_prefill_chunk_attend.argtypes = [_vp, _i32, _i32, _vp, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.im_decode_step.argtypes = [_vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.im_decode_stack.argtypes = [_vp, _i32, _vp, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.im_decode_stack_events.argtypes = [_vp, _i32, _vp, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.im_set_weights.argtypes = [_vp, _i32, _i32, _vp, _sz]
_lib.im_get_weights.argtypes = [_vp, _i32, _i32, _vp, _sz]
_lib.im_state_export.argtypes = [_vp, _i32, _i32, _i32, _vp, _sz]
_lib.im_state_import.argtypes = [_vp, _i32, _i32, _i32, _vp, _sz]
_lib.im_topb_select.argtypes = [_vp, _vp, _i32, _i32, _i32, _i32, _vp, _vp, _vp]
_lib.im_set_scores.argtypes = [_vp, _i32, _i32, _vp, C.c_int64]
_lib.im_state_export_head.argtypes = [_vp, _i32, _i32, _i32, _i32, _vp, _sz]
_lib.im_state_import_head.argtypes = [_vp, _i32, _i32, _i32, _i32, _vp, _sz]
_lib.im_status.argtypes = [_vp, _vp, C.POINTER(C.c_int32)]
_lib.im_launch_count.argtypes = [_vp]
_lib.im_launch_count.restype = C.c_int64
_lib.im_get_config.argtypes = [_vp, C.POINTER(im_config), C.POINTER(C.c_int32)]
_lib.im_profile_begin.argtypes = [_vp, _i32]
_lib.im_profile_end.argtypes = [_vp, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
_lib.im_set_option.argtypes = [_vp, _i32, _i32]
_lib.im_event_count.argtypes = [_vp, _i32, C.POINTER(C.c_int64)]
_lib.im_attention_noalloc.argtypes = [_vp, _vp, _vp, _i32, _i32, _i32, _i32, C.c_float, _vp, _vp]
_lib.im_last_error.restype = C.c_char_p

EXPORTED = ("im_workspace_bytes", "im_create", "im_destroy", "im_reset", "im_prefill_chunk", "im_decode_step",
            "im_set_weights", "im_get_weights", "im_state_export", "im_state_import", "im_topb_select",
            "im_status", "im_launch_count", "im_get_config", "im_last_error", "im_profile_begin", "im_profile_end", "im_set_option", "im_attention_noalloc", "im_event_count", "im_prefill_chunk_attend",
            "im_set_scores", "im_state_export_head", "im_state_import_head", "im_decode_stack",
            "im_decode_stack_events")


def _check(rc: int):
    if rc != IM_OK:
        raise IndexMemError(rc, _lib.im_last_error().decode())


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dev(t: torch.Tensor, dtype, numel: int, name: str) -> int:
    if not (t.is_cuda and t.is_contiguous() and t.dtype == dtype and t.numel() == numel):
        raise ValueError(f"{name}: need a contiguous CUDA {dtype} tensor with {numel} elements, got "
                         f"{tuple(t.shape)} {t.dtype} {t.device}")
    return t.data_ptr()


def _ids(seq_ids) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(seq_ids, dtype=np.int32))


# ------------------------------------------------------------------ C entry points
def im_workspace_bytes(cfg: im_config) -> int:
    return int(_lib.im_workspace_bytes(C.byref(cfg)))


def im_create(cfg: im_config, workspace: torch.Tensor) -> int:
    """Returns the context handle (an integer address)."""
    h = _vp()
    _check(_lib.im_create(C.byref(cfg), workspace.data_ptr(), workspace.numel() * workspace.element_size(), C.byref(h)))
    return h.value


def im_destroy(ctx: int):
    _check(_lib.im_destroy(ctx))


def im_reset(ctx: int, layer: int = -1, seq: int = -1):
    _check(_lib.im_reset(ctx, layer, seq, _stream()))


def _ptr(t):
    return 0 if t is None else t.data_ptr()


def im_prefill_chunk(ctx, layer, seq_ids, chunk_len, x, q_pre, k, v):
    ids = _ids(seq_ids)
    _check(_lib.im_prefill_chunk(ctx, layer, ids.size, ids.ctypes.data, chunk_len, _ptr(x), _ptr(q_pre),
                                 k.data_ptr(), v.data_ptr(), _stream()))


def im_prefill_chunk_attend(ctx, layer, seq_ids, chunk_len, x, q_pre, q, k, v, out):
    ids = _ids(seq_ids)
    _check(_lib.im_prefill_chunk_attend(ctx, layer, ids.size, ids.ctypes.data, chunk_len, x.data_ptr(),
                                        q_pre.data_ptr(), q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                                        _stream()))


def im_decode_step(ctx, layer, seq_ids, x, q_pre, q, k_new, v_new, out):
    ids = _ids(seq_ids)
    _check(_lib.im_decode_step(ctx, layer, ids.size, ids.ctypes.data, _ptr(x), _ptr(q_pre), q.data_ptr(),
                               k_new.data_ptr(), v_new.data_ptr(), out.data_ptr(), _stream()))


def im_decode_stack(ctx, layers, seq_ids, x, q_pre, q, k_new, v_new, out):
    """x .. out: one tensor per layer (sequences of tensors, or tensors stacked over the layers)."""
    ids, lay = _ids(seq_ids), _ids(layers)
    lists = [np.asarray([t.data_ptr() for t in ts], dtype=np.uint64) for ts in (x, q_pre, q, k_new, v_new, out)]
    assert all(a.size == lay.size for a in lists)
    _check(_lib.im_decode_stack(ctx, lay.size, lay.ctypes.data, ids.size, ids.ctypes.data, *[a.ctypes.data for a in lists],
                                _stream()))


def _event_handles(events, n):
    """torch.cuda.Event objects (already recorded once, so that they exist), raw handles or None -> uint64 array."""
    if events is None:
        return None
    assert len(events) == n
    h = []
    for e in events:
        v = 0 if e is None else (e.cuda_event if hasattr(e, "cuda_event") else int(e))
        if e is not None and not v:
            raise ValueError("a CUDA event that has never been recorded has no handle yet: record it once first")
        h.append(v)
    return np.asarray(h, dtype=np.uint64)


def im_decode_stack_events(ctx, layers, seq_ids, x, q_pre, q, k_new, v_new, out, ready_events=None, done_events=None):
    """im_decode_stack with one event per layer for inputs that arrive and outputs that leave while the call runs."""
    ids, lay = _ids(seq_ids), _ids(layers)
    lists = [np.asarray([t.data_ptr() for t in ts], dtype=np.uint64) for ts in (x, q_pre, q, k_new, v_new, out)]
    assert all(a.size == lay.size for a in lists)
    rdy, don = _event_handles(ready_events, lay.size), _event_handles(done_events, lay.size)
    _check(_lib.im_decode_stack_events(ctx, lay.size, lay.ctypes.data, ids.size, ids.ctypes.data,
                                       *[a.ctypes.data for a in lists], None if rdy is None else rdy.ctypes.data,
                                       None if don is None else don.ctypes.data, _stream()))


def im_set_weights(ctx, layer, which, host: np.ndarray):
    host = np.ascontiguousarray(host)
    _check(_lib.im_set_weights(ctx, layer, which, host.ctypes.data, host.nbytes))


def im_get_weights(ctx, layer, which, host: np.ndarray):
    _check(_lib.im_get_weights(ctx, layer, which, host.ctypes.data, host.nbytes))


def im_state_export(ctx, layer, seq, which, host: np.ndarray):
    _check(_lib.im_state_export(ctx, layer, seq, which, host.ctypes.data, host.nbytes))


def im_state_import(ctx, layer, seq, which, host: np.ndarray):
    host = np.ascontiguousarray(host)
    _check(_lib.im_state_import(ctx, layer, seq, which, host.ctypes.data, host.nbytes))


def im_set_scores(ctx, layer, scores: torch.Tensor):
    """scores float32 [n_seq, Hkv, n_positions] (CUDA, contiguous): the importance of every token position per KV head
    for the next compressing call on `layer`; must stay alive until that call's kernels have run."""
    n_seq, _, n_pos = scores.shape
    _dev(scores, torch.float32, scores.numel(), "scores")
    _check(_lib.im_set_scores(ctx, layer, n_seq, scores.data_ptr(), n_pos))


def im_state_export_head(ctx, layer, seq, head, which, host: np.ndarray):
    _check(_lib.im_state_export_head(ctx, layer, seq, head, which, host.ctypes.data, host.nbytes))


def im_state_import_head(ctx, layer, seq, head, which, host: np.ndarray):
    host = np.ascontiguousarray(host)
    _check(_lib.im_state_import_head(ctx, layer, seq, head, which, host.ctypes.data, host.nbytes))


def im_topb_select(scores: torch.Tensor, pos: torch.Tensor, budget: int, n_sink: int):
    """scores float32 [rows, n], pos int32 [rows, n] (CUDA) -> (keep uint8 [rows, n], n_evict int32 [rows])."""
    rows, n = scores.shape
    _dev(scores, torch.float32, rows * n, "scores")
    _dev(pos, torch.int32, rows * n, "pos")
    keep = torch.empty((rows, n), dtype=torch.uint8, device=scores.device)
    nev = torch.empty((rows,), dtype=torch.int32, device=scores.device)
    _check(_lib.im_topb_select(scores.data_ptr(), pos.data_ptr(), rows, n, budget, n_sink, keep.data_ptr(),
                               nev.data_ptr(), _stream()))
    return keep, nev


def im_status(ctx) -> int:
    st = C.c_int32(0)
    _check(_lib.im_status(ctx, _stream(), C.byref(st)))
    return st.value


def im_profile_begin(ctx, max_records: int):
    _check(_lib.im_profile_begin(ctx, max_records))


def im_profile_end(ctx):
    """Returns (total_ms, n_records) of the attention + readout launches recorded since im_profile_begin."""
    ms, n = C.c_double(0.0), C.c_int64(0)
    _check(_lib.im_profile_end(ctx, C.byref(ms), C.byref(n)))
    return ms.value, n.value


IM_OPT_CONCURRENCY, IM_OPT_PREFETCH_NEXT, IM_OPT_PREFILL_TENSOR, IM_OPT_PROFILE_TARGET, IM_OPT_DECODE_TENSOR, IM_OPT_READOUT_STAGES, IM_OPT_WAIT_LIMIT, IM_OPT_LAYER_OVERLAP = 0, 1, 2, 3, 4, 5, 6, 7
IM_OPT_STACK_PIPELINE, IM_OPT_STACK_RESERVED, IM_OPT_STACK_CHUNKS, IM_OPT_FOLD_TENSOR, IM_OPT_PREFILL_PIPELINE = 8, 9, 10, 11, 12


def im_set_option(ctx, option: int, value: int):
    _check(_lib.im_set_option(ctx, option, value))


def im_attention_noalloc(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, softmax_scale: float = 0.0,
                         out: torch.Tensor | None = None) -> torch.Tensor:
    """Attention of one query token over k / v without any allocation inside the library.

    q bf16 [H, d], k and v bf16 [Hkv, n, d] (CUDA, contiguous).  The scratch is a fixed 4 MiB array
    inside the library, so H * ceil(n / 256) * (d + 2) must not exceed 1,048,576; calls must not
    overlap on the GPU.  Pass `out` (bf16 [H, d]) to keep this wrapper from allocating the result.
    """
    H, d = q.shape
    Hkv, n, d2 = k.shape
    bf = torch.bfloat16
    _dev(q, bf, H * d, "q"); _dev(k, bf, Hkv * n * d, "k"); _dev(v, bf, Hkv * n * d, "v")
    if d2 != d:
        raise ValueError("head_dim mismatch")
    if out is None:
        out = torch.empty((H, d), dtype=bf, device=q.device)
    _dev(out, bf, H * d, "out")
    _check(_lib.im_attention_noalloc(q.data_ptr(), k.data_ptr(), v.data_ptr(), H, Hkv, d, n, softmax_scale,
                                     out.data_ptr(), _stream()))
    return out


IM_COUNT_MERGE_RECOMPUTE = 0


def im_event_count(ctx, counter: int) -> int:
    v = C.c_int64(0)
    _check(_lib.im_event_count(ctx, counter, C.byref(v)))
    return int(v.value)


def im_launch_count(ctx) -> int:
    return int(_lib.im_launch_count(ctx))


# ------------------------------------------------------------------ object wrapper
@dataclass
class Config:
    """Python mirror of ``im_config`` (zero = the paper's default, see the header)."""
    n_layers: int
    max_seqs: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    budget: int
    n_index_heads: int = 0
    index_dim: int = 0
    mem_dim: int = 0
    compress_interval: int = 1
    max_chunk: int = 1
    n_sink: int = 4
    act: int = 0
    enable_memory: int = 1
    out_f32: int = 0
    pending_slots: int = 0
    chunk_outputs: int = 0
    score_share: int = 0
    scorer: int = 0
    softmax_scale: float = 0.0
    lambda_: float = 0.0
    eta: float = 0.0
    eps: float = 0.0
    norm_eps: float = 0.0
    init_std: float = 0.0
    seed: int = 0

    def to_c(self) -> im_config:
        c = im_config()
        for f in fields(self):
            setattr(c, f.name, getattr(self, f.name))
        return c


def _bf16_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.bfloat16).contiguous().view(torch.int16).numpy()


def _from_bf16_bits(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16)


class IndexMem:
    """Owns the workspace tensor and the context; methods map one-to-one onto the C calls."""

    def __init__(self, cfg: Config, device="cuda:0"):
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.ccfg = cfg.to_c()
        nbytes = im_workspace_bytes(self.ccfg)
        if nbytes == 0:
            raise IndexMemError(IM_ERR_ARG, "invalid configuration")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        self.ctx = im_create(self.ccfg, self.workspace)
        cap = C.c_int32(0)
        _check(_lib.im_get_config(self.ctx, C.byref(self.ccfg), C.byref(cap)))
        self.capacity = cap.value
        c = self.ccfg
        self.H, self.Hkv, self.d = c.n_q_heads, c.n_kv_heads, c.head_dim
        self.D, self.Dkv = self.H * self.d, self.Hkv * self.d
        self.HI, self.dI, self.dM = c.n_index_heads, c.index_dim, c.mem_dim
        self.out_dtype = torch.float32 if c.out_f32 else torch.bfloat16

    def close(self):
        if getattr(self, "ctx", None):
            im_destroy(self.ctx)
            self.ctx = None
            self.workspace = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- hot calls
    def prefill_chunk(self, layer, seq_ids, x, q_pre, k, v):
        """x and q_pre feed the indexer; with a retained set per KV head (cfg.scorer != 0) they may be None."""
        n, Cn = len(seq_ids), k.shape[-3]
        bf = torch.bfloat16
        if not self.ccfg.scorer:
            _dev(x, bf, n * Cn * self.D, "x"); _dev(q_pre, bf, n * Cn * self.D, "q_pre")
        _dev(k, bf, n * Cn * self.Dkv, "k"); _dev(v, bf, n * Cn * self.Dkv, "v")
        im_prefill_chunk(self.ctx, layer, seq_ids, Cn, x, q_pre, k, v)

    def prefill_chunk_attend(self, layer, seq_ids, x, q_pre, q, k, v, out=None):
        """prefill_chunk that also returns the layer outputs [n, C, H, d] of the chunk's own queries."""
        n, Cn = len(seq_ids), x.shape[-2]
        bf = torch.bfloat16
        _dev(x, bf, n * Cn * self.D, "x"); _dev(q_pre, bf, n * Cn * self.D, "q_pre"); _dev(q, bf, n * Cn * self.D, "q")
        _dev(k, bf, n * Cn * self.Dkv, "k"); _dev(v, bf, n * Cn * self.Dkv, "v")
        if out is None:
            out = torch.empty((n, Cn, self.H, self.d), dtype=self.out_dtype, device=x.device)
        _dev(out, self.out_dtype, n * Cn * self.D, "out")
        im_prefill_chunk_attend(self.ctx, layer, seq_ids, Cn, x, q_pre, q, k, v, out)
        return out

    def decode_step(self, layer, seq_ids, x, q_pre, q, k_new, v_new, out=None):
        n = len(seq_ids)
        bf = torch.bfloat16
        if not self.ccfg.scorer:
            _dev(x, bf, n * self.D, "x"); _dev(q_pre, bf, n * self.D, "q_pre")
        _dev(q, bf, n * self.D, "q")
        _dev(k_new, bf, n * self.Dkv, "k_new"); _dev(v_new, bf, n * self.Dkv, "v_new")
        if out is None:
            out = torch.empty((n, self.H, self.d), dtype=self.out_dtype, device=self.device)
        else:
            _dev(out, self.out_dtype, n * self.D, "out")
        im_decode_step(self.ctx, layer, seq_ids, x, q_pre, q, k_new, v_new, out)
        return out

    def decode_stack(self, layers, seq_ids, x, q_pre, q, k_new, v_new, out=None, ready_events=None, done_events=None):
        """One decode token for every layer of `layers` in one call; x .. v_new (and out) hold one tensor per layer.
        ready_events / done_events: one torch.cuda.Event per layer (or None) for inputs that arrive and outputs that are
        fetched while the call runs (im_decode_stack_events)."""
        n, nl = len(seq_ids), len(layers)
        bf = torch.bfloat16
        for j in range(nl):
            _dev(x[j], bf, n * self.D, "x"); _dev(q_pre[j], bf, n * self.D, "q_pre"); _dev(q[j], bf, n * self.D, "q")
            _dev(k_new[j], bf, n * self.Dkv, "k_new"); _dev(v_new[j], bf, n * self.Dkv, "v_new")
        if out is None:
            out = torch.empty((nl, n, self.H, self.d), dtype=self.out_dtype, device=self.device)
        for j in range(nl):
            _dev(out[j], self.out_dtype, n * self.D, "out")
        if ready_events is None and done_events is None:
            im_decode_stack(self.ctx, layers, seq_ids, x, q_pre, q, k_new, v_new, out)
        else:
            im_decode_stack_events(self.ctx, layers, seq_ids, x, q_pre, q, k_new, v_new, out, ready_events, done_events)
        return out

    def reset(self, layer=-1, seq=-1):
        im_reset(self.ctx, layer, seq)

    def status(self) -> int:
        return im_status(self.ctx)

    def launch_count(self) -> int:
        return im_launch_count(self.ctx)

    # ---- weights
    def weight_shapes(self):
        return {"U_q": (self.HI * self.dI, self.D), "U_k": (self.dI, self.D), "G": (self.HI, self.D),
                "W_theta": (self.dM, self.D), "w_g": (self.D,), "b_g": (1,)}

    def set_weights(self, layer: int, weights: dict):
        for name, t in weights.items():
            if name == "b_g":
                im_set_weights(self.ctx, layer, IM_W_BG, np.asarray(t.detach().cpu().numpy() if torch.is_tensor(t) else t, np.float32).reshape(1))
            else:
                assert tuple(t.shape) == self.weight_shapes()[name], (name, tuple(t.shape))
                im_set_weights(self.ctx, layer, WEIGHT_IDS[name], _bf16_bits(t))

    def get_weights(self, layer: int) -> dict:
        out = {}
        for name, shape in self.weight_shapes().items():
            if name == "b_g":
                a = np.empty(1, np.float32)
                im_get_weights(self.ctx, layer, IM_W_BG, a)
                out[name] = torch.from_numpy(a)
            else:
                a = np.empty(shape, np.int16)
                im_get_weights(self.ctx, layer, WEIGHT_IDS[name], a)
                out[name] = _from_bf16_bits(a).reshape(shape)
        return out

    # ---- state
    def counts(self, layer, seq) -> dict:
        a = np.zeros(8, np.int32)
        im_state_export(self.ctx, layer, seq, IM_S_COUNTS, a)
        return {"n": int(a[0]), "T": int(a[1]), "since": int(a[2]), "evict_steps": int(a[3]),
                "n_evicted": int(a[4]), "n_pending": int(a[5]), "n_sel": int(a[7])}

    def export(self, layer, seq, which):
        """numpy array of one state piece (bf16 pieces come back as float32 values)."""
        n = self.counts(layer, seq)["n"]
        if which == IM_S_POS:
            a = np.empty(n, np.int32)
        elif which == IM_S_IMP:
            a = np.empty(n, np.float32)
        elif which == IM_S_KIDX:
            a = np.empty((n, self.dI), np.int16)
        elif which in (IM_S_K, IM_S_V):
            a = np.empty((n, self.Hkv, self.d), np.int16)
        elif which == IM_S_M:
            a = np.empty((self.dM, self.Dkv), np.float32)
        elif which == IM_S_B:
            a = np.empty(self.dM, np.float32)
        elif which == IM_S_EVICTED:
            a = np.empty(self.counts(layer, seq)["n_evicted"], np.int32)
        elif which == IM_S_SEL_POS:
            a = np.empty(self.counts(layer, seq)["n_sel"], np.int32)
        elif which == IM_S_SEL_IMP:
            a = np.empty(self.counts(layer, seq)["n_sel"], np.float32)
        else:
            raise ValueError(which)
        if a.size:
            im_state_export(self.ctx, layer, seq, which, a)
        if a.dtype == np.int16:
            return _from_bf16_bits(a).to(torch.float32).numpy().reshape(a.shape)
        return a

    # ---- a retained set per KV head (cfg.scorer != 0)
    def set_scores(self, layer, scores: torch.Tensor):
        im_set_scores(self.ctx, layer, scores)

    def export_head(self, layer, seq, head, which):
        """One KV head's piece of the state: IM_S_POS, IM_S_IMP (scores), IM_S_K / IM_S_V ([n, d]), IM_S_EVICTED,
        IM_S_SEL_POS, IM_S_SEL_IMP."""
        c = self.counts(layer, seq)
        n = c["n"]
        if which == IM_S_POS:
            a = np.empty(n, np.int32)
        elif which == IM_S_IMP:
            a = np.empty(n, np.float32)
        elif which in (IM_S_K, IM_S_V):
            a = np.empty((n, self.d), np.int16)
        elif which == IM_S_EVICTED:
            a = np.empty(c["n_evicted"], np.int32)
        elif which == IM_S_SEL_POS:
            a = np.empty(c["n_sel"], np.int32)
        elif which == IM_S_SEL_IMP:
            a = np.empty(c["n_sel"], np.float32)
        else:
            raise ValueError(which)
        if a.size:
            im_state_export_head(self.ctx, layer, seq, head, which, a)
        if a.dtype == np.int16:
            return _from_bf16_bits(a).to(torch.float32).numpy().reshape(a.shape)
        return a

    def import_head_state(self, layer, seq, *, heads, M_kv, b, T, since=0, evict_steps=0):
        """Replaces one sequence's state in per-head mode.  heads: one dict(pos, score, K [n, d], V [n, d]) per KV head,
        all with the same number of entries."""
        n = len(heads[0]["pos"])
        ctr = np.zeros(8, np.int32)
        ctr[0], ctr[1], ctr[2], ctr[3] = n, T, since, evict_steps
        im_state_import(self.ctx, layer, seq, IM_S_M, np.asarray(M_kv, np.float32))
        im_state_import(self.ctx, layer, seq, IM_S_B, np.asarray(b, np.float32))
        im_state_import(self.ctx, layer, seq, IM_S_COUNTS, ctr)
        for h, e in enumerate(heads):
            assert len(e["pos"]) == n
            if n:
                im_state_import_head(self.ctx, layer, seq, h, IM_S_POS, np.asarray(e["pos"], np.int32))
                im_state_import_head(self.ctx, layer, seq, h, IM_S_IMP, np.asarray(e["score"], np.float32))
                im_state_import_head(self.ctx, layer, seq, h, IM_S_K, _bf16_bits(torch.from_numpy(np.asarray(e["K"], np.float32))))
                im_state_import_head(self.ctx, layer, seq, h, IM_S_V, _bf16_bits(torch.from_numpy(np.asarray(e["V"], np.float32))))

    def import_state(self, layer, seq, *, pos, imp, kidx, K, V, M_kv, b, T, since=0, evict_steps=0):
        """Replaces one sequence's state.  kidx/K/V are float arrays holding bf16 values."""
        n = len(pos)
        ctr = np.zeros(8, np.int32)
        ctr[0], ctr[1], ctr[2], ctr[3] = n, T, since, evict_steps
        im_state_import(self.ctx, layer, seq, IM_S_M, np.asarray(M_kv, np.float32))
        im_state_import(self.ctx, layer, seq, IM_S_B, np.asarray(b, np.float32))
        im_state_import(self.ctx, layer, seq, IM_S_COUNTS, ctr)
        if n:
            im_state_import(self.ctx, layer, seq, IM_S_POS, np.asarray(pos, np.int32))
            im_state_import(self.ctx, layer, seq, IM_S_IMP, np.asarray(imp, np.float32))
            im_state_import(self.ctx, layer, seq, IM_S_KIDX, _bf16_bits(torch.from_numpy(np.asarray(kidx, np.float32))))
            im_state_import(self.ctx, layer, seq, IM_S_K, _bf16_bits(torch.from_numpy(np.asarray(K, np.float32))))
            im_state_import(self.ctx, layer, seq, IM_S_V, _bf16_bits(torch.from_numpy(np.asarray(V, np.float32))))
