"""Seeded synthetic workloads for the IndexMem hot path.

This module only *draws inputs*: shapes, value distributions and planted structure of the five
benchmark configurations.  It holds none of the method's arithmetic, imports neither the CUDA
binding nor the CPU oracle, and is the one module both sides of a parity test are fed from.

The inputs stand in for what a backbone (Qwen3-8B, Mistral-7B, Llama-3.1-8B) would hand one
attention layer on the paper's long-context prompts; those prompts, backbones and the trained
indexer/memory weights are not available, so hidden states, queries, keys and values are
N(0,1) draws rounded to bf16, with two kinds of planted structure:

* needles: a few key positions per sequence whose key points along the mean direction of the
  decode queries, so they carry a large share of the softmax mass;
* heavy-tailed key norms: every (token, KV head) key is scaled by exp(sigma * xi), xi ~ N(0,1).

Weights are N(0, init_std^2) rounded to bf16; the gate bias b_g is 0.
"""
from __future__ import annotations

import dataclasses
import math
import zlib
from dataclasses import dataclass

import torch

BASE_SEED = 20260525


@dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    n_seq: int
    H: int
    Hkv: int
    d: int
    ctx: int            # cached context tokens ingested before decoding
    chunk: int          # ingestion chunk length (ctx == chunk: one-shot compression)
    B: int              # KV budget
    steps: int          # decode steps
    tau: int = 1
    n_sink: int = 4
    key_norm_sigma: float = 0.0
    n_needles: int = 0
    init_std: float = 0.02

    @property
    def D(self):
        return self.H * self.d

    @property
    def Dkv(self):
        return self.Hkv * self.d

    @property
    def HI(self):
        return max(1, self.H // 4)

    @property
    def dI(self):
        return max(1, self.d // 8)

    @property
    def dM(self):
        return max(1, self.D // 8)

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


# The five benchmark configurations (context lengths, budgets, head shapes and step counts).
CONFIGS = {
    "tiny": Workload("tiny", 1, 1, 4, 1, 64, 1024, 1024, 256, 64, n_needles=16),
    "llama8b_b1": Workload("llama8b_b1", 1, 1, 32, 8, 128, 4096, 4096, 512, 256, key_norm_sigma=0.5),
    "qwen7b_b8": Workload("qwen7b_b8", 1, 8, 28, 4, 128, 16384, 16384, 1024, 128, n_needles=64),
    "mistral7b_prefill": Workload("mistral7b_prefill", 1, 1, 32, 8, 128, 32768, 2048, 2048, 0),
    "llama8b_stack": Workload("llama8b_stack", 32, 32, 32, 8, 128, 16384, 2048, 2048, 64, key_norm_sigma=0.5),
}

WEIGHT_NAMES = ("U_q", "U_k", "G", "W_theta", "w_g", "b_g")


def _seed(*parts) -> int:
    s = "/".join(str(p) for p in parts)
    return (BASE_SEED * 1000003 + zlib.crc32(s.encode())) % (2 ** 63 - 1)


def _gen(device, *parts) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(_seed(*parts))
    return g


def _randn(shape, device, *parts) -> torch.Tensor:
    return torch.randn(shape, generator=_gen(device, *parts), device=device, dtype=torch.float32)


def weight_shapes(wl: Workload) -> dict:
    return {"U_q": (wl.HI * wl.dI, wl.D), "U_k": (wl.dI, wl.D), "G": (wl.HI, wl.D),
            "W_theta": (wl.dM, wl.D), "w_g": (wl.D,), "b_g": (1,)}


def make_weights(wl: Workload, layer: int, device="cpu") -> dict:
    """bf16 tensors, N(0, init_std^2); b_g = 0 (float32 scalar tensor)."""
    out = {}
    for name, shape in weight_shapes(wl).items():
        if name == "b_g":
            out[name] = torch.zeros(1, dtype=torch.float32, device=device)
        else:
            out[name] = (_randn(shape, device, wl.name, "w", layer, name) * wl.init_std).to(torch.bfloat16)
    return out


def needle_dirs(wl: Workload, layer: int, device="cpu") -> torch.Tensor:
    """Unit vectors u[n_seq, Hkv, d]: the planted mean direction of the decode queries."""
    u = _randn((wl.n_seq, wl.Hkv, wl.d), device, wl.name, "needle_dir", layer)
    return u / u.norm(dim=-1, keepdim=True)


def needle_positions(wl: Workload, layer: int) -> torch.Tensor:
    """int64 [n_seq, n_needles], uniform in [n_sink, ctx), distinct per sequence (CPU tensor)."""
    if wl.n_needles == 0:
        return torch.zeros((wl.n_seq, 0), dtype=torch.int64)
    rows = []
    for s in range(wl.n_seq):
        g = _gen("cpu", wl.name, "needle_pos", layer, s)
        perm = torch.randperm(wl.ctx - wl.n_sink, generator=g)[: wl.n_needles] + wl.n_sink
        rows.append(perm.sort().values)
    return torch.stack(rows)


def rotate_queries(Q: torch.Tensor, positions: torch.Tensor, base: float = 10000.0) -> torch.Tensor:
    """The backbone's rotary position embedding applied to query rows: Q [..., T, H, d] float32, positions [T].

    Pairs (i, i + d/2) of every head are rotated by positions * base^(-2i/d).  This belongs to the backbone,
    not to the method: it only makes the attention query a different tensor from the pre-RoPE query.
    """
    d = Q.shape[-1]
    half = d // 2
    inv = base ** (-torch.arange(half, device=Q.device, dtype=torch.float32) * 2.0 / d)
    ang = positions.to(Q.device, torch.float32)[:, None] * inv[None, :]          # [T, d/2]
    cos, sin = torch.cos(ang)[:, None, :], torch.sin(ang)[:, None, :]            # [T, 1, d/2]
    a, b = Q[..., :half], Q[..., half:]
    return torch.cat([a * cos - b * sin, a * sin + b * cos], dim=-1)


def prefill_inputs(wl: Workload, layer: int, chunk_idx: int, device="cpu", seqs=None):
    """Inputs of ingestion chunk ``chunk_idx`` for sequences ``seqs`` (default all).

    Returns bf16 tensors X [n, C, D], Q_pre [n, C, H, d], Q [n, C, H, d], K [n, C, Hkv, d], V [n, C, Hkv, d].
    Q_pre is the pre-RoPE query (what the indexer reads), Q the same rows after the backbone's rotary
    embedding at their positions (what attention, Linear_theta and the gate read).
    """
    seqs = list(range(wl.n_seq)) if seqs is None else list(seqs)
    C, t0 = wl.chunk, chunk_idx * wl.chunk
    Xs, Qps, Qs, Ks, Vs = [], [], [], [], []
    npos = needle_positions(wl, layer)
    udir = needle_dirs(wl, layer, device) if wl.n_needles else None
    for s in seqs:
        tag = (wl.name, "prefill", layer, chunk_idx, s)
        X = _randn((C, wl.D), device, *tag, "x")
        Qp = _randn((C, wl.H, wl.d), device, *tag, "q")
        Q = rotate_queries(Qp, torch.arange(t0, t0 + C))
        K = _randn((C, wl.Hkv, wl.d), device, *tag, "k")
        V = _randn((C, wl.Hkv, wl.d), device, *tag, "v")
        if wl.key_norm_sigma > 0:
            xi = _randn((C, wl.Hkv, 1), device, *tag, "knorm")
            K = K * torch.exp(wl.key_norm_sigma * xi)
        if wl.n_needles:
            for p in npos[s].tolist():
                if t0 <= p < t0 + C:
                    K[p - t0] = 3.0 * math.sqrt(wl.d) * udir[s]
        Xs.append(X); Qps.append(Qp); Qs.append(Q); Ks.append(K); Vs.append(V)
    bf = lambda ts: torch.stack(ts).to(torch.bfloat16)
    return bf(Xs), bf(Qps), bf(Qs), bf(Ks), bf(Vs)


def decode_inputs(wl: Workload, layer: int, step: int, device="cpu"):
    """Inputs of decode step ``step`` for all sequences.

    Returns bf16 tensors x [n_seq, D], q_pre [n_seq, H, d], q [n_seq, H, d], k_new [n_seq, Hkv, d],
    v_new [n_seq, Hkv, d].  q_pre ~ N(0,1) is the pre-RoPE query; q is q_pre rotated at position ctx + step,
    plus, with needles, sqrt(d) * u with u the planted direction of the query head's KV group.
    """
    tag = (wl.name, "decode", layer, step)
    n = wl.n_seq
    x = _randn((n, wl.D), device, *tag, "x")
    q_pre = _randn((n, wl.H, wl.d), device, *tag, "q")
    q = rotate_queries(q_pre[:, None], torch.tensor([wl.ctx + step]))[:, 0]
    k = _randn((n, wl.Hkv, wl.d), device, *tag, "k")
    v = _randn((n, wl.Hkv, wl.d), device, *tag, "v")
    if wl.key_norm_sigma > 0:
        xi = _randn((n, wl.Hkv, 1), device, *tag, "knorm")
        k = k * torch.exp(wl.key_norm_sigma * xi)
    if wl.n_needles:
        u = needle_dirs(wl, layer, device)                      # [n, Hkv, d]
        q = q + math.sqrt(wl.d) * u.repeat_interleave(wl.H // wl.Hkv, dim=1)
    bf = lambda t: t.to(torch.bfloat16)
    return bf(x), bf(q_pre), bf(q), bf(k), bf(v)


def f32(t: torch.Tensor):
    """bf16 (or any) tensor -> contiguous float32 numpy array holding the same values."""
    return t.detach().to("cpu", torch.float32).contiguous().numpy()
