"""The allocation-free attention entry point.

Hosts that cannot allocate device memory while they run (a serving loop under stream capture, a
plug-in confined to a fixed arena, a process whose memory is fully committed to its KV pool) can
still call ``im_attention_noalloc``: its scratch is a fixed array inside the library.  This test
calls it through the C ABI twice in a row and checks each result against ``im_decode_step`` (memory
disabled, budget never reached, so that call is plain attention over everything cached) and against a
float64 softmax attention written out in numpy over the same cached keys and values, at the ordinary
output bound (2e-3 of the tensor's max-abs plus half a bf16 ulp of storage rounding).  Shapes with a
last split of one to three keys and with a head_dim that is not a multiple of 32 are checked against
the numpy attention alone.  The file sorts last, so a run that stops at the first failure has already
run the rest.
"""
import numpy as np
import pytest
import torch

from paper_2605_25475_b200 import synth

pytestmark = pytest.mark.gpu


def _softmax_attention(q, K, V, scale):
    """q [H, d], K, V [Hkv, n, d] (float64) -> [H, d]: query head j attends over KV head j // (H / Hkv)."""
    H, Gq = q.shape[0], q.shape[0] // K.shape[0]
    out = np.empty_like(q)
    for j in range(H):
        s = (K[j // Gq] @ q[j]) * scale
        p = np.exp(s - s.max())
        out[j] = (p / p.sum()) @ V[j // Gq]
    return out


def _assert_close(got, want, what):
    from tests.parity import bf16_ulp
    scale = np.abs(want).max()
    half_ulp = 0.5 * bf16_ulp(np.maximum(np.abs(want), np.abs(got)))
    err = np.abs(got - want)
    assert np.all(err <= 2e-3 * scale + half_ulp), f"{what}: {err.max():.3e} vs max-abs {scale:.3e}"


def test_noalloc_attention_matches_decode_step_twice():
    from paper_2605_25475_b200 import binding as im
    wl = synth.Workload("noalloc", 1, 1, 8, 2, 64, 700, 700, 4096, 2)
    g = im.IndexMem(im.Config(n_layers=1, max_seqs=1, n_q_heads=wl.H, n_kv_heads=wl.Hkv, head_dim=wl.d, budget=wl.B,
                              max_chunk=wl.chunk, enable_memory=0), "cuda:0")
    dev = g.device
    X, Qp, _, K, V = [t.to(dev) for t in synth.prefill_inputs(wl, 0, 0)]
    g.prefill_chunk(0, [0], X, Qp, K, V)
    out2 = torch.empty((wl.H, wl.d), dtype=torch.bfloat16, device=dev)   # reused: the second call allocates nothing
    for step in range(2):
        x, qp, q, k, v = [t.to(dev) for t in synth.decode_inputs(wl, 0, step)]
        want = g.decode_step(0, [0], x, qp, q, k, v)[0].float().cpu().numpy().astype(np.float64)
        assert g.status() == 0
        n = g.counts(0, 0)["n"]
        assert n == wl.ctx + step + 1
        # the cached keys / values as the library holds them, [n, Hkv, d] -> one slab per KV head
        order = np.argsort(g.export(0, 0, im.IM_S_POS))
        Kh = np.ascontiguousarray(g.export(0, 0, im.IM_S_K)[order].transpose(1, 0, 2))
        Vh = np.ascontiguousarray(g.export(0, 0, im.IM_S_V)[order].transpose(1, 0, 2))
        Kc = torch.tensor(Kh).to(torch.bfloat16).to(dev)
        Vc = torch.tensor(Vh).to(torch.bfloat16).to(dev)
        got = im.im_attention_noalloc(q[0].contiguous(), Kc, Vc, out=out2)
        torch.cuda.synchronize()
        got = got.float().cpu().numpy().astype(np.float64)
        ref = _softmax_attention(q[0].float().cpu().numpy().astype(np.float64), Kh.astype(np.float64),
                                 Vh.astype(np.float64), 1.0 / np.sqrt(wl.d))
        _assert_close(got, ref, f"step {step}, against the numpy attention")
        # the existing entry point computed the same attention: both are bf16 roundings of float32 results,
        # so the two may sit one rounding step apart on top of the common bound
        scale = np.abs(want).max()
        assert np.abs(got - want).max() <= 2e-3 * scale + scale * 2.0 ** -8, f"step {step}: {np.abs(got - want).max()} vs {scale}"
    # sizes beyond the built-in scratch are refused with a clear message, nothing is launched
    big_k = torch.zeros((1, 300000, 64), dtype=torch.bfloat16, device=dev)
    with pytest.raises(im.IndexMemError) as e:
        im.im_attention_noalloc(torch.zeros((64, 64), dtype=torch.bfloat16, device=dev), big_k, big_k)
    assert e.value.code == im.IM_ERR_CAPACITY and "1048576" in str(e.value)


@pytest.mark.parametrize("H,Hkv,d,n", [(6, 3, 80, 2 * 256 + 1), (4, 1, 48, 256 + 3), (14, 2, 128, 5 * 256 + 2), (3, 3, 200, 7)])
def test_noalloc_attention_ragged_splits_and_odd_head_dims(H, Hkv, d, n):
    from paper_2605_25475_b200 import binding as im
    dev = torch.device("cuda:0")
    gen = torch.Generator().manual_seed(1000 * H + n)
    q = torch.randn((H, d), generator=gen).to(torch.bfloat16)
    K = torch.randn((Hkv, n, d), generator=gen).to(torch.bfloat16)
    V = torch.randn((Hkv, n, d), generator=gen).to(torch.bfloat16)
    K[:, n - 1] *= 4.0                                   # weight on the ragged tail
    for call in range(2):
        got = im.im_attention_noalloc(q.to(dev), K.to(dev), V.to(dev))
        torch.cuda.synchronize()
        ref = _softmax_attention(q.double().numpy(), K.double().numpy(), V.double().numpy(), 1.0 / np.sqrt(d))
        _assert_close(got.float().cpu().numpy().astype(np.float64), ref, f"call {call}")
