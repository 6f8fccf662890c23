"""The allocation-free attention entry point against the ordinary decode call.

Hosts that cannot allocate device memory while they run (a serving loop under stream capture, a
plug-in confined to a fixed arena, a process whose memory is fully committed to its KV pool) can
still call ``im_attention_noalloc``: its scratch is a fixed array inside the library.  This test
calls it through the C ABI twice in a row and checks each result against ``im_decode_step`` (memory
disabled, budget never reached, so that call is plain attention over everything cached).  It sits in
a file of its own that sorts last, so a run that stops at the first failure has already run the rest.
"""
import numpy as np
import pytest
import torch

from paper_2605_25475_b200 import synth

pytestmark = pytest.mark.gpu


def test_noalloc_attention_matches_decode_step_twice():
    from paper_2605_25475_b200 import binding as im
    wl = synth.Workload("noalloc", 1, 1, 8, 2, 64, 700, 700, 4096, 2)
    g = im.IndexMem(im.Config(n_layers=1, max_seqs=1, n_q_heads=wl.H, n_kv_heads=wl.Hkv, head_dim=wl.d, budget=wl.B,
                              max_chunk=wl.chunk, enable_memory=0), "cuda:0")
    dev = g.device
    X, Q, K, V = [t.to(dev) for t in synth.prefill_inputs(wl, 0, 0)]
    g.prefill_chunk(0, [0], X, Q, K, V)
    out2 = torch.empty((wl.H, wl.d), dtype=torch.bfloat16, device=dev)   # reused: the second call allocates nothing
    for step in range(2):
        x, q, k, v = [t.to(dev) for t in synth.decode_inputs(wl, 0, step)]
        want = g.decode_step(0, [0], x, q, q, k, v)[0].float().cpu().numpy()
        assert g.status() == 0
        n = g.counts(0, 0)["n"]
        assert n == wl.ctx + step + 1
        # the cached keys / values as the library holds them, [n, Hkv, d] -> one slab per KV head
        order = np.argsort(g.export(0, 0, im.IM_S_POS))
        Kc = torch.tensor(g.export(0, 0, im.IM_S_K)[order]).to(torch.bfloat16).permute(1, 0, 2).contiguous().to(dev)
        Vc = torch.tensor(g.export(0, 0, im.IM_S_V)[order]).to(torch.bfloat16).permute(1, 0, 2).contiguous().to(dev)
        got = im.im_attention_noalloc(q[0].contiguous(), Kc, Vc, out=out2)
        torch.cuda.synchronize()
        got = got.float().cpu().numpy()
        scale = np.abs(want).max()
        # both are bf16 roundings of float32 results that agree to ~1e-6: allow one bf16 ulp of the largest value
        assert np.abs(got - want).max() <= 2e-3 * scale + scale * 2.0 ** -8, f"step {step}: {np.abs(got - want).max()} vs {scale}"
    # sizes beyond the built-in scratch are refused with a clear message, nothing is launched
    big_k = torch.zeros((1, 300000, 64), dtype=torch.bfloat16, device=dev)
    with pytest.raises(im.IndexMemError) as e:
        im.im_attention_noalloc(torch.zeros((64, 64), dtype=torch.bfloat16, device=dev), big_k, big_k)
    assert e.value.code == im.IM_ERR_CAPACITY and "1048576" in str(e.value)
