"""The give-up path of the bounded device-side waits (``-m gpu``).

No copy is broken and nothing is left to hang: the test only lowers the number of attempts a consumer gets to wait
for its copies (IM_OPT_WAIT_LIMIT = 1: none), so every such wait gives up at once.  The kernels must then set the
sticky status word, wait with the full limit for the copies they have in flight, free their tensor memory and
return; ``im_status`` reports IM_ERR_TIMEOUT and nothing else, and after the limit is restored and the context
reset the same context computes correct results again (checked against the oracle).
"""
import pytest
import torch

from paper_2605_25475_b200 import synth

pytestmark = pytest.mark.gpu

LLAMA = synth.CONFIGS["llama8b_b1"]


def _expect_timeout(im, g):
    with pytest.raises(im.IndexMemError) as e:
        g.status()
    assert e.value.code == im.IM_ERR_TIMEOUT, str(e.value)
    assert "status 4)" in str(e.value)          # the time-out bit alone: no count mismatch, no non-finite score


@pytest.mark.parametrize("kernel", ["attn_mma", "attn_tc", "readout_ring", "chunk_attn_tc"])
def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable(kernel):
    from paper_2605_25475_b200 import binding as im
    from tests.parity import Pair
    wl = LLAMA.replace(name="timeout_" + kernel, n_seq=2, ctx=300, chunk=150, B=200, steps=4, n_needles=0)
    p = Pair(wl, chunk_outputs=1)
    g = p.g
    if kernel == "attn_tc":
        im.im_set_option(g.ctx, im.IM_OPT_DECODE_TENSOR, 1)
    if kernel == "readout_ring":
        im.im_set_option(g.ctx, im.IM_OPT_READOUT_STAGES, 2)
    p.prefill(0)
    p.prefill(1)
    p.decode(0)                                  # a good step first
    assert g.status() == 0

    im.im_set_option(g.ctx, im.IM_OPT_WAIT_LIMIT, 1)          # zero attempts
    dev = p.device
    if kernel == "chunk_attn_tc":
        X, Qp, Q, K, V = [t.to(dev) for t in synth.prefill_inputs(wl, 0, 1)]
        g.prefill_chunk_attend(0, p.seq_ids, X, Qp, Q, K, V)
    else:
        x, qp, q, k, v = [t.to(dev) for t in synth.decode_inputs(wl, 0, 1)]
        g.decode_step(0, p.seq_ids, x, qp, q, k, v)
    torch.cuda.synchronize()
    _expect_timeout(im, g)
    _expect_timeout(im, g)                       # sticky until cleared

    # restore, clear, run again from scratch on the same context: results are right again
    im.im_set_option(g.ctx, im.IM_OPT_WAIT_LIMIT, 0)
    g.reset()
    assert g.status() == 0
    p2 = Pair(wl.replace(name="timeout_again_" + kernel), chunk_outputs=1)
    p2.g.close()
    p2.g = g                                     # the context that saw the time-out, against a fresh oracle
    p2.g.set_weights(0, p2.weights)
    p2.prefill_attend(0)
    p2.prefill_attend(1)
    for s in range(wl.steps):
        p2.decode(s)
    assert p2.stats["max_out_err"] <= 2e-3 and p2.stats["max_M_err"] <= 2e-3
    assert g.status() == 0
