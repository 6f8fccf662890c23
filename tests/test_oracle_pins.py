"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Every expected value is computed here with
numpy/python from a definition that is independent of the oracle's code path: a textbook softmax
attention, a brute-force sort, closed forms of Eq. 5-7, invariants of the update rule, and the one
number the paper prints that depends on the layer widths (19.92M indexer parameters).
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import indexmem_oracle as orc
from paper_2605_25475_b200 import synth


def bf16(a):
    return torch.tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16).to(torch.float32).numpy()


def small_cfg(**kw):
    base = dict(H=4, Hkv=2, d=8, B=12, HI=2, dI=4, dM=6, tau=1, n_sink=2)
    base.update(kw)
    return orc.OracleConfig(**base)


def rand_weights(L, rng, std=0.3):
    w = {}
    for name, shape in L.weight_shapes().items():
        w[name] = bf16(rng.standard_normal(shape) * std) if name != "b_g" else np.zeros(1, np.float32)
    L.set_weights(w)
    return w


def rand_tokens(L, rng, n):
    c = L.cfg
    X = bf16(rng.standard_normal((n, L.D)))
    Q = bf16(rng.standard_normal((n, c.H, c.d)))
    K = bf16(rng.standard_normal((n, c.Hkv, c.d)))
    V = bf16(rng.standard_normal((n, c.Hkv, c.d)))
    return X, Q, K, V


def softmax_attention(q, K, V, Gq, scale):
    """Textbook definition: o_j = softmax(q_j K_g^T * scale) V_g, in float64."""
    H, d = q.shape
    o = np.zeros((H, d))
    for j in range(H):
        g = j // Gq
        s = (K[:, g, :].astype(np.float64) @ q[j].astype(np.float64)) * scale
        p = np.exp(s - s.max())
        p /= p.sum()
        o[j] = p @ V[:, g, :].astype(np.float64)
    return o


# ------------------------------------------------------------------ rounding helper
def test_bf16_round_matches_torch():
    rng = np.random.default_rng(0)
    vals = np.concatenate([rng.standard_normal(2000), rng.standard_normal(2000) * 1e-3,
                           rng.standard_normal(500) * 1e4, [0.0, 1.0, -1.0, 1.00390625, 1.01171875]])
    vals = vals.astype(np.float32)          # exactly representable in fp32 -> single rounding in torch too
    want = bf16(vals)
    got = np.array([orc.bf16_round(float(v)) for v in vals], dtype=np.float32)
    assert np.array_equal(want, got)
    # ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert orc.bf16_round(1.0 + 2.0 ** -8) == 1.0
    assert orc.bf16_round(1.0 + 3 * 2.0 ** -8) == 1.0 + 2 * 2.0 ** -7


# ------------------------------------------------------------------ widths (efficiency paragraph)
def test_indexer_parameter_count_llama31_8b():
    wl = synth.Workload("llama31", 32, 1, 32, 8, 128, 8, 8, 8, 1)
    shp = synth.weight_shapes(wl)
    per_layer = math.prod(shp["U_q"]) + math.prod(shp["U_k"]) + math.prod(shp["G"])
    assert 32 * per_layer == 19_922_944          # "19.92M"
    # the figure as the paper prints it (tests/golden, with its citation)
    golden = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "indexer_parameters_llama31_8b.txt")
    printed = [ln.split()[1] for ln in open(golden) if ln.startswith("printed_millions")]
    assert printed == ["%.2f" % (32 * per_layer / 1e6)]
    L = orc.OracleLayer(orc.OracleConfig(H=32, Hkv=8, d=128, B=8))
    assert L.weight_shapes()["U_q"] == shp["U_q"] == (8 * 16, 4096)
    assert L.weight_shapes()["U_k"] == shp["U_k"] == (16, 4096)
    assert L.weight_shapes()["G"] == shp["G"] == (8, 4096)
    assert L.weight_shapes()["W_theta"] == shp["W_theta"] == (512, 4096)


# ------------------------------------------------------------------ indexer features
def test_index_features_against_numpy():
    rng = np.random.default_rng(1)
    L = orc.OracleLayer(small_cfg())
    w = rand_weights(L, rng)
    c = L.cfg
    x = bf16(rng.standard_normal(L.D))
    qp = bf16(rng.standard_normal(L.D))
    # k = RMSNorm(U_k x)
    u = w["U_k"].astype(np.float64) @ x
    k = u / np.sqrt((u ** 2).mean() + c.norm_eps)
    assert np.array_equal(L.index_key(x), bf16(k))
    assert abs(np.sqrt((k ** 2).mean()) - 1.0) < 1e-5
    # q = RMSNorm per indexer head of U_q flatten(Q); alpha = G x / sqrt(H_I d_I)
    y = (w["U_q"].astype(np.float64) @ qp).reshape(c.HI, c.dI)
    y = y / np.sqrt((y ** 2).mean(axis=1, keepdims=True) + c.norm_eps)
    al = (w["G"].astype(np.float64) @ x) / math.sqrt(c.HI * c.dI)
    qf, alpha = L.index_query(x, qp)
    np.testing.assert_allclose(qf, y, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(alpha, al, rtol=1e-12, atol=1e-14)
    # the indexer query comes from q_pre, the gate and the key from x: swapping must change them
    qf2, alpha2 = L.index_query(qp, x)
    assert not np.allclose(qf2, qf) and not np.allclose(alpha2, alpha)


def test_index_query_invariants():
    """What fixes the indexer query and the head gate without restating their formula (Sec. 3.1, Alg. 1): the
    normalisation is per indexer head over d_I (unit RMS per head; a head's features depend only on its own rows of
    U_q; rescaling q_pre changes nothing), and with one-hot rows the projections pick single inputs."""
    rng = np.random.default_rng(11)
    L = orc.OracleLayer(small_cfg(norm_eps=1e-12))
    c = L.cfg
    w = rand_weights(L, rng)
    x = bf16(rng.standard_normal(L.D))
    qp = bf16(rng.standard_normal(L.D))
    qf, alpha = L.index_query(x, qp)
    # unit RMS per indexer head, not over the whole H_I * d_I vector (the heads' raw norms differ)
    np.testing.assert_allclose(np.sqrt((qf ** 2).mean(axis=1)), np.ones(c.HI), rtol=1e-9)
    raw = (w["U_q"].astype(np.float64) @ qp).reshape(c.HI, c.dI)
    assert abs(np.sqrt((raw[0] ** 2).mean()) / np.sqrt((raw[1] ** 2).mean()) - 1.0) > 1e-3
    # scale invariance in q_pre (a power of two is exact in bf16); alpha does not depend on q_pre, nor qf on x
    qf2, alpha2 = L.index_query(x, 4.0 * qp)
    np.testing.assert_allclose(qf2, qf, rtol=1e-9)
    np.testing.assert_array_equal(alpha2, alpha)
    qf3, alpha3 = L.index_query(bf16(rng.standard_normal(L.D)), qp)
    np.testing.assert_array_equal(qf3, qf)
    assert not np.allclose(alpha3, alpha)
    # heads are normalised independently: doubling head 0's rows of U_q leaves every head's features unchanged
    w2 = dict(w)
    w2["U_q"] = w["U_q"].copy()
    w2["U_q"][: c.dI] *= 2.0
    L.set_weights(w2)
    qf4, _ = L.index_query(x, qp)
    np.testing.assert_allclose(qf4, qf, rtol=1e-9)
    # one-hot rows: feature r of head h reads q_pre[col], the gate reads x[col] / sqrt(H_I d_I)
    Uq = np.zeros((c.HI * c.dI, L.D), np.float32)
    cols = rng.permutation(L.D)[: c.HI * c.dI]
    Uq[np.arange(c.HI * c.dI), cols] = 1.0
    G = np.zeros((c.HI, L.D), np.float32)
    gcols = rng.permutation(L.D)[: c.HI]
    G[np.arange(c.HI), gcols] = 1.0
    w3 = dict(w, U_q=Uq, G=G)
    L.set_weights(w3)
    qf5, alpha5 = L.index_query(x, qp)
    picked = qp.astype(np.float64)[cols].reshape(c.HI, c.dI)
    for h in range(c.HI):
        np.testing.assert_allclose(qf5[h], picked[h] / np.sqrt((picked[h] ** 2).mean()), rtol=1e-9)
    np.testing.assert_allclose(alpha5, x.astype(np.float64)[gcols] / math.sqrt(c.HI * c.dI), rtol=1e-12)
    # flatten(Q) is head-major: column j * d + c of U_q reads component c of query head j
    Q = qp.reshape(c.H, c.d)
    j, cc = 2, 5
    Uq1 = np.zeros_like(Uq)
    Uq1[0, j * c.d + cc] = 1.0
    Uq1[1, 0] = 1.0
    L.set_weights(dict(w, U_q=Uq1))
    qf6, _ = L.index_query(x, qp)
    assert abs(qf6[0, 0] / qf6[0, 1] - float(Q[j, cc]) / float(Q[0, 0])) < 1e-9


def test_score_relu_hand_computed_two_heads():
    """A_t = sum_h alpha_h ReLU(q_h . k_t) on numbers small enough to do by hand (H_I = 2, d_I = 4)."""
    L = orc.OracleLayer(small_cfg(act=0))
    qf = np.array([[1.0, 2.0, 0.0, 0.0], [0.0, 0.0, -1.0, 1.0]])
    alpha = np.array([0.5, -2.0])
    kidx = np.array([[1, 1, 1, 1],      # head dots 3, 0   -> 0.5 * 3            = 1.5
                     [-1, -1, 2, 0],    # head dots -3, -2 -> both clipped        = 0
                     [0, 0, 0, 2],      # head dots 0, 2   -> -2 * 2              = -4
                     [2, 0.5, -3, 1]],  # head dots 3, 4   -> 0.5 * 3 - 2 * 4     = -6.5
                    np.float32)
    np.testing.assert_array_equal(L.index_scores(qf, alpha, kidx), np.array([1.5, 0.0, -4.0, -6.5]))
    # without the clipping the second key would score 0.5 * -3 - 2 * -2 = 2.5
    Li = orc.OracleLayer(small_cfg(act=1))
    np.testing.assert_array_equal(Li.index_scores(qf, alpha, kidx), np.array([1.5, 2.5, -4.0, -6.5]))


def test_score_relu_and_identity_closed_form():
    rng = np.random.default_rng(2)
    for act in (0, 1):
        L = orc.OracleLayer(small_cfg(act=act))
        c = L.cfg
        qf = rng.standard_normal((c.HI, c.dI))
        alpha = rng.standard_normal(c.HI)
        kidx = bf16(rng.standard_normal((50, c.dI)))
        A = L.index_scores(qf, alpha, kidx)
        if act == 1:
            # identity: the head sum folds into one dot product
            want = kidx.astype(np.float64) @ (alpha[:, None] * qf).sum(axis=0)
        else:
            z = np.maximum(kidx.astype(np.float64) @ qf.T, 0.0)       # [n, HI]
            want = z @ alpha
            # a head whose dot products are all negative contributes exactly nothing
            assert (z == 0).any()
        np.testing.assert_allclose(A, want, rtol=1e-12, atol=1e-13)


# ------------------------------------------------------------------ selection
def brute_force_keep(score, pos, B, n_sink):
    n = len(score)
    key = [(-(math.inf if pos[i] < n_sink else float(score[i]) + 0.0), int(pos[i])) for i in range(n)]
    order = sorted(range(n), key=lambda i: key[i])
    keep = np.zeros(n, np.uint8)
    keep[order[: min(B, n)]] = 1
    return keep


@pytest.mark.parametrize("seed", range(6))
def test_select_brute_force(seed):
    rng = np.random.default_rng(100 + seed)
    n = int(rng.integers(5, 40))
    B = int(rng.integers(3, n + 3))
    n_sink = int(rng.integers(0, 3))
    # few distinct values => many ties; include both zeros and -inf (never scored)
    score = rng.choice(np.array([0.0, -0.0, 0.5, -0.25, 1.5, -np.inf], np.float32), size=n)
    pos = rng.permutation(n * 2)[:n].astype(np.int32)            # slot order != position order
    got = orc.select_top_b(score, pos, B, n_sink)
    assert np.array_equal(got, brute_force_keep(score, pos, B, n_sink))
    assert got.sum() == min(B, n)


def test_select_all_ties_keeps_lowest_positions_and_sinks():
    n, B = 20, 7
    pos = np.arange(n, dtype=np.int32)[::-1].copy()
    keep = orc.select_top_b(np.zeros(n, np.float32), pos, B, 0)
    assert sorted(pos[keep == 1].tolist()) == list(range(B))
    # sinks survive even with the lowest scores
    score = np.linspace(1.0, 2.0, n).astype(np.float32)
    pos = np.arange(n, dtype=np.int32)
    keep = orc.select_top_b(score, pos, 6, 4)
    assert sorted(pos[keep == 1].tolist()) == [0, 1, 2, 3, 18, 19]
    # signed zeros compare equal: position decides
    keep = orc.select_top_b(np.array([-0.0, 0.0, -0.0, 0.0], np.float32), np.array([3, 2, 1, 0], np.int32), 2, 0)
    assert keep.tolist() == [0, 0, 1, 1]


def test_alpha_zero_keeps_first_positions():
    """G = 0 => alpha = 0 => every score ties at 0 => the B lowest positions stay."""
    rng = np.random.default_rng(3)
    L = orc.OracleLayer(small_cfg(B=9, n_sink=2))
    w = rand_weights(L, rng)
    w["G"] = np.zeros_like(w["G"])
    L.set_weights(w)
    X, Q, K, V = rand_tokens(L, rng, 30)
    L.prefill_chunk(0, X, Q, K, V)
    assert L.positions().tolist() == list(range(9))
    assert L.last_evicted().tolist() == list(range(9, 30))


# ------------------------------------------------------------------ prefill pooling
def test_prefill_pooled_importance_causal_max():
    n = 17
    L = orc.OracleLayer(small_cfg(B=1000))
    rand_weights(L, np.random.default_rng(4))
    X, Q, K, V = rand_tokens(L, np.random.default_rng(44), n)
    # stage functions (pinned above) give the per-query features; the pooling is re-done here
    qfs, als, kid = [], [], []
    for s in range(n):
        qf, al = L.index_query(X[s], Q[s].reshape(-1))
        qfs.append(qf); als.append(al); kid.append(L.index_key(X[s]))
    kid = np.stack(kid)
    A = np.stack([L.index_scores(qfs[s], als[s], kid) for s in range(n)])        # [s, t]
    A[np.triu_indices(n, 1)] = -np.inf                                            # key t > query s masked
    # ... but the pooled value is exported before the reset only through selection: use B < n
    L2 = orc.OracleLayer(small_cfg(B=5, n_sink=0))
    rand_weights(L2, np.random.default_rng(4))            # same draws as L's weights
    L2.prefill_chunk(0, X, Q, K, V)
    imp = A.max(axis=0).astype(np.float32)
    want = brute_force_keep(imp, np.arange(n), 5, 0)
    assert L2.positions().tolist() == np.nonzero(want)[0].tolist()
    # the last token is scored by its own query only
    assert imp[n - 1] == np.float32(A[n - 1, n - 1])


def test_decode_interval_pooling_and_reset():
    rng = np.random.default_rng(5)
    tau, B = 4, 10
    L = orc.OracleLayer(small_cfg(B=B, tau=tau, n_sink=1))
    rand_weights(L, rng)
    X, Q, K, V = rand_tokens(L, rng, B)
    L.prefill_chunk(0, X, Q, K, V)
    assert L.count() == B and np.all(L.entries()["acc"] == -np.inf)
    qfs, als = [], []
    for s in range(2 * tau):
        x, q, k, v = [a[0] for a in rand_tokens(L, rng, 1)]
        L.decode_step(0, x, q.reshape(-1), q, k, v)
        qfs.append(L.index_query(x, q.reshape(-1)))
        if (s + 1) % tau:
            # inside an interval nothing is evicted and acc is the running max over the interval's queries
            assert L.count() == B + (s + 1) % tau and L.since() == (s + 1) % tau
            e = L.entries()
            lo = s - (s % tau)
            want = np.full(L.count(), -np.inf)
            for j in range(lo, s + 1):
                a = L.index_scores(qfs[j][0], qfs[j][1], e["kidx"]).astype(np.float32)
                a[e["pos"] > B + j] = -np.inf           # entries appended after query j
                want = np.maximum(want, a)
            np.testing.assert_array_equal(e["acc"], want.astype(np.float32))
        else:
            assert L.count() == B and L.since() == 0 and len(L.last_evicted()) == tau
            assert np.all(L.entries()["acc"] == -np.inf)
    assert L.evict_steps() == 2


# ------------------------------------------------------------------ attention / budget invariants
def test_infinite_budget_is_exact_softmax_attention():
    rng = np.random.default_rng(6)
    L = orc.OracleLayer(small_cfg(B=10 ** 6))
    rand_weights(L, rng)
    c = L.cfg
    X, Q, K, V = rand_tokens(L, rng, 40)
    L.prefill_chunk(0, X[:30], Q[:30], K[:30], V[:30])
    for s in range(30, 40):
        ob, od = L.decode_step(0, X[s], Q[s].reshape(-1), Q[s], K[s], V[s])
        want = softmax_attention(Q[s], K[: s + 1], V[: s + 1], L.Gq, 1.0 / math.sqrt(c.d))
        np.testing.assert_allclose(od, want, rtol=1e-12, atol=1e-13)
        assert np.array_equal(ob, bf16(od))
    M, b = L.memory()
    assert not M.any() and not b.any() and L.evict_steps() == 0


def test_memory_disabled_is_attention_over_retained_set():
    rng = np.random.default_rng(7)
    L = orc.OracleLayer(small_cfg(B=8, enable_memory=0))
    rand_weights(L, rng)
    c = L.cfg
    X, Q, K, V = rand_tokens(L, rng, 40)
    L.prefill_chunk(0, X[:25], Q[:25], K[:25], V[:25])
    for s in range(25, 40):
        ob, od = L.decode_step(0, X[s], Q[s].reshape(-1), Q[s], K[s], V[s])
        keep = L.positions()
        assert len(keep) == 8 and set(range(c.n_sink)) <= set(keep.tolist())
        want = softmax_attention(Q[s], K[keep], V[keep], L.Gq, 1.0 / math.sqrt(c.d))
        np.testing.assert_allclose(od, want, rtol=1e-12, atol=1e-13)
    M, b = L.memory()
    assert not M.any() and not b.any()


def test_gqa_head_mapping():
    """Query head j must read KV head j // G_q: make one KV head's values constant and check."""
    rng = np.random.default_rng(8)
    L = orc.OracleLayer(small_cfg(B=100, enable_memory=0))
    rand_weights(L, rng)
    X, Q, K, V = rand_tokens(L, rng, 10)
    V[:, 0, :] = 1.0
    V[:, 1, :] = -2.0
    L.prefill_chunk(0, X[:9], Q[:9], K[:9], V[:9])
    _, od = L.decode_step(0, X[9], Q[9].reshape(-1), Q[9], K[9], V[9])
    np.testing.assert_allclose(od[:2], 1.0, atol=1e-12)
    np.testing.assert_allclose(od[2:], -2.0, atol=1e-12)


# ------------------------------------------------------------------ memory write / read
def model_space(kv, Gq):
    """[.., Hkv, d] -> [.., H*d] with query head j reading KV head j // G_q."""
    return np.repeat(kv, Gq, axis=-2).reshape(*kv.shape[:-2], -1)


def test_memory_additive_order_invariant_lambda_one():
    """At lambda = 1 the state is eta * sum over everything ever evicted, however it was split."""
    rng = np.random.default_rng(9)
    eta = 0.5
    L = orc.OracleLayer(small_cfg(B=6, eta=eta))
    w = rand_weights(L, rng)
    X, Q, K, V = rand_tokens(L, rng, 40)
    L.prefill_chunk(0, X[:10], Q[:10], K[:10], V[:10])       # evicts 4 at once
    L.prefill_chunk(0, X[10:25], Q[10:25], K[10:25], V[10:25])  # evicts 15 at once
    for s in range(25, 40):                                   # evicts one per step
        L.decode_step(0, X[s], Q[s].reshape(-1), Q[s], K[s], V[s])
    gone = sorted(set(range(40)) - set(L.positions().tolist()))
    assert len(gone) == 34
    Wt = w["W_theta"].astype(np.float64)
    for order in (gone, gone[::-1]):
        Phi = model_space(K[order], L.Gq).astype(np.float64) @ Wt.T            # [N, dM]
        Mw = eta * Phi.T @ model_space(V[order], L.Gq).astype(np.float64)     # [dM, D]
        bw = eta * (Phi ** 2).sum(axis=0)
        M, b = L.memory()
        np.testing.assert_allclose(M, Mw, rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(b, bw, rtol=1e-11, atol=1e-12)
    # KV-space view: columns of query heads in one group are equal
    Mkv, _ = L.memory_kv()
    c = L.cfg
    M3 = M.reshape(c.dM, c.H, c.d)
    for j in range(c.H):
        np.testing.assert_array_equal(M3[:, j], Mkv.reshape(c.dM, c.Hkv, c.d)[:, j // L.Gq])
    np.testing.assert_allclose(L.phi_kv(K[3]), Wt @ model_space(K[3], L.Gq), rtol=1e-12, atol=1e-13)


def test_memory_decay_lambda_power():
    """A write made j evict steps ago is scaled by lambda^j; steps without eviction do not decay."""
    rng = np.random.default_rng(10)
    lam, eta = 0.8, 1.0
    L = orc.OracleLayer(small_cfg(B=6, lambda_=lam, eta=eta, tau=2, n_sink=1))
    w = rand_weights(L, rng)
    X, Q, K, V = rand_tokens(L, rng, 30)
    Wt = w["W_theta"].astype(np.float64)
    M_want = np.zeros((L.cfg.dM, L.D))
    b_want = np.zeros(L.cfg.dM)
    L.prefill_chunk(0, X[:10], Q[:10], K[:10], V[:10])
    seen = 10
    prev = set(range(10))

    def account(evicted):
        nonlocal M_want, b_want
        Phi = model_space(K[evicted], L.Gq).astype(np.float64) @ Wt.T
        M_want = lam * M_want + eta * Phi.T @ model_space(V[evicted], L.Gq).astype(np.float64)
        b_want = lam * b_want + eta * (Phi ** 2).sum(axis=0)

    account(sorted(prev - set(L.positions().tolist())))
    for s in range(10, 30):
        L.decode_step(0, X[s], Q[s].reshape(-1), Q[s], K[s], V[s])
        ev = L.last_evicted().tolist()
        if (s - 10 + 1) % 2 == 0:
            assert len(ev) == 2
            account(ev)
        else:
            assert len(ev) == 0 or L.since() == 1
        M, b = L.memory()
        np.testing.assert_allclose(M, M_want, rtol=1e-11, atol=1e-13)
        np.testing.assert_allclose(b, b_want, rtol=1e-11, atol=1e-13)
    assert L.evict_steps() == 11


def test_single_pair_rank_one_closed_form():
    """d_M = 1, one evicted pair, lambda = eta = 1: m(q) = phi_q phi_k v / (phi_q^2 phi_k^2 + eps)."""
    rng = np.random.default_rng(11)
    eps = 1e-3
    L = orc.OracleLayer(small_cfg(B=3, dM=1, n_sink=0, eps=eps))
    w = rand_weights(L, rng, std=0.5)
    c = L.cfg
    X, Q, K, V = rand_tokens(L, rng, 5)
    L.prefill_chunk(0, X[:4], Q[:4], K[:4], V[:4])
    ev = L.last_evicted().tolist()
    assert len(ev) == 1
    wt = w["W_theta"].astype(np.float64)[0]
    phi_k = wt @ model_space(K[ev[0]], L.Gq)
    q = Q[4]
    phi_q = wt @ q.reshape(-1)
    m_want = phi_q * phi_k * model_space(V[ev[0]], L.Gq) / (phi_q ** 2 * phi_k ** 2 + eps)
    m, gate = L.mem_read(0, q.reshape(-1))
    np.testing.assert_allclose(m, m_want, rtol=1e-12, atol=1e-14)
    g_want = 1.0 / (1.0 + math.exp(-(w["w_g"].astype(np.float64) @ q.reshape(-1))))
    assert 0.0 <= gate <= 1.0 and abs(gate - g_want) < 1e-14
    # Eq. 4 on a decode step with B large enough that nothing more is evicted
    L2 = orc.OracleLayer(small_cfg(B=3, dM=1, n_sink=0, eps=eps, tau=100))
    L2.set_weights(w)
    L2.prefill_chunk(0, X[:4], Q[:4], K[:4], V[:4])
    _, od = L2.decode_step(0, X[4], q.reshape(-1), q, K[4], V[4])
    keep = L2.positions()
    o_attn = softmax_attention(q, np.concatenate([K[:4], K[4:5]])[keep], np.concatenate([V[:4], V[4:5]])[keep],
                               L2.Gq, 1.0 / math.sqrt(c.d))
    np.testing.assert_allclose(od.reshape(-1), o_attn.reshape(-1) + g_want * m_want, rtol=1e-12, atol=1e-14)


def test_gate_bias_and_range():
    rng = np.random.default_rng(12)
    L = orc.OracleLayer(small_cfg(B=3, n_sink=0))
    w = rand_weights(L, rng)
    X, Q, K, V = rand_tokens(L, rng, 6)
    L.prefill_chunk(0, X[:5], Q[:5], K[:5], V[:5])
    for bg, lo, hi in ((-40.0, 0.0, 1e-15), (40.0, 1 - 1e-15, 1.0)):
        w["b_g"] = np.array([bg], np.float32)
        L.set_weights(w)
        _, g = L.mem_read(0, Q[5].reshape(-1))
        assert lo <= g <= hi


# ------------------------------------------------------------------ layer outputs of a prefill chunk's own queries
def test_chunk_outputs_with_infinite_budget_are_causal_softmax_attention():
    """Nothing is ever evicted and the memory is off: the outputs of a prompt fed in three ragged chunks are
    textbook causal attention over the whole prompt (numpy, float64), row by row."""
    rng = np.random.default_rng(31)
    L = orc.OracleLayer(small_cfg(B=10_000, enable_memory=0))
    rand_weights(L, rng)
    c = L.cfg
    n = 23
    X, Q, K, V = rand_tokens(L, rng, n)
    outs = []
    for a, b in ((0, 7), (7, 8), (8, 23)):
        ob, od = L.prefill_chunk_out(0, X[a:b], Q[a:b], Q[a:b], K[a:b], V[a:b])
        outs.append(od)
        assert np.array_equal(ob, bf16(od))
    got = np.concatenate(outs)
    for s in range(n):
        want = softmax_attention(Q[s], K[:s + 1], V[:s + 1], c.H // c.Hkv, 1.0 / math.sqrt(c.d))
        np.testing.assert_allclose(got[s], want, rtol=1e-12, atol=1e-13)
    # the mask is causal: a later token must not change an earlier row
    L2 = orc.OracleLayer(small_cfg(B=10_000, enable_memory=0))
    rand_weights(L2, np.random.default_rng(31))
    K2 = K.copy()
    K2[-1] += 1.0
    _, od2 = L2.prefill_chunk_out(0, X, Q, Q, K2, V)
    np.testing.assert_allclose(od2[:-1], got[:-1], rtol=1e-12, atol=1e-13)
    assert not np.allclose(od2[-1], got[-1])


def test_chunk_outputs_attend_to_the_retained_prefix_and_read_the_memory_of_before_the_chunk():
    """After evictions: a chunk's query s sees exactly (entries retained when the chunk arrives) + (chunk tokens
    up to s), and Eq. 4 adds g(q) m(q) with the memory as it was BEFORE the chunk's own evict step.  Expected
    values: numpy softmax over the exported retained set plus the chunk, and Eq. 5 evaluated in numpy on the
    exported (M, b); the evict step of the chunk itself must not leak into its outputs."""
    rng = np.random.default_rng(32)
    L = orc.OracleLayer(small_cfg(B=9, n_sink=1))
    w = rand_weights(L, rng)
    c = L.cfg
    Gq = c.H // c.Hkv
    X, Q, K, V = rand_tokens(L, rng, 30)
    L.prefill_chunk(0, X[:14], Q[:14], K[:14], V[:14])          # evicts 5
    assert L.count(0) == 9 and L.evict_steps(0) == 1
    e = L.entries(0)
    M, b = L.memory(0)
    Cn = 11
    xs, qs, ks, vs = X[14:14 + Cn], Q[14:14 + Cn], K[14:14 + Cn], V[14:14 + Cn]
    ob, od = L.prefill_chunk_out(0, xs, qs, qs, ks, vs)
    assert L.evict_steps(0) == 2                                   # the chunk was compressed afterwards
    for s in range(Cn):
        Ks = np.concatenate([e["K"], ks[:s + 1]])
        Vs = np.concatenate([e["V"], vs[:s + 1]])
        o = softmax_attention(qs[s], Ks, Vs, Gq, 1.0 / math.sqrt(c.d))
        qd = qs[s].reshape(-1).astype(np.float64)
        phi = w["W_theta"].astype(np.float64) @ qd
        m = (phi @ M) / ((phi ** 2) @ b + c.eps)
        gate = 1.0 / (1.0 + math.exp(-float(w["w_g"].astype(np.float64).reshape(-1) @ qd)))
        want = o + gate * m.reshape(c.H, c.d)
        np.testing.assert_allclose(od[s], want, rtol=1e-10, atol=1e-12)
    # and the state after the call is the one the plain call leaves
    L2 = orc.OracleLayer(small_cfg(B=9, n_sink=1))
    L2.set_weights(w)
    L2.prefill_chunk(0, X[:14], Q[:14], K[:14], V[:14])
    L2.prefill_chunk(0, xs, qs, ks, vs)
    assert np.array_equal(L2.positions(0), L.positions(0))
    np.testing.assert_array_equal(L2.memory(0)[0], L.memory(0)[0])


def test_single_token_chunk_output_equals_decode_output_when_nothing_is_evicted():
    rng = np.random.default_rng(33)
    La, Lb = orc.OracleLayer(small_cfg(B=50, tau=1)), orc.OracleLayer(small_cfg(B=50, tau=1))
    w = rand_weights(La, rng)
    Lb.set_weights(w)
    X, Q, K, V = rand_tokens(La, rng, 12)
    for L in (La, Lb):
        L.prefill_chunk(0, X[:8], Q[:8], K[:8], V[:8])
    for t in range(8, 12):
        _, oa = La.prefill_chunk_out(0, X[t:t + 1], Q[t:t + 1], Q[t:t + 1], K[t:t + 1], V[t:t + 1])
        _, ob = Lb.decode_step(0, X[t], Q[t], Q[t], K[t], V[t])
        np.testing.assert_allclose(oa[0], ob, rtol=1e-13, atol=1e-14)


# ------------------------------------------------------------------ score reuse across neighbouring layers (App. B)
def _leader_and_follower(rng, same=False, **kw):
    lead = orc.OracleLayer(small_cfg(**kw))
    foll = orc.OracleLayer(small_cfg(**kw))
    wl = rand_weights(lead, rng)
    if same:
        foll.set_weights(wl)
        wf = wl
    else:
        wf = rand_weights(foll, rng)
    return lead, foll, wl, wf


def test_score_reuse_follower_keeps_the_leaders_positions_and_attends_to_its_own_cache():
    """IndexCache-style reuse: the following layer makes the leading layer's decisions (same retained positions
    after every call) but everything it computes comes from its own keys, values and queries: with the memory
    disabled its output is the textbook softmax attention over its own K / V at the positions the leader kept."""
    rng = np.random.default_rng(21)
    lead, foll, _, _ = _leader_and_follower(rng, B=9, tau=3, n_sink=2, enable_memory=0)
    n0, steps = 14, 13
    X, Q, K, V = rand_tokens(lead, rng, n0 + steps)
    _, Q2, K2, V2 = rand_tokens(foll, rng, n0 + steps)
    lead.prefill_chunk(0, X[:n0], Q[:n0], K[:n0], V[:n0])
    foll.prefill_chunk_follow(0, lead, 0, K2[:n0], V2[:n0])
    assert foll.positions().tolist() == lead.positions().tolist() and len(lead.positions()) == 9
    for s in range(n0, n0 + steps):
        lead.decode_step(0, X[s], Q[s].reshape(-1), Q[s], K[s], V[s])
        _, od = foll.decode_step_follow(0, lead, 0, Q2[s], K2[s], V2[s])
        pos = lead.positions()
        assert foll.positions().tolist() == pos.tolist()
        assert foll.since() == lead.since() and foll.evict_steps() == lead.evict_steps()
        want = softmax_attention(Q2[s], K2[pos], V2[pos], foll.Gq, foll.cfg.scale)
        np.testing.assert_allclose(od, want, rtol=1e-11, atol=1e-13)
        # the follower's cache holds its OWN rows at those positions
        e = foll.entries()
        assert np.array_equal(e["K"], K2[pos]) and np.array_equal(e["V"], V2[pos])
    assert lead.evict_steps() == 1 + steps // 3


def test_score_reuse_follower_writes_its_own_evicted_pairs_to_its_own_memory():
    """lambda = 1: the follower's (M, b) is the sum over every position evicted so far of phi(k) v^T / phi(k)^2 formed
    with the follower's weights, keys and values - the leader decides which positions, nothing else."""
    rng = np.random.default_rng(22)
    lead, foll, _, wf = _leader_and_follower(rng, B=7, tau=1, n_sink=1)
    n = 22
    X, Q, K, V = rand_tokens(lead, rng, n)
    _, Q2, K2, V2 = rand_tokens(foll, rng, n)
    lead.prefill_chunk(0, X[:10], Q[:10], K[:10], V[:10])
    foll.prefill_chunk_follow(0, lead, 0, K2[:10], V2[:10])
    for s in range(10, n):
        lead.decode_step(0, X[s], Q[s].reshape(-1), Q[s], K[s], V[s])
        foll.decode_step_follow(0, lead, 0, Q2[s], K2[s], V2[s])
    gone = sorted(set(range(n)) - set(lead.positions().tolist()))
    assert len(gone) == n - 7
    Wt = wf["W_theta"].astype(np.float64)
    Phi = model_space(K2[gone], foll.Gq).astype(np.float64) @ Wt.T
    M, b = foll.memory()
    np.testing.assert_allclose(M, Phi.T @ model_space(V2[gone], foll.Gq).astype(np.float64), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(b, (Phi ** 2).sum(axis=0), rtol=1e-10, atol=1e-12)
    Ml, _ = lead.memory()
    assert not np.allclose(M, Ml)


def test_score_reuse_follower_with_the_leaders_inputs_reproduces_the_leader():
    """A follower given the leader's weights, keys, values and queries is the leader: outputs, cache and memory agree
    to the last bit (reusing the scores changes who computes them, not what is selected), also for the layer outputs
    of a prefill chunk's own queries."""
    rng = np.random.default_rng(23)
    lead, foll, _, _ = _leader_and_follower(rng, same=True, B=8, tau=2, n_sink=2, lambda_=0.9, eta=0.5)
    X, Q, K, V = rand_tokens(lead, rng, 30)
    for c in range(2):
        sl = slice(6 * c, 6 * c + 6)
        _, od_l = lead.prefill_chunk_out(0, X[sl], Q[sl], Q[sl], K[sl], V[sl])
        _, od_f = foll.prefill_chunk_follow(0, lead, 0, K[sl], V[sl], Q=Q[sl])
        assert np.array_equal(od_l, od_f)
    for s in range(12, 30):
        _, od_l = lead.decode_step(0, X[s], Q[s].reshape(-1), Q[s], K[s], V[s])
        _, od_f = foll.decode_step_follow(0, lead, 0, Q[s], K[s], V[s])
        assert np.array_equal(od_l, od_f)
    for a, b in zip(lead.memory(), foll.memory()):
        assert np.array_equal(a, b)
    el, ef = lead.entries(), foll.entries()
    assert np.array_equal(el["pos"], ef["pos"]) and np.array_equal(el["K"], ef["K"]) and np.array_equal(el["V"], ef["V"])


def test_score_reuse_needs_the_leaders_call_first():
    rng = np.random.default_rng(24)
    lead, foll, _, _ = _leader_and_follower(rng, B=5, tau=1)
    X, Q, K, V = rand_tokens(lead, rng, 8)
    lead.prefill_chunk(0, X[:7], Q[:7], K[:7], V[:7])
    foll.prefill_chunk_follow(0, lead, 0, K[:7], V[:7])
    with pytest.raises(AssertionError):            # the leader has not seen token 7 yet
        foll.decode_step_follow(0, lead, 0, Q[7], K[7], V[7])


# ------------------------------------------------------------------ a retained set per KV head (Sec. 2.2 framework)
def _dense_scores(pos, acc, n_pos, Hkv):
    """[Hkv, n_pos] score table by token position with the same row for every head."""
    row = np.full(n_pos, -np.inf, np.float32)
    row[pos] = acc
    return np.tile(row, (Hkv, 1))


def test_per_head_knorm_keeps_the_largest_key_norms_of_every_head():
    """Knorm (Sec. 2.2: S_t = ||K_t||_2): every KV head keeps its sinks and then the B - n_sink entries with the
    largest key norm of THAT head (ties to the lower position) - a brute-force sort per head; the heads' sets differ."""
    rng = np.random.default_rng(31)
    L = orc.OracleLayer(small_cfg(Hkv=2, B=7, tau=3, n_sink=2, scorer=1, enable_memory=0))
    rand_weights(L, rng)
    _, Q, K, V = rand_tokens(L, rng, 40)
    K = bf16(K * np.exp(0.6 * rng.standard_normal((40, 2, 1))))          # norms differ between heads
    L.ph_prefill_chunk(0, K[:12], V[:12])
    alive = [list(range(12)) for _ in range(2)]

    def compress(h):
        norm = lambda t: np.float32(np.sqrt((K[t, h].astype(np.float64) ** 2).sum()))
        order = sorted(alive[h], key=lambda t: (-(math.inf if t < 2 else float(norm(t))), t))
        alive[h] = sorted(order[:7])

    for h in range(2):
        compress(h)
        assert L.ph_entries(0, h)["pos"].tolist() == alive[h]
    for s in range(12, 40):
        _, od = L.ph_decode_step(0, Q[s], K[s], V[s])
        for h in range(2):
            alive[h].append(s)
            if (s - 12 + 1) % 3 == 0:
                compress(h)
            e = L.ph_entries(0, h)
            assert e["pos"].tolist() == alive[h]
            assert np.array_equal(e["K"], K[alive[h], h]) and np.array_equal(e["V"], V[alive[h], h])
        # attention of query head j over the set of ITS KV head (memory disabled): textbook softmax per head
        for j in range(L.cfg.H):
            g = j // L.Gq
            sc = (K[alive[g], g].astype(np.float64) @ Q[s, j].astype(np.float64)) * L.cfg.scale
            pr = np.exp(sc - sc.max())
            np.testing.assert_allclose(od[j], (pr / pr.sum()) @ V[alive[g], g].astype(np.float64), rtol=1e-11, atol=1e-13)
    assert alive[0] != alive[1]


def test_per_head_memory_write_assembles_the_evicted_slices_of_a_token():
    """The evict step's memory write with per-head sets (Alg. 1, "summed across heads per token"): a token that loses
    the slices of some heads in this step contributes ONE pair (k~, v~) in model space, holding those slices at their
    query heads' places and zeros elsewhere.  Scores from the caller make head 0 evict positions {1, 3} and head 1
    evict {3, 4}: three pairs - position 1 (head 0 only), 3 (both), 4 (head 1 only) - against numpy."""
    rng = np.random.default_rng(32)
    L = orc.OracleLayer(small_cfg(Hkv=2, B=3, n_sink=0, scorer=2, lambda_=0.5, eta=2.0))
    w = rand_weights(L, rng)
    c = L.cfg
    _, Q, K, V = rand_tokens(L, rng, 6)
    ext = np.array([[5, 0, 4, 1, 3], [5, 4, 3, 0, 1]], np.float32)        # by position, per head
    L.ph_prefill_chunk(0, K[:5], V[:5], ext=ext)
    assert L.ph_entries(0, 0)["pos"].tolist() == [0, 2, 4] and L.ph_entries(0, 1)["pos"].tolist() == [0, 1, 2]
    assert L.ph_last_evicted(0, 0).tolist() == [1, 3] and L.ph_last_evicted(0, 1).tolist() == [3, 4]
    Wt = w["W_theta"].astype(np.float64)
    M_want, b_want = np.zeros((c.dM, L.D)), np.zeros(c.dM)
    for t, heads in ((1, [0]), (3, [0, 1]), (4, [1])):
        ku, vu = np.zeros((c.H, c.d)), np.zeros((c.H, c.d))
        for h in heads:
            ku[h * L.Gq:(h + 1) * L.Gq] = K[t, h]
            vu[h * L.Gq:(h + 1) * L.Gq] = V[t, h]
        phi = Wt @ ku.reshape(-1)
        M_want += np.outer(phi, vu.reshape(-1))
        b_want += phi ** 2
    M, b = L.memory()
    np.testing.assert_allclose(M, 2.0 * M_want, rtol=1e-11, atol=1e-13)     # eta = 2, first evict step: lambda * 0
    np.testing.assert_allclose(b, 2.0 * b_want, rtol=1e-11, atol=1e-13)
    # a second evict step decays the first: one more token, every head evicts its lowest score
    ext2 = np.array([[5, 0, 4, 1, 3, 2], [5, 4, 3, 0, 1, 9]], np.float32)
    L.ph_decode_step(0, Q[5], K[5], V[5], ext=ext2)
    assert L.ph_last_evicted(0, 0).tolist() == [5] and L.ph_last_evicted(0, 1).tolist() == [2]
    M2_want, b2_want = 0.5 * 2.0 * M_want, 0.5 * 2.0 * b_want
    for t, h in ((2, 1), (5, 0)):
        ku, vu = np.zeros((c.H, c.d)), np.zeros((c.H, c.d))
        ku[h * L.Gq:(h + 1) * L.Gq] = K[t, h]
        vu[h * L.Gq:(h + 1) * L.Gq] = V[t, h]
        phi = Wt @ ku.reshape(-1)
        M2_want += 2.0 * np.outer(phi, vu.reshape(-1))
        b2_want += 2.0 * phi ** 2
    M, b = L.memory()
    np.testing.assert_allclose(M, M2_want, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(b, b2_want, rtol=1e-11, atol=1e-13)


def test_per_head_sets_with_identical_rows_reduce_to_the_shared_row_path():
    """Handed the indexer's own pooled scores as the row of every head, the per-head path makes the indexer path's
    selections, memory writes and outputs to the last bit (a token then loses all its slices at once and the
    assembled pair is the plain lifted key / value)."""
    rng = np.random.default_rng(33)
    kw = dict(B=8, tau=2, n_sink=1, lambda_=0.9, eta=0.7)
    A = orc.OracleLayer(small_cfg(**kw))
    P = orc.OracleLayer(small_cfg(scorer=2, **kw))
    w = rand_weights(A, rng)
    P.set_weights(w)
    X, Q, K, V = rand_tokens(A, rng, 34)
    Hkv = A.cfg.Hkv
    _, od_a = A.prefill_chunk_out(0, X[:14], Q[:14], Q[:14], K[:14], V[:14])
    _, od_p = P.ph_prefill_chunk(0, K[:14], V[:14], Q=Q[:14], ext=_dense_scores(*A.last_selection(), 14, Hkv))
    assert np.array_equal(od_a, od_p)
    for s in range(14, 34):
        _, od_a = A.decode_step(0, X[s], Q[s].reshape(-1), Q[s], K[s], V[s])
        ext = _dense_scores(*A.last_selection(), s + 1, Hkv) if A.since() == 0 else None
        _, od_p = P.ph_decode_step(0, Q[s], K[s], V[s], ext=ext)
        assert np.array_equal(od_a, od_p), s
        for h in range(Hkv):
            assert P.ph_entries(0, h)["pos"].tolist() == A.positions().tolist()
    for a, b in zip(A.memory(), P.memory()):
        assert np.array_equal(a, b)
    assert A.evict_steps() == P.evict_steps() == 1 + 10


def test_per_head_scores_from_the_caller_are_required():
    rng = np.random.default_rng(34)
    L = orc.OracleLayer(small_cfg(B=3, scorer=2))
    rand_weights(L, rng)
    _, Q, K, V = rand_tokens(L, rng, 5)
    with pytest.raises(AssertionError):
        L.ph_prefill_chunk(0, K[:5], V[:5])                               # no scores
    L2 = orc.OracleLayer(small_cfg(B=3, scorer=2))
    with pytest.raises(AssertionError):
        L2.ph_prefill_chunk(0, K[:5], V[:5], ext=np.zeros((2, 4), np.float32))   # position 4 not covered
