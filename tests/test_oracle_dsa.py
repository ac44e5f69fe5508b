"""Pins for the sparse (DSA) replay oracle: brute force, hand values, the dense limit, the
two-level (per-shard, then global) selection of Eq. glm-global-dsa, and finite differences."""
import math

import numpy as np

from oracle import attention as oa
from oracle import dsa
from oracle import pages as op


def make(seed, P=11, R=5, pg=4, dk=6, dv=4, hi=3, di=5, n_extra_pages=2):
    rng = np.random.default_rng(seed)
    n_pages = (P + pg - 1) // pg
    nphys = n_pages + n_extra_pages
    table = rng.permutation(nphys)[:n_pages]
    k_pool = rng.standard_normal((nphys, pg, 1, dk))
    ki_pool = rng.standard_normal((nphys, pg, 1, di))
    k_resp = rng.standard_normal((R, 1, dk))
    ki_resp = rng.standard_normal((R, di))
    q = rng.standard_normal((R, dk))
    qi = rng.standard_normal((R, hi, di))
    w = rng.standard_normal((R, hi))
    d_o = rng.standard_normal((R, dv))
    return dict(P=P, R=R, pg=pg, dk=dk, dv=dv, table=table, k_pool=k_pool, ki_pool=ki_pool, k_resp=k_resp,
                ki_resp=ki_resp, q=q, qi=qi, w=w, d_o=d_o)


def key_at(c, s, pool="k_pool", resp="k_resp"):
    if s < c["P"]:
        return c[pool][c["table"][s // c["pg"]], s % c["pg"], 0]
    r = c[resp][s - c["P"]]
    return r[0] if r.ndim == 2 else r


def test_index_scores_against_scalar_loops():
    c = make(1)
    t_rows = np.arange(c["R"])
    got = dsa.index_scores(c["qi"], c["w"], t_rows, c["ki_pool"], c["table"], c["P"], c["pg"], c["ki_resp"])
    for t in range(c["R"]):
        for s in range(c["P"] + c["R"]):
            if s - c["P"] > t:
                assert got[t, s] == -np.inf
                continue
            ki = key_at(c, s, "ki_pool", "ki_resp")
            want = 0.0
            for j in range(c["qi"].shape[1]):
                dot = sum(c["qi"][t, j, d] * ki[d] for d in range(len(ki)))
                want += c["w"][t, j] * max(dot, 0.0)
            assert abs(got[t, s] - want) < 1e-12


def test_index_score_hand_example():
    # one index head, weight 2: scores are 2 ReLU(<q, k>); a negative dot product scores exactly 0
    qi = np.array([[[1.0, -1.0]]])
    w = np.array([[2.0]])
    pool = np.array([[[[3.0, 1.0]], [[1.0, 4.0]]]])          # one page of two tokens
    got = dsa.index_scores(qi, w, np.array([0]), pool, np.array([0]), 2, 2, np.array([[0.5, 0.25]]))
    assert got.tolist() == [[4.0, 0.0, 0.5]]


def test_topk_rule():
    s = np.array([1.0, 5.0, 3.0, 5.0, -np.inf, 3.0, 0.0])
    assert dsa.topk_select(s, 1).tolist() == [1]                 # tie between 1 and 3: lower position
    assert dsa.topk_select(s, 2).tolist() == [1, 3]
    assert dsa.topk_select(s, 3).tolist() == [1, 2, 3]           # tie between 2 and 5: lower position
    assert dsa.topk_select(s, 4).tolist() == [1, 2, 3, 5]
    assert dsa.topk_select(s, 6).tolist() == [0, 1, 2, 3, 5, 6]  # exactly the visible ones
    assert dsa.topk_select(s, 100).tolist() == [0, 1, 2, 3, 5, 6]
    assert dsa.topk_select(np.full(4, -np.inf), 2).tolist() == []


def test_per_shard_candidates_then_global_topk_equals_global_topk():
    # Eq. glm-global-dsa: every shard's top-k candidates, merged and re-ranked, give the global top-k,
    # for any ownership policy -- with ties decided by global position
    rng = np.random.default_rng(3)
    P, pg = 64 * 7 + 5, 64
    for policy in (op.CONTIGUOUS, op.CYCLIC, op.ZIGZAG):
        for S in (1, 3, 8):
            scores = np.round(rng.standard_normal(P + 4), 1)       # rounding makes ties common
            shards = op.shard_positions(P, pg, S, policy) + [np.arange(P, P + 4)]
            for k in (1, 5, 64, 1000):
                a = dsa.topk_select(scores, k)
                b = dsa.merge_shard_candidates(scores, shards, k)
                assert np.array_equal(a, b), (policy, S, k)


def test_selecting_everything_is_the_dense_operator():
    c = make(4)
    t_rows = np.arange(c["R"])
    sel = [np.arange(c["P"] + t + 1) for t in t_rows]
    v_resp = c["k_resp"][..., :c["dv"]]
    o, lse, dq, dk, dv = dsa.sparse_backward_rows(c["q"], sel, c["k_pool"], c["table"], c["P"], c["pg"], c["k_resp"],
                                                  c["dv"], 0.41, c["d_o"])
    o2, lse2, dq2, dk2, dv2 = oa.backward_rows(c["q"], t_rows, 0, c["k_pool"], c["k_pool"], c["table"], c["P"],
                                               c["pg"], c["k_resp"], v_resp, 0.41, c["d_o"])
    for a, b in ((o, o2), (lse, lse2), (dq, dq2), (dk, dk2), (dv, dv2)):
        assert np.abs(a - b).max() < 1e-12


def test_sparse_forward_against_scalar_loops_and_one_hot_limit():
    c = make(5)
    t_rows = np.arange(c["R"])
    I = dsa.index_scores(c["qi"], c["w"], t_rows, c["ki_pool"], c["table"], c["P"], c["pg"], c["ki_resp"])
    sel = [dsa.topk_select(I[t], 4) for t in t_rows]
    scale = 0.3
    o, lse, _ = dsa.sparse_forward_rows(c["q"], sel, c["k_pool"], c["table"], c["P"], c["pg"], c["k_resp"], c["dv"], scale)
    for t in t_rows:
        s = [scale * sum(c["q"][t, d] * key_at(c, int(j))[d] for d in range(c["dk"])) for j in sel[t]]
        m = max(s)
        z = sum(math.exp(x - m) for x in s)
        assert abs(lse[t] - (m + math.log(z))) < 1e-12
        for ch in range(c["dv"]):
            want = sum(math.exp(x - m) / z * key_at(c, int(j))[ch] for x, j in zip(s, sel[t]))
            assert abs(o[t, ch] - want) < 1e-12
    # k = 1: the output is the selected latent's value, the log-normaliser its score
    one = [dsa.topk_select(I[t], 1) for t in t_rows]
    o1, lse1, _ = dsa.sparse_forward_rows(c["q"], one, c["k_pool"], c["table"], c["P"], c["pg"], c["k_resp"], c["dv"], scale)
    for t in t_rows:
        kk = key_at(c, int(one[t][0]))
        assert np.allclose(o1[t], kk[:c["dv"]]) and abs(lse1[t] - scale * float(c["q"][t] @ kk)) < 1e-12


def test_two_key_hand_example():
    # two selected keys with scores 0 and ln 3 (scale 1): p = (1/4, 3/4), LSE = ln 4
    q = np.array([[1.0, 0.0]])
    pool = np.array([[[[0.0, 2.0]], [[math.log(3.0), -2.0]]]])
    o, lse, probs = dsa.sparse_forward_rows(q, [np.array([0, 1])], pool, np.array([0]), 2, 2, np.zeros((1, 1, 2)), 2, 1.0)
    assert abs(lse[0] - math.log(4.0)) < 1e-12 and np.allclose(probs[0], [0.25, 0.75])
    assert np.allclose(o[0], [0.75 * math.log(3.0), 0.5 - 1.5])


def test_backward_by_finite_differences_with_the_selection_held_fixed():
    c = make(6, P=9, R=4)
    t_rows = np.arange(c["R"])
    I = dsa.index_scores(c["qi"], c["w"], t_rows, c["ki_pool"], c["table"], c["P"], c["pg"], c["ki_resp"])
    sel = [dsa.topk_select(I[t], 5) for t in t_rows]
    assert any((s >= c["P"]).any() for s in sel), "some response positions must be selected"
    scale, dvv = 0.37, c["dv"]

    def loss(q, k_resp):
        o, _, _ = dsa.sparse_forward_rows(q, sel, c["k_pool"], c["table"], c["P"], c["pg"], k_resp, dvv, scale)
        return float((o * c["d_o"]).sum())

    _, _, dq, dk, dv = dsa.sparse_backward_rows(c["q"], sel, c["k_pool"], c["table"], c["P"], c["pg"], c["k_resp"], dvv,
                                                scale, c["d_o"])
    h = 1e-6
    for idx in np.ndindex(*c["q"].shape):
        qp, qm = c["q"].copy(), c["q"].copy()
        qp[idx] += h
        qm[idx] -= h
        assert abs((loss(qp, c["k_resp"]) - loss(qm, c["k_resp"])) / (2 * h) - dq[idx]) < 1e-7
    # the latent row of a response token is key (all channels) and value (first dv channels) at once:
    # its total derivative is dK + dV padded to the key width
    total = dk.copy()
    total[:, :dvv] += dv
    for j in range(c["R"]):
        for ch in range(c["dk"]):
            kp, km = c["k_resp"].copy(), c["k_resp"].copy()
            kp[j, 0, ch] += h
            km[j, 0, ch] -= h
            assert abs((loss(c["q"], kp) - loss(c["q"], km)) / (2 * h) - total[j, ch]) < 1e-7
