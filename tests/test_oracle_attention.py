"""Pins for the fp64 attention oracle: hand-derived closed forms, brute force with
scalar loops, central finite differences, merge = unsharded, page-permutation
bit-identity, and the P = 0 / masked cases against a library attention."""
import math

import numpy as np
import pytest
import torch

from oracle import attention as oa
from oracle import pages as op


def rand_case(seed, P, pg, R, Hq, Hkv, Dk, Dv, extra=1, scale=None):
    rng = np.random.default_rng(seed)
    Np = op.num_pages(P, pg)
    nphys = Np + extra
    k_pool = rng.standard_normal((nphys, pg, Hkv, Dk))
    v_pool = rng.standard_normal((nphys, pg, Hkv, Dv))
    table = rng.permutation(nphys)[:Np].astype(np.int32)
    q = rng.standard_normal((R, Hq, Dk))
    k_resp = rng.standard_normal((R, Hkv, Dk))
    v_resp = rng.standard_normal((R, Hkv, Dv))
    d_o = rng.standard_normal((R, Hq, Dv))
    scale = 1.0 / math.sqrt(Dk) if scale is None else scale
    return dict(q=q, k_pool=k_pool, v_pool=v_pool, page_table=table, P=P, pg=pg,
                k_resp=k_resp, v_resp=v_resp, scale=scale), d_o


def logical(pool, table, P, pg):
    """Test-side gather of the prefix in logical order (scalar indexing)."""
    out = np.zeros((P,) + pool.shape[2:])
    for j in range(P):
        out[j] = pool[table[j // pg], j % pg]
    return out


# ------------------------------------------------------------------ closed forms

def test_two_key_hand_example():
    # One prefix key k=0 (score 0), response key k=ln3 (score ln3) with q=1, scale=1:
    # weights 1/4 and 3/4, LSE = ln 4.
    k_pool = np.zeros((1, 1, 1, 1))
    v_pool = np.array([[[[10.0]]]])
    q = np.ones((1, 1, 1))
    k_resp = np.full((1, 1, 1), math.log(3.0))
    v_resp = np.array([[[2.0]]])
    o, lse = oa.replay_forward(q, k_pool, v_pool, np.array([0]), 1, 1, k_resp, v_resp, 1.0)
    assert abs(lse[0, 0] - math.log(4.0)) < 1e-15
    assert abs(o[0, 0, 0] - (10.0 * 0.25 + 2.0 * 0.75)) < 1e-14
    # dO = 1: Delta = 4, dp = (10, 2), ds = p(dp - Delta) = (1.5, -1.5);
    # dq = 0*1.5 + ln3*(-1.5); dK_resp = ds_resp * q = -1.5; dV_resp = p_resp = 0.75
    _, _, dq, dk, dv = oa.replay_backward(q, k_pool, v_pool, np.array([0]), 1, 1, k_resp, v_resp, 1.0,
                                          np.ones((1, 1, 1)))
    assert abs(dq[0, 0, 0] + 1.5 * math.log(3.0)) < 1e-14
    assert abs(dk[0, 0, 0] + 1.5) < 1e-14
    assert abs(dv[0, 0, 0] - 0.75) < 1e-14


def test_identical_keys_give_mean_of_values():
    rng = np.random.default_rng(3)
    P, pg, R, Hq, Hkv, Dk, Dv = 37, 8, 5, 4, 2, 6, 3
    c, d_o = rand_case(4, P, pg, R, Hq, Hkv, Dk, Dv)
    kvec = rng.standard_normal((Hkv, Dk))
    c["k_pool"][:] = kvec
    c["k_resp"][:] = kvec
    o, lse, dq, dk, dv = oa.replay_backward(**c, d_o=d_o)
    vlog = logical(c["v_pool"], c["page_table"], P, pg)
    g = Hq // Hkv
    for t in range(R):
        for h in range(Hq):
            kv = h // g
            n = P + t + 1
            mean = (vlog[:, kv].sum(0) + c["v_resp"][:t + 1, kv].sum(0)) / n
            s = c["scale"] * c["q"][t, h] @ kvec[kv]
            assert np.allclose(o[t, h], mean, atol=1e-13)
            assert abs(lse[t, h] - (s + math.log(n))) < 1e-12
    # softmax is flat in q when all keys coincide: sum_j ds_j k_j = k * sum_j ds_j = 0
    assert np.abs(dq).max() < 1e-12


def test_one_hot_limit_returns_the_needle_value():
    c, _ = rand_case(5, 64, 16, 4, 2, 1, 8, 8)
    t, h, pos = 2, 1, 41
    c["k_pool"][c["page_table"][pos // 16], pos % 16, 0] = 40.0 * c["q"][t, h] / c["scale"] / (c["q"][t, h] @ c["q"][t, h])
    o, lse = oa.replay_forward(**c)
    v_needle = c["v_pool"][c["page_table"][pos // 16], pos % 16, 0]
    assert np.allclose(o[t, h], v_needle, atol=1e-9)
    assert abs(lse[t, h] - 40.0) < 1e-9


def test_lse_statistics_for_gaussian_scores():
    # given q, scores are N(0, sigma^2) with sigma = scale |q|: E exp(s) = e^{sigma^2/2},
    # so LSE ~ ln(n) + sigma^2 / 2 (~ ln n + 1/2 for N(0,1) q and scale 1/sqrt(D))
    c, _ = rand_case(6, 8192, 64, 2, 1, 1, 64, 4)
    _, lse = oa.replay_forward(**c)
    sig2 = (c["scale"] ** 2) * (c["q"][:, 0] ** 2).sum(-1)
    assert np.allclose(lse[:, 0], math.log(8192) + sig2 / 2, atol=0.08)


# ------------------------------------------------------------------ brute force

def brute_forward(c):
    q, kr, vr = c["q"], c["k_resp"], c["v_resp"]
    P, pg, sc = c["P"], c["pg"], c["scale"]
    R, Hq, Dk = q.shape
    Hkv, Dv = vr.shape[1], vr.shape[2]
    g = Hq // Hkv
    O = np.zeros((R, Hq, Dv))
    L = np.zeros((R, Hq))
    for t in range(R):
        for h in range(Hq):
            kv = h // g
            scores, vals = [], []
            for j in range(P):
                kj = c["k_pool"][c["page_table"][j // pg]][j % pg][kv]
                scores.append(sc * sum(q[t, h, d] * kj[d] for d in range(Dk)))
                vals.append(c["v_pool"][c["page_table"][j // pg]][j % pg][kv])
            for j in range(t + 1):
                scores.append(sc * sum(q[t, h, d] * kr[j, kv, d] for d in range(Dk)))
                vals.append(vr[j, kv])
            z = sum(math.exp(s) for s in scores)
            L[t, h] = math.log(z)
            for s, v in zip(scores, vals):
                for d in range(Dv):
                    O[t, h, d] += math.exp(s) / z * v[d]
    return O, L


@pytest.mark.parametrize("P,pg", [(0, 2), (1, 2), (5, 2), (8, 4)])
def test_forward_brute_force(P, pg):
    c, _ = rand_case(10 + P, P, pg, 3, 4, 2, 6, 4)
    o, lse = oa.replay_forward(**c)
    bo, bl = brute_forward(c)
    assert np.abs(o - bo).max() < 1e-13
    assert np.abs(lse - bl).max() < 1e-13


# ------------------------------------------------------------------ backward

def loss(c, d_o):
    o, _ = oa.replay_forward(**c)
    return float((o * d_o).sum())


@pytest.mark.parametrize("P,pg,Hq,Hkv", [(7, 4, 4, 2), (0, 4, 2, 2), (12, 4, 3, 1)])
def test_backward_finite_differences(P, pg, Hq, Hkv):
    c, d_o = rand_case(20 + P, P, pg, 4, Hq, Hkv, 5, 3)
    _, _, dq, dk, dv = oa.replay_backward(**c, d_o=d_o)
    eps = 1e-6
    for name, grad in (("q", dq), ("k_resp", dk), ("v_resp", dv)):
        num = np.zeros_like(grad)
        it = np.nditer(c[name], flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            old = c[name][idx]
            c[name][idx] = old + eps
            lp = loss(c, d_o)
            c[name][idx] = old - eps
            lm = loss(c, d_o)
            c[name][idx] = old
            num[idx] = (lp - lm) / (2 * eps)
        assert np.abs(num - grad).max() < 1e-7, name


def test_backward_matches_library_autograd_with_prefix():
    # library masked attention + autograd; prefix K/V enter as constants (stop-gradient)
    P, pg, R, Hq, Hkv, Dk, Dv = 21, 4, 6, 4, 2, 8, 5
    c, d_o = rand_case(31, P, pg, R, Hq, Hkv, Dk, Dv)
    kp = torch.tensor(logical(c["k_pool"], c["page_table"], P, pg))
    vp = torch.tensor(logical(c["v_pool"], c["page_table"], P, pg))
    q = torch.tensor(c["q"], requires_grad=True)
    kr = torch.tensor(c["k_resp"], requires_grad=True)
    vr = torch.tensor(c["v_resp"], requires_grad=True)
    g = Hq // Hkv
    k_all = torch.cat([kp, kr], 0).repeat_interleave(g, dim=1).permute(1, 0, 2)   # [Hq, P+R, Dk]
    v_all = torch.cat([vp, vr], 0).repeat_interleave(g, dim=1).permute(1, 0, 2)
    mask = torch.ones(R, P + R, dtype=torch.bool)
    mask[:, P:] = torch.tril(torch.ones(R, R, dtype=torch.bool))
    out = torch.nn.functional.scaled_dot_product_attention(
        q.permute(1, 0, 2), k_all, v_all, attn_mask=mask, scale=c["scale"]).permute(1, 0, 2)
    (out * torch.tensor(d_o)).sum().backward()
    o, lse, dq, dk, dv = oa.replay_backward(**c, d_o=d_o)
    assert np.abs(o - out.detach().numpy()).max() < 1e-12
    assert np.abs(dq - q.grad.numpy()).max() < 1e-12
    assert np.abs(dk - kr.grad.numpy()).max() < 1e-12
    assert np.abs(dv - vr.grad.numpy()).max() < 1e-12


def test_p0_reduces_to_causal_self_attention():
    c, d_o = rand_case(41, 0, 4, 9, 4, 4, 8, 8)
    q = torch.tensor(c["q"], requires_grad=True)
    kr = torch.tensor(c["k_resp"], requires_grad=True)
    vr = torch.tensor(c["v_resp"], requires_grad=True)
    out = torch.nn.functional.scaled_dot_product_attention(
        q.permute(1, 0, 2), kr.permute(1, 0, 2), vr.permute(1, 0, 2), is_causal=True,
        scale=c["scale"]).permute(1, 0, 2)
    (out * torch.tensor(d_o)).sum().backward()
    o, _, dq, dk, dv = oa.replay_backward(**c, d_o=d_o)
    assert np.abs(o - out.detach().numpy()).max() < 1e-12
    assert np.abs(dq - q.grad.numpy()).max() < 1e-12
    assert np.abs(dk - kr.grad.numpy()).max() < 1e-12
    assert np.abs(dv - vr.grad.numpy()).max() < 1e-12
    # scale invariance q -> a q, k -> k / a leaves the loss unchanged: sum q.dq = sum k.dk
    assert abs((c["q"] * dq).sum() - (c["k_resp"] * dk).sum()) < 1e-10
    # each row's probabilities sum to one: sum_j dV_j = sum_{t,h in group} dO
    assert np.allclose(dv.sum(0), d_o.sum(0), atol=1e-12)


def test_rows_subset_matches_full():
    c, d_o = rand_case(51, 19, 4, 8, 4, 2, 6, 6)
    o, lse, dq, dk, dv = oa.replay_backward(**c, d_o=d_o)
    T = 3
    t_rows = np.repeat(np.arange(8 - T, 8), 2)
    heads = np.tile(np.array([2, 3]), T)           # KV group 1
    args = {k: v for k, v in c.items() if k != "q"}
    o2, l2, dq2, dk2, dv2 = oa.backward_rows(c["q"][t_rows, heads], t_rows, 1, d_o_rows=d_o[t_rows, heads], **args)
    assert np.abs(o2 - o[t_rows, heads]).max() < 1e-13
    assert np.abs(l2 - lse[t_rows, heads]).max() < 1e-13
    assert np.abs(dq2 - dq[t_rows, heads]).max() < 1e-13
    # keys j >= R-T receive gradient only from the tail rows
    assert np.abs(dk2[8 - T:] - dk[8 - T:, 1]).max() < 1e-13
    assert np.abs(dv2[8 - T:] - dv[8 - T:, 1]).max() < 1e-13


# ------------------------------------------------------------------ merge and pages

@pytest.mark.parametrize("policy", [op.CONTIGUOUS, op.CYCLIC, op.ZIGZAG])
@pytest.mark.parametrize("S", [1, 2, 5, 16])
def test_merge_of_any_split_equals_unsharded(policy, S):
    P, pg, R, Hq, Hkv, Dk, Dv = 45, 4, 5, 4, 2, 6, 5     # ragged last page; S=16 > Np leaves empty shards
    c, _ = rand_case(61, P, pg, R, Hq, Hkv, Dk, Dv)
    o, lse = oa.replay_forward(**c)
    g = Hq // Hkv
    t = np.arange(R)
    for h in range(Hq):
        kv = h // g
        parts_o, parts_l = [], []
        for pos in op.shard_positions(P, pg, S, policy):
            po, pl = oa.local_attention(c["q"][:, h], kv, c["k_pool"], c["v_pool"], c["page_table"], pg, pos, c["scale"])
            parts_o.append(po)
            parts_l.append(pl)
        po, pl = oa.local_attention_response(c["q"][:, h], t, kv, c["k_resp"], c["v_resp"], c["scale"])
        parts_o.append(po)
        parts_l.append(pl)
        mo, ml = oa.merge(np.stack(parts_o), np.stack(parts_l))
        assert np.abs(mo - o[:, h]).max() < 1e-12
        assert np.abs(ml - lse[:, h]).max() < 1e-12
        assert np.isfinite(mo).all() and np.isfinite(ml).all()


def test_merge_hand_example_and_empty_part():
    # parts with l = ln1, ln3: weights 1/4, 3/4 ; a third part with l = -inf weighs 0
    o, l = oa.merge(np.array([[[4.0]], [[8.0]], [[123.0]]]), np.array([[0.0], [math.log(3.0)], [-np.inf]]))
    assert abs(o[0, 0] - 7.0) < 1e-14 and abs(l[0] - math.log(4.0)) < 1e-15


def test_physical_page_permutation_is_bit_identical():
    c, d_o = rand_case(71, 40, 8, 4, 4, 2, 8, 8, extra=3)
    ref = oa.replay_backward(**c, d_o=d_o)
    rng = np.random.default_rng(0)
    nphys = c["k_pool"].shape[0]
    perm = rng.permutation(nphys)                 # new physical slot of old page i is perm[i]
    k2 = np.empty_like(c["k_pool"]); v2 = np.empty_like(c["v_pool"])
    k2[perm] = c["k_pool"]; v2[perm] = c["v_pool"]
    c2 = dict(c, k_pool=k2, v_pool=v2, page_table=perm[c["page_table"]].astype(np.int32))
    out = oa.replay_backward(**c2, d_o=d_o)
    for a, b in zip(ref, out):
        assert np.array_equal(a, b)


def test_widen_is_exact_for_bf16_bits():
    bits = np.array([0x3F80, 0xBF80, 0x4049, 0x0000, 0x3DCD], dtype=np.uint16)
    want = torch.tensor(bits.view(np.int16)).view(torch.bfloat16).double().numpy()
    assert np.array_equal(oa.widen(bits), want)


def test_mla_alias_value_is_prefix_of_key_page():
    # V = first Dv channels of the K page (shared latent): passing the K pool as the V pool
    c, _ = rand_case(81, 24, 8, 3, 4, 1, 12, 8)
    c["v_pool"] = c["k_pool"]
    o, lse = oa.replay_forward(**c)
    c2 = dict(c, v_pool=np.ascontiguousarray(c["k_pool"][..., :8]))
    o2, lse2 = oa.replay_forward(**c2)
    assert np.array_equal(o, o2) and np.array_equal(lse, lse2)


def test_local_attention_value_slice_of_the_key_page():
    # shared-latent pages: V is the first dv channels of the K page.  Brute force with scalar loops.
    rng = np.random.default_rng(5)
    pg, n_pages, dk, dv = 4, 3, 8, 5
    pool = rng.standard_normal((n_pages, pg, 1, dk))
    table = np.array([2, 0, 1])
    q = rng.standard_normal((3, dk))
    positions = np.array([1, 4, 5, 9, 10])
    scale = 0.37
    o, l = oa.local_attention(q, 0, pool, pool, table, pg, positions, scale, dv=dv)
    assert o.shape == (3, dv)
    for i in range(3):
        s = []
        for pos in positions:
            key = pool[table[pos // pg], pos % pg, 0]
            s.append(scale * sum(q[i, c] * key[c] for c in range(dk)))
        m = max(s)
        z = sum(np.exp(x - m) for x in s)
        assert abs(l[i] - (m + np.log(z))) < 1e-12
        for c in range(dv):
            want = sum(np.exp(x - m) / z * pool[table[pos // pg], pos % pg, 0, c] for x, pos in zip(s, positions))
            assert abs(o[i, c] - want) < 1e-12
    # without dv the whole page would be the value: the slice is what makes the shapes differ
    o_full, _ = oa.local_attention(q, 0, pool, pool, table, pg, positions, scale)
    assert o_full.shape == (3, dk) and np.allclose(o_full[:, :dv], o)


def test_round_bf16_against_bit_patterns_and_ties():
    # every bf16 value is a float32 whose low 16 bits are zero: rounding must land on such a value, be the
    # nearest one, and send exact halves to the even neighbour
    rng = np.random.default_rng(5)
    x = np.concatenate([rng.standard_normal(2000) * 10.0 ** rng.integers(-6, 6, 2000), [0.0, 1.0, -3.5, 2.0 ** -20]])
    r = oa.round_bf16(x)
    bits = r.astype(np.float32).view(np.uint32)
    assert (r.astype(np.float32).astype(np.float64) == r).all() and (bits & 0xFFFF == 0).all()
    ulp = np.exp2(np.floor(np.log2(np.abs(np.where(x == 0, 1.0, x)))) - 7)
    assert (np.abs(r - x) <= ulp / 2 + 1e-300).all()
    # 1 + 2^-8 is halfway between 1 and 1 + 2^-7: even neighbour 1; 1 + 3 * 2^-8 is halfway: even neighbour 1 + 2^-6
    assert oa.round_bf16(np.array([1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, 1 + 2.0 ** -8 + 2.0 ** -20])).tolist() == \
        [1.0, 1 + 2.0 ** -6, 1 + 2.0 ** -7]


def test_merge_bf16_numerator_hand_example_and_bounds():
    # two shards of equal weight, o = 1 and 2^-9: the fp32 numerator 1 + 2^-9 is below half a bf16 step
    # above 1, so the bf16 numerator is 1 and o = 1/2, where the full-precision merge gives (1 + 2^-9)/2
    o = np.array([[[1.0]], [[2.0 ** -9]]])
    l = np.array([[0.3], [0.3]])
    got, lse = oa.merge_bf16_numerator(o, l)
    assert got[0, 0] == 0.5 and abs(lse[0] - (0.3 + np.log(2.0))) < 1e-15
    assert oa.merge(o, l)[0][0, 0] == (1 + 2.0 ** -9) / 2
    # one shard: the output is that shard's o rounded to bf16; LSE untouched
    rng = np.random.default_rng(8)
    o1 = rng.standard_normal((1, 7, 5))
    g1, l1 = oa.merge_bf16_numerator(o1, rng.standard_normal((1, 7)))
    assert (g1 == oa.round_bf16(o1[0])).all()
    # S shards: within S + 1 roundings of the exact merge (each 2^-9 relative to the running magnitude), same LSE
    S = 9
    o = rng.standard_normal((S, 50, 16))
    l = rng.standard_normal((S, 50)) * 3.0
    l[2, ::5] = -np.inf
    got, lse = oa.merge_bf16_numerator(o, l)
    ref, lref = oa.merge(o, l)
    w = np.exp(l - l.max(axis=0))
    bound = (S + 1) * 2.0 ** -9 * (w[..., None] * np.abs(o)).sum(axis=0) / w.sum(axis=0)[..., None]
    assert (np.abs(got - ref) <= bound).all() and np.array_equal(lse, lref)
    assert np.abs(got - ref).max() > 0          # the rounding is really there
