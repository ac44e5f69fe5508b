"""The five workloads at full size, in the launch configuration bench.py times, against the
fp64 oracle on a seeded sample of (row, head) pairs (all heads of one KV group at rows
{0,127,128,R/2,R-1} and the last rows, seeded random pairs, every needle-matched row) and, for
dK/dV, on the last response keys, whose contributing rows are all inside the sample."""
import numpy as np
import pytest
import torch

from paper_2607_14952_b200 import binding as B
from paper_2607_14952_b200 import workloads as W
from paper_2607_14952_b200.workloads import CONFIGS

import parity

pytestmark = pytest.mark.gpu


def _free(case):
    case.pages.close()
    del case
    torch.cuda.empty_cache()


def test_config2_p128k_two_members():
    cfg = CONFIGS["p128k"]
    case = parity.Case(cfg)
    for member in range(cfg.G):                      # G = 2 replays against the same resident prefix
        fw = parity.check_forward(case, member=member, kv_groups=[member, 3], full=False, per_shard=False,
                                  strict_abs=True)
        parity.check_backward(case, fw, kv_groups=[member, 3], full=False, tail=16, strict_abs=True)
    _free(case)


def test_config3_p2m_all_members_and_every_needle():
    # G = 8 members replayed one after the other against the one resident prefix.  Every member's
    # needle-matched rows (all 16 over the loop, whatever their KV group) plus seeded rows are checked
    # against the oracle; member 0 also gets the full row sample and the dK / dV tail of one KV group.
    cfg = CONFIGS["p2m"]
    case = parity.Case(cfg)
    plan = W.needle_plan(cfg)
    assert len(plan) == 16 and {m for _, m, _, _ in plan} == set(range(cfg.G))
    g = cfg.Hq // cfg.Hkv
    before = B.ls_prefix_pages_checksum(case.pages)
    S = cfg.num_shards
    o_part = torch.empty((S + 1, cfg.R, cfg.Hq, cfg.Dv), dtype=torch.float32, device="cuda")
    lse_part = torch.empty((S + 1, cfg.R, cfg.Hq), dtype=torch.float32, device="cuda")
    ws = torch.empty(B.ls_replay_attn_workspace_bytes(case.pages, cfg.R, cfg.Hq, cfg.scale, B.LS_WORKSPACE_BWD),
                     dtype=torch.uint8, device="cuda")
    fws = torch.empty(max(16, B.ls_replay_attn_workspace_bytes(case.pages, cfg.R, cfg.Hq, cfg.scale, B.LS_WORKSPACE_FWD)),
                      dtype=torch.uint8, device="cuda")
    rng = np.random.default_rng(77)
    tail = 16
    kv0 = plan[0][3] // g
    samples, got = {}, {}
    for member in range(cfg.G):
        # rows to check, per KV group
        rows = {kv: set() for kv in range(cfg.Hkv)}
        for _, m, t, h in plan:
            if m == member:
                rows[h // g].add((t, h))
        for _ in range(4):
            h = int(rng.integers(cfg.Hq))
            rows[h // g].add((int(rng.integers(cfg.R)), h))
        if member == 0:
            t0, h0 = parity.sampled_rows(cfg, kv0, tail=tail)
            rows[kv0] |= set(zip(t0.tolist(), h0.tolist()))
        q, k, v, d_o = case.member(member)
        B.ls_replay_attn_fwd(case.pages, q, k, v, cfg.scale, o_part=o_part, lse_part=lse_part, status=case.status,
                             workspace=fws)
        o_bf16, o_f32, lse = B.ls_lse_merge(o_part, lse_part, status=case.status)
        _, m_f32, m_lse = B.ls_replay_attn_fwd_merged(case.pages, q, k, v, cfg.scale, status=case.status,
                                                      want_bf16=False)
        dq, dk, dv = B.ls_replay_attn_bwd(case.pages, q, k, v, o_f32, lse, d_o, cfg.scale, workspace=ws,
                                          status=case.status)
        case.check_status()
        assert B.ls_prefix_pages_checksum(case.pages) == before, "prefix modified by member %d" % member
        samples[member] = rows
        for kv in range(cfg.Hkv):
            if rows[kv]:
                pairs = sorted(rows[kv])
                tt, hh = np.array([p[0] for p in pairs]), np.array([p[1] for p in pairs])
                got[(member, kv)] = (tt, hh, parity.f64(lse[tt, hh]), parity.f64(o_f32[tt, hh]), parity.f64(o_bf16[tt, hh]),
                                     parity.f64(m_lse[tt, hh]), parity.f64(m_f32[tt, hh]), parity.f64(dq[tt, hh]),
                                     parity.f64(dk[cfg.R - tail:, kv]), parity.f64(dv[cfg.R - tail:, kv]),
                                     W.bf16_bits(q[tt, hh]), W.bf16_bits(d_o[tt, hh]), W.bf16_bits(k[:, kv:kv + 1]),
                                     W.bf16_bits(v[:, kv:kv + 1]))
        if member == 0:
            # statistical sanity on every row: LSE ~ ln(P + t + 1) + |q|^2 scale^2 / 2 away from needle keys
            want = np.log(cfg.P + np.arange(cfg.R) + 1.0)[:, None] + 0.5 * (cfg.scale ** 2) * (q.double().cpu().numpy() ** 2).sum(-1)
            assert np.median(np.abs(lse.double().cpu().numpy() - want)) < 0.02
        del q, k, v, d_o, dq, dk, dv, o_bf16, o_f32, lse, m_f32, m_lse
    del o_part, lse_part, ws
    torch.cuda.empty_cache()
    # ---- oracle, one KV head on the host at a time
    needle_rows_checked = 0
    for kv in range(cfg.Hkv):
        kp, vp = case.host_pool(kv)
        for member in range(cfg.G):
            if (member, kv) not in got:
                continue
            tt, hh, g_lse, g_o32, g_o16, f_lse, f_o32, g_dq, g_dk, g_dv, qr, dor, kr, vr = got[(member, kv)]
            o_ref, lse_ref, dq_ref, dk_ref, dv_ref = parity.oa.backward_rows(
                qr, tt, 0, kp, vp, case.table, cfg.P, cfg.page_size, kr, vr, float(np.float32(cfg.scale)), dor)
            assert np.abs(g_lse - lse_ref).max() <= parity.LSE_TOL, ("LSE", member, kv)
            assert np.abs(f_lse - lse_ref).max() <= parity.LSE_TOL, ("merged LSE", member, kv)
            assert parity.abs_excess(g_o16, o_ref, True) <= 1.0
            assert parity.rel_gate(g_o32, o_ref, cfg.Dv) <= 1.0 and parity.rel_gate(f_o32, o_ref, cfg.Dv) <= 1.0
            assert parity.abs_excess(g_dq, dq_ref, True) <= 1.0
            extra = np.zeros(len(tt))
            for pos, m, t, h in plan:
                if m == member and h // g == kv:        # peaked row: O ~ V[needle], LSE ~ 4 |q|^2 / 16
                    i = int(np.where((tt == t) & (hh == h))[0][0])
                    page, slot = int(case.table[pos // cfg.page_size]), pos % cfg.page_size
                    k_needle, v_needle = parity.oa.widen(kp[page, slot, 0]), parity.oa.widen(vp[page, slot, 0])
                    assert np.abs(g_o32[i] - v_needle).max() < 2e-2 and g_lse[i] > 40
                    assert np.abs(g_dq[i]).max() < 1e-3                      # ds = p (dp - Delta) cancels
                    # the true dQ of such a row is ~1e-20: what the kernel returns is the rounding of dp - Delta
                    extra[i] = parity.needle_row_model(float(np.float32(cfg.scale)), k_needle, v_needle,
                                                       parity.oa.widen(dor[i]))
                    needle_rows_checked += 1
            assert parity.rel_gate(g_dq, dq_ref, cfg.Dk, extra) <= 1.0, ("dQ", member, kv)
            if member == 0 and kv == kv0:               # the tail window is complete: dK / dV of the last keys
                assert parity.abs_excess(g_dk, dk_ref[cfg.R - tail:], True) <= 1.0
                assert parity.abs_excess(g_dv, dv_ref[cfg.R - tail:], True) <= 1.0
                assert parity.rel_gate(g_dk, dk_ref[cfg.R - tail:], cfg.Dk) <= 1.0
                assert parity.rel_gate(g_dv, dv_ref[cfg.R - tail:], cfg.Dv) <= 1.0
        case._host.clear()
    assert needle_rows_checked == 16
    _free(case)


def test_config4_p4m_cycles_keep_the_prefix_intact():
    cfg = CONFIGS["p4m"]
    case = parity.Case(cfg)
    before = B.ls_prefix_pages_checksum(case.pages)
    S = cfg.num_shards
    o_part = torch.empty((S + 1, cfg.R, cfg.Hq, cfg.Dv), dtype=torch.float32, device="cuda")
    lse_part = torch.empty((S + 1, cfg.R, cfg.Hq), dtype=torch.float32, device="cuda")
    ws = torch.empty(B.ls_replay_attn_workspace_bytes(case.pages, cfg.R, cfg.Hq, cfg.scale, B.LS_WORKSPACE_BWD),
                     dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    first = None
    for cycle in range(cfg.cycles):                   # 8 cycles x G = 8 replays = 64 passes, one prefix
        for member in range(cfg.G):
            q, k, v, d_o = case.member(member, cycle)
            B.ls_replay_attn_fwd(case.pages, q, k, v, cfg.scale, o_part=o_part, lse_part=lse_part, status=status)
            _, o_f32, lse = B.ls_lse_merge(o_part, lse_part, want_bf16=False)
            dq, dk, dv = B.ls_replay_attn_bwd(case.pages, q, k, v, o_f32, lse, d_o, cfg.scale, workspace=ws,
                                              status=status)
            if cycle == 0 and member == 0:
                first = (lse.clone(), dq.clone(), dk.clone(), dv.clone())
        assert B.ls_prefix_pages_checksum(case.pages) == before, "prefix modified in cycle %d" % cycle
    assert int(status.item()) == 0
    # cycle 0 / member 0 is reproducible from its seeds after 64 passes, bit for bit
    q, k, v, d_o = case.member(0, 0)
    B.ls_replay_attn_fwd(case.pages, q, k, v, cfg.scale, o_part=o_part, lse_part=lse_part)
    _, o_f32, lse = B.ls_lse_merge(o_part, lse_part, want_bf16=False)
    again = B.ls_replay_attn_bwd(case.pages, q, k, v, o_f32, lse, d_o, cfg.scale, workspace=ws)
    torch.cuda.synchronize()
    assert torch.equal(lse, first[0])
    for a, b in zip(again, first[1:]):
        assert torch.equal(a, b)
    # and it matches the oracle on a sample of one KV group
    del o_part, lse_part, ws
    orig = parity.sampled_rows
    try:
        parity.sampled_rows = lambda c, kv, tail=8, n_random=8, seed=0, extra=(): orig(c, kv, tail=8, n_random=8,
                                                                                     seed=seed, extra=extra)
        fw = parity.check_forward(case, member=0, kv_groups=[2], full=False, per_shard=False, strict_abs=True)
        parity.check_backward(case, fw, kv_groups=[2], full=False, tail=8, strict_abs=True)
    finally:
        parity.sampled_rows = orig
    _free(case)


def test_config5_mla1m_shared_latent():
    cfg = CONFIGS["mla1m"]
    case = parity.Case(cfg)
    orig = parity.sampled_rows
    try:
        # 64 heads share the one latent KV head: sample rows over a few heads only
        def few(c, kv, tail=8, n_random=24, seed=0, extra=()):
            t, h = orig(c, kv, tail=tail, n_random=n_random, seed=seed, extra=extra)
            keep = (h < 3) | (np.arange(len(h)) % 11 == 0)
            # the tail rows must stay complete for dK/dV: keep every head there
            keep |= t >= c.R - tail
            return t[keep], h[keep]
        parity.sampled_rows = few
        for member in range(cfg.G):
            fw = parity.check_forward(case, member=member, kv_groups=[0], full=False, per_shard=False,
                                      strict_abs=True)
            parity.check_backward(case, fw, kv_groups=[0], full=False, tail=8, strict_abs=True)
    finally:
        parity.sampled_rows = orig
    _free(case)


@pytest.mark.parametrize("R", [16, 64])
def test_short_responses_at_the_2m_prefix(R):
    # the launch configuration of `bench.py --small-r R`: the 2M prefix in 64 shards, Q tiles that pack the
    # rows of several heads (R = 16: one tile per KV group; R = 64: four tiles of 21 tokens x 6 heads)
    cfg = W.scaled(CONFIGS["p2m"], name="p2m-R%d" % R, R=R, num_shards=64, needles=0)
    case = parity.Case(cfg)
    fw = parity.check_forward(case, kv_groups=[2], full=False, per_shard=False, strict_abs=True)
    parity.check_backward(case, fw, kv_groups=[2], full=False, tail=4, strict_abs=True)
    _free(case)


def test_short_response_over_the_1m_shared_latent():
    # `bench.py --workload mla1m --small-r 4`: four row blocks of 64 heads, the parts spread over CTA pairs
    cfg = W.scaled(CONFIGS["mla1m"], name="mla1m-R4", R=4, num_shards=64, needles=0)
    case = parity.Case(cfg)
    orig = parity.sampled_rows
    try:
        def few(c, kv, tail=4, n_random=8, seed=0, extra=()):
            t, h = orig(c, kv, tail=tail, n_random=n_random, seed=seed, extra=extra)
            keep = (h % 9 == 0) | (t >= c.R - 1)          # every head at the last row (dK / dV of the last key)
            return t[keep], h[keep]
        parity.sampled_rows = few
        fw = parity.check_forward(case, kv_groups=[0], full=False, per_shard=False, strict_abs=True)
        parity.check_backward(case, fw, kv_groups=[0], full=False, tail=1, strict_abs=True)
    finally:
        parity.sampled_rows = orig
    _free(case)
