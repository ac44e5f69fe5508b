"""The BASELINE configs at full size, in the launch configuration bench.py times, against the
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


def test_config3_p2m_needles():
    cfg = CONFIGS["p2m"]
    case = parity.Case(cfg)
    plan = W.needle_plan(cfg)
    g = cfg.Hq // cfg.Hkv
    member = 0
    needles = [(t, h) for _, m, t, h in plan if m == member]
    assert needles
    kv = needles[0][1] // g                           # the KV group of this member's first needle
    fw = parity.check_forward(case, member=member, kv_groups=[kv], full=False, per_shard=False,
                              extra_rows=needles, strict_abs=True)
    for pos, m, t, h in plan:
        if m == member and h // g == kv:              # peaked row: O ~ V[needle], LSE ~ 4 |q|^2 / 16
            v_needle = case.v_pool[int(case.table[pos // cfg.page_size]), pos % cfg.page_size, kv].float()
            assert (fw["o_f32"][t, h] - v_needle).abs().max() < 2e-2
            assert fw["lse"][t, h] > 40
    parity.check_backward(case, fw, kv_groups=[kv], full=False, tail=16, extra_rows=needles, strict_abs=True)
    # statistical sanity on every row: LSE ~ ln(P + t + 1) + |q|^2 scale^2 / 2 away from needle keys
    lse = fw["lse"].double().cpu().numpy()
    q = fw["q"].double().cpu().numpy()
    want = np.log(cfg.P + np.arange(cfg.R) + 1.0)[:, None] + 0.5 * (cfg.scale ** 2) * (q ** 2).sum(-1)
    assert np.median(np.abs(lse - want)) < 0.02
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
