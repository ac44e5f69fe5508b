"""Sparse (DSA) replay over the shared latent on the GPU against the fp64 oracle: index scores
(Eq. dsa-index), global top-k with the position tie rule (Eq. glm-global-dsa; bit-exact on the
scores the GPU produced), and attention / backward over the selected rows plus the causal
response block (Eq. dsa-attention)."""
import numpy as np
import pytest
import torch

from oracle import attention as oa
from oracle import dsa
from paper_2607_14952_b200 import binding as B
from paper_2607_14952_b200 import workloads as W
from paper_2607_14952_b200.workloads import ReplayConfig

import parity

pytestmark = pytest.mark.gpu


def latent(name, **kw):
    base = dict(name=name, P=64 * 40 + 9, R=70, Hq=8, Hkv=1, Dk=576, Dv=512, page_size=64, num_shards=4, G=1,
                v_aliases_k=True, seed=601)
    base.update(kw)
    return ReplayConfig(**base)


class DsaCase:
    def __init__(self, cfg, hi, top_k, extra_phys_pages=2):
        self.case = parity.Case(cfg, extra_phys_pages=extra_phys_pages)
        self.cfg, self.hi, self.top_k = cfg, hi, top_k
        nphys = self.case.k_pool.shape[0]
        self.ki_pool, self.q_index, self.w_index = W.make_index_inputs(cfg, hi, 0, "cuda", num_phys_pages=nphys)
        self.plan = B.ls_dsa_plan_create(self.case.pages, self.ki_pool, cfg.R, cfg.Hq, hi, top_k)
        q, k, _, d_o = self.case.member(0)
        self.q, self.k_resp, self.d_o = q, k, d_o
        self.v_resp = k[..., :cfg.Dv].contiguous()       # the latent row of a response token is key and value at once

    def scores(self):
        s = B.ls_dsa_index_scores(self.plan, self.q_index, self.w_index, status=self.case.status)
        self.case.check_status()
        return s

    def oracle_scores(self, rows):
        c = self.cfg
        ki = W.bf16_bits(self.ki_pool).reshape(self.ki_pool.shape[0], c.page_size, 1, -1)
        I = dsa.index_scores(W.bf16_bits(self.q_index[rows]), self.w_index[rows].double().cpu().numpy(), rows, ki,
                             self.case.table, c.P, c.page_size, np.zeros((c.R, ki.shape[-1])))
        return I[:, :c.P]


@pytest.mark.parametrize("cfg,hi", [
    (latent("idx_pg64"), 32),
    (latent("idx_pg256_ragged", P=256 * 9 + 100, page_size=256, R=37), 32),
    (latent("idx_h8", P=64 * 13 + 1, R=200), 8),
    (latent("idx_h16_short", P=100, R=9), 16),
    (latent("idx_h64_pg512", P=512 * 3 + 5, page_size=512, R=64), 64),
], ids=lambda x: x.name if isinstance(x, ReplayConfig) else str(x))
def test_index_scores_match_the_oracle(cfg, hi):
    dc = DsaCase(cfg, hi, 64)
    got = dc.scores().double().cpu().numpy()
    rows = np.arange(cfg.R)
    want = dc.oracle_scores(rows)
    assert np.isfinite(got).all()
    # bf16 products are exact in fp32; what differs is fp32 accumulation of 128 + H_I terms
    assert np.abs(got - want).max() <= 1e-4 * (1.0 + np.abs(want).max())


def test_topk_is_bit_exact_including_ties():
    cfg = latent("topk", P=64 * 50 + 3, R=40)
    dc = DsaCase(cfg, 32, 128)
    s = dc.scores()
    # make ties common in some rows: rounded scores, an all-equal row, a row with +-inf-free negatives only
    s[1] = torch.round(s[1] / 8.0) * 8.0
    s[2] = 1.5
    s[3] = -torch.abs(s[3]) - 1.0
    s[4] = torch.round(s[4])
    sel = B.ls_dsa_topk(dc.plan, s).cpu().numpy()
    torch.cuda.synchronize()
    host = s.double().cpu().numpy()
    for t in range(cfg.R):
        want = dsa.topk_select(host[t], 128)
        assert np.array_equal(sel[t], want), t
    # fewer prefix positions than top_k: every position is selected
    small = DsaCase(latent("topk_all", P=100, R=5), 16, 2048)
    sel = B.ls_dsa_topk(small.plan, small.scores()).cpu().numpy()
    assert sel.shape == (5, 100) and (sel == np.arange(100)[None, :]).all()


@pytest.mark.parametrize("P", [64 * 9400, 64 * 9400 + 37])          # rows of 16-byte aligned and unaligned length
def test_topk_over_a_long_row(P):
    # long rows take the selection's shortcut (a lower bound on the threshold from the row's first 64K
    # positions); rows are built so that the bound is tight, loose, or sits in a crowd of equal scores
    cfg = latent("topk_long", P=P, R=7, Hq=2, num_shards=2)
    dc = DsaCase(cfg, 8, 2048)
    g = torch.Generator(device="cuda").manual_seed(77)
    s = torch.randn(cfg.R, P, device="cuda", generator=g)
    s[1] = torch.round(s[1] * 2.0) / 2.0                                  # few distinct values: ties everywhere
    s[2] = 0.25                                                           # all equal: the first 2048 positions
    s[3, :65536] -= 100.0                                                 # head far below the rest: loose bound
    s[4, :65536] += 100.0                                                 # every selected score sits in the head
    s[5] = torch.where(torch.rand(P, device="cuda", generator=g) < 0.5, s[5], -s[5].abs() * 1e-30)
    s[6, 70000:70000 + 3000] = float("inf")                               # more infinities than top_k
    sel = B.ls_dsa_topk(dc.plan, s).cpu().numpy()
    torch.cuda.synchronize()
    host = s.double().cpu().numpy()
    for t in range(cfg.R):
        assert np.array_equal(sel[t], dsa.topk_select(host[t], 2048)), t


def run_sparse(dc):
    cfg = dc.cfg
    sel = B.ls_dsa_topk(dc.plan, dc.scores())
    o_bf16, o_f32, lse = B.ls_dsa_attn_fwd(dc.plan, sel, dc.q, dc.k_resp, dc.v_resp, cfg.scale, status=dc.case.status)
    dq, dk, dv = B.ls_dsa_attn_bwd(dc.plan, dc.q, dc.k_resp, dc.v_resp, o_f32, lse, dc.d_o, cfg.scale,
                                   status=dc.case.status)
    dc.case.check_status()
    return sel.cpu().numpy(), o_bf16, o_f32, lse, dq, dk, dv


def check_sparse(dc, got, t_rows, heads, check_kv):
    """Rows (t, h) against the oracle with the GPU's selection; dK / dV when the row set is complete."""
    cfg = dc.cfg
    sel, o_bf16, o_f32, lse, dq, dk, dv = got
    kp, _ = dc.case.host_pool(0)
    kr = W.bf16_bits(dc.k_resp)
    sels = [np.concatenate([sel[t], cfg.P + np.arange(t + 1)]) for t in t_rows]
    scale = float(np.float32(cfg.scale))
    o_ref, lse_ref, dq_ref, dk_ref, dv_ref = dsa.sparse_backward_rows(
        W.bf16_bits(dc.q[t_rows, heads]), sels, kp, dc.case.table, cfg.P, cfg.page_size, kr, cfg.Dv, scale,
        W.bf16_bits(dc.d_o[t_rows, heads]))
    assert np.abs(parity.f64(lse[t_rows, heads]) - lse_ref).max() <= parity.LSE_TOL
    assert parity.abs_excess(parity.f64(o_bf16[t_rows, heads]), o_ref, False) <= 1.0
    assert parity.rel_gate(parity.f64(o_f32[t_rows, heads]), o_ref, cfg.Dv) <= 1.0
    g_dq = parity.f64(dq[t_rows, heads])
    assert parity.abs_excess(g_dq, dq_ref, False) <= 1.0
    assert parity.rel_gate(g_dq, dq_ref, cfg.Dk) <= 1.0
    if check_kv:
        g_dk, g_dv = parity.f64(dk[:, 0]), parity.f64(dv[:, 0])
        assert parity.abs_excess(g_dk, dk_ref, False) <= 1.0 and parity.abs_excess(g_dv, dv_ref, False) <= 1.0
        assert parity.rel_gate(g_dk, dk_ref, cfg.Dk) <= 1.0 and parity.rel_gate(g_dv, dv_ref, cfg.Dv) <= 1.0


@pytest.mark.parametrize("cfg,hi,top_k", [
    (latent("sparse_pg64", P=64 * 40 + 9, R=70, Hq=8), 32, 256),
    (latent("sparse_pg256", P=256 * 12 + 77, page_size=256, R=33, Hq=4), 16, 192),
    (latent("sparse_all", P=150, R=20, Hq=4), 8, 2048),              # top_k >= P: the dense operator
    (latent("sparse_64heads", P=64 * 64, R=16, Hq=64), 32, 512),
], ids=lambda x: x.name if isinstance(x, ReplayConfig) else str(x))
def test_sparse_replay_forward_and_backward(cfg, hi, top_k):
    dc = DsaCase(cfg, hi, top_k)
    before = B.ls_prefix_pages_checksum(dc.case.pages)
    got = run_sparse(dc)
    t_rows = np.repeat(np.arange(cfg.R), cfg.Hq)
    heads = np.tile(np.arange(cfg.Hq), cfg.R)
    check_sparse(dc, got, t_rows, heads, check_kv=True)
    assert B.ls_prefix_pages_checksum(dc.case.pages) == before
    if top_k >= cfg.P:      # every prefix position selected: the dense replay of the same inputs agrees
        fw = dc.case.forward(dc.q, dc.k_resp, dc.v_resp)
        assert (got[3] - fw[4]).abs().max() < 1e-4
        # (different key tilings round the bf16 probabilities differently: 2^-9 relative per term)
        assert (got[2] - fw[3]).abs().max() < 5e-3
    # bit-reproducible
    again = run_sparse(dc)
    assert np.array_equal(got[0], again[0])
    for a, b in zip(got[1:], again[1:]):
        assert torch.equal(a, b)


def test_sparse_replay_at_a_64k_prefix():
    # the paper's indexer shape (32 heads of 128, top-2,048) over 65,536 latent positions, 64 heads
    cfg = latent("sparse_64k", P=65536, R=96, Hq=64, num_shards=8, seed=611)
    dc = DsaCase(cfg, 32, 2048, extra_phys_pages=0)
    got = run_sparse(dc)
    sel = got[0]
    assert sel.shape == (cfg.R, 2048) and (np.diff(sel, axis=1) > 0).all() and sel.max() < cfg.P
    # scores and selection of a few rows against the oracle's fp64 scores: the sets may differ only where
    # fp32 and fp64 scores order near-ties differently, so compare through the threshold
    rows = np.array([0, 17, cfg.R - 1])
    want = dc.oracle_scores(rows)
    gpu = dc.scores().double().cpu().numpy()[rows]
    assert np.abs(gpu - want).max() <= 1e-4 * (1.0 + np.abs(want).max())
    for i, t in enumerate(rows):
        assert np.array_equal(sel[t], dsa.topk_select(gpu[i], 2048))
        kth = np.sort(want[i])[-2048]
        assert (want[i][sel[t]] >= kth - 1e-3).all()
    # attention and gradients on sampled rows, every head
    t_s = np.array([0, 1, 50, cfg.R - 1])
    t_rows = np.repeat(t_s, cfg.Hq)
    heads = np.tile(np.arange(cfg.Hq), len(t_s))
    check_sparse(dc, got, t_rows, heads, check_kv=False)


def test_sparse_replay_at_the_1m_workload():
    # the launch configuration of `bench.py --mode dsa`: 1,048,576 latent positions, 1,024 response tokens,
    # 64 heads, 32 index heads of 128, top-2,048
    cfg = W.CONFIGS["mla1m"]
    dc = DsaCase(cfg, 32, 2048, extra_phys_pages=0)
    got = run_sparse(dc)
    sel = got[0]
    assert sel.shape == (cfg.R, 2048) and (np.diff(sel, axis=1) > 0).all() and sel.max() < cfg.P
    rows = np.array([0, 511, cfg.R - 1])
    want = dc.oracle_scores(rows)
    gpu = dc.scores()[torch.as_tensor(rows, device="cuda")].double().cpu().numpy()
    assert np.abs(gpu - want).max() <= 1e-4 * (1.0 + np.abs(want).max())
    for i, t in enumerate(rows):
        assert np.array_equal(sel[t], dsa.topk_select(gpu[i], 2048))         # bit-exact on the GPU's scores
        kth = np.sort(want[i])[-2048]
        assert (want[i][sel[t]] >= kth - 1e-3).all()                         # and the right set up to fp32 near-ties
    t_s = np.array([0, 1, 700, cfg.R - 1])
    heads_s = np.array([0, 5, 31, 63])
    t_rows = np.repeat(t_s, len(heads_s))
    heads = np.tile(heads_s, len(t_s))
    check_sparse(dc, got, t_rows, heads, check_kv=False)
