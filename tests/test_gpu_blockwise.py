"""Blockwise response replay with a paged suffix (Sec. "Four-Block Response Replay", Sec. "Lazy
Gradient Pages") against the dense oracle.

The response is cut into B blocks.  A no-grad suffix pass scores each block (forward with the
merge folded in) and appends its K/V as temporary pages; the policy pass walks the blocks in
reverse: pop the block, replay it against prefix + earlier blocks + its own causal part, run
the backward -- which adds the block's contribution to the fp32 gradient pages of the earlier
blocks and returns dQ plus the block's own dK/dV with what later blocks left for it.  The
oracle's arithmetic does not change: the dense replay at R = B * Rb is the expected result
(O / LSE / dQ of block b are its rows, dK / dV after the sweep are the dense ones).
"""
import numpy as np
import pytest
import torch

from paper_2607_14952_b200 import binding as B
from paper_2607_14952_b200 import workloads as W
from paper_2607_14952_b200.workloads import CONFIGS, ReplayConfig

import parity

pytestmark = pytest.mark.gpu


def blockwise_replay(case, q, k, v, d_o, nblocks, rb):
    """Runs the suffix pass and the reverse policy pass; returns dense-shaped O, LSE, dQ, dK, dV."""
    cfg = case.cfg
    pg = cfg.page_size
    pages_per_block = (rb + pg - 1) // pg
    mapped = set(int(x) for x in case.table)
    free = [p for p in range(case.k_pool.shape[0]) if p not in mapped]
    assert len(free) >= nblocks * pages_per_block
    dk_grad = torch.full((nblocks * pages_per_block, pg, cfg.Hkv, cfg.Dk), float("nan"), device="cuda")
    dv_grad = torch.full((nblocks * pages_per_block, pg, cfg.Hkv, cfg.Dv), float("nan"), device="cuda")
    B.ls_suffix_pages_reserve(case.pages, nblocks, nblocks * pages_per_block, dk_grad, dv_grad)
    blk = lambda x, b: x[b * rb:(b + 1) * rb].contiguous()
    o_sfx = torch.empty((cfg.R, cfg.Hq, cfg.Dv), dtype=torch.float32, device="cuda")
    lse_sfx = torch.empty((cfg.R, cfg.Hq), dtype=torch.float32, device="cuda")
    # ---- no-grad suffix pass: score block b, then append its pages
    for b in range(nblocks):
        gen = B.ls_pages_generation(case.pages)
        _, o_b, l_b = B.ls_replay_attn_fwd_merged(case.pages, blk(q, b), blk(k, b), blk(v, b), cfg.scale,
                                                  status=case.status, generation=gen)
        o_sfx[b * rb:(b + 1) * rb], lse_sfx[b * rb:(b + 1) * rb] = o_b, l_b
        ids = free[b * pages_per_block:(b + 1) * pages_per_block]
        B.ls_suffix_pages_append(case.pages, ids, blk(k, b), None if cfg.v_aliases_k else blk(v, b))
        assert B.ls_pages_generation(case.pages) == gen + 1
    assert B.ls_suffix_pages_tokens(case.pages) == nblocks * rb
    case.check_status()
    # ---- policy pass, blocks in reverse
    o = torch.empty_like(o_sfx)
    lse = torch.empty_like(lse_sfx)
    dq = torch.empty_like(q)
    dk = torch.empty_like(k)
    dv = torch.empty_like(v)
    for b in reversed(range(nblocks)):
        stale = B.ls_pages_generation(case.pages)
        B.ls_suffix_pages_pop(case.pages)
        gen = B.ls_pages_generation(case.pages)
        with pytest.raises(B.LsError) as e:          # a call planned before the pop is refused on the host
            B.ls_replay_attn_fwd_merged(case.pages, blk(q, b), blk(k, b), blk(v, b), cfg.scale, generation=stale)
        assert e.value.status == B.LS_ERR_STALE
        _, o_b, l_b = B.ls_replay_attn_fwd_merged(case.pages, blk(q, b), blk(k, b), blk(v, b), cfg.scale,
                                                  status=case.status, generation=gen)
        dq_b, dk_b, dv_b = B.ls_replay_attn_bwd(case.pages, blk(q, b), blk(k, b), blk(v, b), o_b, l_b, blk(d_o, b),
                                                cfg.scale, status=case.status, flags=B.LS_FLAG_ADD_SUFFIX_GRAD,
                                                generation=gen)
        o[b * rb:(b + 1) * rb], lse[b * rb:(b + 1) * rb] = o_b, l_b
        dq[b * rb:(b + 1) * rb], dk[b * rb:(b + 1) * rb], dv[b * rb:(b + 1) * rb] = dq_b, dk_b, dv_b
    case.check_status()
    assert B.ls_suffix_pages_tokens(case.pages) == 0
    # the policy pass recomputes what the suffix pass scored: same kernels, same order, same bits
    assert torch.equal(o, o_sfx) and torch.equal(lse, lse_sfx)
    return o, lse, dq, dk, dv


def check_against_dense_oracle(case, q, k, v, d_o, got, kv_groups, rows=None, key_lo=0):
    """got = (O, LSE, dQ, dK, dV) in the dense layout.  rows: (t, h) pairs per KV group or None = all."""
    cfg = case.cfg
    o, lse, dq, dk, dv = got
    for kv in kv_groups:
        t_rows, heads = parity.all_rows_of_group(cfg, kv) if rows is None else rows(kv)
        o_ref, lse_ref, dq_ref, dk_ref, dv_ref = case.oracle_rows(kv, t_rows, heads, q, k, v, d_o)
        assert np.abs(parity.f64(lse[t_rows, heads]) - lse_ref).max() <= parity.LSE_TOL
        assert parity.rel_gate(parity.f64(o[t_rows, heads]), o_ref, cfg.Dv) <= 1.0
        g_dq = parity.f64(dq[t_rows, heads])
        assert parity.abs_excess(g_dq, dq_ref, False) <= 1.0
        # (a response behind an empty prefix: its first rows see one or two keys, see parity.dq_rounding_model)
        extra = parity.dq_rounding_model(case, kv, t_rows, heads, q, k, v, d_o) if cfg.P <= 1 else None
        assert parity.rel_gate(g_dq, dq_ref, cfg.Dk, extra) <= 1.0
        g_dk, g_dv = parity.f64(dk[key_lo:, kv]), parity.f64(dv[key_lo:, kv])
        assert parity.abs_excess(g_dk, dk_ref[key_lo:], False) <= 1.0
        assert parity.abs_excess(g_dv, dv_ref[key_lo:], False) <= 1.0
        assert parity.rel_gate(g_dk, dk_ref[key_lo:], cfg.Dk) <= 1.0, "dK"
        assert parity.rel_gate(g_dv, dv_ref[key_lo:], cfg.Dv) <= 1.0, "dV"


@pytest.mark.parametrize("cfg,nblocks", [
    (ReplayConfig(name="b4x512", P=2048 + 77, R=2048, Hq=4, Hkv=2, Dk=256, Dv=256, page_size=256, num_shards=3, G=1,
                  seed=311), 4),
    (ReplayConfig(name="b3x300_ragged_pages", P=64 * 11 + 5, R=900, Hq=6, Hkv=2, Dk=256, Dv=256, page_size=64,
                  num_shards=2, G=1, seed=312), 3),
    (ReplayConfig(name="b2x200_d128", P=128 * 5, R=400, Hq=4, Hkv=1, Dk=128, Dv=128, page_size=128, num_shards=2, G=1,
                  seed=313), 2),
    (ReplayConfig(name="b4x130_p0", P=0, R=520, Hq=2, Hkv=1, Dk=256, Dv=256, page_size=512, num_shards=1, G=1,
                  seed=314), 4),
    # blocks shorter than a Q tile: the rows of a KV group share one tile, and the dQ pass walks the response
    # block, the prefix parts and the earlier blocks' suffix pages as ranges of one list of key tiles
    (ReplayConfig(name="b3x20_short_blocks", P=64 * 37 + 9, R=60, Hq=8, Hkv=2, Dk=256, Dv=256, page_size=64,
                  num_shards=3, G=1, seed=315), 3),
    (ReplayConfig(name="b2x9_short_blocks_d128", P=128 * 21 + 50, R=18, Hq=12, Hkv=2, Dk=128, Dv=128, page_size=128,
                  num_shards=4, G=1, seed=316), 2),
], ids=lambda x: x.name if isinstance(x, ReplayConfig) else str(x))
def test_blockwise_replay_equals_the_dense_replay(cfg, nblocks):
    rb = cfg.R // nblocks
    pg = cfg.page_size
    case = parity.Case(cfg, extra_phys_pages=nblocks * ((rb + pg - 1) // pg) + 1)
    before = B.ls_prefix_pages_checksum(case.pages)
    q, k, v, d_o = case.member(0)
    got = blockwise_replay(case, q, k, v, d_o, nblocks, rb)
    assert B.ls_prefix_pages_checksum(case.pages) == before          # the prefix is never written
    check_against_dense_oracle(case, q, k, v, d_o, got, range(cfg.Hkv))
    # the one-block replay of the same response through the dense entry points agrees
    _, _, _, o_f32, lse = case.forward(q, k, v)
    dq1, dk1, dv1 = case.backward(q, k, v, o_f32, lse, d_o)
    assert (got[1] - lse).abs().max() < 1e-4
    assert (got[2].float() - dq1.float()).abs().max() < 2e-2
    assert (got[3].float() - dk1.float()).abs().max() <= 2e-2 + 2.0 ** -7 * dk1.float().abs().max()
    assert (got[4].float() - dv1.float()).abs().max() <= 2e-2 + 2.0 ** -7 * dv1.float().abs().max()


def test_blockwise_replay_at_the_128k_prefix():
    # 4 x 2,048 response tokens behind the 131,072-position prefix (the paper's block shape):
    # sampled rows for O / LSE / dQ, and dK / dV on the last keys of the LAST block and of block 2 --
    # the latter collect gradient from the later block through the gradient pages
    base = CONFIGS["p128k"]
    nblocks, rb = 4, 2048
    cfg = W.scaled(base, name="p128k-4x2048", R=nblocks * rb)
    case = parity.Case(cfg, extra_phys_pages=nblocks * (rb // cfg.page_size))
    before = B.ls_prefix_pages_checksum(case.pages)
    q, k, v, d_o = case.member(0)
    got = blockwise_replay(case, q, k, v, d_o, nblocks, rb)
    assert B.ls_prefix_pages_checksum(case.pages) == before
    kv = 1
    g = cfg.Hq // cfg.Hkv
    heads = list(range(kv * g, (kv + 1) * g))
    tail = 8

    def rows(_kv):
        ts = sorted({0, rb - 1, rb, 2 * rb + 5, 3 * rb - 1} | set(range(cfg.R - tail, cfg.R)))
        pairs = sorted({(t, h) for t in ts for h in heads})
        return np.array([p[0] for p in pairs]), np.array([p[1] for p in pairs])

    check_against_dense_oracle(case, q, k, v, d_o, got, [kv], rows=rows, key_lo=cfg.R - tail)
    # keys at the end of block 2: their gradient is the block's own causal part plus what block 3 left
    # in the gradient pages; every row t >= j of the group contributes, so the oracle runs on all of them
    # (about 12k rows over 139k keys, in slabs to bound host memory)
    tail2 = 4
    j0, j1 = 3 * rb - tail2, 3 * rb
    t_all = np.repeat(np.arange(j0, cfg.R), g)
    h_all = np.tile(np.array(heads), cfg.R - j0)
    step = 768
    dk_ref = np.zeros((cfg.R, cfg.Dk))
    dv_ref = np.zeros((cfg.R, cfg.Dv))
    for lo in range(0, len(t_all), step):
        _, _, _, dk_p, dv_p = case.oracle_rows(kv, t_all[lo:lo + step], h_all[lo:lo + step], q, k, v, d_o)
        dk_ref += dk_p
        dv_ref += dv_p
    g_dk, g_dv = parity.f64(got[3][j0:j1, kv]), parity.f64(got[4][j0:j1, kv])
    assert parity.abs_excess(g_dk, dk_ref[j0:j1], True) <= 1.0
    assert parity.abs_excess(g_dv, dv_ref[j0:j1], True) <= 1.0
    assert parity.rel_gate(g_dk, dk_ref[j0:j1], cfg.Dk) <= 1.0
    assert parity.rel_gate(g_dv, dv_ref[j0:j1], cfg.Dv) <= 1.0


def test_suffix_page_checks():
    cfg = ReplayConfig(name="sfx", P=256 * 3, R=256, Hq=2, Hkv=1, Dk=256, Dv=256, page_size=256, num_shards=2, G=1, seed=9)
    case = parity.Case(cfg, extra_phys_pages=3)
    q, k, v, _ = case.member(0)
    mapped = [int(x) for x in case.table]
    free = [p for p in range(case.k_pool.shape[0]) if p not in mapped]
    st = lambda fn: parity_status(fn)
    assert st(lambda: B.ls_suffix_pages_append(case.pages, free[:1], k, v)) == B.LS_ERR_INVALID_ARG   # nothing reserved
    B.ls_suffix_pages_reserve(case.pages, 2, 2)                                                        # forward only
    assert st(lambda: B.ls_suffix_pages_append(case.pages, mapped[:1], k, v)) == B.LS_ERR_BAD_PAGE_TABLE   # a prefix page
    assert st(lambda: B.ls_suffix_pages_append(case.pages, [case.k_pool.shape[0]], k, v)) == B.LS_ERR_BAD_PAGE_TABLE
    B.ls_suffix_pages_append(case.pages, free[:1], k, v)
    assert st(lambda: B.ls_suffix_pages_append(case.pages, free[:1], k, v)) == B.LS_ERR_BAD_PAGE_TABLE     # already in the suffix
    # the per-shard forward describes the prefix only
    assert st(lambda: B.ls_replay_attn_fwd(case.pages, q, k, v, cfg.scale)) == B.LS_ERR_INVALID_ARG
    # a backward over suffix blocks needs gradient pages
    o = torch.zeros((cfg.R, cfg.Hq, cfg.Dv), device="cuda")
    l = torch.zeros((cfg.R, cfg.Hq), device="cuda")
    assert st(lambda: B.ls_replay_attn_bwd(case.pages, q, k, v, o, l, q, cfg.scale)) == B.LS_ERR_INVALID_ARG
    B.ls_suffix_pages_append(case.pages, free[1:2], k, v)
    assert st(lambda: B.ls_suffix_pages_append(case.pages, free[2:3], k, v)) == B.LS_ERR_INVALID_ARG      # capacity
    B.ls_suffix_pages_pop(case.pages)
    B.ls_suffix_pages_pop(case.pages)
    assert st(lambda: B.ls_suffix_pages_pop(case.pages)) == B.LS_ERR_INVALID_ARG
    torch.cuda.synchronize()


def parity_status(fn):
    with pytest.raises(B.LsError) as e:
        fn()
    return e.value.status
