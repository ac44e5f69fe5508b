"""Seeded random small shapes through the whole path against the oracle: forward partials, merge, the
forward with the merge folded in, backward (tests/parity.py gates), the blockwise replay with a paged
suffix against the dense oracle, and the sparse replay (index scores, top-k, attention over the selected
latent rows and its backward) against the sparse oracle.  The draws cover what the hand-picked cases pair up only sparsely: head
dims x page sizes x shard policies x stream budgets (shards walked as sub-ranges) x responses of 1 .. 300
tokens (packed Q tiles, one or several per KV group) x prefixes of 0 .. 4,113 positions (empty shards, ragged
last pages, more shards than pages)."""
import random

import pytest

from paper_2607_14952_b200 import binding as B
from paper_2607_14952_b200.workloads import ReplayConfig

import parity
import test_gpu_blockwise as blockwise

pytestmark = pytest.mark.gpu

POLICIES = [B.LS_SHARD_CONTIGUOUS, B.LS_SHARD_CONTIGUOUS, B.LS_SHARD_CYCLIC, B.LS_SHARD_ZIGZAG]


def draw_dense(seed):
    rng = random.Random(seed)
    shape = rng.choice(["d128", "d256", "d256", "mla"])
    pg = rng.choice([64, 128, 256, 512])
    if shape == "mla":
        pg = rng.choice([64, 256])
        hkv, hq, dk, dv, alias = 1, rng.choice([1, 2, 4, 8, 16, 64]), 576, 512, True
    else:
        hkv = rng.choice([1, 2, 4])
        hq = hkv * rng.choice([1, 2, 3, 4, 6])
        dk = dv = 128 if shape == "d128" else 256
        alias = False
    r = rng.choice([1, 2, 3, 5, 9, 16, 21, 33, 64, 100, 128, 129, 200, 300])
    p = rng.choice([0, 1, 63, 64, 65, 200, 777, 1024, 1500, 2048, 3001, 4096 + 17])
    if shape == "mla" and hq >= 16:
        r = min(r, 64)
    if p <= 1:          # (hundreds of rows over one or two keys make dK / dV sums of magnitude ~30 in bf16)
        hq = min(hq, 16) // hkv * hkv or hkv
    cfg = ReplayConfig(name="rnd%d" % seed, P=p, R=r, Hq=hq, Hkv=hkv, Dk=dk, Dv=dv, page_size=pg,
                       num_shards=rng.choice([1, 2, 3, 5, 8]), G=1, seed=7000 + seed, v_aliases_k=alias)
    return cfg, rng.choice(POLICIES), rng.choice([0, 0, 64, 256]), rng.choice([0, 2]) if p > 0 else 2


def draw_blockwise(seed):
    rng = random.Random(10_000 + seed)
    d = rng.choice([128, 256, 256])
    hkv = rng.choice([1, 2, 4])
    nblocks = rng.choice([2, 3, 4])
    rb = rng.choice([1, 3, 8, 20, 33, 64, 100, 128, 130, 200])
    cfg = ReplayConfig(name="rndb%d" % seed, P=rng.choice([0, 1, 65, 200, 777, 1024, 2048, 3001]), R=nblocks * rb,
                       Hq=hkv * rng.choice([1, 2, 3, 4, 6]), Hkv=hkv, Dk=d, Dv=d, page_size=rng.choice([64, 128, 256, 512]),
                       num_shards=rng.choice([1, 2, 3, 5]), G=1, seed=8000 + seed)
    return cfg, nblocks, rb, rng.choice(POLICIES), rng.choice([0, 0, 64, 256])


@pytest.mark.parametrize("seed", range(128))
def test_random_shape_forward_and_backward(seed):
    cfg, policy, budget_kib, extra_pages = draw_dense(seed)
    case = parity.Case(cfg, policy=policy, extra_phys_pages=extra_pages, stream_budget_kib=budget_kib)
    before = B.ls_prefix_pages_checksum(case.pages)
    fw = parity.check_forward(case, per_shard=(budget_kib == 0))
    parity.check_backward(case, fw, dq_model=cfg.P <= 1)
    assert B.ls_prefix_pages_checksum(case.pages) == before


@pytest.mark.parametrize("seed", range(48))
def test_random_shape_blockwise_replay(seed):
    cfg, nblocks, rb, policy, budget_kib = draw_blockwise(seed)
    pg = cfg.page_size
    case = parity.Case(cfg, policy=policy, extra_phys_pages=nblocks * ((rb + pg - 1) // pg) + 1,
                       stream_budget_kib=budget_kib)
    before = B.ls_prefix_pages_checksum(case.pages)
    q, k, v, d_o = case.member(0)
    got = blockwise.blockwise_replay(case, q, k, v, d_o, nblocks, rb)
    assert B.ls_prefix_pages_checksum(case.pages) == before
    blockwise.check_against_dense_oracle(case, q, k, v, d_o, got, range(cfg.Hkv))


def draw_sparse(seed):
    rng = random.Random(20_000 + seed)
    pg = rng.choice([64, 256])
    p = rng.choice([63, 64, 65, 150, 64 * 9 + 7, 777, 1500, 64 * 40 + 9, 256 * 12 + 77])
    cfg = ReplayConfig(name="rnds%d" % seed, P=p, R=rng.choice([1, 2, 5, 16, 20, 33, 70, 129]),
                       Hq=rng.choice([1, 2, 4, 8, 16, 64]), Hkv=1, Dk=576, Dv=512, page_size=pg,
                       num_shards=rng.choice([1, 2, 4, 5]), G=1, seed=9000 + seed, v_aliases_k=True)
    return cfg, rng.choice([8, 16, 32]), rng.choice([16, 64, 192, 256, 512, 2048])


@pytest.mark.parametrize("seed", range(32))
def test_random_shape_sparse_replay(seed):
    import numpy as np
    import test_gpu_dsa as sparse
    cfg, index_heads, top_k = draw_sparse(seed)
    dc = sparse.DsaCase(cfg, index_heads, top_k)
    before = B.ls_prefix_pages_checksum(dc.case.pages)
    got = sparse.run_sparse(dc)
    t_rows = np.repeat(np.arange(cfg.R), cfg.Hq)
    heads = np.tile(np.arange(cfg.Hq), cfg.R)
    sparse.check_sparse(dc, got, t_rows, heads, check_kv=True)
    assert B.ls_prefix_pages_checksum(dc.case.pages) == before


def draw_mid_size(seed):
    rng = random.Random(30_000 + seed)
    shape = rng.choice(["d128", "d256", "d256", "mla"])
    if shape == "mla":
        pg, hkv, hq, dk, dv, alias = rng.choice([64, 256]), 1, rng.choice([8, 16, 64]), 576, 512, True
        r = rng.choice([1, 4, 16, 70, 200, 512])
    else:
        pg = rng.choice([64, 128, 256, 512])
        hkv = rng.choice([1, 2, 4])
        hq = hkv * rng.choice([1, 4, 6])
        dk = dv = 128 if shape == "d128" else 256
        alias = False
        r = rng.choice([1, 7, 16, 64, 100, 300, 777, 1024])
    cfg = ReplayConfig(name="rndm%d" % seed, P=rng.randrange(20000, 400000), R=r, Hq=hq, Hkv=hkv, Dk=dk, Dv=dv,
                       page_size=pg, num_shards=rng.choice([1, 3, 8, 16, 33]), G=1, seed=9500 + seed, v_aliases_k=alias)
    return cfg, rng.choice(POLICIES), rng.choice([0, 1024, 4096, 16384]), rng.randrange(hkv)


@pytest.mark.parametrize("seed", range(12))
def test_random_mid_size_shape_sampled_rows(seed):
    # prefixes of 20,000 .. 400,000 positions: launches of hundreds of CTAs that hand their sums over to one
    # another; sampled rows of one KV group against the oracle
    cfg, policy, budget_kib, kv = draw_mid_size(seed)
    case = parity.Case(cfg, policy=policy, extra_phys_pages=3, stream_budget_kib=budget_kib)
    fw = parity.check_forward(case, kv_groups=[kv], full=False, per_shard=(budget_kib == 0))
    parity.check_backward(case, fw, kv_groups=[kv], full=False, tail=8)
