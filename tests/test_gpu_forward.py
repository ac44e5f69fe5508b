"""Replay forward + merge on the GPU against the fp64 oracle, element by element."""
import numpy as np
import pytest
import torch

from paper_2607_14952_b200 import binding as B
from paper_2607_14952_b200 import workloads as W
from paper_2607_14952_b200.workloads import CONFIGS, ReplayConfig

import parity

pytestmark = pytest.mark.gpu


def small(name, **kw):
    base = dict(name=name, P=2048, R=256, Hq=4, Hkv=2, Dk=256, Dv=256, page_size=256, num_shards=3, G=1, seed=77)
    base.update(kw)
    return ReplayConfig(**base)


def test_config1_tiny_full():
    case = parity.Case(CONFIGS["tiny"])
    parity.check_forward(case, strict_abs=True)


@pytest.mark.parametrize("cfg", [
    small("d256_basic"),
    small("d256_ragged", P=1000, R=200, num_shards=2),                 # partial last page, R not a tile multiple
    small("d256_pg64", P=64 * 13 + 7, page_size=64, num_shards=4, R=130),     # odd page count per shard, ragged tail
    small("d256_pg512", P=4096 + 300, page_size=512, num_shards=2),
    small("d128_pg128", Dk=128, Dv=128, P=128 * 9, page_size=128, num_shards=4, Hq=6, Hkv=2, R=384),
    small("d128_small_p", Dk=128, Dv=128, P=50, page_size=64, num_shards=2, R=64),   # prefix below one tile
    small("d256_empty_shards", P=512, page_size=256, num_shards=5),      # S > Np leaves empty partials
    small("d256_p0", P=0, num_shards=2, R=300),                          # pure causal response block
    # shared-latent shape: 576-wide key page whose first 512 channels are the value
    small("mla_pg64", Dk=576, Dv=512, v_aliases_k=True, Hq=8, Hkv=1, P=64 * 20 + 5, page_size=64, num_shards=3, R=130),
    small("mla_pg256", Dk=576, Dv=512, v_aliases_k=True, Hq=4, Hkv=1, P=2048, page_size=256, num_shards=2, R=256),
    # short responses: every (head, token) row of a KV group shares one Q tile
    small("short_r5", P=3000, page_size=128, num_shards=5, R=5, Hq=6, Hkv=2),
    small("short_r16", P=4096, page_size=256, num_shards=4, R=16, Hq=24, Hkv=4),
    small("short_r1", P=1500, page_size=64, num_shards=3, R=1, Hq=8, Hkv=2, Dk=128, Dv=128),
    small("short_r32_full_tile", P=2048, page_size=256, num_shards=2, R=32, Hq=8, Hkv=2),
    # responses shorter than a Q tile whose KV group needs several tiles of (tokens x heads) rows
    small("short_r40_two_tiles", P=2048 + 77, page_size=256, num_shards=3, R=40, Hq=8, Hkv=2),
    small("short_r100_d128", Dk=128, Dv=128, P=64 * 21 + 3, page_size=64, num_shards=4, R=100, Hq=16, Hkv=2),
    small("mla_short_r5_64heads", Dk=576, Dv=512, v_aliases_k=True, Hq=64, Hkv=1, P=64 * 23 + 11, page_size=64,
          num_shards=4, R=5),
], ids=lambda c: c.name)
def test_forward_small_cases(cfg):
    case = parity.Case(cfg, extra_phys_pages=2)
    parity.check_forward(case)


@pytest.mark.parametrize("policy", [B.LS_SHARD_CYCLIC, B.LS_SHARD_ZIGZAG])
def test_forward_shard_policies(policy):
    cfg = small("policy", P=64 * 21 + 9, page_size=64, num_shards=4, Dk=128, Dv=128, R=128)
    case = parity.Case(cfg, policy=policy)
    parity.check_forward(case)


def test_forward_is_deterministic_and_page_permutation_invariant():
    cfg = small("det", P=3000, page_size=128, num_shards=4)
    case = parity.Case(cfg, extra_phys_pages=3)
    q, k, v, _ = case.member(0)
    a = case.forward(q, k, v)
    b = case.forward(q, k, v)
    torch.cuda.synchronize()
    for x, y in zip(a, b):
        assert torch.equal(x, y)
    # move every page to a new physical slot: same logical content, bit-identical result
    nphys = case.k_pool.shape[0]
    perm = torch.randperm(nphys, generator=torch.Generator().manual_seed(5))
    k2 = torch.empty_like(case.k_pool); v2 = torch.empty_like(case.v_pool)
    k2[perm.cuda()] = case.k_pool; v2[perm.cuda()] = case.v_pool
    table2 = perm.numpy()[case.table].astype(np.int32)
    pages2 = B.ls_prefix_pages_build(cfg.P, cfg.page_size, cfg.num_shards, cfg.Hkv, cfg.Dk, cfg.Dv, nphys,
                                     page_table=table2, k_pool=k2, v_pool=v2)
    o_part, lse_part = B.ls_replay_attn_fwd(pages2, q, k, v, cfg.scale)
    torch.cuda.synchronize()
    assert torch.equal(o_part, a[0]) and torch.equal(lse_part, a[1])


def test_merged_forward_is_bit_reproducible_and_close_to_the_two_step_path():
    # the forward with the merge folded in hands its partial results over between CTAs in a fixed
    # order: two runs agree bit for bit (also with sub-ranges forced by a small stream budget), and the
    # result agrees with forward + ls_lse_merge up to fp32 rounding of a different summation order
    for budget in (0, 256):
        cfg = small("merged_det", P=256 * 19 + 77, page_size=256, num_shards=3, R=300, Hq=6, Hkv=2)
        case = parity.Case(cfg, stream_budget_kib=budget)
        q, k, v, _ = case.member(0)
        a = case.forward_merged(q, k, v)
        b = case.forward_merged(q, k, v)
        for x, y in zip(a, b):
            assert torch.equal(x, y)
        _, _, o_bf16, o_f32, lse = case.forward(q, k, v)
        assert (a[2] - lse).abs().max() < 1e-5
        assert (a[1] - o_f32).abs().max() < 1e-5
        assert (a[0].float() - o_bf16.float()).abs().max() <= 2.0 ** -8 * o_bf16.float().abs().max()


def test_packed_tiles_are_bit_reproducible_after_other_work():
    # a packed short-response tile fills only g * R of the 128 Q rows; the rest of the tile holds
    # whatever the previous CTA left in shared memory and must not influence the real rows
    cfg = small("packed_det", P=4096, page_size=256, num_shards=4, R=3, Hq=24, Hkv=4)
    case = parity.Case(cfg)
    q, k, v, _ = case.member(0)
    a = case.forward(q, k, v)
    other = parity.Case(small("noise", P=2048, R=256, seed=5))      # different bytes through the same SMs
    oq, ok_, ov, _ = other.member(0)
    other.forward(oq * 37.0, ok_ * 11.0, ov)
    b = case.forward(q, k, v)
    for x, y in zip(a, b):
        assert torch.equal(x, y)


def test_forward_split_count_does_not_change_the_merge():
    outs = []
    for S in (1, 2, 4, 8, 32):
        cfg = small("split%d" % S, P=64 * 40, page_size=64, num_shards=S, Dk=128, Dv=128, R=128, Hq=2, Hkv=1)
        case = parity.Case(cfg)
        q, k, v, _ = case.member(0)
        outs.append(case.forward(q, k, v))
    torch.cuda.synchronize()
    for o in outs[1:]:
        assert (o[4] - outs[0][4]).abs().max() < 1e-4          # LSE
        assert (o[3] - outs[0][3]).abs().max() < 2e-3          # O fp32


def test_forward_needle_rows_rescale_path():
    # a key equal to 4x a query vector: that row's maximum jumps from ~5 to ~64 mid-stream
    cfg = small("needle", P=4096, page_size=256, num_shards=2, needles=6, R=256, G=1)
    case = parity.Case(cfg)
    plan = W.needle_plan(cfg)
    fw = parity.check_forward(case, extra_rows=[(t, h) for _, _, t, h in plan])
    for pos, _, t, h in plan:
        kvh = h // (cfg.Hq // cfg.Hkv)
        v_needle = case.v_pool[int(case.table[pos // cfg.page_size]), pos % cfg.page_size, kvh].float()
        assert (fw["o_f32"][t, h] - v_needle).abs().max() < 2e-2
        assert fw["lse"][t, h] > 40


def test_prefix_pool_is_not_modified():
    cfg = small("checksum", P=2048)
    case = parity.Case(cfg)
    before = B.ls_prefix_pages_checksum(case.pages)
    q, k, v, _ = case.member(0)
    case.forward(q, k, v)
    assert B.ls_prefix_pages_checksum(case.pages) == before
    case.k_pool[int(case.table[3]), 5, 0, 7] += 1.0
    assert B.ls_prefix_pages_checksum(case.pages) != before
