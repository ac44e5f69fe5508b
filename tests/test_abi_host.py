"""Host side of the C ABI (no GPU): the library loads, exports every declared symbol,
and its page/shard planner agrees bit for bit with the oracle's integer arithmetic."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import pages as op
from paper_2607_14952_b200 import binding as B
from paper_2607_14952_b200.workloads import CONFIGS, page_permutation

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "ls.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = set(re.findall(r"\b(ls_[a-z_0-9]+)\s*\(", header))
    assert {"ls_prefix_pages_build", "ls_replay_attn_fwd", "ls_lse_merge", "ls_replay_attn_bwd"} <= names
    L = B.lib()
    for n in sorted(names):
        assert hasattr(L, n), n


def test_struct_layout_matches_header():
    assert C.sizeof(B.ls_pages_desc_t) == 8 + 8 * 4 + 8 + 8 * 2 + 8 * 6
    assert C.sizeof(B.ls_attn_params_t) == 24


POLICIES = [(B.LS_SHARD_CONTIGUOUS, op.CONTIGUOUS), (B.LS_SHARD_CYCLIC, op.CYCLIC), (B.LS_SHARD_ZIGZAG, op.ZIGZAG)]


def plan_matches_oracle(P, pg, S, pol, opol, table, nphys, Hkv=4, Dk=256, Dv=256):
    pages = B.ls_prefix_pages_build(P, pg, S, Hkv, Dk, Dv, nphys, page_table=table, shard_policy=pol)
    ex = B.ls_prefix_pages_export(pages)
    Np = op.num_pages(P, pg)
    want_table = np.arange(Np, dtype=np.int32) if table is None else np.asarray(table, np.int32)
    assert np.array_equal(ex["page_table"], want_table)
    assert np.array_equal(ex["shard_of_page"], op.shard_of_page(Np, S, opol))
    lists = op.shard_page_lists(Np, S, opol)
    assert np.array_equal(ex["shard_page_offset"], np.concatenate([[0], np.cumsum([len(l) for l in lists])]))
    flat = np.concatenate(lists).astype(np.int32) if Np else np.zeros(0, np.int32)
    assert np.array_equal(ex["shard_logical_pages"], flat)
    assert np.array_equal(ex["shard_tokens"], op.shard_tokens(P, pg, S, opol))
    pages.close()


@pytest.mark.parametrize("name", list(CONFIGS))
def test_plan_of_the_five_configs(name):
    c = CONFIGS[name]
    table = page_permutation(c.num_pages, c.num_pages, c.seed + 2)
    assert op.check_page_table(table, c.num_pages, c.num_pages)
    plan_matches_oracle(c.P, c.page_size, c.num_shards, B.LS_SHARD_CONTIGUOUS, op.CONTIGUOUS, table, c.num_pages,
                        c.Hkv, c.Dk, c.Dv)


@pytest.mark.parametrize("pol,opol", POLICIES)
@pytest.mark.parametrize("P,pg,S", [(4096, 64, 4), (1000, 64, 3), (63, 64, 4), (0, 64, 2), (130, 128, 8),
                                     (2088960, 64, 8), (2097152, 64, 32), (64 * 7 + 5, 64, 2)])
def test_plan_policies_and_ragged_sizes(pol, opol, P, pg, S):
    Np = op.num_pages(P, pg)
    plan_matches_oracle(P, pg, S, pol, opol, None, Np + 3)


def test_paper_worked_examples_through_the_abi():
    # 2,088,960 prompt tokens / 64 = 32,640 pages, 4,080 per rank under owner(p) = p mod 8
    pages = B.ls_prefix_pages_build(2088960, 64, 8, 4, 256, 256, 32640, shard_policy=B.LS_SHARD_CYCLIC)
    ex = B.ls_prefix_pages_export(pages)
    assert pages.num_logical_pages == 32640
    assert (np.diff(ex["shard_page_offset"]) == 4080).all()
    assert (ex["shard_of_page"] == np.arange(32640) % 8).all()
    # zigzag over 32 ranks: rank 0 holds pages 0-511 then 32,256-32,767
    pages = B.ls_prefix_pages_build(2097152, 64, 32, 1, 576, 512, 32768, shard_policy=B.LS_SHARD_ZIGZAG,
                                    v_aliases_k=True)
    ex = B.ls_prefix_pages_export(pages)
    r0 = ex["shard_logical_pages"][:1024]
    assert r0[0] == 0 and r0[511] == 511 and r0[512] == 32256 and r0[1023] == 32767
    r31 = ex["shard_logical_pages"][31 * 1024:32 * 1024]
    assert r31[0] == 15872 and r31[511] == 16383 and r31[512] == 16384 and r31[1023] == 16895
    assert (ex["shard_tokens"] == 65536).all()


def status_of(fn):
    with pytest.raises(B.LsError) as e:
        fn()
    return e.value.status


def test_error_paths_before_any_launch():
    ok = dict(prefix_len=256, page_size=64, num_shards=2, num_kv_heads=1, dim_k=128, dim_v=128, num_phys_pages=4)
    bld = lambda **kw: B.ls_prefix_pages_build(**{**ok, **kw})
    assert status_of(lambda: bld(page_table=np.array([0, 1, 1, 2]))) == B.LS_ERR_BAD_PAGE_TABLE     # duplicate
    assert status_of(lambda: bld(page_table=np.array([0, 1, 4, 2]))) == B.LS_ERR_BAD_PAGE_TABLE     # out of range
    assert status_of(lambda: bld(page_table=np.array([0, -1, 3, 2]))) == B.LS_ERR_BAD_PAGE_TABLE
    assert status_of(lambda: bld(num_phys_pages=3)) == B.LS_ERR_INVALID_ARG                         # pool too small
    assert status_of(lambda: bld(page_size=48)) == B.LS_ERR_UNSUPPORTED_SHAPE
    assert status_of(lambda: bld(dim_k=96)) == B.LS_ERR_UNSUPPORTED_SHAPE
    assert status_of(lambda: bld(num_shards=0)) == B.LS_ERR_INVALID_ARG
    assert status_of(lambda: bld(prefix_len=-1)) == B.LS_ERR_INVALID_ARG
    assert status_of(lambda: bld(shard_policy=7)) == B.LS_ERR_INVALID_ARG
    pages = bld(page_table=np.array([3, 0, 2, 1]), num_phys_pages=6)          # pool larger than Np is fine
    assert B.ls_prefix_pages_export(pages)["page_table"].tolist() == [3, 0, 2, 1]
    assert B.lib().ls_status_string(B.LS_ERR_TIMEOUT) != b"unknown status"


def _ctl(chains):
    return ((4 + chains) * 4 + 15) // 16 * 16


def test_workspace_sizes():
    # backward: Delta, the hand-over counters (one per Q tile) and ONE fp32 running dQ, whatever
    # the number of shards; the 576/512 shape with a V pool of its own keeps one dQ per partial
    R, Hq = 96, 8
    rows = R * Hq
    head = rows * 4 + _ctl(Hq * 1)
    plain = B.ls_prefix_pages_build(256 * 12, 256, 3, 2, 256, 256, 12)
    assert B.ls_replay_attn_workspace_bytes(plain, R, Hq, 0.0625, B.LS_WORKSPACE_BWD) == head + rows * 256 * 4
    assert B.ls_replay_attn_workspace_bytes(plain, R, Hq, 0.0625, B.LS_WORKSPACE_FWD) == 0
    assert B.ls_replay_attn_workspace_bytes(plain, R, Hq, 0.0625, B.LS_WORKSPACE_FWD_MERGED) == _ctl(2 * 4)
    many = B.ls_prefix_pages_build(256 * 12, 256, 12, 2, 256, 256, 12)
    assert B.ls_replay_attn_workspace_bytes(many, R, Hq, 0.0625, B.LS_WORKSPACE_BWD) == head + rows * 256 * 4
    # a tiny stream budget walks every shard as sub-ranges: the forward then needs its counters, nothing more
    cut = B.ls_prefix_pages_build(256 * 12, 256, 3, 2, 256, 256, 12, stream_budget_kib=512)
    # (R = 96 < 128 with 4 heads per KV head: 3 Q tiles of 32 tokens x 4 heads per KV head, not 4 of one head)
    assert B.ls_replay_attn_workspace_bytes(cut, R, Hq, 0.0625, B.LS_WORKSPACE_FWD) == _ctl(2 * 3 * 3)
    assert B.ls_replay_attn_workspace_bytes(cut, R, Hq, 0.0625, B.LS_WORKSPACE_BWD) == head + rows * 256 * 4
    # a short response whose KV group is one Q tile (16 tokens x 4 heads): the key tiles of a KV head are cut
    # into one range per CTA, each with an fp32 sum of its own -- 148 / 2 KV heads = 74 CTAs per KV head at a
    # long prefix, one per four 128-key tiles at a short one (3,072 positions: 7)
    Rs = 16
    rs = Rs * Hq
    assert B.ls_replay_attn_workspace_bytes(plain, Rs, Hq, 0.0625, B.LS_WORKSPACE_BWD) == \
        rs * 4 + _ctl(Hq * 1) + (1 + 7) * rs * 256 * 4
    long_prefix = B.ls_prefix_pages_build(256 * 4096, 256, 8, 2, 256, 256, 4096)
    assert B.ls_replay_attn_workspace_bytes(long_prefix, Rs, Hq, 0.0625, B.LS_WORKSPACE_BWD) == \
        rs * 4 + _ctl(Hq * 1) + (1 + 74) * rs * 256 * 4
    mla = B.ls_prefix_pages_build(64 * 40, 64, 4, 1, 576, 512, 40, v_aliases_k=True)
    # 16 row blocks of 64 are too few to fill the GPU: the 4 parts go to 4 CTA pairs per block, each with an
    # fp32 sum of its own beside the response block's
    # (this shape's dQ kernel works on 64-row blocks: 16 hand-over counters, not 8; the response dK / dV of
    # a short response are summed over 8 head ranges, each with an fp32 [R, 576] sum)
    kv = 8 * R * 576 * 4
    assert B.ls_replay_attn_workspace_bytes(mla, R, Hq, 1 / 24, B.LS_WORKSPACE_BWD) == \
        rows * 4 + _ctl(16) + kv + (1 + 4) * rows * 576 * 4
    # many row blocks: the parts fold into the one running dQ in order, no partials
    assert B.ls_replay_attn_workspace_bytes(mla, 4096, 64, 1 / 24, B.LS_WORKSPACE_BWD) == \
        4096 * 64 * 4 + _ctl(64 * 64) + 4096 * 64 * 576 * 4
    # forward: 6 Q tiles of 16 tokens x 8 heads, two 256-channel halves of O each
    assert B.ls_replay_attn_workspace_bytes(mla, R, Hq, 1 / 24, B.LS_WORKSPACE_FWD_MERGED) == _ctl(6 * 2) + rows * 4
    sep = B.ls_prefix_pages_build(64 * 40, 64, 4, 1, 576, 512, 40, v_aliases_k=False)
    assert B.ls_replay_attn_workspace_bytes(sep, R, Hq, 1 / 24, B.LS_WORKSPACE_BWD) == head + kv + (4 + 1) * rows * 576 * 4
    empty = B.ls_prefix_pages_build(0, 64, 1, 1, 576, 512, 1, v_aliases_k=True)
    assert B.ls_replay_attn_workspace_bytes(empty, R, Hq, 1 / 24, B.LS_WORKSPACE_BWD) == head + kv + (1 + 1) * rows * 576 * 4


def test_suffix_bookkeeping_needs_a_device_handle():
    # a host-only plan has no pool to append pages to
    plan = B.ls_prefix_pages_build(256, 64, 2, 1, 128, 128, 8)
    assert B.ls_pages_generation(plan) == 1 and B.ls_suffix_pages_tokens(plan) == 0
    assert status_of(lambda: B.ls_suffix_pages_reserve(plan, 2, 4)) == B.LS_ERR_INVALID_ARG
    assert status_of(lambda: B.ls_suffix_pages_pop(plan)) == B.LS_ERR_INVALID_ARG
