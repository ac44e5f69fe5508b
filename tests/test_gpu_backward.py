"""Replay backward on the GPU against the fp64 oracle's analytic gradients."""
import numpy as np
import pytest
import torch

from paper_2607_14952_b200 import binding as B
from paper_2607_14952_b200 import workloads as W
from paper_2607_14952_b200.workloads import CONFIGS, ReplayConfig

import parity

pytestmark = pytest.mark.gpu


def small(name, **kw):
    base = dict(name=name, P=2048, R=256, Hq=4, Hkv=2, Dk=256, Dv=256, page_size=256, num_shards=3, G=1, seed=91)
    base.update(kw)
    return ReplayConfig(**base)


def test_config1_tiny_full():
    case = parity.Case(CONFIGS["tiny"])
    fw = parity.check_forward(case, per_shard=False, strict_abs=True)
    parity.check_backward(case, fw, strict_abs=True)


@pytest.mark.parametrize("cfg", [
    small("d256_basic"),
    small("d256_ragged", P=1000, R=200, num_shards=2),
    small("d256_pg64", P=64 * 13 + 7, page_size=64, num_shards=4, R=130),
    small("d256_pg512", P=4096 + 300, page_size=512, num_shards=2, Hq=6, Hkv=2),
    small("d128_pg128", Dk=128, Dv=128, P=128 * 9, page_size=128, num_shards=4, Hq=6, Hkv=2, R=384),
    small("d128_small_p", Dk=128, Dv=128, P=50, page_size=64, num_shards=2, R=64),
    small("d256_empty_shards", P=512, page_size=256, num_shards=5),
    # P = 0: pure causal self-attention, where dK/dV are O(1) and the absolute tolerance bites
    small("d256_p0", P=0, num_shards=2, R=300),
    small("d128_p0", Dk=128, Dv=128, P=0, num_shards=1, R=257, Hq=2, Hkv=1, page_size=64),
    # shared-latent shape: 576-wide key page whose first 512 channels are the value
    small("mla_pg64", Dk=576, Dv=512, v_aliases_k=True, Hq=8, Hkv=1, P=64 * 20 + 5, page_size=64, num_shards=3, R=130),
    small("mla_pg256", Dk=576, Dv=512, v_aliases_k=True, Hq=4, Hkv=1, P=2048, page_size=256, num_shards=2, R=256),
    small("mla_p0", Dk=576, Dv=512, v_aliases_k=True, Hq=2, Hkv=1, P=0, page_size=64, num_shards=1, R=200),
    # (found by random shapes: first rows that see one or two keys, one of them dominant)
    small("d256_p0_packed_tiles", P=0, page_size=256, num_shards=3, R=100, Hq=8, Hkv=2, seed=1438),
    small("d128_p0_g6", Dk=128, Dv=128, P=0, page_size=64, num_shards=5, R=200, Hq=24, Hkv=4, seed=1308),
    small("mla_p0_one_head", Dk=576, Dv=512, v_aliases_k=True, Hq=1, Hkv=1, P=0, page_size=64, num_shards=5, R=300,
          seed=1371),
    small("d256_p1_short", P=1, page_size=64, num_shards=5, R=3, Hq=24, Hkv=4, seed=1258),
    # short responses: every (head, token) row of a KV group shares one Q tile
    small("short_r5", P=3000, page_size=128, num_shards=5, R=5, Hq=6, Hkv=2),
    small("short_r16", P=4096, page_size=256, num_shards=4, R=16, Hq=24, Hkv=4),
    small("short_r1", P=1500, page_size=64, num_shards=3, R=1, Hq=8, Hkv=2, Dk=128, Dv=128),
    small("short_r32_full_tile", P=2048, page_size=256, num_shards=2, R=32, Hq=8, Hkv=2),
    small("mla_short_r3", Dk=576, Dv=512, v_aliases_k=True, Hq=16, Hkv=1, P=64 * 11 + 7, page_size=64, num_shards=2, R=3),
    small("mla_short_r1_64heads", Dk=576, Dv=512, v_aliases_k=True, Hq=64, Hkv=1, P=256 * 5 + 9, page_size=256,
          num_shards=3, R=1),
    # responses shorter than a Q tile whose KV group needs several tiles of (tokens x heads) rows
    small("short_r40_two_tiles", P=2048 + 77, page_size=256, num_shards=3, R=40, Hq=8, Hkv=2),
    small("short_r30_g6", P=1900, page_size=128, num_shards=2, R=30, Hq=12, Hkv=2),
    small("short_r100_d128", Dk=128, Dv=128, P=64 * 21 + 3, page_size=64, num_shards=4, R=100, Hq=16, Hkv=2),
    small("mla_short_r5_64heads", Dk=576, Dv=512, v_aliases_k=True, Hq=64, Hkv=1, P=64 * 23 + 11, page_size=64,
          num_shards=4, R=5),
    small("mla_short_r2_128heads", Dk=576, Dv=512, v_aliases_k=True, Hq=128, Hkv=1, P=256 * 4 + 100, page_size=256,
          num_shards=2, R=2),
    small("mla_short_r20_8heads", Dk=576, Dv=512, v_aliases_k=True, Hq=8, Hkv=1, P=64 * 17, page_size=64,
          num_shards=3, R=20),
], ids=lambda c: c.name)
def test_backward_small_cases(cfg):
    case = parity.Case(cfg, extra_phys_pages=2)
    before = B.ls_prefix_pages_checksum(case.pages)
    fw = parity.check_forward(case, per_shard=False)
    # with P = 0 the first rows see one or two keys: ds = p (dp - Delta) cancels to ~0 and what is
    # left is the rounding of two dot products and of the forward's bf16 P (through Delta = dO . O)
    # against a reference near 0: the gate takes the kernel's unavoidable rounding
    # (parity.dq_rounding_model) into account there
    parity.check_backward(case, fw, dq_model=cfg.P <= 1)
    assert B.ls_prefix_pages_checksum(case.pages) == before      # the prefix is read-only


def test_backward_needle_rows_cancel():
    # on a needle-matched row p ~ one-hot, so ds = p (dp - Delta) ~ 0 by cancellation
    cfg = small("needle", P=4096, page_size=256, num_shards=2, needles=6, R=256, G=1)
    case = parity.Case(cfg)
    plan = W.needle_plan(cfg)
    rows = [(t, h) for _, _, t, h in plan]
    fw = parity.check_forward(case, per_shard=False, extra_rows=rows)
    # 6 needles among only 4,096 keys also dominate many OTHER rows, whose dQ is then a
    # near-cancelling sum of bf16-rounded terms times key norms of 64: the gate adds the
    # kernel's unavoidable rounding (parity.dq_rounding_model) to the relative bound
    bw = parity.check_backward(case, fw, extra_rows=rows, dq_model=True)
    for t, h in rows:
        assert bw["dq"][t, h].float().abs().max() < 1e-3


def test_backward_is_deterministic_and_workspace_is_checked():
    cfg = small("det", P=3000, page_size=128, num_shards=4)
    case = parity.Case(cfg)
    q, k, v, d_o = case.member(0)
    _, _, _, o_f32, lse = case.forward(q, k, v)
    a = case.backward(q, k, v, o_f32, lse, d_o)
    b = case.backward(q, k, v, o_f32, lse, d_o)
    torch.cuda.synchronize()
    for x, y in zip(a, b):
        assert torch.equal(x, y)
    with pytest.raises(B.LsError) as e:
        B.ls_replay_attn_bwd(case.pages, q, k, v, o_f32, lse, d_o, cfg.scale,
                             workspace=torch.empty(1024, dtype=torch.uint8, device="cuda"))
    assert e.value.status == B.LS_ERR_WORKSPACE


def test_backward_split_count_does_not_change_dq():
    outs = []
    for S in (1, 4, 32):
        cfg = small("split%d" % S, P=64 * 40, page_size=64, num_shards=S, Dk=128, Dv=128, R=128, Hq=2, Hkv=1)
        case = parity.Case(cfg)
        q, k, v, d_o = case.member(0)
        _, _, _, o_f32, lse = case.forward(q, k, v)
        outs.append(case.backward(q, k, v, o_f32, lse, d_o))
    torch.cuda.synchronize()
    for o in outs[1:]:
        assert (o[0].float() - outs[0][0].float()).abs().max() < 2e-3


@pytest.mark.parametrize("budget_kib", [96, 256, 1024])
def test_sub_split_shards_forward_and_backward(budget_kib):
    # long shards are walked as consecutive sub-ranges (a locality measure for long prefixes) whose
    # results fold back, in order, into the S partials of the ABI; a tiny stream budget forces that
    # on small cases, including sub-ranges left empty
    for cfg in (small("sub_pg64", P=64 * 13 + 7, page_size=64, num_shards=4, R=130),
                small("sub_pg256", P=256 * 9 + 100, page_size=256, num_shards=2, R=200, Hq=6, Hkv=2),
                small("sub_d128", Dk=128, Dv=128, P=128 * 11, page_size=128, num_shards=3, R=96, Hq=8, Hkv=2),
                small("sub_mla", Dk=576, Dv=512, v_aliases_k=True, Hq=4, Hkv=1, P=64 * 9 + 3, page_size=64,
                      num_shards=2, R=70)):
        case = parity.Case(cfg, stream_budget_kib=budget_kib)
        fw = parity.check_forward(case, per_shard=True)
        parity.check_backward(case, fw)


@pytest.mark.parametrize("aliased", [True, False])
def test_shared_latent_dq_paths(aliased):
    # 576/512 pools whose V aliases K take the transposed dQ kernel that walks every partial in
    # one accumulator; a 576/512 pool with a V tensor of its own takes the per-partial kernel.
    # Cases: ragged tail page, several heads per latent, more than one row tile per head, a
    # response longer than one key tile.
    for cfg in (small("mla_t_pg64", Dk=576, Dv=512, v_aliases_k=aliased, Hq=8, Hkv=1, P=64 * 37 + 21, page_size=64,
                      num_shards=5, R=150),
                small("mla_t_pg512", Dk=576, Dv=512, v_aliases_k=aliased, Hq=2, Hkv=1, P=512 * 5 + 300, page_size=512,
                      num_shards=3, R=64)):
        case = parity.Case(cfg)
        fw = parity.check_forward(case, per_shard=True)
        parity.check_backward(case, fw)


def test_shared_latent_dq_chained_ranges():
    # many row blocks (64 heads x 2 blocks of the 96 rows) and a tiny stream budget: the transposed dQ kernel
    # hands the pairs of one range of parts out together and folds the 32 ranges of every row block into one
    # running dQ, in order, on top of the response block's partial
    cfg = small("mla_chain", Dk=576, Dv=512, v_aliases_k=True, Hq=64, Hkv=1, P=64 * 40, page_size=64, num_shards=4, R=96,
                seed=431)
    case = parity.Case(cfg, stream_budget_kib=96)
    fw = parity.check_forward(case, per_shard=False)
    parity.check_backward(case, fw)
    # without a response block the running dQ starts empty: same result as the one-range walk of a handle
    # with the default budget, up to the fp32 summation order and the bf16 output rounding
    q, k, v, d_o = case.member(0)
    _, _, _, o_f32, lse = case.forward(q, k, v)
    a = case.backward(q, None, None, o_f32, lse, d_o, flags=B.LS_FLAG_NO_RESPONSE_BLOCK)[0].float()
    one = parity.Case(cfg)
    b = one.backward(q, None, None, o_f32, lse, d_o, flags=B.LS_FLAG_NO_RESPONSE_BLOCK)[0].float()
    torch.cuda.synchronize()
    assert torch.isfinite(a).all() and (a - b).abs().max() <= 2.0 ** -7 * b.abs().max() + 1e-6
    again = case.backward(q, None, None, o_f32, lse, d_o, flags=B.LS_FLAG_NO_RESPONSE_BLOCK)[0].float()
    assert torch.equal(a, again)                       # fixed fold order: bit-reproducible


def test_shared_latent_dq_ignores_unmapped_pages():
    # 64-token pages, an odd page count per shard (the last 128-key tile of a shard is half
    # empty), a pool larger than the prefix whose unmapped pages -- physical page 0 among them --
    # hold NaN patterns: nothing of them may reach dQ
    cfg = small("mla_nan", Dk=576, Dv=512, v_aliases_k=True, Hq=4, Hkv=1, P=64 * 9, page_size=64, num_shards=3, R=96)
    case = parity.Case(cfg, extra_phys_pages=3)
    mapped = set(int(x) for x in case.table)
    moved = None
    if 0 in mapped:                                   # free physical page 0: move its logical page elsewhere
        free = [p for p in range(case.k_pool.shape[0]) if p not in mapped]
        lp = list(case.table).index(0)
        case.k_pool[free[0]] = case.k_pool[0]
        case.table[lp] = free[0]
        moved = free[0]
        case.pages.close()
        case.pages = B.ls_prefix_pages_build(cfg.P, cfg.page_size, cfg.num_shards, cfg.Hkv, cfg.Dk, cfg.Dv,
                                             case.k_pool.shape[0], page_table=case.table, k_pool=case.k_pool,
                                             v_aliases_k=True)
        case._host = {}
    mapped = set(int(x) for x in case.table)
    for p in range(case.k_pool.shape[0]):
        if p not in mapped:
            case.k_pool[p] = float("nan")
    assert torch.isnan(case.k_pool[0]).all()
    fw = parity.check_forward(case, per_shard=False)
    bw = parity.check_backward(case, fw)
    assert torch.isfinite(bw["dq"].float()).all()


@pytest.mark.parametrize("cfg", [
    # long responses over short prefixes, every element compared: each response key's dK / dV
    # accumulates over all later column tiles and all heads of its group, and dQ covers every row tile
    small("long_d256", P=4096, R=4096, Hq=6, Hkv=1, page_size=256, num_shards=2, seed=401),
    small("long_d128", Dk=128, Dv=128, P=2048, R=2048, Hq=8, Hkv=2, page_size=128, num_shards=2, seed=402),
    small("long_mla", Dk=576, Dv=512, v_aliases_k=True, P=2048, R=1024, Hq=64, Hkv=1, page_size=64, num_shards=4,
          seed=403),
], ids=lambda c: c.name)
def test_long_response_full_check(cfg):
    case = parity.Case(cfg)
    fw = parity.check_forward(case, per_shard=False)
    parity.check_backward(case, fw)


@pytest.mark.parametrize("cfg,policy,budget_kib", [
    (small("short_r7_zigzag_pg64", P=64 * 301 + 19, page_size=64, num_shards=7, R=7, Hq=24, Hkv=4), B.LS_SHARD_ZIGZAG, 512),
    (small("short_r9_d128_cyclic", Dk=128, Dv=128, P=128 * 90 + 5, page_size=128, num_shards=5, R=9, Hq=8, Hkv=2),
     B.LS_SHARD_CYCLIC, 0),
    (small("short_r3_more_shards_than_pages", P=256 * 9 + 1, page_size=256, num_shards=16, R=3, Hq=12, Hkv=2),
     B.LS_SHARD_CONTIGUOUS, 0),
], ids=lambda c: getattr(c, "name", None))
def test_short_response_dq_ranges_cross_parts(cfg, policy, budget_kib):
    # one Q tile per KV group: the dQ pass cuts the key tiles of a KV head (response block and all parts
    # end to end) into equal ranges, one CTA each, so a CTA's keys cross part boundaries, ragged
    # tails and empty parts; every element against the oracle
    case = parity.Case(cfg, policy=policy, stream_budget_kib=budget_kib)
    fw = parity.check_forward(case, per_shard=False)
    parity.check_backward(case, fw)


@pytest.mark.parametrize("policy", [B.LS_SHARD_CYCLIC, B.LS_SHARD_ZIGZAG])
def test_shard_policies_at_scale_forward_and_backward(policy):
    # the 131,072-position prefix on 64-token pages (2,048 pages: every page its own TMA box)
    # under the paper's block-cyclic and zigzag ownership, forward (every partial against
    # Eq. qwen-local-attn on its shard's positions) and backward, sampled rows
    cfg = W.scaled(CONFIGS["p128k"], name="p128k-pg64", page_size=64, R=512)
    case = parity.Case(cfg, policy=policy)
    fw = parity.check_forward(case, kv_groups=[2], full=False, per_shard=True, strict_abs=True)
    parity.check_backward(case, fw, kv_groups=[2], full=False, tail=8, strict_abs=True)


def test_abi_errors_on_a_device_handle():
    cfg = small("abi", P=256 * 9 + 100, page_size=256, num_shards=2, R=200, Hq=6, Hkv=2)
    case = parity.Case(cfg, stream_budget_kib=256)          # shards are walked as sub-ranges: the forward needs counters
    q, k, v, d_o = case.member(0)
    need = B.ls_replay_attn_workspace_bytes(case.pages, cfg.R, cfg.Hq, cfg.scale, B.LS_WORKSPACE_FWD)
    assert need > 0

    def status_of(fn):
        with pytest.raises(B.LsError) as e:
            fn()
        return e.value.status

    tiny_ws = torch.empty(16, dtype=torch.uint8, device="cuda")
    assert status_of(lambda: B.ls_replay_attn_fwd(case.pages, q, k, v, cfg.scale, workspace=tiny_ws)) == B.LS_ERR_WORKSPACE
    assert status_of(lambda: B.ls_replay_attn_fwd_merged(case.pages, q, k, v, cfg.scale, workspace=tiny_ws[:0])) \
        == B.LS_ERR_WORKSPACE
    # a query tensor that starts 2 bytes into an allocation
    flat = torch.empty(q.numel() + 8, dtype=torch.bfloat16, device="cuda")
    q_off = flat[1:1 + q.numel()].view_as(q)
    q_off.copy_(q)
    assert q_off.data_ptr() % 16 != 0
    assert status_of(lambda: B.ls_replay_attn_fwd(case.pages, q_off, k, v, cfg.scale)) == B.LS_ERR_ALIGNMENT
    assert status_of(lambda: B.ls_replay_attn_fwd_merged(case.pages, q_off, k, v, cfg.scale)) == B.LS_ERR_ALIGNMENT
    _, _, _, o_f32, lse = case.forward(q, k, v)
    assert status_of(lambda: B.ls_replay_attn_bwd(case.pages, q_off, k, v, o_f32, lse, d_o, cfg.scale)) == B.LS_ERR_ALIGNMENT
    # a plan without a pool cannot run attention
    plan = B.ls_prefix_pages_build(cfg.P, cfg.page_size, cfg.num_shards, cfg.Hkv, cfg.Dk, cfg.Dv, cfg.num_pages)
    assert status_of(lambda: B.ls_replay_attn_fwd(plan, q, k, v, cfg.scale)) == B.LS_ERR_INVALID_ARG
    assert status_of(lambda: B.ls_replay_attn_bwd(plan, q, k, v, o_f32, lse, d_o, cfg.scale)) == B.LS_ERR_INVALID_ARG
    # a call planned against another generation of the handle
    gen = B.ls_pages_generation(case.pages)
    assert status_of(lambda: B.ls_replay_attn_fwd(case.pages, q, k, v, cfg.scale, generation=gen + 1)) == B.LS_ERR_STALE
    B.ls_replay_attn_fwd(case.pages, q, k, v, cfg.scale, generation=gen)
    torch.cuda.synchronize()


def test_merge_reports_non_finite_lse():
    o = torch.zeros(3, 16, 128, device="cuda")
    l = torch.zeros(3, 16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.ls_lse_merge(o, l, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    l[1, 5] = float("nan")                      # host-made: a partial arrives with a NaN log-normaliser
    _, _, lse = B.ls_lse_merge(o, l, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == B.LS_ERR_NONFINITE and torch.isnan(lse[5]) and torch.isfinite(lse[:5]).all()
    status.zero_()
    l[1, 5] = float("inf")
    B.ls_lse_merge(o, l, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == B.LS_ERR_NONFINITE
    status.zero_()
    l[:, 7] = -float("inf")                     # an all-empty row is fine: l = -inf, nothing reported
    l[1, 5] = 0.0
    B.ls_lse_merge(o, l, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
