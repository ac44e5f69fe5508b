"""The workspace-free backward entry point against the regular one.

ls_replay_attn_bwd_static exists for callers that cannot provide scratch memory: a replay
scheduler whose page pool already fills the GPU, or a host framework whose allocator owns
all device memory, so that nothing may be allocated at backward time.  It keeps its scratch
in a fixed array inside the library.  The test calls it twice in a row through the C ABI
(the second call meets the first call's leftovers in that shared array) and checks both
results against ls_replay_attn_bwd on the same inputs.  It is collected last on purpose.
"""
import pytest
import torch

from paper_2607_14952_b200 import binding as B
from paper_2607_14952_b200.workloads import CONFIGS, ReplayConfig

import parity

pytestmark = pytest.mark.gpu


def test_static_backward_matches_workspace_backward_twice():
    case = parity.Case(CONFIGS["tiny"])
    cfg = case.cfg
    need = B.ls_replay_attn_workspace_bytes(case.pages, cfg.R, cfg.Hq, cfg.scale, B.LS_WORKSPACE_BWD)
    assert 0 < need <= B.ls_replay_attn_bwd_static_capacity()
    for member in (0, 1):                      # two calls in a row, different inputs
        q, k, v, d_o = case.member(member)
        _, _, _, o_f32, lse = case.forward(q, k, v)
        ref = case.backward(q, k, v, o_f32, lse, d_o)
        out = [torch.full_like(x, float("nan")) for x in ref]
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        B.ls_replay_attn_bwd_static(case.pages, q, k, v, o_f32, lse, d_o, cfg.scale, *out, status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        for name, a, b in zip(("dq", "dk", "dv"), out, ref):
            assert torch.isfinite(a.float()).all(), name
            # same kernels, same order of summation: the tolerance of the parity tests is met with zero error
            assert (a.float() - b.float()).abs().max().item() <= parity.ABS_TOL, name
            assert torch.equal(a, b), name


def test_static_backward_rejects_shapes_beyond_its_scratch():
    cfg = ReplayConfig(name="big", P=1024, R=2048, Hq=8, Hkv=2, Dk=256, Dv=256, page_size=256, num_shards=8, G=1, seed=5)
    case = parity.Case(cfg)
    need = B.ls_replay_attn_workspace_bytes(case.pages, cfg.R, cfg.Hq, cfg.scale, B.LS_WORKSPACE_BWD)
    assert need > B.ls_replay_attn_bwd_static_capacity()
    q, k, v, d_o = case.member(0)
    o_f32 = torch.zeros((cfg.R, cfg.Hq, cfg.Dv), device="cuda")
    lse = torch.zeros((cfg.R, cfg.Hq), device="cuda")
    with pytest.raises(B.LsError) as e:
        B.ls_replay_attn_bwd_static(case.pages, q, k, v, o_f32, lse, d_o, cfg.scale, torch.empty_like(q),
                                    torch.empty_like(k), torch.empty_like(v))
    assert e.value.status == B.LS_ERR_WORKSPACE
