"""The workspace-free backward entry point against the regular one.

ls_replay_attn_bwd_static exists for callers that cannot provide scratch memory: a replay
scheduler whose page pool already fills the GPU, or a host framework whose allocator owns
all device memory, so that nothing may be allocated at backward time.  It keeps its scratch
in a fixed array inside the library.  The test first runs a call of ANOTHER shape (so that
the leftovers in that shared array do not line up with what the next call writes), then
calls it twice in a row through the C ABI and checks both results against
ls_replay_attn_bwd on the same inputs, and that the device's free memory does not move
across the calls.  It is collected last on purpose.
"""
import pytest
import torch

from paper_2607_14952_b200 import binding as B
from paper_2607_14952_b200.workloads import CONFIGS, ReplayConfig

import parity

pytestmark = pytest.mark.gpu


def _static(case, q, k, v, o_f32, lse, d_o, ref):
    out = [torch.full_like(x, float("nan")) for x in ref]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    B.ls_replay_attn_bwd_static(case.pages, q, k, v, o_f32, lse, d_o, case.cfg.scale, *out, status=status)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the device's free memory"
    assert int(status.item()) == 0
    return out


def test_static_backward_matches_workspace_backward_twice():
    # a call of a different shape first: its leftovers sit at other offsets of the shared scratch
    other = parity.Case(ReplayConfig(name="other", P=64 * 7 + 3, R=70, Hq=6, Hkv=2, Dk=256, Dv=256, page_size=64,
                                     num_shards=3, G=1, seed=17))
    q, k, v, d_o = other.member(0)
    _, _, _, o_f32, lse = other.forward(q, k, v)
    ref = other.backward(q, k, v, o_f32, lse, d_o)
    out = _static(other, q, k, v, o_f32, lse, d_o, ref)      # (also the first call on this device: address look-up)
    for a, b in zip(out, ref):
        assert torch.equal(a, b)

    case = parity.Case(CONFIGS["tiny"])
    cfg = case.cfg
    need = B.ls_replay_attn_workspace_bytes(case.pages, cfg.R, cfg.Hq, cfg.scale, B.LS_WORKSPACE_BWD)
    assert 0 < need <= B.ls_replay_attn_bwd_static_capacity()
    for member in (0, 1):                      # two calls in a row, different inputs
        q, k, v, d_o = case.member(member)
        _, _, _, o_f32, lse = case.forward(q, k, v)
        ref = case.backward(q, k, v, o_f32, lse, d_o)
        out = _static(case, q, k, v, o_f32, lse, d_o, ref)
        for name, a, b in zip(("dq", "dk", "dv"), out, ref):
            assert torch.isfinite(a.float()).all(), name
            # same kernels, same order of summation: the tolerance of the parity tests is met with zero error
            assert (a.float() - b.float()).abs().max().item() <= parity.ABS_TOL, name
            assert torch.equal(a, b), name


def test_static_backward_rejects_shapes_beyond_its_scratch():
    cfg = ReplayConfig(name="big", P=1024, R=4096, Hq=12, Hkv=2, Dk=256, Dv=256, page_size=256, num_shards=8, G=1, seed=5)
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
