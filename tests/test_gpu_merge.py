"""ls_lse_merge against the oracle's merge (Eq. qwen-lse-parts, Eq. qwen-global-attn)."""
import numpy as np
import pytest
import torch

from oracle import attention as oa
from paper_2607_14952_b200 import binding as B

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("parts", [1, 2, 5, 9, 33])
@pytest.mark.parametrize("dv", [128, 256, 512])
def test_merge_matches_oracle(parts, dv):
    g = torch.Generator(device="cuda").manual_seed(parts * 1000 + dv)
    rows = 1000 + parts                     # not a multiple of the warps per block
    o = torch.randn(parts, rows, dv, generator=g, device="cuda")
    l = torch.randn(parts, rows, generator=g, device="cuda") * 20.0          # spread of ~60 between partials
    if parts > 1:
        l[1, ::3] = -float("inf")           # empty partials
        o[1, ::3] = 0.0
    o_bf16, o_f32, lse = B.ls_lse_merge(o, l)
    torch.cuda.synchronize()
    ro, rl = oa.merge(o.double().cpu().numpy(), l.double().cpu().numpy())
    assert np.abs(lse.double().cpu().numpy() - rl).max() < 1e-4
    assert np.abs(o_f32.double().cpu().numpy() - ro).max() < 1e-4
    assert np.abs(o_bf16.double().cpu().numpy() - ro).max() < 2e-2
    assert torch.equal(o_f32.to(torch.bfloat16), o_bf16)


def test_merge_all_empty_and_dominant_partial():
    o = torch.zeros(3, 8, 128, device="cuda")
    l = torch.full((3, 8), -float("inf"), device="cuda")
    l[2, 4:] = 64.0
    o[2, 4:] = 3.0
    l[0, 4:] = 15.0                        # e^{-49} relative weight: vanishes without NaN
    o[0, 4:] = -7.0
    _, o_f32, lse = B.ls_lse_merge(o, l)
    torch.cuda.synchronize()
    assert torch.isinf(lse[:4]).all() and (lse[:4] < 0).all() and (o_f32[:4] == 0).all()
    assert torch.allclose(lse[4:], torch.full_like(lse[4:], 64.0)) and torch.allclose(o_f32[4:], torch.full_like(o_f32[4:], 3.0))
    assert torch.isfinite(o_f32).all()


def test_bounded_wait_gives_up_and_reports_timeout():
    # a barrier that nothing completes: the wait must run out (2 ms budget), the kernel must return,
    # the status word must say LS_ERR_TIMEOUT and the context must stay usable
    import time
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    t0 = time.perf_counter()
    B.ls_selftest_bounded_wait(status, 2_000_000)
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 1.0
    assert int(status.item()) == B.LS_ERR_TIMEOUT
    x = torch.ones(4, device="cuda") * 2                      # the context still works
    assert float(x.sum()) == 8.0


@pytest.mark.parametrize("parts,dv", [(1, 128), (9, 256), (33, 512)])
def test_merge_with_the_numerator_summed_in_bf16(parts, dv):
    # ls_lse_merge_bf16_numerator against the oracle's emulation of the same roundings; the two form the
    # products w * o in fp32 and fp64, so a term may now and then fall on the other side of a bf16 rounding
    # boundary: one bf16 step of the running magnitude per element is allowed, the typical error must be far less
    g = torch.Generator(device="cuda").manual_seed(parts * 77 + dv)
    rows = 300 + parts
    o = torch.randn(parts, rows, dv, generator=g, device="cuda")
    l = torch.randn(parts, rows, generator=g, device="cuda") * 4.0
    if parts > 1:
        l[1, ::4] = -float("inf")
        o[1, ::4] = 0.0
    o_bf16, o_f32, lse = B.ls_lse_merge(o, l, bf16_numerator=True)
    _, o_plain, lse_plain = B.ls_lse_merge(o, l)
    torch.cuda.synchronize()
    od, ld = o.double().cpu().numpy(), l.double().cpu().numpy()
    ro, rl = oa.merge_bf16_numerator(od, ld)
    assert torch.equal(lse, lse_plain) and np.abs(lse.double().cpu().numpy() - rl).max() < 1e-4
    got = o_f32.double().cpu().numpy()
    w = np.exp(ld - ld.max(axis=0))
    step = 2.0 ** -7 * (w[..., None] * np.abs(od)).sum(axis=0) / w.sum(axis=0)[..., None]
    err = np.abs(got - ro)
    assert (err <= step + 1e-6).all()
    assert (err <= 1e-6).mean() > 0.98                     # almost every element takes identical roundings
    assert torch.equal(o_f32.to(torch.bfloat16), o_bf16)
    if parts > 1:                                          # and it is not the fp32 merge
        assert (o_f32 != o_plain).any()
