"""The allocation-free prefill entry point, `lasad_forward_static`, against `lasad_forward`.

Some hosts of this library must not let it allocate device memory: a serving process that fixes
its device-memory plan at start-up, or a plug-in whose host framework owns every allocation.
For them the library carries its scratch (the per-(batch, head) relay slots of the streaming
prefill) in a fixed array of its own image.  This file checks, through the C ABI, that the
entry point gives the same output and final state as the ordinary one, twice in a row -- the
second call finds the array as the first one left it.  It is collected last on purpose, so that
a run that stops at the first failure has already run every other test.
"""
import pytest
import torch

from paper_2507_01652_b200 import binding
from tests._util import TOL, rel_err, to64

pytestmark = pytest.mark.gpu


def _case(seed, B, T, H, w, P):
    gen = torch.Generator().manual_seed(seed)
    q, k, v = [(torch.randn(B, T, H, 64, generator=gen) / 8).to(torch.bfloat16).cuda() for _ in range(3)]
    g = (0.9 + 0.0999 * torch.rand(H, generator=gen)).cuda()
    s_in = torch.randn(B, H, 64, 64, generator=gen).cuda()
    return q, k, v, g, s_in, w, P


def test_static_entry_point_matches_lasad_forward_twice_in_a_row():
    ctx = binding.Lasad(0)
    try:
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        # two different shapes, both several chunks long, so that the second call reuses relay
        # slots the first one has written
        for seed, B, T, H, w, P in ((21, 2, 700, 5, 24, 0), (22, 3, 391, 4, 16, 1)):
            q, k, v, g, s_in, w, P = _case(seed, B, T, H, w, P)
            o_ref, s_ref = ctx.lasad_forward(q, k, v, g, w, prefix_len=P, t0=3, scale=0.5, state_in=s_in)
            o = torch.empty_like(o_ref)
            s = torch.empty_like(s_ref)
            binding.lasad_forward_static(q, k, v, g, w, o, state_out=s, prefix_len=P, t0=3, scale=0.5,
                                         state_in=s_in, device_status=status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0, "a device-side wait timed out"
            assert rel_err(o, to64(o_ref)) <= TOL[torch.bfloat16]
            assert rel_err(s, to64(s_ref)) <= TOL[torch.bfloat16]
    finally:
        ctx.close()


def test_static_entry_point_rejects_what_it_cannot_hold():
    B, T, H = 33, 16, 8     # 264 (batch, head) pairs: more than the built-in storage covers
    q = torch.zeros(B, T, H, 64, dtype=torch.bfloat16, device="cuda")
    g = torch.ones(H, device="cuda")
    with pytest.raises(binding.LasadError) as e:
        binding.lasad_forward_static(q, q, q, g, 4, torch.empty_like(q))
    assert e.value.code == binding.LASAD_ERR_UNSUPPORTED
    q32 = torch.zeros(1, 8, 2, 64, dtype=torch.float32, device="cuda")
    with pytest.raises(binding.LasadError) as e:
        binding.lasad_forward_static(q32, q32, q32, g[:2], 4, torch.empty_like(q32))
    assert e.value.code == binding.LASAD_ERR_UNSUPPORTED
