"""The allocation-free prefill entry point, `lasad_forward_static`, against `lasad_forward` and
against the CPU oracle.

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
from tests._util import TOL, oracle, rel_err, to64

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
            # and against the oracle: the two entry points may share a kernel, so agreement
            # between them alone would not show a fault common to both
            o_orc, s_orc = oracle(q, k, v, g, w, P, 3, 0.5, s_in)
            assert rel_err(o, o_orc) <= TOL[torch.bfloat16]
            assert rel_err(s, s_orc) <= TOL[torch.bfloat16]
    finally:
        ctx.close()


def test_static_entry_point_allocates_nothing_at_its_limit():
    """B * H = 256, the most the built-in storage holds, without a status word of the caller's: the
    driver's count of free device memory must not move over further calls, and the result must
    match the oracle on sampled chains."""
    B, T, H, w = 16, 300, 16, 10
    q, k, v, g, s_in, w, P = _case(23, B, T, H, w, 0)
    o = torch.empty_like(v)
    s = torch.empty(B, H, 64, 64, device="cuda")
    binding.lasad_forward_static(q, k, v, g, w, o, state_out=s, state_in=s_in)     # the device's first-call set-up, if still due
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        binding.lasad_forward_static(q, k, v, g, w, o, state_out=s, state_in=s_in)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, "device memory was allocated or freed by lasad_forward_static"
    for b, h in ((0, 0), (7, 9), (15, 15)):
        sl = (slice(b, b + 1), slice(None), slice(h, h + 1))
        o_orc, s_orc = oracle(q[sl], k[sl], v[sl], g[h:h + 1], w, 0, 0, 1.0, s_in[b:b + 1, h:h + 1])
        assert rel_err(o[sl], o_orc) <= TOL[torch.bfloat16], (b, h)
        assert rel_err(s[b:b + 1, h:h + 1], s_orc) <= TOL[torch.bfloat16], (b, h)


def test_static_entry_point_refuses_a_stream_that_is_being_captured():
    """The kernel tells its calls apart by a number counted on the host, which a replayed recording
    would repeat; so the entry point must refuse to be recorded rather than replay wrongly."""
    q, k, v, g, s_in, w, P = _case(24, 1, 300, 2, 10, 0)
    o = torch.empty_like(v)
    binding.lasad_forward_static(q, k, v, g, w, o)          # set-up outside the capture
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            with pytest.raises(binding.LasadError) as e:
                binding.lasad_forward_static(q, k, v, g, w, o, stream=stream.cuda_stream)
    assert e.value.code == binding.LASAD_ERR_UNSUPPORTED
    torch.cuda.synchronize()
    o_orc, _ = oracle(q, k, v, g, w)
    binding.lasad_forward_static(q, k, v, g, w, o)          # and it still works afterwards
    torch.cuda.synchronize()
    assert rel_err(o, o_orc) <= TOL[torch.bfloat16]


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
