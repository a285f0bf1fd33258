"""GPU parity at the full benchmark sizes, in the launch configuration bench.py times (default
implementation, whole workload in one call): the outputs and final states of sampled (batch,
head) chains against the CPU oracle run on exactly those chains.  Every chain is independent of
the others (the SAD recurrence of Section 3.4 has no cross-head or cross-batch term), so a chain's
oracle result is the expected value of that slice of the full launch."""
import pytest
import torch

from paper_2507_01652_b200 import binding, workloads
from tests._util import TOL, oracle, rel_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = binding.Lasad(0)
    yield c
    c.close()


def _sampled_chains(wl, n):
    """First, last and a spread of (b, h) pairs, deterministic."""
    gen = torch.Generator().manual_seed(wl.seed + 31)
    picks = {(0, 0), (wl.B - 1, wl.H - 1)}
    while len(picks) < n:
        picks.add((int(torch.randint(wl.B, (1,), generator=gen)), int(torch.randint(wl.H, (1,), generator=gen))))
    return sorted(picks)


@pytest.mark.parametrize("name", ["config2", "config3", "config5a", "config5b"])
def test_prefill_full_size_sampled_chains(ctx, name):
    wl = workloads.WORKLOADS[name]
    q, k, v = workloads.make_qkv(wl)
    g = workloads.make_decay(wl)
    o, s = ctx.lasad_forward(q.cuda(), k.cuda(), v.cuda(), g.cuda(), wl.grid_w, prefix_len=wl.prefix_len)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    o, s = o.cpu(), s.cpu()
    assert torch.isfinite(o.float()).all() and torch.isfinite(s).all()
    for b, h in _sampled_chains(wl, 5):
        sl = (slice(b, b + 1), slice(None), slice(h, h + 1))
        o_ref, s_ref = oracle(q[sl], k[sl], v[sl], g[h:h + 1], wl.grid_w, wl.prefix_len)
        assert rel_err(o[sl], o_ref) <= TOL[torch.bfloat16], (b, h)
        assert rel_err(s[b:b + 1, h:h + 1], s_ref) <= TOL[torch.bfloat16], (b, h)


@pytest.mark.parametrize("name", ["config3", "config5b"])
def test_gated_prefill_full_size_sampled_chains(ctx, name):
    wl = workloads.WORKLOADS[name]
    q, k, v = workloads.make_qkv(wl)
    lam = workloads.make_gate(wl)
    o, s = ctx.lasad_forward_gated(q.cuda(), k.cuda(), v.cuda(), lam.cuda(), wl.grid_w, prefix_len=wl.prefix_len)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    o, s = o.cpu(), s.cpu()
    for b, h in _sampled_chains(wl, 5):
        sl = (slice(b, b + 1), slice(None), slice(h, h + 1))
        o_ref, s_ref = oracle(q[sl], k[sl], v[sl], lam[sl], wl.grid_w, wl.prefix_len)
        assert rel_err(o[sl], o_ref) <= TOL[torch.bfloat16], (b, h)
        assert rel_err(s[b:b + 1, h:h + 1], s_ref) <= TOL[torch.bfloat16], (b, h)


@pytest.mark.parametrize("name", ["config3", "config5b"])
def test_fused_prefill_full_size_sampled_chains(ctx, name):
    """The fused call (Algorithm 1's loop body: SiLU, Sigmoid, key tied to the gate, operator, RMS
    norm) as bench.py times it -- pre-activations q~ ~ N(0,1), gate~ ~ N(2,1), the workload's v --
    on sampled chains against the oracle's layer_core."""
    from oracle import lasad_oracle as orc
    from tests._util import to64
    wl = workloads.WORKLOADS[name]
    gen = torch.Generator().manual_seed(wl.seed + 11)
    qp = torch.randn(wl.B, wl.T, wl.H, wl.d, generator=gen).to(torch.bfloat16)
    gp = (torch.randn(wl.B, wl.T, wl.H, wl.d, generator=gen) + 2.0).to(torch.bfloat16)
    v = workloads.make_qkv(wl)[2]
    o, s = ctx.lasad_forward_fused(qp.cuda(), None, v.cuda(), gp.cuda(), wl.grid_w, prefix_len=wl.prefix_len)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    o, s = o.cpu(), s.cpu()
    for b, h in _sampled_chains(wl, 4):
        sl = (slice(b, b + 1), slice(None), slice(h, h + 1))
        o_ref, s_ref = orc.layer_core(to64(qp[sl]), None, to64(v[sl]), to64(gp[sl]), wl.grid_w, wl.prefix_len, 0, 1.0, None,
                                      1e-6)
        assert rel_err(o[sl], o_ref) <= TOL[torch.bfloat16], (b, h)
        assert rel_err(s[b:b + 1, h:h + 1], s_ref) <= TOL[torch.bfloat16], (b, h)


def test_decode_full_size_config4_sampled_chains(ctx):
    """Config 4 as the bench runs it: one prefill call for the class token, then one decode step per
    grid token (all 256 of them) on all 256 x 20 states; sampled chains against the oracle over the
    whole 257-token sequence."""
    wl = workloads.WORKLOADS["config4"]
    T = wl.T                                   # class token + all 256 grid positions
    q, k, v = workloads.make_qkv(wl, T)
    g = workloads.make_decay(wl)
    dq, dk, dv, dg = q.cuda(), k.cuda(), v.cuda(), g.cuda()
    P = wl.prefix_len
    o0, state = ctx.lasad_forward(dq[:, :P], dk[:, :P], dv[:, :P], dg, wl.grid_w, prefix_len=P)
    outs = [o0]
    for t in range(P, T):
        outs.append(ctx.lasad_decode_step(dq[:, t], dk[:, t], dv[:, t], dg, state, wl.grid_w, P, t).unsqueeze(1))
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    o, s = torch.cat(outs, 1).cpu(), state.cpu()
    for b, h in _sampled_chains(wl, 6):
        sl = (slice(b, b + 1), slice(None), slice(h, h + 1))
        o_ref, s_ref = oracle(q[sl], k[sl], v[sl], g[h:h + 1], wl.grid_w, P)
        assert rel_err(o[sl], o_ref) <= TOL[torch.bfloat16], (b, h)
        assert rel_err(s[b:b + 1, h:h + 1], s_ref) <= TOL[torch.bfloat16], (b, h)
