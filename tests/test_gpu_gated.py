"""GPU parity of the data-dependent (gated) form of the operator -- the paper's own decay, a
vector lambda_t per token (Algorithm 1), with the SAD rule -- against the CPU oracle run on the
same gate tensor.  Tolerances as for the constant-decay path."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2507_01652_b200 import binding, workloads
from tests._util import TOL, oracle, rel_err, to64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = binding.Lasad(0)
    yield c
    c.close()


def _dev(*ts):
    return [None if t is None else t.cuda() for t in ts]


def _inputs(seed, B, T, H, d, dtype, gate_lo=None):
    gen = torch.Generator().manual_seed(seed)
    q, k, v = [(torch.randn(B, T, H, d, generator=gen) / d ** 0.5).to(dtype) for _ in range(3)]
    lam = torch.sigmoid(torch.randn(B, T, H, d, generator=gen) + 2.0)
    if gate_lo is not None:        # a few hard zeros, ones and tiny gates
        sel = torch.rand(B, T, H, d, generator=gen)
        lam = torch.where(sel < 0.02, torch.zeros_like(lam), lam)
        lam = torch.where((sel >= 0.02) & (sel < 0.04), torch.ones_like(lam), lam)
        lam = torch.where((sel >= 0.04) & (sel < 0.06), torch.full_like(lam, gate_lo), lam)
    return q, k, v, lam.to(dtype)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("d", [32, 64])
@pytest.mark.parametrize("T,w,P", [(1, 4, 0), (16, 4, 0), (17, 5, 1), (100, 7, 0), (257, 16, 1), (300, 0, 0)])
def test_gated_prefill_matches_oracle(ctx, dtype, d, T, w, P):
    B, H = 2, 3
    q, k, v, lam = _inputs(500 + T + d, B, T, H, d, dtype)
    s_in = torch.randn(B, H, d, d, generator=torch.Generator().manual_seed(T))
    o_ref, s_ref = oracle(q, k, v, lam, w, P, 5, 0.5, s_in)
    o, s = ctx.lasad_forward_gated(*_dev(q, k, v, lam), w, prefix_len=P, t0=5, scale=0.5, state_in=s_in.cuda())
    torch.cuda.synchronize()
    assert rel_err(o, o_ref) <= TOL[dtype]
    assert rel_err(s, s_ref) <= TOL[dtype]


@pytest.mark.parametrize("T,w,P", [(1, 4, 0), (100, 7, 0), (128, 16, 0), (257, 16, 1), (700, 24, 0)])
def test_gated_prefill_both_implementations(ctx, T, w, P):
    """bf16, d = 64: the default, the CUDA-core kernel (option 1), the CTA-per-chain tensor-core kernel
    (option 2) and the balanced tensor-core kernel (option 5) against the oracle on the same inputs."""
    B, H, d = 3, 5, 64
    q, k, v, lam = _inputs(900 + T, B, T, H, d, torch.bfloat16)
    s_in = torch.randn(B, H, d, d, generator=torch.Generator().manual_seed(T))
    o_ref, s_ref = oracle(q, k, v, lam, w, P, 3, 0.25, s_in)
    for impl in (0, 1, 2, 5):
        ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, impl)
        try:
            o, s = ctx.lasad_forward_gated(*_dev(q, k, v, lam), w, prefix_len=P, t0=3, scale=0.25, state_in=s_in.cuda())
            torch.cuda.synchronize()
        finally:
            ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, 0)
        assert ctx.device_status() == 0
        assert rel_err(o, o_ref) <= TOL[torch.bfloat16], impl
        assert rel_err(s, s_ref) <= TOL[torch.bfloat16], impl


@pytest.mark.parametrize("impl", [2, 5])
@pytest.mark.parametrize("level,tied", [(0.35, False), (0.05, False), (0.003, True), (1e-5, False), (0.0, False)])
def test_gated_tensor_core_path_strong_decay(ctx, impl, level, tied):
    """Gates so small that a 128-token chunk cannot be scaled around one reference point: the
    tensor-core kernel cuts such chunks into segments of 64, 32, 16 or single tokens.  The middle
    chunk of three is the strong one, with exact zeros sprinkled in; the others are ordinary."""
    B, T, H, d, w = 2, 330, 3, 64, 11
    q, k, v, lam = _inputs(1200 + int(level * 1e6), B, T, H, d, torch.bfloat16)
    gen = torch.Generator().manual_seed(5)
    strong = torch.full((B, 128, H, d), level) * (1.0 + 0.3 * torch.rand(B, 128, H, d, generator=gen))
    strong = torch.where(torch.rand(B, 128, H, d, generator=gen) < 0.01, torch.zeros_like(strong), strong)
    lam[:, 128:256] = strong.to(torch.bfloat16)
    k_used = torch.from_numpy(1.0 - to64(lam)) if tied else k
    o_ref, s_ref = oracle(q, k_used, v, lam, w)
    ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, impl)
    try:
        o, s = ctx.lasad_forward_gated(q.cuda(), None if tied else k.cuda(), v.cuda(), lam.cuda(), w)
        torch.cuda.synchronize()
    finally:
        ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, 0)
    assert ctx.device_status() == 0
    assert torch.isfinite(o.float()).all() and torch.isfinite(s).all()
    assert rel_err(o, o_ref) <= TOL[torch.bfloat16]
    assert rel_err(s, s_ref) <= TOL[torch.bfloat16]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_gated_prefill_key_tied_to_gate(ctx, dtype):
    """k = NULL: the key is 1 - lambda (the paper's base decay lambda = 1 - k)."""
    B, T, H, d, w = 2, 150, 4, 64, 10
    q, _, v, lam = _inputs(77, B, T, H, d, dtype)
    k_ref = 1.0 - to64(lam)                    # from the gate the kernel sees, in fp64
    o_ref, s_ref = oracle(q, torch.from_numpy(k_ref), v, lam, w)
    o, s = ctx.lasad_forward_gated(q.cuda(), None, v.cuda(), lam.cuda(), w)
    torch.cuda.synchronize()
    assert rel_err(o, o_ref) <= TOL[dtype]
    assert rel_err(s, s_ref) <= TOL[dtype]


def test_gated_prefill_extreme_gates(ctx):
    """Gates of exactly 0 and 1 and tiny ones: nothing overflows, zeros cut the history."""
    B, T, H, d, w = 1, 90, 2, 32, 9
    q, k, v, lam = _inputs(78, B, T, H, d, torch.float32, gate_lo=1e-6)
    o_ref, s_ref = oracle(q, k, v, lam, w)
    o, s = ctx.lasad_forward_gated(*_dev(q, k, v, lam), w)
    torch.cuda.synchronize()
    assert torch.isfinite(o).all() and torch.isfinite(s).all()
    assert rel_err(o, o_ref) <= TOL[torch.float32]
    assert rel_err(s, s_ref) <= TOL[torch.float32]


def test_constant_gate_reduces_to_the_per_head_path(ctx):
    """A gate that is the same number everywhere in a head is the data-independent decay."""
    wl = workloads.WORKLOADS["config2"].scaled(B=2, H=4)
    q, k, v = workloads.make_qkv(wl)
    g = workloads.make_decay(wl)
    lam = g.view(1, 1, wl.H, 1).expand(wl.B, wl.T, wl.H, wl.d).to(torch.bfloat16).contiguous()
    g_seen = lam[0, 0, :, 0].float()           # the per-head value after rounding to bf16
    o_ref, s_ref = oracle(q, k, v, g_seen, wl.grid_w)
    o, s = ctx.lasad_forward_gated(*_dev(q, k, v, lam), wl.grid_w)
    o2, s2 = ctx.lasad_forward(*_dev(q, k, v, g_seen), wl.grid_w)
    torch.cuda.synchronize()
    assert rel_err(o, o_ref) <= TOL[torch.bfloat16] and rel_err(s, s_ref) <= TOL[torch.bfloat16]
    assert rel_err(o2, o_ref) <= TOL[torch.bfloat16] and rel_err(s2, s_ref) <= TOL[torch.bfloat16]


@pytest.mark.parametrize("dtype,d", [(torch.float32, 32), (torch.bfloat16, 64)])
@pytest.mark.parametrize("tied", [False, True])
def test_gated_decode_matches_oracle_and_prefill(ctx, dtype, d, tied):
    B, T, H, w, P = 2, 40, 3, 6, 1
    q, k, v, lam = _inputs(90 + d, B, T, H, d, dtype)
    k_used = torch.from_numpy(1.0 - to64(lam)) if tied else k
    o_ref, s_ref = oracle(q, k_used, v, lam, w, P)
    dq, dk_, dv_, dl = _dev(q, k, v, lam)
    state = torch.zeros(B, H, d, d, device="cuda")
    outs = []
    for t in range(T):
        outs.append(ctx.lasad_decode_step_gated(dq[:, t], None if tied else dk_[:, t], dv_[:, t], dl[:, t], state,
                                                w, P, t))
    torch.cuda.synchronize()
    assert rel_err(torch.stack(outs, 1), o_ref) <= TOL[dtype]
    assert rel_err(state, s_ref) <= TOL[dtype]
    _, s_pre = ctx.lasad_forward_gated(dq, None if tied else dk_, dv_, dl, w, prefix_len=P)
    torch.cuda.synchronize()
    assert rel_err(state, to64(s_pre)) <= TOL[dtype]


def test_gated_state_handoff(ctx):
    wl = dataclasses.replace(workloads.WORKLOADS["config3"], B=1, H=2)
    q, k, v = workloads.make_qkv(wl)
    lam = workloads.make_gate(wl)
    o_ref, s_ref = oracle(q, k, v, lam, wl.grid_w)
    dq, dk_, dv_, dl = _dev(q, k, v, lam)
    for m in (1, 37, 300):
        o1, s1 = ctx.lasad_forward_gated(dq[:, :m], dk_[:, :m], dv_[:, :m], dl[:, :m], wl.grid_w)
        o2, s2 = ctx.lasad_forward_gated(dq[:, m:], dk_[:, m:], dv_[:, m:], dl[:, m:], wl.grid_w, t0=m,
                                         state_in=s1, state_out=s1)
        torch.cuda.synchronize()
        assert rel_err(torch.cat([o1, o2], 1), o_ref) <= TOL[torch.bfloat16]
        assert rel_err(s2, s_ref) <= TOL[torch.bfloat16]


@pytest.mark.parametrize("impl", [2, 5])
def test_gated_dependent_calls_enqueued_without_a_synchronise_in_between(ctx, impl):
    """As the test of the same name for the scalar decay: the gated kernels (and the CUDA-core kernel
    launched behind them) are programmatic dependents of whatever precedes them; three calls on 160
    sequences, each from the state the call before leaves, with a gated decode step in between and
    nothing else on the stream."""
    B, H, T, d, w = 1, 160, 1501, 64, 11
    gen = torch.Generator().manual_seed(94)
    q, k, v = [(torch.randn(B, T, H, d, generator=gen) / 8).to(torch.bfloat16) for _ in range(3)]
    lam = torch.sigmoid(2.0 + torch.randn(B, T, H, d, generator=gen)).to(torch.bfloat16)
    o_ref, s_ref = oracle(q, k, v, lam, w)
    dq, dk_, dv_, dl = _dev(q, k, v, lam)
    a, b = 500, 1000
    o = torch.empty_like(dv_)
    s = torch.empty(B, H, d, d, device="cuda")
    ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, impl)
    try:
        for rep in range(2):
            ctx.lasad_forward_gated(dq[:, :a], dk_[:, :a], dv_[:, :a], dl[:, :a], w, o=o[:, :a], state_out=s)
            ctx.lasad_forward_gated(dq[:, a:b], dk_[:, a:b], dv_[:, a:b], dl[:, a:b], w, t0=a, o=o[:, a:b], state_in=s,
                                    state_out=s)
            ctx.lasad_decode_step_gated(dq[:, b], dk_[:, b], dv_[:, b], dl[:, b], s, w, 0, b, o=o[:, b])
            ctx.lasad_forward_gated(dq[:, b + 1:], dk_[:, b + 1:], dv_[:, b + 1:], dl[:, b + 1:], w, t0=b + 1,
                                    o=o[:, b + 1:], state_in=s, state_out=s)
            torch.cuda.synchronize()
            assert ctx.device_status() == 0
            assert rel_err(o, o_ref) <= TOL[torch.bfloat16], rep
            assert rel_err(s, s_ref) <= TOL[torch.bfloat16], rep
    finally:
        ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, 0)


@pytest.mark.parametrize("impl,H", [(2, 3), (5, 3), (5, 80)])
def test_gated_prefill_recorded_into_a_cuda_graph_and_replayed(ctx, impl, H):
    """Both launches of the gated prefill (tensor-core kernel, CUDA-core kernel for flagged chains)
    captured into a CUDA graph and replayed on new inputs; the second replay has a strong-decay
    stretch, so the replayed CUDA-core launch has chains to redo (and, with the balanced kernel and
    160 chains, chains that were given up on one CTA and finished on another)."""
    B, T, d, w = 2, (1100 if H > 3 else 300), 64, 10
    dq, dk, dv, dl = [torch.empty(B, T, H, d, dtype=torch.bfloat16, device="cuda") for _ in range(4)]
    o = torch.empty_like(dv)
    s = torch.empty(B, H, d, d, device="cuda")
    q, k, v, lam = _inputs(31, B, T, H, d, torch.bfloat16)
    for dst, src in ((dq, q), (dk, k), (dv, v), (dl, lam)):
        dst.copy_(src)
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, impl)
    try:
        with torch.cuda.stream(stream):
            ctx.lasad_forward_gated(dq, dk, dv, dl, w, o=o, state_out=s)     # warm-up outside the capture
            torch.cuda.synchronize()
            with torch.cuda.graph(graph, stream=stream):
                ctx.lasad_forward_gated(dq, dk, dv, dl, w, o=o, state_out=s)
    finally:
        ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, 0)
    for rep in range(3):
        q, k, v, lam = _inputs(32 + rep, B, T, H, d, torch.bfloat16)
        if rep == 1:
            lam[:, 130:250] = 0.004
        for dst, src in ((dq, q), (dk, k), (dv, v), (dl, lam)):
            dst.copy_(src)
        graph.replay()
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        o_ref, s_ref = oracle(q, k, v, lam, w)
        assert rel_err(o, o_ref) <= TOL[torch.bfloat16], rep
        assert rel_err(s, s_ref) <= TOL[torch.bfloat16], rep


@pytest.mark.parametrize("B,H,T,tied", [(1, 160, 1100, False), (2, 163, 700, True), (1, 151, 260, False), (1, 149, 2500, True)])
def test_gated_balanced_prefill_left_over_chains(ctx, B, H, T, tied):
    """The balanced gated kernel (option 5) with more chains than SMs: left-over chains cut into
    pieces whose state crosses CTAs; some heads with a decay too strong for the kernel's scaling in
    the second half of the sequence only, so that a chain is given up on one CTA after an earlier
    piece of it was taken normally, and the mark has to travel with the state; an incoming state,
    state_out aliasing state_in; twice in a row."""
    d, w = 64, 13
    q, k, v, lam = _inputs(2100 + H + T, B, T, H, d, torch.bfloat16)
    lam[:, T // 2:, 0] = 0.01
    lam[:, :, H - 1] = 0.02
    lam[:, T // 3:, H // 2] = 0.0
    k_used = torch.from_numpy(1.0 - to64(lam)) if tied else k
    s_in = torch.randn(B, H, d, d, generator=torch.Generator().manual_seed(T)) * 0.3
    o_ref, s_ref = oracle(q, k_used, v, lam, w, 1, 5, 0.5, s_in)
    dq, dk, dv, dl = _dev(q, k, v, lam)
    ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, 5)
    try:
        for rep in range(2):
            ds = s_in.cuda()
            o, s = ctx.lasad_forward_gated(dq, None if tied else dk, dv, dl, w, prefix_len=1, t0=5, scale=0.5,
                                           state_in=ds, state_out=ds)
            torch.cuda.synchronize()
            assert ctx.device_status() == 0
            assert rel_err(o, o_ref) <= TOL[torch.bfloat16], rep
            assert rel_err(s, s_ref) <= TOL[torch.bfloat16], rep
    finally:
        ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, 0)
