"""GPU parity of the fused entry points -- Algorithm 1's loop body as one call: SiLU on the query,
Sigmoid on the gate, key tied to the gate, the SAD recurrence, a weight-free RMS norm on the
output -- against the oracle's `layer_core`, which is written from Algorithm 1 and pinned on the CPU.
Tolerances as for the other paths (max|err| / max|ref|: 1e-4 fp32 I/O, 2e-2 bf16 I/O)."""
import numpy as np
import pytest
import torch

from oracle import lasad_oracle as orc
from paper_2507_01652_b200 import binding, workloads
from tests._util import TOL, rel_err, to64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = binding.Lasad(0)
    yield c
    c.close()


def _pre(seed, B, T, H, d, dtype, gate_shift=2.0, gate_scale=1.0):
    """Pre-activations: q~ ~ N(0,1), gate~ ~ N(shift, scale) (Sigmoid puts its mass near 1, where the
    forget gates of trained gated linear attention layers sit), v ~ N(0,1)/sqrt(d), key ~ N(0,1)/sqrt(d)."""
    gen = torch.Generator().manual_seed(seed)
    q = torch.randn(B, T, H, d, generator=gen).to(dtype)
    g = (gate_scale * torch.randn(B, T, H, d, generator=gen) + gate_shift).to(dtype)
    v = (torch.randn(B, T, H, d, generator=gen) / d ** 0.5).to(dtype)
    k = (torch.randn(B, T, H, d, generator=gen) / d ** 0.5).to(dtype)
    return q, k, v, g


def _oracle(q, k, v, g, w, P=0, t0=0, scale=1.0, s_in=None, eps=1e-6):
    return orc.layer_core(to64(q), to64(k), to64(v), to64(g), w, P, t0, scale, to64(s_in), eps)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("d", [32, 64])
@pytest.mark.parametrize("tied", [True, False])
@pytest.mark.parametrize("T,w,P", [(1, 4, 0), (17, 5, 1), (130, 7, 0), (300, 16, 1)])
def test_fused_prefill_matches_layer_core(ctx, dtype, d, tied, T, w, P):
    B, H = 2, 3
    q, k, v, g = _pre(700 + T + d, B, T, H, d, dtype)
    s_in = torch.randn(B, H, d, d, generator=torch.Generator().manual_seed(T)) * 0.2
    kk = None if tied else k
    o_ref, s_ref = _oracle(q, kk, v, g, w, P, 5, 0.5, s_in, 1e-5)
    o, s = ctx.lasad_forward_fused(q.cuda(), None if tied else k.cuda(), v.cuda(), g.cuda(), w, prefix_len=P, t0=5,
                                   scale=0.5, state_in=s_in.cuda(), norm_eps=1e-5)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    assert rel_err(o, o_ref) <= TOL[dtype]
    assert rel_err(s, s_ref) <= TOL[dtype]


@pytest.mark.parametrize("T,w", [(700, 24), (1153, 32)])
def test_fused_prefill_both_implementations_and_gates_close_to_one(ctx, T, w):
    """bf16, d = 64, several chunks: the tensor-core kernel (default) and the CUDA-core kernel
    (option 1) against the oracle; half of the heads get gate pre-activations around 7 (lambda
    within 1e-3 of 1: a memory of a thousand tokens, where a rounding of lambda itself to bf16
    would be felt), the others around 1."""
    B, H, d = 2, 4, 64
    q, k, v, g = _pre(1700 + T, B, T, H, d, torch.bfloat16)
    gen = torch.Generator().manual_seed(T)
    g[:, :, ::2] = (7.0 + 0.5 * torch.randn(B, T, H // 2, d, generator=gen)).to(torch.bfloat16)
    g[:, :, 1::2] = (1.0 + torch.randn(B, T, H // 2, d, generator=gen)).to(torch.bfloat16)
    o_ref, s_ref = _oracle(q, None, v, g, w, 0, 0, 1.0, None, 1e-6)
    for impl in (0, 1):
        ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, impl)
        try:
            o, s = ctx.lasad_forward_fused(q.cuda(), None, v.cuda(), g.cuda(), w)
            torch.cuda.synchronize()
        finally:
            ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, 0)
        assert ctx.device_status() == 0
        assert rel_err(o, o_ref) <= TOL[torch.bfloat16], impl
        assert rel_err(s, s_ref) <= TOL[torch.bfloat16], impl


@pytest.mark.parametrize("H,T,tied", [(160, 1100, True), (151, 1300, False)])
def test_fused_balanced_prefill_with_states_crossing_ctas(ctx, H, T, tied):
    """The fused form on the balanced kernel (option 5) with more chains than SMs: left-over chains
    are cut into pieces whose state crosses CTAs; an incoming state, a prefix token, a start in
    mid-row; twice in a row (the hand-off packets of the first call must not pass for the second's)."""
    B, d, w = 1, 64, 11
    q, k, v, g = _pre(2300 + H, B, T, H, d, torch.bfloat16)
    s_in = torch.randn(B, H, d, d, generator=torch.Generator().manual_seed(H)) * 0.2
    o_ref, s_ref = _oracle(q, None if tied else k, v, g, w, 1, 7, 0.5, s_in, 1e-6)
    dq, dk, dv, dg, ds = q.cuda(), (None if tied else k.cuda()), v.cuda(), g.cuda(), s_in.cuda()
    ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, 5)
    try:
        for rep in range(2):
            o, s = ctx.lasad_forward_fused(dq, dk, dv, dg, w, prefix_len=1, t0=7, scale=0.5, state_in=ds)
            torch.cuda.synchronize()
            assert ctx.device_status() == 0
            assert rel_err(o, o_ref) <= TOL[torch.bfloat16], rep
            assert rel_err(s, s_ref) <= TOL[torch.bfloat16], rep
    finally:
        ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, 0)


def test_fused_prefill_strong_decay_takes_the_exact_path(ctx):
    """Gate pre-activations far below zero (lambda down to e^-20): the tensor-core kernel gives such
    chains up and the CUDA-core kernel behind it computes them; the entry point stays exact."""
    B, T, H, d, w = 2, 300, 3, 64, 10
    q, k, v, g = _pre(1800, B, T, H, d, torch.bfloat16)
    g[:, :, 0] = -20.0
    g[:, :, 1] = (-3.0 + torch.randn(B, T, d, generator=torch.Generator().manual_seed(5))).to(torch.bfloat16)
    o_ref, s_ref = _oracle(q, None, v, g, w)
    o, s = ctx.lasad_forward_fused(q.cuda(), None, v.cuda(), g.cuda(), w)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    assert rel_err(o, o_ref) <= TOL[torch.bfloat16]
    assert rel_err(s, s_ref) <= TOL[torch.bfloat16]


@pytest.mark.parametrize("dtype,d", [(torch.float32, 32), (torch.bfloat16, 64)])
def test_fused_decode_equals_fused_prefill(ctx, dtype, d):
    """T fused decode steps give the outputs and the final state of one fused prefill, and both match
    the oracle (the decode state after N steps = the prefill's final state)."""
    B, T, H, w, P = 2, 40, 3, 6, 1
    q, k, v, g = _pre(1900 + d, B, T, H, d, dtype)
    o_ref, s_ref = _oracle(q, None, v, g, w, P, 0, 1.0, None, 1e-6)
    dq, dv, dg = q.cuda(), v.cuda(), g.cuda()
    o_pre, s_pre = ctx.lasad_forward_fused(dq, None, dv, dg, w, prefix_len=P)
    state = torch.zeros(B, H, d, d, device="cuda")
    outs = [ctx.lasad_decode_step_fused(dq[:, t], None, dv[:, t], dg[:, t], state, w, P, t) for t in range(T)]
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    o_dec = torch.stack(outs, 1)
    for o, s in ((o_pre, s_pre), (o_dec, state)):
        assert rel_err(o, o_ref) <= TOL[dtype]
        assert rel_err(s, s_ref) <= TOL[dtype]


def test_fused_equals_the_unfused_sequence(ctx):
    """One fused call against torch's element-wise kernels around lasad_forward_gated (fp32 I/O, so
    that the intermediate tensors of the unfused sequence lose nothing): same numbers."""
    B, T, H, d, w = 2, 150, 3, 32, 8
    q, k, v, g = _pre(2000, B, T, H, d, torch.float32)
    dq, dv, dg = q.cuda(), v.cuda(), g.cuda()
    o_f, s_f = ctx.lasad_forward_fused(dq, None, dv, dg, w, norm_eps=1e-6)
    lam = torch.sigmoid(dg)
    o_u, s_u = ctx.lasad_forward_gated(torch.nn.functional.silu(dq), 1.0 - lam, dv, lam, w)
    o_u = o_u * torch.rsqrt(o_u.pow(2).mean(-1, keepdim=True) + 1e-6)
    torch.cuda.synchronize()
    assert rel_err(o_f, to64(o_u)) <= 1e-4
    assert rel_err(s_f, to64(s_u)) <= 1e-4


def test_fused_argument_errors(ctx):
    q = torch.zeros(1, 8, 2, 64, dtype=torch.bfloat16, device="cuda")
    n0 = ctx.launch_count
    with pytest.raises(binding.LasadError) as e:
        ctx.lasad_forward_fused(q, None, q, q, 4, norm_eps=-1.0)
    assert e.value.code == binding.LASAD_ERR_INVALID_ARG
    with pytest.raises(binding.LasadError) as e:
        ctx.lasad_forward_fused(q, None, q, q, 4, norm_eps=float("nan"))
    assert e.value.code == binding.LASAD_ERR_INVALID_ARG
    assert ctx.launch_count == n0
