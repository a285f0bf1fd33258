"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle.

Tolerances (max|err| / max|ref| over the whole tensor): 1e-4 for fp32 I/O, 2e-2 for bf16 I/O
with fp32 accumulation; the same bounds for the fp32 state.
"""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2507_01652_b200 import binding, workloads
from tests._util import TOL, oracle, rel_err, to64

pytestmark = pytest.mark.gpu

IMPLS = [1, 2, 3, 4, 5]  # 1 = CUDA-core fp32 kernel, 2 = tcgen05 kernel (CTA per chain), 3 = tcgen05 task-streaming kernel,
                      # 4 = as 2, few long chains cut into segments


@pytest.fixture(scope="module")
def ctx():
    c = binding.Lasad(0)
    yield c
    c.close()


def _dev(*ts):
    return [None if t is None else t.cuda() for t in ts]


def _supported(impl, dtype, d):
    return impl == 1 or (dtype == torch.bfloat16 and d == 64)


def _forward(ctx, impl, *args, chunk=0, **kw):
    ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, impl)
    ctx.set_option(binding.LASAD_OPT_PREFILL_CHUNK, chunk)
    try:
        out = ctx.lasad_forward(*args, **kw)
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        return out
    finally:
        ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, 0)
        ctx.set_option(binding.LASAD_OPT_PREFILL_CHUNK, 0)


def _small(name, B, H):
    return workloads.WORKLOADS[name].scaled(B=B, H=H)


# ------------------------------------------------------------------------------------------
# config 1 in full: fp32 prefill, 256 decode steps, state agreement
# ------------------------------------------------------------------------------------------
def test_config1_prefill_and_decode_full(ctx):
    wl = workloads.WORKLOADS["config1"]
    q, k, v = workloads.make_qkv(wl)
    g = workloads.make_decay(wl)
    o_ref, s_ref = oracle(q, k, v, g, wl.grid_w, form="recurrent")
    o_quad, s_quad = oracle(q, k, v, g, wl.grid_w, form="quadratic")
    np.testing.assert_allclose(o_ref, o_quad, rtol=1e-10, atol=1e-12)
    dq, dk_, dv_, dg = _dev(q, k, v, g)
    o, s = _forward(ctx, 1, dq, dk_, dv_, dg, wl.grid_w)
    assert rel_err(o, o_ref) <= TOL[torch.float32]
    assert rel_err(s, s_ref) <= TOL[torch.float32]
    # decode from the zero state, token by token
    state = torch.zeros(wl.B, wl.H, wl.d, wl.d, device="cuda")
    outs = []
    for t in range(wl.T):
        outs.append(ctx.lasad_decode_step(dq[:, t], dk_[:, t], dv_[:, t], dg, state, wl.grid_w, 0, t))
    torch.cuda.synchronize()
    od = torch.stack(outs, 1)
    assert rel_err(od, o_ref) <= TOL[torch.float32]
    assert rel_err(state, s_ref) <= TOL[torch.float32]
    # decode state after N steps equals prefill's final state
    assert rel_err(state, to64(s)) <= TOL[torch.float32]


# ------------------------------------------------------------------------------------------
# the bf16 configurations at oracle-sized batch, every prefill kernel
# ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("name,B,H", [("config2", 2, 12), ("config3", 2, 4), ("config4", 3, 5),
                                      ("config5a", 1, 2)])
def test_bf16_configs_prefill(ctx, impl, name, B, H):
    wl = _small(name, B, H)
    q, k, v = workloads.make_qkv(wl)
    g = workloads.make_decay(wl)
    o_ref, s_ref = oracle(q, k, v, g, wl.grid_w, wl.prefix_len)
    o, s = _forward(ctx, impl, *_dev(q, k, v, g), wl.grid_w, prefix_len=wl.prefix_len)
    assert rel_err(o, o_ref) <= TOL[torch.bfloat16]
    assert rel_err(s, s_ref) <= TOL[torch.bfloat16]


@pytest.mark.parametrize("name,B,H", [("config2", 2, 12), ("config4", 2, 20)])
def test_bf16_decode_sweep_matches_oracle_and_prefill(ctx, name, B, H):
    wl = _small(name, B, H)
    q, k, v = workloads.make_qkv(wl)
    g = workloads.make_decay(wl)
    o_ref, s_ref = oracle(q, k, v, g, wl.grid_w, wl.prefix_len)
    dq, dk_, dv_, dg = _dev(q, k, v, g)
    P = wl.prefix_len
    # class-token prefix through prefill (T = P), then one decode step per grid token
    if P:
        o0, state = _forward(ctx, 1, dq[:, :P], dk_[:, :P], dv_[:, :P], dg, wl.grid_w, prefix_len=P)
        assert rel_err(o0, o_ref[:, :P]) <= TOL[torch.bfloat16]
    else:
        state = torch.zeros(wl.B, wl.H, wl.d, wl.d, device="cuda")
    outs = []
    for t in range(P, wl.T):
        outs.append(ctx.lasad_decode_step(dq[:, t], dk_[:, t], dv_[:, t], dg, state, wl.grid_w, P, t))
    torch.cuda.synchronize()
    od = torch.stack(outs, 1)
    assert rel_err(od, o_ref[:, P:]) <= TOL[torch.bfloat16]
    assert rel_err(state, s_ref) <= TOL[torch.bfloat16]
    for impl in IMPLS:
        _, s_pre = _forward(ctx, impl, dq, dk_, dv_, dg, wl.grid_w, prefix_len=P)
        assert rel_err(state, to64(s_pre)) <= TOL[torch.bfloat16]


# ------------------------------------------------------------------------------------------
# ragged lengths, several tiles, both head sizes, both dtypes, every chunk size
# ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("d", [32, 64])
@pytest.mark.parametrize("T,w,P", [(1, 4, 0), (2, 2, 0), (3, 1, 0), (17, 5, 0), (64, 8, 0),
                                   (100, 7, 1), (129, 16, 0), (257, 16, 1), (300, 0, 0), (391, 23, 3)])
def test_ragged_shapes(ctx, impl, dtype, d, T, w, P):
    if not _supported(impl, dtype, d):
        pytest.skip("tensor-core prefill covers bf16, d = 64")
    gen = torch.Generator().manual_seed(1000 + T + d)
    B, H = 2, 3
    q, k, v = [(torch.randn(B, T, H, d, generator=gen) / d ** 0.5).to(dtype) for _ in range(3)]
    g = torch.tensor([0.8, 0.95, 0.999])
    s_in = torch.randn(B, H, d, d, generator=gen)
    o_ref, s_ref = oracle(q, k, v, g, w, P, 5, 0.5, s_in)
    for chunk in ([0, 16, 32, 64] if impl == 1 else [0]):
        o, s = _forward(ctx, impl, *_dev(q, k, v, g), w, prefix_len=P, t0=5, scale=0.5,
                        state_in=s_in.cuda(), chunk=chunk)
        assert rel_err(o, o_ref) <= TOL[dtype], f"chunk {chunk}"
        assert rel_err(s, s_ref) <= TOL[dtype], f"chunk {chunk}"


@pytest.mark.parametrize("impl", IMPLS)
def test_decay_edge_cases(ctx, impl):
    """gamma = 0 (state wiped except across boundary steps), gamma = 1 (plain causal linear
    attention), and a mix, on a grid whose rows straddle chunk borders."""
    B, T, H, d, w = 1, 150, 4, 64, 9
    gen = torch.Generator().manual_seed(7)
    q, k, v = [(torch.randn(B, T, H, d, generator=gen) / 8).to(torch.bfloat16) for _ in range(3)]
    g = torch.tensor([0.0, 1.0, 0.5, 0.9999])
    o_ref, s_ref = oracle(q, k, v, g, w)
    o, s = _forward(ctx, impl, *_dev(q, k, v, g), w)
    assert torch.isfinite(o.float()).all() and torch.isfinite(s).all()
    for h in range(H):
        assert rel_err(o[:, :, h], o_ref[:, :, h]) <= TOL[torch.bfloat16], f"head {h}"
        assert rel_err(s[:, h], s_ref[:, h]) <= TOL[torch.bfloat16], f"head {h}"


@pytest.mark.parametrize("impl", IMPLS)
def test_state_handoff_mid_row(ctx, impl):
    """forward(0..T) == forward(0..m) then forward(m..T) from the carried state (t0 = m)."""
    wl = _small("config3", 1, 3)
    q, k, v = workloads.make_qkv(wl)
    g = workloads.make_decay(wl)
    dq, dk_, dv_, dg = _dev(q, k, v, g)
    o_ref, s_ref = oracle(q, k, v, g, wl.grid_w)
    for m in (1, 37, 128, 300, 575):
        o1, s1 = _forward(ctx, impl, dq[:, :m], dk_[:, :m], dv_[:, :m], dg, wl.grid_w)
        o2, s2 = _forward(ctx, impl, dq[:, m:], dk_[:, m:], dv_[:, m:], dg, wl.grid_w, t0=m, state_in=s1,
                          state_out=s1)  # in-place state
        assert rel_err(torch.cat([o1, o2], 1), o_ref) <= TOL[torch.bfloat16]
        assert rel_err(s2, s_ref) <= TOL[torch.bfloat16]


@pytest.mark.parametrize("impl", [1, 2, 5])
def test_dependent_calls_enqueued_without_a_synchronise_in_between(ctx, impl):
    """The kernels are launched as programmatic dependents: a call's CTAs may come onto the SMs while
    the call before it is still running, and must wait for it before they read what it wrote.  Three
    calls are enqueued back to back on one stream with nothing in between -- the first third of 160
    sequences, the second third from the state the first call leaves (in place), then one decode
    step per sequence on that state, and the last third -- large enough for each call to find its
    predecessor still at work; outputs and final state against the oracle on the whole sequence."""
    B, H, T, d, w = 1, 160, 2101, 64, 11
    gen = torch.Generator().manual_seed(93)
    q, k, v = [(torch.randn(B, T, H, d, generator=gen) / 8).to(torch.bfloat16) for _ in range(3)]
    g = 0.9 + 0.0999 * torch.rand(H, generator=gen)
    o_ref, s_ref = oracle(q, k, v, g, w)
    dq, dk, dv, dg = _dev(q, k, v, g)
    a, b = 700, 1400
    o = torch.empty_like(dv)
    s = torch.empty(B, H, d, d, device="cuda")
    ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, impl)
    try:
        for rep in range(2):
            ctx.lasad_forward(dq[:, :a], dk[:, :a], dv[:, :a], dg, w, o=o[:, :a], state_out=s)
            ctx.lasad_forward(dq[:, a:b], dk[:, a:b], dv[:, a:b], dg, w, t0=a, o=o[:, a:b], state_in=s, state_out=s)
            ctx.lasad_decode_step(dq[:, b], dk[:, b], dv[:, b], dg, s, w, 0, b, o=o[:, b])
            ctx.lasad_forward(dq[:, b + 1:], dk[:, b + 1:], dv[:, b + 1:], dg, w, t0=b + 1, o=o[:, b + 1:], state_in=s,
                              state_out=s)
            torch.cuda.synchronize()
            assert ctx.device_status() == 0
            assert rel_err(o, o_ref) <= TOL[torch.bfloat16], rep
            assert rel_err(s, s_ref) <= TOL[torch.bfloat16], rep
    finally:
        ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, 0)


@pytest.mark.parametrize("impl", IMPLS)
def test_head_major_layout_through_strides(ctx, impl):
    """[B,H,T,d] storage viewed as [B,T,H,d]: only the strides change."""
    B, T, H, d, w = 2, 96, 3, 64, 12
    gen = torch.Generator().manual_seed(11)
    q, k, v = [(torch.randn(B, H, T, d, generator=gen) / 8).to(torch.bfloat16).cuda().transpose(1, 2)
               for _ in range(3)]
    g = torch.tensor([0.9, 0.99, 0.7])
    o_ref, _ = oracle(q, k, v, g, w)
    o_store = torch.empty(B, H, T, d, dtype=torch.bfloat16, device="cuda").transpose(1, 2)
    o, _ = _forward(ctx, impl, q, k, v, g.cuda(), w, o=o_store)
    assert not q.is_contiguous()
    assert rel_err(o, o_ref) <= TOL[torch.bfloat16]


@pytest.mark.parametrize("impl", IMPLS)
def test_outputs_stay_inside_their_buffers_and_are_deterministic(ctx, impl):
    B, T, H, d, w = 2, 77, 3, 64, 8
    gen = torch.Generator().manual_seed(12)
    q, k, v = [(torch.randn(B, T, H, d, generator=gen) / 8).to(torch.bfloat16).cuda() for _ in range(3)]
    g = torch.tensor([0.9, 0.99, 0.7]).cuda()
    pad = 4096
    obuf = torch.full((B * T * H * d + 2 * pad,), 7.0, dtype=torch.bfloat16, device="cuda")
    sbuf = torch.full((B * H * d * d + 2 * pad,), 7.0, dtype=torch.float32, device="cuda")
    o = obuf[pad:-pad].view(B, T, H, d)
    s = sbuf[pad:-pad].view(B, H, d, d)
    _forward(ctx, impl, q, k, v, g, w, o=o, state_out=s)
    assert (obuf[:pad] == 7).all() and (obuf[-pad:] == 7).all()
    assert (sbuf[:pad] == 7).all() and (sbuf[-pad:] == 7).all()
    o2, s2 = _forward(ctx, impl, q, k, v, g, w)
    assert torch.equal(o, o2) and torch.equal(s, s2)


def test_decode_every_thread_mapping(ctx):
    B, H, w = 3, 5, 4
    gen = torch.Generator().manual_seed(13)
    for dtype in (torch.float32, torch.bfloat16):
        for d in (32, 64):
            q, k, v = [(torch.randn(B, 1, H, d, generator=gen) / d ** 0.5).to(dtype) for _ in range(3)]
            g = torch.rand(H, generator=gen)
            s_in = torch.randn(B, H, d, d, generator=gen)
            for t in (2, 3):  # t = 3 is a boundary step for w = 4
                o_ref, s_ref = oracle(q, k, v, g, w, 0, t, 0.25, s_in)
                for tpu in (0, 32, 64, 128, 256):
                    ctx.set_option(binding.LASAD_OPT_DECODE_TPU, tpu)
                    state = s_in.clone().cuda()
                    dq, dk_, dv_, dg = _dev(q[:, 0], k[:, 0], v[:, 0], g)
                    o = ctx.lasad_decode_step(dq, dk_, dv_, dg, state, w, 0, t, scale=0.25)
                    torch.cuda.synchronize()
                    assert rel_err(o, o_ref[:, 0]) <= TOL[dtype]
                    assert rel_err(state, s_ref) <= 1e-6
    ctx.set_option(binding.LASAD_OPT_DECODE_TPU, 0)


def test_argument_errors_launch_nothing(ctx):
    B, T, H, d = 1, 8, 2, 64
    q = torch.zeros(B, T, H, d, dtype=torch.bfloat16, device="cuda")
    g = torch.ones(H, device="cuda")
    n0 = ctx.launch_count
    with pytest.raises(binding.LasadError) as e:
        ctx.lasad_forward(q, q, q, g, -1)
    assert e.value.code == binding.LASAD_ERR_INVALID_ARG
    q48 = torch.zeros(B, T, H, 48, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.LasadError) as e:
        ctx.lasad_forward(q48, q48, q48, g, 4)
    assert e.value.code == binding.LASAD_ERR_UNSUPPORTED
    with pytest.raises(binding.LasadError) as e:  # misaligned base pointer
        flat = torch.zeros(B * T * H * d + 8, dtype=torch.bfloat16, device="cuda")
        qm = flat[1:1 + B * T * H * d].view(B, T, H, d)
        ctx.lasad_forward(qm, q, q, g, 4)
    assert e.value.code == binding.LASAD_ERR_INVALID_ARG
    with pytest.raises(ValueError):
        ctx.lasad_forward(q.cpu(), q, q, g, 4)
    # a zero stride over a dimension with more than one element (a broadcast view) is refused
    qb = torch.zeros(1, T, H, d, dtype=torch.bfloat16, device="cuda").expand(3, T, H, d)
    q3 = torch.zeros(3, T, H, d, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.LasadError) as e:
        ctx.lasad_forward(qb, q3, q3, g, 4)
    assert e.value.code == binding.LASAD_ERR_INVALID_ARG
    assert ctx.launch_count == n0


# ------------------------------------------------------------------------------------------
# task-streaming prefill (implementation 3): paths the shared cases above do not reach
# ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("T", [100, 129, 300])
def test_more_chains_than_resident_ctas(ctx, T):
    """More (batch, head) pairs than CTAs that fit on the device: the CTA-per-chain kernel keeps its
    CTAs and hands them further chains from its work counter.  Heads on the normal and on the exact
    path alternate (a CTA changes path from one chain to the next), with an incoming state; the call
    is repeated, so the counter must have returned to zero."""
    B, H, d, w = 47, 13, 64, 7
    gen = torch.Generator().manual_seed(300 + T)
    q, k, v = [(torch.randn(B, T, H, d, generator=gen) / 8).to(torch.bfloat16) for _ in range(3)]
    g = torch.tensor([0.95, 0.0, 0.999, 0.3, 0.6, 0.59, 1.0, 0.9, 0.5, 0.97, 0.2, 0.99, 0.8])
    s_in = torch.randn(B, H, d, d, generator=gen)
    o_ref, s_ref = oracle(q, k, v, g, w, 0, 3, 0.5, s_in)
    dq, dk, dv, dg, ds = _dev(q, k, v, g, s_in)
    for rep in range(2):
        o, s = _forward(ctx, 2, dq, dk, dv, dg, w, t0=3, scale=0.5, state_in=ds)
        assert rel_err(o, o_ref) <= TOL[torch.bfloat16], rep
        assert rel_err(s, s_ref) <= TOL[torch.bfloat16], rep
    # a smaller call afterwards (fewer chains than CTAs) starts from a clean counter as well
    o, s = _forward(ctx, 2, dq[:2], dk[:2], dv[:2], dg, w, t0=3, scale=0.5, state_in=ds[:2])
    assert rel_err(o, o_ref[:2]) <= TOL[torch.bfloat16]
    assert rel_err(s, s_ref[:2]) <= TOL[torch.bfloat16]


@pytest.mark.parametrize("B,H,T", [(1, 5, 2000), (2, 12, 1500), (1, 1, 9216), (3, 16, 1153)])
def test_few_long_chains_cut_into_segments(ctx, B, H, T):
    """Implementation 4: a first launch gets every segment's own contribution to the state from K and
    V and a scan hands every segment its starting state; a second launch runs the segments side by side.
    Ragged last chunk, heads on both decay paths, an incoming state, a prefix token, a start in
    mid-row, state_out aliasing state_in; twice in a row."""
    d, w = 64, 13
    gen = torch.Generator().manual_seed(900 + T)
    q, k, v = [(torch.randn(B, T, H, d, generator=gen) / 8).to(torch.bfloat16) for _ in range(3)]
    g = 0.9 + 0.0999 * torch.rand(H, generator=gen)
    g[0] = 0.45
    if H > 3:
        g[1], g[2], g[3] = 0.0, 1.0, 0.59
    s_in = torch.randn(B, H, d, d, generator=gen)
    o_ref, s_ref = oracle(q, k, v, g, w, 1, 5, 0.5, s_in)
    dq, dk, dv, dg = _dev(q, k, v, g)
    for rep in range(2):
        ds = s_in.cuda()
        o, s = _forward(ctx, 4, dq, dk, dv, dg, w, prefix_len=1, t0=5, scale=0.5, state_in=ds, state_out=ds)
        assert rel_err(o, o_ref) <= TOL[torch.bfloat16], rep
        assert rel_err(s, s_ref) <= TOL[torch.bfloat16], rep


def test_default_prefill_picks_a_kernel_by_the_number_of_chains(ctx):
    """Option 0: few (batch, head) pairs with several chunks each go to the task-streaming kernel,
    long sequences that do not fill whole rounds of CTA slots to the balanced kernel, everything else
    in bf16 / d = 64 to the CTA-per-chain kernel; whichever runs, the result is that kernel's bit for
    bit, and right."""
    d, w = 64, 12
    gen = torch.Generator().manual_seed(4242)
    g_all = 0.9 + 0.0999 * torch.rand(100, generator=gen)
    for B, H, T, expect in ((1, 16, 700, 3), (12, 16, 700, 2), (1, 100, 4000, 5)):
        q, k, v = [(torch.randn(B, T, H, d, generator=gen) / 8).to(torch.bfloat16) for _ in range(3)]
        g = g_all[:H]
        o_ref, s_ref = oracle(q, k, v, g, w)
        dq, dk, dv, dg = _dev(q, k, v, g)
        o0, s0 = _forward(ctx, 0, dq, dk, dv, dg, w)
        o1, s1 = _forward(ctx, expect, dq, dk, dv, dg, w)
        assert torch.equal(o0, o1) and torch.equal(s0, s1), (B, H)
        assert rel_err(o0, o_ref) <= TOL[torch.bfloat16]
        assert rel_err(s0, s_ref) <= TOL[torch.bfloat16]


@pytest.mark.parametrize("B,H,T", [(1, 160, 1100), (2, 163, 1100), (1, 151, 260), (40, 5, 130), (1, 149, 2500),
                                   (3, 7, 900), (1, 150, 100), (2, 148, 300)])
def test_balanced_prefill_left_over_chains_cut_into_pieces(ctx, B, H, T):
    """Implementation 5 with more chains than SMs: every CTA takes whole chains in rounds and one
    piece of a left-over chain, whose state travels from CTA to CTA (pieces of 4 chunks, two or three
    to a chain, some shares straddling two chains: 160 x 9 chunks; two rounds: 326 chains; chains too
    short to be cut: 1, 2 and 3 chunks; one long left-over chain over many CTAs: 149 x 20 chunks;
    whole rounds with nothing left over: 296 chains), and with fewer chains than SMs (one chain per CTA).  Heads on both decay paths, an incoming state, a
    prefix token, a start in mid-row, state_out aliasing state_in; twice in a row (the packet tags
    must tell the launches apart)."""
    d, w = 64, 13
    gen = torch.Generator().manual_seed(1200 + H + T)
    q, k, v = [(torch.randn(B, T, H, d, generator=gen) / 8).to(torch.bfloat16) for _ in range(3)]
    g = 0.9 + 0.0999 * torch.rand(H, generator=gen)
    g[0], g[1], g[2], g[3] = 0.45, 0.0, 1.0, 0.59
    g[H - 1] = 0.3
    s_in = torch.randn(B, H, d, d, generator=gen)
    o_ref, s_ref = oracle(q, k, v, g, w, 1, 5, 0.5, s_in)
    dq, dk, dv, dg = _dev(q, k, v, g)
    for rep in range(2):
        ds = s_in.cuda()
        o, s = _forward(ctx, 5, dq, dk, dv, dg, w, prefix_len=1, t0=5, scale=0.5, state_in=ds, state_out=ds)
        assert rel_err(o, o_ref) <= TOL[torch.bfloat16], rep
        assert rel_err(s, s_ref) <= TOL[torch.bfloat16], rep


def test_expired_wait_while_states_cross_ctas_is_reported_and_the_next_call_is_right(ctx):
    """Implementation 5 on 160 chains of 9 chunks (left-over chains in pieces, their states handed
    from CTA to CTA) with the poll limit of the device-side waits set to 1: some wait -- on a barrier
    or on a hand-off packet -- runs out, every CTA must still leave through its normal exit (so the
    launch counters are put back), the status word must say so, and the next call with the default
    limit must be correct: the packets the aborted launch left behind carry its tag, not the next one's."""
    B, H, T, d, w = 1, 160, 1100, 64, 9
    gen = torch.Generator().manual_seed(81)
    q, k, v = [(torch.randn(B, T, H, d, generator=gen) / 8).to(torch.bfloat16) for _ in range(3)]
    g = 0.9 + 0.0999 * torch.rand(H, generator=gen)
    o_ref, s_ref = oracle(q, k, v, g, w)
    dq, dk, dv, dg = _dev(q, k, v, g)
    ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, 5)
    try:
        ctx.set_option(binding.LASAD_OPT_WAIT_LIMIT, 1)
        ctx.lasad_forward(dq, dk, dv, dg, w)
        torch.cuda.synchronize()
        assert ctx.device_status() == binding.LASAD_ERR_TIMEOUT
        ctx.set_option(binding.LASAD_OPT_WAIT_LIMIT, 0)
        for rep in range(2):
            o, s = ctx.lasad_forward(dq, dk, dv, dg, w)
            torch.cuda.synchronize()
            assert ctx.device_status() == 0, rep
            assert rel_err(o, o_ref) <= TOL[torch.bfloat16], rep
            assert rel_err(s, s_ref) <= TOL[torch.bfloat16], rep
    finally:
        ctx.set_option(binding.LASAD_OPT_WAIT_LIMIT, 0)
        ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, 0)


def test_balanced_prefill_recorded_into_a_cuda_graph_and_replayed(ctx):
    """Implementation 5 numbers its launches on the device, so a recorded launch may be replayed: the
    hand-off packets of one replay must not pass for the next one's (160 chains of 9 chunks: the
    left-over chains' states cross CTAs)."""
    B, H, T, d, w = 1, 160, 1100, 64, 9
    gen = torch.Generator().manual_seed(78)
    g = 0.9 + 0.0999 * torch.rand(H, generator=gen)
    dg = g.cuda()
    dq, dk, dv = [torch.empty(B, T, H, d, dtype=torch.bfloat16, device="cuda") for _ in range(3)]
    o = torch.empty_like(dv)
    s = torch.empty(B, H, d, d, device="cuda")
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, 5)
    try:
        with torch.cuda.stream(stream):
            ctx.lasad_forward(dq, dk, dv, dg, w, o=o, state_out=s)          # warm-up outside the capture
            torch.cuda.synchronize()
            with torch.cuda.graph(graph, stream=stream):
                ctx.lasad_forward(dq, dk, dv, dg, w, o=o, state_out=s)
    finally:
        ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, 0)
    for rep in range(3):
        q, k, v = [(torch.randn(B, T, H, d, generator=gen) / 8).to(torch.bfloat16) for _ in range(3)]
        dq.copy_(q); dk.copy_(k); dv.copy_(v)
        graph.replay()
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        o_ref, s_ref = oracle(q, k, v, g, w)
        assert rel_err(o, o_ref) <= TOL[torch.bfloat16], rep
        assert rel_err(s, s_ref) <= TOL[torch.bfloat16], rep


@pytest.mark.parametrize("T", [700, 2300])
def test_prefill_recorded_into_a_cuda_graph_and_replayed(ctx, T):
    """A prefill call captured into a CUDA graph and replayed on new inputs.  With few chains the
    default would take the task-streaming kernel (T = 700), whose packets carry a host-side launch
    number; under capture it must fall back, and asking for that kernel by option must be refused.
    T = 2300 records the two launches of the segment-parallel mode."""
    B, H, d, w = 1, 4, 64, 9
    gen = torch.Generator().manual_seed(77 + T)
    g = torch.tensor([0.93, 0.5, 0.999, 0.97])
    dg = g.cuda()
    dq, dk, dv = [torch.empty(B, T, H, d, dtype=torch.bfloat16, device="cuda") for _ in range(3)]
    o = torch.empty_like(dv)
    s = torch.empty(B, H, d, d, device="cuda")
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        ctx.lasad_forward(dq, dk, dv, dg, w, o=o, state_out=s)          # warm-up outside the capture
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=stream):
            ctx.lasad_forward(dq, dk, dv, dg, w, o=o, state_out=s)
            ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, 3)
            try:
                with pytest.raises(binding.LasadError):
                    ctx.lasad_forward(dq, dk, dv, dg, w, o=o, state_out=s)
            finally:
                ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, 0)
    for rep in range(3):
        q, k, v = [(torch.randn(B, T, H, d, generator=gen) / 8).to(torch.bfloat16) for _ in range(3)]
        dq.copy_(q); dk.copy_(k); dv.copy_(v)
        graph.replay()
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        o_ref, s_ref = oracle(q, k, v, g, w)
        assert rel_err(o, o_ref) <= TOL[torch.bfloat16], rep
        assert rel_err(s, s_ref) <= TOL[torch.bfloat16], rep


def test_streaming_prefill_many_heads_and_relay_growth(ctx):
    """More heads than the kernel's shared-memory decay cache holds (H > 256) and more (batch,
    head) pairs than the context's initial relay storage (B * H > 1024, so the call grows it)."""
    B, T, H, d, w = 4, 300, 260, 64, 10
    gen = torch.Generator().manual_seed(31)
    q, k, v = [(torch.randn(B, T, H, d, generator=gen) / 8).to(torch.bfloat16) for _ in range(3)]
    g = 0.85 + 0.1499 * torch.rand(H, generator=gen)
    o_ref, s_ref = oracle(q, k, v, g, w)
    o, s = _forward(ctx, 3, *_dev(q, k, v, g), w)
    assert rel_err(o, o_ref) <= TOL[torch.bfloat16]
    assert rel_err(s, s_ref) <= TOL[torch.bfloat16]


def test_streaming_prefill_without_final_state_and_repeated_calls(ctx):
    """state_out = NULL, and many launches in a row over the same relay slots (each launch must
    ignore the packets the previous one left behind)."""
    wl = _small("config3", 2, 3)
    q, k, v = workloads.make_qkv(wl)
    g = workloads.make_decay(wl)
    o_ref, _ = oracle(q, k, v, g, wl.grid_w)
    dq, dk_, dv_, dg = _dev(q, k, v, g)
    ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, 3)
    try:
        outs = []
        for _ in range(50):
            o, s = ctx.lasad_forward(dq, dk_, dv_, dg, wl.grid_w, want_state=False)
            assert s is None
            outs.append(o)
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
    finally:
        ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, 0)
    assert rel_err(outs[0], o_ref) <= TOL[torch.bfloat16]
    assert all(torch.equal(outs[0], x) for x in outs[1:])


def test_streaming_prefill_launch_counter_wraps(ctx):
    """The relay tags hold the launch number modulo 65535: run past the wrap (the library clears
    the slots there) and check the result on both sides of it."""
    B, T, H, d, w = 1, 256, 2, 64, 16
    gen = torch.Generator().manual_seed(32)
    q, k, v = [(torch.randn(B, T, H, d, generator=gen) / 8).to(torch.bfloat16) for _ in range(3)]
    g = torch.tensor([0.9, 0.99])
    o_ref, s_ref = oracle(q, k, v, g, w)
    dq, dk_, dv_, dg = _dev(q, k, v, g)
    o = torch.empty_like(dq)
    s = torch.empty(B, H, d, d, device="cuda")
    ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, 3)
    try:
        for it in range(66000):
            ctx.lasad_forward(dq, dk_, dv_, dg, w, o=o, state_out=s)
            if it % 8192 == 0 or it > 65990:
                torch.cuda.synchronize()
                assert ctx.device_status() == 0
                assert rel_err(o, o_ref) <= TOL[torch.bfloat16], f"launch {it}"
                assert rel_err(s, s_ref) <= TOL[torch.bfloat16], f"launch {it}"
    finally:
        ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, 0)


# ------------------------------------------------------------------------------------------
# host-buffer entry point: the pipelined copies must not change the result
# ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype,d,B,T", [(torch.bfloat16, 64, 5, 333), (torch.float32, 32, 3, 333),
                                         (torch.bfloat16, 64, 1, 333), (torch.bfloat16, 64, 3, 2100)])
def test_forward_host_equals_device_path(ctx, dtype, d, B, T):
    """(T = 333 with few chains runs the task-streaming kernel under the default option, T = 2100 the
    segment-parallel mode: the host entry point must take the same one as the device entry point.)"""
    H, w, P = 3, 12, 1
    gen = torch.Generator().manual_seed(41 + B)
    q, k, v = [(torch.randn(B, T, H, d, generator=gen) / d ** 0.5).to(dtype).pin_memory() for _ in range(3)]
    g = torch.tensor([0.9, 0.97, 0.999]).pin_memory()
    s_in = torch.randn(B, H, d, d, generator=gen).pin_memory()
    o_h = torch.empty(B, T, H, d, dtype=dtype).pin_memory()
    s_h = torch.empty(B, H, d, d).pin_memory()
    for _ in range(2):      # twice: the second call reuses the staging slots and events
        o_h.zero_()
        s_h.zero_()
        ctx.lasad_forward_host(q, k, v, g, w, o_h, prefix_len=P, t0=2, scale=0.5, state_in=s_in, state_out=s_h)
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        o_d, s_d = ctx.lasad_forward(q.cuda(), k.cuda(), v.cuda(), g.cuda(), w, prefix_len=P, t0=2, scale=0.5,
                                     state_in=s_in.cuda())
        torch.cuda.synchronize()
        assert torch.equal(o_h, o_d.cpu()) and torch.equal(s_h, s_d.cpu())
    o_ref, s_ref = oracle(q, k, v, g, w, P, 2, 0.5, s_in)
    assert rel_err(o_h, o_ref) <= TOL[dtype] and rel_err(s_h, s_ref) <= TOL[dtype]


def test_decode_per_sequence_positions_and_widths(ctx):
    """Every sequence at its own position and on its own grid width: each batch element must
    equal a single-sequence oracle run at that position."""
    B, H, d = 5, 3, 64
    gen = torch.Generator().manual_seed(51)
    q, k, v = [(torch.randn(B, 1, H, d, generator=gen) / 8).to(torch.bfloat16) for _ in range(3)]
    g = torch.tensor([0.8, 0.95, 0.999])
    s_in = torch.randn(B, H, d, d, generator=gen)
    pos = torch.tensor([3, 4, 7, 11, 0], dtype=torch.int32)       # with P = 0: 3, 7, 11 end a row of width 4
    widths = torch.tensor([4, 4, 8, 6, 1], dtype=torch.int32)     # element 4: width 1, every step is a boundary
    for use_widths in (False, True):
        state = s_in.clone().cuda()
        o = ctx.lasad_decode_step_pos(q[:, 0].cuda(), k[:, 0].cuda(), v[:, 0].cuda(), g.cuda(), state, pos.cuda(),
                                      prefix_len=0, grid_w=4, widths=widths.cuda() if use_widths else None)
        torch.cuda.synchronize()
        for b in range(B):
            w = int(widths[b]) if use_widths else 4
            o_ref, s_ref = oracle(q[b:b + 1], k[b:b + 1], v[b:b + 1], g, w, 0, int(pos[b]), 1.0, s_in[b:b + 1])
            assert rel_err(o[b:b + 1], o_ref[:, 0]) <= TOL[torch.bfloat16], (b, use_widths)
            assert rel_err(state[b:b + 1], s_ref) <= 1e-6, (b, use_widths)


# ------------------------------------------------------------------------------------------
# bounded waits: a wait that runs out is reported, nothing hangs, the context stays usable
# ------------------------------------------------------------------------------------------
@pytest.mark.parametrize("impl", [2, 3, 4, 5])
def test_expired_device_wait_is_reported_and_context_survives(ctx, impl):
    """With the poll limit of the device-side waits set to 1, some wait runs out before its
    barrier completes: the kernel must leave through its normal exit, the status word must say
    so, and the next call (default limit) must be correct again."""
    wl = _small("config3", 1, 2)
    q, k, v = workloads.make_qkv(wl)
    g = workloads.make_decay(wl)
    o_ref, s_ref = oracle(q, k, v, g, wl.grid_w)
    dq, dk_, dv_, dg = _dev(q, k, v, g)
    ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, impl)
    try:
        ctx.set_option(binding.LASAD_OPT_WAIT_LIMIT, 1)
        ctx.lasad_forward(dq, dk_, dv_, dg, wl.grid_w)
        torch.cuda.synchronize()                       # returns: no wait is unbounded
        assert ctx.device_status() == binding.LASAD_ERR_TIMEOUT
        assert ctx.device_status() == 0                # the query clears the flag
        ctx.set_option(binding.LASAD_OPT_WAIT_LIMIT, 0)
        o, s = ctx.lasad_forward(dq, dk_, dv_, dg, wl.grid_w)
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        assert rel_err(o, o_ref) <= TOL[torch.bfloat16]
        assert rel_err(s, s_ref) <= TOL[torch.bfloat16]
    finally:
        ctx.set_option(binding.LASAD_OPT_WAIT_LIMIT, 0)
        ctx.set_option(binding.LASAD_OPT_PREFILL_IMPL, 0)
