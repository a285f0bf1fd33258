"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle.

Each test names the passage it rests on.  None of the expected values comes from the oracle or
from the CUDA path: they are hand-derived fixtures (tests/golden), closed forms, library
matmuls for the special cases that reduce to one, or invariants of the recurrence.
"""
import os

import numpy as np
import pytest

from oracle import lasad_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
FORMS = [orc.recurrent, orc.quadratic]
FORM_IDS = ["recurrent", "quadratic"]


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def _read_golden(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            t, coef, val = [p.strip() for p in line.split(":")]
            rows.append((int(t), [float(c) for c in coef.split()], float(val)))
    return rows


# ---------------------------------------------------------------------------------------------
# hand-derived tiny grids (Section 3.4: SAD recurrence + SAD rule, evaluated symbolically)
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("form", FORMS, ids=FORM_IDS)
@pytest.mark.parametrize("fixture,w", [("grid2x2_allones.txt", 2), ("grid3x3_allones.txt", 3)])
def test_golden_small_grids(form, fixture, w):
    rows = _read_golden(fixture)
    T = len(rows)
    ones = np.ones((1, T, 1, 1))
    for g in (0.5, 0.9, 0.0, 1.0, 0.37):
        o, s = form(ones, ones, ones, np.array([g]), grid_w=w)
        for t, coef, val in rows:
            expect = sum(c * g ** p for p, c in enumerate(coef))
            if g == 0.5:
                assert expect == pytest.approx(val, abs=1e-15)
            assert o[0, t - 1, 0, 0] == pytest.approx(expect, rel=1e-14, abs=1e-14)
        # final state equals the last output when q = 1, d = 1
        assert s[0, 0, 0, 0] == pytest.approx(o[0, -1, 0, 0], rel=1e-14)


# ---------------------------------------------------------------------------------------------
# decay = 1 reduces to plain causal linear attention (Section 3.2 recurrence vs Section 3.3)
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("form", FORMS, ids=FORM_IDS)
def test_all_decays_one_is_causal_linear_attention(form):
    B, T, H, dk, dv = 2, 37, 3, 8, 5
    q, k, v = _rand((B, T, H, dk), 1), _rand((B, T, H, dk), 2), _rand((B, T, H, dv), 3)
    o, s = form(q, k, v, np.ones(H), grid_w=6)
    for b in range(B):
        for h in range(H):
            A = np.tril(q[b, :, h] @ k[b, :, h].T)
            np.testing.assert_allclose(o[b, :, h], A @ v[b, :, h], rtol=1e-12, atol=1e-12)
            np.testing.assert_allclose(s[b, h], k[b, :, h].T @ v[b, :, h], rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------------------------------------
# single column: every step is a boundary, so the decay never acts
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("form", FORMS, ids=FORM_IDS)
def test_single_column_grid_ignores_decay(form):
    B, T, H, d = 1, 9, 2, 4
    q, k, v = _rand((B, T, H, d), 4), _rand((B, T, H, d), 5), _rand((B, T, H, d), 6)
    o, s = form(q, k, v, np.array([0.3, 0.0]), grid_w=1)
    for h in range(H):
        A = np.tril(q[0, :, h] @ k[0, :, h].T)
        np.testing.assert_allclose(o[0, :, h], A @ v[0, :, h], rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(s[0, h], k[0, :, h].T @ v[0, :, h], rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------------------------------------
# single row / rule off: ordinary 1-D decay (Section 3.3), geometric-series closed form
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("form", FORMS, ids=FORM_IDS)
def test_single_row_closed_form(form):
    T, g = 12, 0.8
    ones = np.ones((1, T, 1, 1))
    geo = np.array([(1 - g ** t) / (1 - g) for t in range(1, T + 1)])
    # rule off: o_t = 1 + g + ... + g^(t-1)
    o, _ = form(ones, ones, ones, np.array([g]), grid_w=0)
    np.testing.assert_allclose(o[0, :, 0, 0], geo, rtol=1e-13)
    # grid wider than the sequence: no boundary is reached, same thing
    o, _ = form(ones, ones, ones, np.array([g]), grid_w=T + 5)
    np.testing.assert_allclose(o[0, :, 0, 0], geo, rtol=1e-13)
    # one row of exactly T tokens: only the last step is a boundary -> o_T = o_{T-1} + 1
    o, _ = form(ones, ones, ones, np.array([g]), grid_w=T)
    np.testing.assert_allclose(o[0, :-1, 0, 0], geo[:-1], rtol=1e-13)
    assert o[0, -1, 0, 0] == pytest.approx(geo[-2] + 1.0, rel=1e-13)


# ---------------------------------------------------------------------------------------------
# 1-D decay as a library matmul: O = (Q K^T o gamma^(t-s) o causal) V  (Section 3.3 unrolled)
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("form", FORMS, ids=FORM_IDS)
def test_rule_off_matches_retention_matrix(form):
    T, d, g = 29, 6, 0.93
    q, k, v = _rand((1, T, 1, d), 7), _rand((1, T, 1, d), 8), _rand((1, T, 1, d), 9)
    o, s = form(q, k, v, np.array([g]), grid_w=0)
    idx = np.arange(T)
    D = np.where(idx[:, None] >= idx[None, :], g ** np.clip(idx[:, None] - idx[None, :], 0, None), 0.0)
    np.testing.assert_allclose(o[0, :, 0], ((q[0, :, 0] @ k[0, :, 0].T) * D) @ v[0, :, 0], rtol=1e-12, atol=1e-12)
    wj = g ** (T - 1 - idx)
    np.testing.assert_allclose(s[0, 0], (k[0, :, 0] * wj[:, None]).T @ v[0, :, 0], rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------------------------------------
# the decay between two tokens is a closed form of their 2-D (row, col) positions
# ---------------------------------------------------------------------------------------------
def _mask_from_rowcol(h, w, g, P=0):
    """D[t,s] = g^m with m counted from grid positions only (no running product).

    A decaying step is any step that does not absorb the last token of a row.  Between tokens
    s < t (grid positions) lie (row_t-row_s)(w-1) + (col_t-col_s) such steps, corrected by one
    when t (resp. s) itself sits in the last column.  Prefix tokens each add one decaying step.
    """
    N = P + h * w
    D = np.zeros((N, N))
    def cnt(i):  # decaying steps among absolute indices 0..i
        if i < P:
            return i + 1
        j = i - P
        row, col = divmod(j, w)
        return P + row * (w - 1) + col + (0 if col == w - 1 else 1)
    for t in range(N):
        for s in range(t + 1):
            D[t, s] = g ** (cnt(t) - cnt(s)) if g > 0 else float(cnt(t) == cnt(s))
    return D


@pytest.mark.parametrize("form", FORMS, ids=FORM_IDS)
@pytest.mark.parametrize("h,w,P", [(2, 2, 0), (3, 3, 0), (4, 5, 0), (5, 4, 1), (3, 7, 3), (8, 8, 0)])
def test_decay_is_function_of_row_col(form, h, w, P):
    d, g = 3, 0.85
    N = P + h * w
    q, k, v = _rand((1, N, 1, d), 10), _rand((1, N, 1, d), 11), _rand((1, N, 1, d), 12)
    o, _ = form(q, k, v, np.array([g]), grid_w=w, prefix_len=P)
    D = _mask_from_rowcol(h, w, g, P)
    np.testing.assert_allclose(o[0, :, 0], ((q[0, :, 0] @ k[0, :, 0].T) * D) @ v[0, :, 0], rtol=1e-12, atol=1e-12)


def test_rowcol_pair_formula():
    """m(t,s) = (row_t-row_s)(w-1) + (col_t-col_s) - [col_t=w-1] + [col_s=w-1] (0-based grid)."""
    for h, w in [(2, 2), (3, 3), (4, 7), (8, 8), (5, 1)]:
        a = [0 if (j + 1) % w == 0 else 1 for j in range(h * w)]   # SAD rule, 1-based t = j+1
        c = np.cumsum(a)
        for t in range(h * w):
            for s in range(t + 1):
                rt, ct = divmod(t, w)
                rs, cs = divmod(s, w)
                m = (rt - rs) * (w - 1) + (ct - cs) - (ct == w - 1) + (cs == w - 1)
                assert m == c[t] - c[s]


# ---------------------------------------------------------------------------------------------
# per-channel (vector) decay: key channels evolve independently (diag(lambda) in Section 3.3)
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("form", FORMS, ids=FORM_IDS)
def test_vector_decay_decomposes_per_channel(form):
    h, w, dk, dv = 3, 4, 3, 2
    N = h * w
    q, k, v = _rand((1, N, 1, dk), 13), _rand((1, N, 1, dk), 14), _rand((1, N, 1, dv), 15)
    lam = np.array([0.5, 0.9, 0.0]).reshape(1, 1, 1, dk)
    o, _ = form(q, k, v, lam, grid_w=w)
    expect = np.zeros((N, dv))
    for c in range(dk):
        D = _mask_from_rowcol(h, w, lam[0, 0, 0, c])
        expect += (np.outer(q[0, :, 0, c], k[0, :, 0, c]) * D) @ v[0, :, 0]
    np.testing.assert_allclose(o[0, :, 0], expect, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("form", FORMS, ids=FORM_IDS)
def test_data_dependent_decay_bruteforce(form):
    """Per-token, per-channel decays: explicit products over the steps between s and t."""
    w, T, dk, dv = 3, 7, 2, 2
    rng = np.random.default_rng(16)
    q, k, v = _rand((1, T, 1, dk), 17), _rand((1, T, 1, dk), 18), _rand((1, T, 1, dv), 19)
    lam = rng.uniform(0.2, 1.0, size=(1, T, 1, dk))
    o, _ = form(q, k, v, lam, grid_w=w)
    for t in range(T):
        acc = np.zeros(dv)
        for s in range(t + 1):
            for c in range(dk):
                p = 1.0
                for u in range(s + 1, t + 1):
                    p *= 1.0 if (u + 1) % w == 0 else lam[0, u, 0, c]
                acc += q[0, t, 0, c] * k[0, s, 0, c] * p * v[0, s, 0]
        np.testing.assert_allclose(o[0, t, 0], acc, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("form", FORMS, ids=FORM_IDS)
def test_data_dependent_decay_with_incoming_state_bruteforce(form):
    """Per-token, per-channel decays on top of a non-zero incoming state, a prefix token and a start
    in mid-row: outputs and the final state from explicit products over the steps (Section 3.4,
    the SAD recurrence unrolled; the boundary step multiplies by exactly 1)."""
    w, T, dk, dv, P, t0, scale = 3, 8, 2, 3, 1, 2, 0.5
    rng = np.random.default_rng(116)
    q, k, v = _rand((1, T, 1, dk), 117), _rand((1, T, 1, dk), 118), _rand((1, T, 1, dv), 119)
    lam = rng.uniform(0.2, 1.0, size=(1, T, 1, dk))
    s_in = _rand((1, 1, dk, dv), 120)
    o, s_out = form(q, k, v, lam, w, P, t0, scale, s_in)

    def step_decay(u, c):       # decay of local step u (absolute index t0 + u), channel c
        i = t0 + u
        boundary = i >= P and (i - P + 1) % w == 0
        return 1.0 if boundary else lam[0, u, 0, c]

    def prod(lo, hi, c):        # product over local steps lo .. hi (inclusive)
        p = 1.0
        for u in range(lo, hi + 1):
            p *= step_decay(u, c)
        return p

    for t in range(T):
        acc = np.zeros(dv)
        for c in range(dk):
            acc += q[0, t, 0, c] * prod(0, t, c) * s_in[0, 0, c]
            for j in range(t + 1):
                acc += q[0, t, 0, c] * k[0, j, 0, c] * prod(j + 1, t, c) * v[0, j, 0]
        np.testing.assert_allclose(o[0, t, 0], scale * acc, rtol=1e-12, atol=1e-13)
    for c in range(dk):
        row = prod(0, T - 1, c) * s_in[0, 0, c]
        for j in range(T):
            row = row + prod(j + 1, T - 1, c) * k[0, j, 0, c] * v[0, j, 0]
        np.testing.assert_allclose(s_out[0, 0, c], row, rtol=1e-12, atol=1e-13)


# ---------------------------------------------------------------------------------------------
# the two statements of the method agree (equation vs algorithm)
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("B,T,H,d,w,P,t0", [(2, 64, 3, 8, 8, 0, 0), (1, 50, 2, 16, 7, 1, 0),
                                             (1, 33, 2, 4, 5, 2, 11), (3, 20, 1, 32, 0, 0, 0)])
def test_quadratic_equals_recurrent(B, T, H, d, w, P, t0):
    q, k, v = _rand((B, T, H, d), 20), _rand((B, T, H, d), 21), _rand((B, T, H, d), 22)
    g = np.random.default_rng(23).uniform(0.5, 1.0, H)
    s_in = _rand((B, H, d, d), 24)
    for sin in (None, s_in):
        o1, s1 = orc.recurrent(q, k, v, g, w, P, t0, 0.7, sin)
        o2, s2 = orc.quadratic(q, k, v, g, w, P, t0, 0.7, sin)
        np.testing.assert_allclose(o1, o2, rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(s1, s2, rtol=1e-11, atol=1e-12)


# ---------------------------------------------------------------------------------------------
# invariants of the recurrence
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("form", FORMS, ids=FORM_IDS)
def test_causality(form):
    T, d = 24, 4
    q, k, v = _rand((1, T, 1, d), 25), _rand((1, T, 1, d), 26), _rand((1, T, 1, d), 27)
    o, _ = form(q, k, v, np.array([0.9]), grid_w=6)
    s = 13
    q2, k2, v2 = q.copy(), k.copy(), v.copy()
    q2[0, s:] += 1.0; k2[0, s:] -= 2.0; v2[0, s:] *= 3.0
    o2, _ = form(q2, k2, v2, np.array([0.9]), grid_w=6)
    np.testing.assert_array_equal(o[0, :s], o2[0, :s])
    assert np.abs(o[0, s:] - o2[0, s:]).max() > 1e-3


@pytest.mark.parametrize("form", FORMS, ids=FORM_IDS)
def test_linearity(form):
    T, d = 18, 4
    q, k = _rand((1, T, 2, d), 28), _rand((1, T, 2, d), 29)
    v1, v2 = _rand((1, T, 2, d), 30), _rand((1, T, 2, d), 31)
    g = np.array([0.8, 0.95])
    oa, _ = form(q, k, v1, g, 6)
    ob, _ = form(q, k, v2, g, 6)
    oc, _ = form(q, k, 2.0 * v1 - 3.0 * v2, g, 6)
    np.testing.assert_allclose(oc, 2.0 * oa - 3.0 * ob, rtol=1e-11, atol=1e-12)
    od, _ = form(2.0 * q, -0.5 * k, v1, g, 6)
    np.testing.assert_allclose(od, -oa, rtol=1e-11, atol=1e-12)
    oe, _ = form(q, k, v1, g, 6, scale=0.125)
    np.testing.assert_allclose(oe, 0.125 * oa, rtol=1e-13)


@pytest.mark.parametrize("form", FORMS, ids=FORM_IDS)
def test_state_handoff_every_split(form):
    """forward(0..T) equals forward(0..m) followed by forward(m..T) from the carried state."""
    T, d, w, P = 21, 4, 5, 1
    q, k, v = _rand((1, T, 2, d), 32), _rand((1, T, 2, d), 33), _rand((1, T, 2, d), 34)
    g = np.array([0.7, 0.97])
    o, s = form(q, k, v, g, w, P)
    for m in range(1, T):
        o1, s1 = form(q[:, :m], k[:, :m], v[:, :m], g, w, P, 0)
        o2, s2 = form(q[:, m:], k[:, m:], v[:, m:], g, w, P, m, 1.0, s1)
        np.testing.assert_allclose(np.concatenate([o1, o2], 1), o, rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(s2, s, rtol=1e-11, atol=1e-12)


def test_decode_steps_equal_prefill():
    """T single-token calls (Algorithm 1's loop body) reproduce one full-sequence call."""
    T, d, w = 16, 4, 4
    q, k, v = _rand((2, T, 2, d), 35), _rand((2, T, 2, d), 36), _rand((2, T, 2, d), 37)
    g = np.array([0.6, 0.99])
    o, s = orc.quadratic(q, k, v, g, w)
    st = None
    for t in range(T):
        ot, st = orc.recurrent(q[:, t:t + 1], k[:, t:t + 1], v[:, t:t + 1], g, w, 0, t, 1.0, st)
        np.testing.assert_allclose(ot[:, 0], o[:, t], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(st, s, rtol=1e-11, atol=1e-12)


@pytest.mark.parametrize("form", FORMS, ids=FORM_IDS)
def test_first_step_decay_is_moot_from_zero_state(form):
    """s_0 = 0, so whether the first step counts as a boundary cannot matter."""
    T, d = 10, 3
    q, k, v = _rand((1, T, 1, d), 38), _rand((1, T, 1, d), 39), _rand((1, T, 1, d), 40)
    lam = np.full((1, T, 1, d), 0.8)
    o1, _ = form(q, k, v, lam, 5)
    lam2 = lam.copy(); lam2[0, 0] = 0.123
    o2, _ = form(q, k, v, lam2, 5)
    np.testing.assert_array_equal(o1, o2)
    # with an incoming state the first step's decay does act
    s_in = _rand((1, 1, d, d), 41)
    o3, _ = form(q, k, v, lam, 5, state_in=s_in)
    o4, _ = form(q, k, v, lam2, 5, state_in=s_in)
    assert np.abs(o3 - o4).max() > 1e-3


@pytest.mark.parametrize("form", FORMS, ids=FORM_IDS)
def test_boundary_is_last_token_of_row_not_first_of_next(form):
    """The exempt step is the one that absorbs the last token of a row (t mod w = 0, 1-based);
    prefix_len = 1 shifts the rule by one position (grid position = index - prefix)."""
    w, T, g = 3, 6, 0.5
    ones = np.ones((1, T, 1, 1))
    o, _ = form(ones, ones, ones, np.array([g]), w, 0)
    # 1-based t=3 is exempt: o_3 = o_2 + 1, while t=4 decays: o_4 = g*o_3 + 1
    assert o[0, 2, 0, 0] == pytest.approx(o[0, 1, 0, 0] + 1.0)
    assert o[0, 3, 0, 0] == pytest.approx(g * o[0, 2, 0, 0] + 1.0)
    o, _ = form(ones, ones, ones, np.array([g]), w, 1)
    # with one prefix token the exempt steps move to 1-based t = 4
    assert o[0, 2, 0, 0] == pytest.approx(g * o[0, 1, 0, 0] + 1.0)
    assert o[0, 3, 0, 0] == pytest.approx(o[0, 2, 0, 0] + 1.0)


@pytest.mark.parametrize("form", FORMS, ids=FORM_IDS)
def test_zero_decay_keeps_only_current_row_segment(form):
    """gamma = 0 wipes the state at every decaying step; a boundary step keeps it (decay 1,
    taken in the linear domain so that 0 * log(0) never appears)."""
    w, T = 3, 6
    ones = np.ones((1, T, 1, 1))
    o, _ = form(ones, ones, ones, np.array([0.0]), w)
    np.testing.assert_array_equal(o[0, :, 0, 0], [1, 1, 2, 1, 1, 2])


# ---------------------------------------------------------------------------------------------
# Algorithm 1's loop body with its neighbours (SiLU, Sigmoid, tied key, Norm)
# ---------------------------------------------------------------------------------------------
def _np_silu(x):
    return x / (1.0 + np.exp(-x))


def _np_sigmoid(x):
    return 1.0 / (1.0 + np.exp(-x))


def test_layer_core_single_token_closed_form():
    """One token from a zero state: s = k v^T, o = (q . k) v, so the normalised output is
    v / rms(v) times the sign of q . k, whatever the gate's decay (s_0 = 0 makes it moot)."""
    dk, dv = 3, 4
    q_pre = np.array([0.3, -1.2, 2.0]).reshape(1, 1, 1, dk)
    g_pre = np.array([1.5, -0.4, 0.0]).reshape(1, 1, 1, dk)
    v = np.array([0.5, -1.0, 2.0, 0.25]).reshape(1, 1, 1, dv)
    o, s = orc.layer_core(q_pre, None, v, g_pre, grid_w=4, eps=0.0)
    q = _np_silu(q_pre[0, 0, 0])
    k = 1.0 - _np_sigmoid(g_pre[0, 0, 0])
    np.testing.assert_allclose(s[0, 0], np.outer(k, v[0, 0, 0]), rtol=1e-13)
    dot = float(q @ k)
    expect = np.sign(dot) * v[0, 0, 0] / np.sqrt(np.mean(v[0, 0, 0] ** 2))
    np.testing.assert_allclose(o[0, 0, 0], expect, rtol=1e-12)
    # known values of the activations: SiLU(0) = 0, Sigmoid(0) = 1/2 -> k = 1/2
    np.testing.assert_allclose(k[2], 0.5, rtol=0, atol=1e-15)
    o0, _ = orc.layer_core(np.zeros((1, 1, 1, dk)), None, v, g_pre, grid_w=4, eps=1.0)
    np.testing.assert_allclose(o0, 0.0, atol=1e-15)      # q = SiLU(0) = 0, and eps keeps 0/0 away


@pytest.mark.parametrize("tied", [True, False])
def test_layer_core_is_activations_then_the_recurrence_then_the_norm(tied):
    """The fused statement against its parts: numpy's SiLU / Sigmoid / RMS norm around the
    (separately pinned) recurrent form with the gate as a per-token, per-channel decay; prefix,
    start in mid-row, incoming state, scale and eps all in play."""
    B, T, H, dk, dv, w, P, t0, scale, eps = 2, 19, 3, 4, 5, 4, 1, 3, 0.7, 1e-3
    q_pre, g_pre, v = _rand((B, T, H, dk), 301) * 2, _rand((B, T, H, dk), 302) * 2 + 1.0, _rand((B, T, H, dv), 303)
    k_in = None if tied else _rand((B, T, H, dk), 304)
    s_in = _rand((B, H, dk, dv), 305)
    o, s = orc.layer_core(q_pre, k_in, v, g_pre, w, P, t0, scale, s_in, eps)
    lam = _np_sigmoid(g_pre)
    k = 1.0 - lam if tied else k_in
    o_raw, s_ref = orc.recurrent(_np_silu(q_pre), k, v, lam, w, P, t0, scale, s_in)
    o_ref = o_raw / np.sqrt(np.mean(o_raw ** 2, axis=-1, keepdims=True) + eps)
    np.testing.assert_allclose(o, o_ref, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(s, s_ref, rtol=1e-11, atol=1e-12)


def test_layer_core_norm_properties():
    """Each head's normalised output has unit RMS when eps = 0, and scaling v (hence o) leaves it
    unchanged; with eps > 0 a small output is shrunk, not blown up."""
    B, T, H, dk, dv = 1, 12, 2, 4, 8
    q_pre, g_pre, v = _rand((B, T, H, dk), 311), _rand((B, T, H, dk), 312) + 2.0, _rand((B, T, H, dv), 313)
    o, _ = orc.layer_core(q_pre, None, v, g_pre, 3, eps=0.0)
    np.testing.assert_allclose(np.sqrt(np.mean(o ** 2, axis=-1)), 1.0, rtol=1e-12)
    o10, _ = orc.layer_core(q_pre, None, 10.0 * v, g_pre, 3, eps=0.0)
    np.testing.assert_allclose(o10, o, rtol=1e-11, atol=1e-13)
    o_eps, _ = orc.layer_core(q_pre, None, 1e-6 * v, g_pre, 3, eps=1.0)
    assert np.abs(o_eps).max() < 1e-4
