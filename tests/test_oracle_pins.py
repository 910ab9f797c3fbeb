"""Pins of the fp64 oracle against things other than itself.

The paper prints no worked numerical example of Eq. 3, so the oracle is pinned to what the
equation and the mathematics fix: the unrolled closed form by brute force, the f == 0 and
f == 1 special cases, the scalar recurrence of Eq. 1 / Eq. 2 at d_k = d_v = 1, the
partition-of-unity identity of tied gates, state passing, exact adjoint identities and
central finite differences.  None of the checks below re-types the oracle's loop.
"""
import itertools

import numpy as np
import pytest

from oracle import ref


def rng_inputs(seed, B, H, N, dk, dv, gamma=0.0, with_state=True):
    r = np.random.default_rng(seed)
    o = r.standard_normal((B, H, N, dk))
    f = gamma + (1 - gamma) / (1 + np.exp(-r.standard_normal((B, H, N, dk))))
    i = r.standard_normal((B, H, N, dv))
    S0 = r.standard_normal((B, H, dk, dv)) if with_state else None
    return o, f, i, S0


# ---------------------------------------------------------------- P1: closed form, brute force
def closed_form(o, f, i, S0):
    """y_t = sum_{s<=t} sum_k o_tk (prod_{r=s+1..t} f_rk)(1-f_sk) i_s + sum_k o_tk (prod_{r<=t} f_rk) S0[k]
    (Eq. 3 unrolled), every product formed explicitly from scratch."""
    B, H, N, dk = o.shape
    dv = i.shape[-1]
    y = np.zeros((B, H, N, dv))
    S = np.zeros((B, H, dk, dv))
    for b, h in itertools.product(range(B), range(H)):
        for t in range(N):
            for v in range(dv):
                acc = 0.0
                for k in range(dk):
                    for s in range(t + 1):
                        w = 1.0
                        for r in range(s + 1, t + 1):
                            w *= f[b, h, r, k]
                        acc += o[b, h, t, k] * w * (1.0 - f[b, h, s, k]) * i[b, h, s, v]
                    w0 = 1.0
                    for r in range(t + 1):
                        w0 *= f[b, h, r, k]
                    if S0 is not None:
                        acc += o[b, h, t, k] * w0 * S0[b, h, k, v]
                y[b, h, t, v] = acc
        for k in range(dk):
            for v in range(dv):
                acc = 0.0
                for s in range(N):
                    w = 1.0
                    for r in range(s + 1, N):
                        w *= f[b, h, r, k]
                    acc += w * (1.0 - f[b, h, s, k]) * i[b, h, s, v]
                w0 = 1.0
                for r in range(N):
                    w0 *= f[b, h, r, k]
                if S0 is not None:
                    acc += w0 * S0[b, h, k, v]
                S[b, h, k, v] = acc
    return y, S


@pytest.mark.parametrize("shape", [(1, 1, 8, 3, 2), (2, 2, 5, 2, 3), (1, 1, 1, 1, 1), (1, 2, 7, 4, 4)])
@pytest.mark.parametrize("with_state", [False, True])
def test_p1_closed_form(shape, with_state):
    o, f, i, S0 = rng_inputs(11, *shape, with_state=with_state)
    y, SN = ref.hgrn2_fwd(o, f, i, S0)
    y_cf, S_cf = closed_form(o, f, i, S0)
    np.testing.assert_allclose(y, y_cf, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(SN, S_cf, rtol=1e-12, atol=1e-13)


# ---------------------------------------------------------------- P2: f == 0
def test_p2_f_zero_forward():
    o, f, i, S0 = rng_inputs(2, 2, 3, 9, 5, 4)
    f[:] = 0.0
    y, SN = ref.hgrn2_fwd(o, f, i, S0)
    expect = o.sum(-1, keepdims=True) * i           # y_t = (sum_k o_tk) i_t, independent of S0
    np.testing.assert_allclose(y, expect, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(SN, np.broadcast_to(i[:, :, -1, None, :], SN.shape), rtol=0, atol=0)


def test_p2_f_zero_backward():
    # With f == 0: y_t = (sum_k o_tk) i_t  =>  d_o_tk = <dy_t, i_t>, d_i_t = (sum_k o_tk) dy_t, dS0 = 0.
    o, f, i, S0 = rng_inputs(3, 1, 2, 6, 3, 4)
    f[:] = 0.0
    dy = np.random.default_rng(4).standard_normal(i.shape)
    d_o, d_f, d_i, dS0 = ref.hgrn2_bwd(o, f, i, S0, dy)
    np.testing.assert_allclose(d_o, np.broadcast_to((dy * i).sum(-1, keepdims=True), o.shape), atol=1e-13)
    np.testing.assert_allclose(d_i, o.sum(-1, keepdims=True) * dy, atol=1e-13)
    np.testing.assert_allclose(dS0, 0.0, atol=0)
    # d_f_tk at f = 0: dL/df through S_t = f S_{t-1} + (1-f) i_t  ->  G_t[k,:].(S_{t-1}[k,:] - i_t),
    # where G_t[k,:] = o_tk dy_t (later steps are cut off by f_{t+1} = 0) and S_{t-1}[k,:] = i_{t-1} (S0 at t=0).
    prev = np.concatenate([S0[:, :, None, :, :], np.broadcast_to(i[:, :, :-1, None, :], (1, 2, 5, 3, 4))], axis=2)
    expect = np.einsum("bhtk,bhtv,bhtkv->bhtk", o, dy, prev - i[:, :, :, None, :])
    np.testing.assert_allclose(d_f, expect, atol=1e-12)


# ---------------------------------------------------------------- P3: f == 1
def test_p3_untied_decay_one_is_causal_linear_attention():
    r = np.random.default_rng(5)
    B, H, N, dk, dv = 2, 2, 12, 5, 3
    q, k = r.standard_normal((2, B, H, N, dk))
    v = r.standard_normal((B, H, N, dv))
    y, SN = ref.gla_fwd(q, k, v, np.ones_like(q))
    expect = np.matmul(np.tril(np.matmul(q, np.swapaxes(k, -1, -2))), v)     # tril(Q K^T) V
    np.testing.assert_allclose(y, expect, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(SN, np.matmul(np.swapaxes(k, -1, -2), v), rtol=1e-12, atol=1e-12)


def test_p3_tied_f_one_freezes_state():
    o, f, i, S0 = rng_inputs(6, 1, 2, 7, 4, 3)
    f[:] = 1.0
    y, SN = ref.hgrn2_fwd(o, f, i, S0)
    np.testing.assert_allclose(y, np.einsum("bhtk,bhkv->bhtv", o, S0), rtol=1e-13, atol=1e-13)
    np.testing.assert_array_equal(SN, S0)


def test_p3_scalar_decay_is_masked_attention():
    # f equal across the key dimension: y = (D * Q K^T) V with D[t,s] = prod_{r=s+1..t} f_r (library matmul).
    r = np.random.default_rng(7)
    B, H, N, dk, dv = 1, 2, 10, 4, 3
    o = r.standard_normal((B, H, N, dk)); i = r.standard_normal((B, H, N, dv))
    fs = 0.3 + 0.7 * r.random((B, H, N))
    f = np.repeat(fs[..., None], dk, axis=-1)
    y, _ = ref.hgrn2_fwd(o, f, i, None)
    c = np.cumsum(np.log(fs), axis=-1)
    D = np.tril(np.exp(c[..., :, None] - c[..., None, :]))
    expect = np.matmul(D * np.matmul(o, np.swapaxes(1 - f, -1, -2)), i)
    np.testing.assert_allclose(y, expect, rtol=1e-11, atol=1e-12)


# ---------------------------------------------------------------- P5: d_k = d_v = 1 is Eq. 1 / Eq. 2
def test_p5_scalar_recurrence():
    r = np.random.default_rng(8)
    N = 20
    o = r.standard_normal((1, 1, N, 1)); i = r.standard_normal((1, 1, N, 1))
    f = r.random((1, 1, N, 1))
    h0 = 0.7
    y, SN = ref.hgrn2_fwd(o, f, i, np.full((1, 1, 1, 1), h0))
    h = h0
    for t in range(N):
        h = f[0, 0, t, 0] * h + (1 - f[0, 0, t, 0]) * i[0, 0, t, 0]      # h_t = f h_{t-1} + (1-f) i_t
        assert abs(y[0, 0, t, 0] - h * o[0, 0, t, 0]) < 1e-14             # y_t = h_t o_t
    assert abs(SN[0, 0, 0, 0] - h) < 1e-14


# ---------------------------------------------------------------- P6: partition of unity
def test_p6_constant_input_fixed_point_and_geometric():
    o, f, i, _ = rng_inputs(9, 1, 2, 15, 3, 4)
    c = np.array([0.5, -1.25, 2.0, 0.125])
    i[:] = c
    S0 = np.broadcast_to(c, (1, 2, 3, 4)).copy()
    y, SN = ref.hgrn2_fwd(o, f, i, S0)
    np.testing.assert_allclose(SN, S0, rtol=1e-14)                        # prod f + sum (prod f)(1-f) = 1
    np.testing.assert_allclose(y, o.sum(-1, keepdims=True) * c, rtol=1e-13, atol=1e-13)
    phi = 0.8
    f[:] = phi
    _, SN = ref.hgrn2_fwd(o, f, i, None)
    np.testing.assert_allclose(SN, (1 - phi ** 15) * np.broadcast_to(c, SN.shape), rtol=1e-13)


def test_p6_convex_combination_bound():
    o, f, i, S0 = rng_inputs(10, 2, 2, 30, 4, 3)
    _, SN = ref.hgrn2_fwd(o, f, i, S0)
    bound = np.maximum(np.abs(S0), np.abs(i).max(axis=2)[:, :, None, :])
    assert np.all(np.abs(SN) <= bound + 1e-15)


# ---------------------------------------------------------------- P8: state passing, step == fwd
@pytest.mark.parametrize("m", [1, 4, 10])
def test_p8_split_sequence(m):
    o, f, i, S0 = rng_inputs(12, 2, 2, 11, 3, 5)
    y, SN = ref.hgrn2_fwd(o, f, i, S0)
    y1, Sm = ref.hgrn2_fwd(o[:, :, :m], f[:, :, :m], i[:, :, :m], S0)
    y2, SN2 = ref.hgrn2_fwd(o[:, :, m:], f[:, :, m:], i[:, :, m:], Sm)
    np.testing.assert_allclose(np.concatenate([y1, y2], axis=2), y, rtol=1e-14, atol=1e-14)
    np.testing.assert_allclose(SN2, SN, rtol=1e-14, atol=1e-14)


def test_p8_step_equals_fwd():
    o, f, i, S0 = rng_inputs(13, 3, 2, 9, 4, 6)
    y, SN = ref.hgrn2_fwd(o, f, i, S0)
    S = S0.copy()
    for t in range(o.shape[2]):
        yt = ref.hgrn2_step(o[:, :, t], f[:, :, t], i[:, :, t], S)
        np.testing.assert_allclose(yt, y[:, :, t], rtol=1e-14, atol=1e-14)
    np.testing.assert_allclose(S, SN, rtol=1e-14, atol=1e-14)


def test_p8_backward_split_sequence():
    # dS passes backwards through a split the way S passes forwards.
    o, f, i, S0 = rng_inputs(14, 1, 2, 10, 3, 4)
    r = np.random.default_rng(15)
    dy = r.standard_normal(i.shape); dSN = r.standard_normal(S0.shape)
    m = 6
    d_o, d_f, d_i, dS0 = ref.hgrn2_bwd(o, f, i, S0, dy, dSN)
    _, Sm = ref.hgrn2_fwd(o[:, :, :m], f[:, :, :m], i[:, :, :m], S0)
    b2 = ref.hgrn2_bwd(o[:, :, m:], f[:, :, m:], i[:, :, m:], Sm, dy[:, :, m:], dSN)
    b1 = ref.hgrn2_bwd(o[:, :, :m], f[:, :, :m], i[:, :, :m], S0, dy[:, :, :m], b2[3])
    for full, a, b in zip((d_o, d_f, d_i), b1[:3], b2[:3]):
        np.testing.assert_allclose(np.concatenate([a, b], axis=2), full, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(b1[3], dS0, rtol=1e-12, atol=1e-13)


# ---------------------------------------------------------------- P7: exact adjoint identities
def test_p7_adjoint_linear_in_i_and_S0():
    o, f, i, S0 = rng_inputs(16, 2, 2, 13, 4, 3)
    dy = np.random.default_rng(17).standard_normal(i.shape)
    y, _ = ref.hgrn2_fwd(o, f, i, S0)
    d_o, d_f, d_i, dS0 = ref.hgrn2_bwd(o, f, i, S0, dy, None)
    lhs = (dy * y).sum()
    np.testing.assert_allclose(lhs, (d_i * i).sum() + (dS0 * S0).sum(), rtol=1e-12)   # y linear in (i, S0)
    np.testing.assert_allclose(lhs, (d_o * o).sum(), rtol=1e-12)                      # y linear in o


def test_p7_adjoint_final_state():
    o, f, i, S0 = rng_inputs(18, 1, 2, 9, 3, 3)
    dSN = np.random.default_rng(19).standard_normal(S0.shape)
    _, SN = ref.hgrn2_fwd(o, f, i, S0)
    d_o, d_f, d_i, dS0 = ref.hgrn2_bwd(o, f, i, S0, np.zeros_like(i), dSN)
    np.testing.assert_allclose((dSN * SN).sum(), (d_i * i).sum() + (dS0 * S0).sum(), rtol=1e-12)
    np.testing.assert_allclose(d_o, 0.0, atol=0)                                       # S_N does not see o


# ---------------------------------------------------------------- P4: central finite differences
def _fd(fun, x, h=1e-6):
    g = np.zeros_like(x)
    it = np.nditer(x, flags=["multi_index"])
    for _ in it:
        idx = it.multi_index
        old = x[idx]
        x[idx] = old + h; lp = fun()
        x[idx] = old - h; lm = fun()
        x[idx] = old
        g[idx] = (lp - lm) / (2 * h)
    return g


@pytest.mark.parametrize("with_state", [True, False])
def test_p4_finite_differences_tied(with_state):
    o, f, i, S0 = rng_inputs(20, 1, 2, 6, 3, 2, gamma=0.1, with_state=with_state)
    r = np.random.default_rng(21)
    dy = r.standard_normal(i.shape); dSN = r.standard_normal((1, 2, 3, 2))

    def loss():
        y, SN = ref.hgrn2_fwd(o, f, i, S0)
        return (dy * y).sum() + (dSN * SN).sum()

    d_o, d_f, d_i, dS0 = ref.hgrn2_bwd(o, f, i, S0, dy, dSN)
    np.testing.assert_allclose(d_o, _fd(loss, o), rtol=1e-6, atol=1e-8)
    np.testing.assert_allclose(d_f, _fd(loss, f), rtol=1e-6, atol=1e-8)
    np.testing.assert_allclose(d_i, _fd(loss, i), rtol=1e-6, atol=1e-8)
    if with_state:
        np.testing.assert_allclose(dS0, _fd(loss, S0), rtol=1e-6, atol=1e-8)


def test_p4_finite_differences_untied():
    r = np.random.default_rng(22)
    B, H, N, dk, dv = 1, 1, 7, 3, 2
    q, k = r.standard_normal((2, B, H, N, dk))
    v = r.standard_normal((B, H, N, dv)); a = 0.2 + 0.8 * r.random((B, H, N, dk))
    S0 = r.standard_normal((B, H, dk, dv))
    dy = r.standard_normal(v.shape); dSN = r.standard_normal(S0.shape)

    def loss():
        y, SN = ref.gla_fwd(q, k, v, a, S0)
        return (dy * y).sum() + (dSN * SN).sum()

    dq, dk_, dv_, da, dS0 = ref.gla_bwd(q, k, v, a, S0, dy, dSN)
    for g, x in ((dq, q), (dk_, k), (dv_, v), (da, a), (dS0, S0)):
        np.testing.assert_allclose(g, _fd(loss, x), rtol=1e-6, atol=1e-8)


def test_checkpointed_backward_long_sequence_matches_adjoint():
    # N large enough for many sqrt(N) segments with a ragged last one.
    o, f, i, S0 = rng_inputs(23, 1, 1, 203, 3, 2, gamma=0.5)
    r = np.random.default_rng(24)
    dy = r.standard_normal(i.shape); dSN = r.standard_normal(S0.shape)
    y, SN = ref.hgrn2_fwd(o, f, i, S0)
    d_o, d_f, d_i, dS0 = ref.hgrn2_bwd(o, f, i, S0, dy, dSN)
    lhs = (dy * y).sum() + (dSN * SN).sum()
    np.testing.assert_allclose(lhs, (d_i * i).sum() + (dS0 * S0).sum(), rtol=1e-11)
    # directional derivative in f
    df_dir = r.standard_normal(f.shape)
    h = 1e-6
    yp, Sp = ref.hgrn2_fwd(o, f + h * df_dir, i, S0)
    ym, Sm = ref.hgrn2_fwd(o, f - h * df_dir, i, S0)
    num = ((dy * (yp - ym)).sum() + (dSN * (Sp - Sm)).sum()) / (2 * h)
    np.testing.assert_allclose((d_f * df_dir).sum(), num, rtol=1e-6)


def test_batch_head_units_are_independent():
    o, f, i, S0 = rng_inputs(25, 3, 2, 8, 3, 2)
    y, SN = ref.hgrn2_fwd(o, f, i, S0)
    for b in range(3):
        yb, Sb = ref.hgrn2_fwd(o[b:b + 1], f[b:b + 1], i[b:b + 1], S0[b:b + 1])
        np.testing.assert_array_equal(yb, y[b:b + 1])
        np.testing.assert_array_equal(Sb, SN[b:b + 1])


def test_packed_batch_equals_the_same_sequences_as_an_ordinary_batch():
    # the packed-batch wrappers add no arithmetic: B sequences of equal length laid end to end must reproduce the
    # [B, H, N, d] result exactly, forward and backward, states included (this pins their indexing)
    rng = np.random.default_rng(5)
    B, H, N, dk, dv = 3, 2, 7, 4, 3
    o = rng.standard_normal((B, H, N, dk)); f = rng.uniform(0.05, 1.0, (B, H, N, dk))
    i = rng.standard_normal((B, H, N, dv)); dy = rng.standard_normal((B, H, N, dv))
    S0 = rng.standard_normal((B, H, dk, dv)); dSN = rng.standard_normal((B, H, dk, dv))
    pack = lambda x: np.ascontiguousarray(np.moveaxis(x, 0, 1).reshape(H, B * N, x.shape[-1]))
    cu = np.arange(B + 1) * N
    y, SN = ref.hgrn2_fwd(o, f, i, S0)
    yp, SNp = ref.hgrn2_fwd_varlen(pack(o), pack(f), pack(i), cu, S0)
    np.testing.assert_array_equal(yp, pack(y)); np.testing.assert_array_equal(SNp, SN)
    g = ref.hgrn2_bwd(o, f, i, S0, dy, dSN)
    gp = ref.hgrn2_bwd_varlen(pack(o), pack(f), pack(i), cu, S0, pack(dy), dSN)
    for a, b in zip(g[:3], gp[:3]):
        np.testing.assert_array_equal(b, pack(a))
    np.testing.assert_array_equal(gp[3], g[3])
    # an empty sequence passes its state (and its state gradient) through
    cu2 = np.array([0, 0, N])
    _, SN2 = ref.hgrn2_fwd_varlen(pack(o)[:, :N], pack(f)[:, :N], pack(i)[:, :N], cu2, S0[:2])
    np.testing.assert_array_equal(SN2[0], S0[0])


def test_gated_wrappers_against_finite_differences():
    # the gate activations of Eq. 1 / Eq. 2 in front of the recurrence: gradients with respect to the three
    # pre-activations and to the lower bound beta against central differences of L = <dy, y> + <dSN, S_N>
    rng = np.random.default_rng(17)
    B, H, N, dk, dv = 2, 2, 5, 3, 2
    zo = rng.standard_normal((B, H, N, dk)); zf = rng.standard_normal((B, H, N, dk))
    zi = rng.standard_normal((B, H, N, dv)); beta = rng.uniform(0.0, 0.9, (H, dk))
    S0 = rng.standard_normal((B, H, dk, dv)); dy = rng.standard_normal((B, H, N, dv))
    dSN = rng.standard_normal((B, H, dk, dv))

    def loss(zo_, zf_, zi_, beta_):
        y, SN = ref.hgrn2_fwd_gated(zo_, zf_, zi_, beta_, S0)
        return float((dy * y).sum() + (dSN * SN).sum())

    got = ref.hgrn2_bwd_gated(zo, zf, zi, beta, S0, dy, dSN)
    args = [zo, zf, zi, beta]
    h = 1e-6
    for which in range(4):
        x = args[which]
        num = np.zeros_like(x)
        it = np.nditer(x, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            xp = x.copy(); xp[idx] += h
            xm = x.copy(); xm[idx] -= h
            ap = list(args); ap[which] = xp
            am = list(args); am[which] = xm
            num[idx] = (loss(*ap) - loss(*am)) / (2 * h)
        assert np.abs(num - got[which]).max() <= 1e-6 * max(1.0, np.abs(num).max()), which
    # the activations themselves: sigmoid(0) = 1/2, silu(0) = 0, f = beta where the sigmoid vanishes
    o, f, i = ref.gates(np.zeros((1, 1, 1, 2)), np.full((1, 1, 1, 2), -700.0), np.zeros((1, 1, 1, 2)), np.array([[0.25, 0.5]]))
    np.testing.assert_allclose(o, 0.5); np.testing.assert_allclose(i, 0.0)
    np.testing.assert_allclose(f[0, 0, 0], [0.25, 0.5])
