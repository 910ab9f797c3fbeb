"""The chunkwise-parallel form that the CUDA kernels implement, checked on the CPU.

The paper does not print the chunkwise algorithm (it points to prior work), so the
formulas are derived from Eq. 3 by unrolling C steps.  This file writes that derivation
out in numpy (fp64), in the notation of the kernels' comments, and compares it with the
step-by-step oracle, so that a mistake in the derivation shows up without a GPU.  It is a
test of the mathematics only; the product never calls it.

Per chunk, with q = o, k = 1 - f, v = i, b_j = sum_{r<=j} log f_r (inclusive, per key
dimension), Lam_j = exp(b_j), S_in the state at the chunk start, dS_out the state gradient
arriving from the right:

  A[t,s]  = sum_k q_tk k_sk exp(b_tk - b_sk)          for s <= t, else 0
  Y       = A V + (q * Lam) S_in
  S_out   = Diag(Lam_C) S_in + (k * Lam_C/Lam)^T V
  dA      = tril(dY V^T)
  dq_tk   = sum_{s<=t} dA[t,s] k_sk exp(b_tk-b_sk) + Lam_tk (dY S_in^T)_tk
  dk_sk   = sum_{t>=s} dA[t,s] q_tk exp(b_tk-b_sk) + (Lam_C/Lam_s)_k (V dS_out^T)_sk
            `---------------- intra ------------'   `------------ inter -----------'
  dV      = A^T dY + (k * Lam_C/Lam) dS_out
  dS_in   = Diag(Lam_C) dS_out + (q * Lam)^T dY
  dg_jk   = sum_{j'>=j} (q dq - k dk_intra)_{j'k} + sum_{s<j} (k dk_inter)_{sk}
            + Lam_Ck sum_v dS_out[k,v] S_in[k,v]                     (gradient w.r.t. log f_j)
  d_o = dq,  d_i = dV,  d_f = dg / f - dk
"""
import numpy as np
import pytest

from oracle import ref


def chunk_fwd(o, f, i, S0, C):
    B, H, N, dk = o.shape
    dv = i.shape[-1]
    y = np.zeros((B, H, N, dv))
    S = np.zeros((B, H, dk, dv)) if S0 is None else S0.copy()
    states = []
    for c0 in range(0, N, C):
        sl = slice(c0, min(c0 + C, N))
        q, fk, v = o[:, :, sl], f[:, :, sl], i[:, :, sl]
        k = 1 - fk
        b = np.cumsum(np.log(fk), axis=2)
        states.append(S.copy())
        D = np.exp(b[:, :, :, None, :] - b[:, :, None, :, :])                 # [t, s, k]
        A = np.tril(np.einsum("bhtk,bhsk,bhtsk->bhts", q, k, D))
        y[:, :, sl] = A @ v + (q * np.exp(b)) @ S
        lamC = np.exp(b[:, :, -1])
        S = lamC[..., None] * S + np.swapaxes(k * np.exp(b[:, :, -1:, :] - b), -1, -2) @ v
    return y, S, states


def chunk_bwd(o, f, i, dy, dSN, states, C):
    B, H, N, dk = o.shape
    dv = i.shape[-1]
    d_o, d_f, d_i = np.zeros_like(o), np.zeros_like(f), np.zeros_like(i)
    dS = np.zeros((B, H, dk, dv)) if dSN is None else dSN.copy()
    starts = list(range(0, N, C))
    for ci in reversed(range(len(starts))):
        c0 = starts[ci]
        sl = slice(c0, min(c0 + C, N))
        q, fk, v, g = o[:, :, sl], f[:, :, sl], i[:, :, sl], dy[:, :, sl]
        S_in = states[ci]
        k = 1 - fk
        b = np.cumsum(np.log(fk), axis=2)
        lam, lamC = np.exp(b), np.exp(b[:, :, -1])
        D = np.exp(b[:, :, :, None, :] - b[:, :, None, :, :])
        A = np.tril(np.einsum("bhtk,bhsk,bhtsk->bhts", q, k, D))
        dA = np.tril(g @ np.swapaxes(v, -1, -2))
        mask = np.tril(np.ones((q.shape[2], q.shape[2])))
        dq = np.einsum("bhts,bhsk,bhtsk->bhtk", dA * mask, k, D) + lam * (g @ np.swapaxes(S_in, -1, -2))
        dk_intra = np.einsum("bhts,bhtk,bhtsk->bhsk", dA * mask, q, D)
        dk_inter = np.exp(b[:, :, -1:, :] - b) * (v @ np.swapaxes(dS, -1, -2))
        dkk = dk_intra + dk_inter
        dV = np.swapaxes(A, -1, -2) @ g + (k * np.exp(b[:, :, -1:, :] - b)) @ dS
        a = q * dq - k * dk_intra
        e = k * dk_inter
        suffix = np.flip(np.cumsum(np.flip(a, 2), axis=2), 2)                  # sum_{j'>=j}
        prefix = np.cumsum(e, axis=2) - e                                      # sum_{s<j}
        R = (dS * S_in).sum(-1)
        dg = suffix + prefix + (lamC * R)[:, :, None, :]
        d_o[:, :, sl] = dq
        d_i[:, :, sl] = dV
        d_f[:, :, sl] = dg / fk - dkk
        dS = lamC[..., None] * dS + np.swapaxes(q * lam, -1, -2) @ g
    return d_o, d_f, d_i, dS


@pytest.mark.parametrize("N,C", [(37, 8), (16, 16), (5, 8), (64, 16), (33, 1)])
@pytest.mark.parametrize("with_state", [False, True])
def test_chunk_form_matches_oracle(N, C, with_state):
    r = np.random.default_rng(100 + N + C)
    B, H, dk, dv = 2, 2, 5, 4
    o = r.standard_normal((B, H, N, dk)); i = r.standard_normal((B, H, N, dv))
    f = 0.05 + 0.95 / (1 + np.exp(-r.standard_normal((B, H, N, dk))))
    dy = r.standard_normal(i.shape)
    S0 = r.standard_normal((B, H, dk, dv)) if with_state else None
    dSN = r.standard_normal((B, H, dk, dv)) if with_state else None
    y, SN, states = chunk_fwd(o, f, i, S0, C)
    y_ref, SN_ref = ref.hgrn2_fwd(o, f, i, S0)
    np.testing.assert_allclose(y, y_ref, rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(SN, SN_ref, rtol=1e-10, atol=1e-11)
    got = chunk_bwd(o, f, i, dy, dSN, states, C)
    want = ref.hgrn2_bwd(o, f, i, S0, dy, dSN)
    for g, w in zip(got, want):
        np.testing.assert_allclose(g, w, rtol=1e-9, atol=1e-10)


# --------------------------------------------------------------------------------------------------
# The mid-chunk reference frame of the tensor-core kernels.  Only two rescaled operands exist,
#   Qs_t = q_t exp(b_t - b_m),  Ks_s = k_s exp(b_m - b_s)      (m = middle of the chunk),
# the state is carried as S' = Pm * S_in (Pm = exp(b_m)) and leaves as S_out = E * (S' + Ks^T V)
# (E = exp(b_C - b_m)).  The decay gradient is formed from products in the same frame:
#   a = Qs*dQs - Ks*dKs_intra,  e = Ks*dKs_inter,  R_k = sum_v dS''[k,v] S'[k,v],  dS'' = E * dS_out
#   dg_t = sum_{j>=t} a_j + sum_{s<t} e_s + R
# --------------------------------------------------------------------------------------------------
def midframe_fwd_bwd(o, f, i, S0, dy, dSN, C):
    B, H, N, dk = o.shape
    dv = i.shape[-1]
    assert N % C == 0
    T = lambda x: np.swapaxes(x, -1, -2)
    y = np.zeros((B, H, N, dv))
    S = np.zeros((B, H, dk, dv)) if S0 is None else S0.copy()
    saved = []
    for c0 in range(0, N, C):
        sl = slice(c0, c0 + C)
        b = np.cumsum(np.log(f[:, :, sl]), axis=2)
        bm = b[:, :, C // 2 - 1:C // 2]
        Qs = o[:, :, sl] * np.exp(b - bm)
        Ks = (1 - f[:, :, sl]) * np.exp(bm - b)
        Pm, E = np.exp(bm[:, :, 0]), np.exp(b[:, :, -1] - bm[:, :, 0])
        Sp = Pm[..., None] * S
        saved.append(Sp)
        y[:, :, sl] = np.tril(Qs @ T(Ks)) @ i[:, :, sl] + Qs @ Sp
        S = E[..., None] * (Sp + T(Ks) @ i[:, :, sl])
    SN = S
    d_o, d_f, d_i = np.zeros_like(o), np.zeros_like(f), np.zeros_like(i)
    dS_out = np.zeros((B, H, dk, dv)) if dSN is None else dSN.copy()
    for ci in reversed(range(N // C)):
        sl = slice(ci * C, ci * C + C)
        fk, v, g = f[:, :, sl], i[:, :, sl], dy[:, :, sl]
        b = np.cumsum(np.log(fk), axis=2)
        bm = b[:, :, C // 2 - 1:C // 2]
        sq, sk = np.exp(b - bm), np.exp(bm - b)
        Qs, Ks = o[:, :, sl] * sq, (1 - fk) * sk
        Pm, E = np.exp(bm[:, :, 0]), np.exp(b[:, :, -1] - bm[:, :, 0])
        Sp = saved[ci]
        dS2 = E[..., None] * dS_out
        A = np.tril(Qs @ T(Ks))
        dA = np.tril(g @ T(v))
        dQs = dA @ Ks + g @ T(Sp)
        dKs_intra = T(dA) @ Qs
        dKs_inter = v @ T(dS2)
        d_i[:, :, sl] = T(A) @ g + Ks @ dS2
        a = Qs * dQs - Ks * dKs_intra
        e = Ks * dKs_inter
        R = (dS2 * Sp).sum(-1)
        dg = np.flip(np.cumsum(np.flip(a, 2), 2), 2) + (np.cumsum(e, 2) - e) + R[:, :, None, :]
        dkk = (dKs_intra + dKs_inter) * sk
        d_o[:, :, sl] = dQs * sq
        d_f[:, :, sl] = dg / fk - dkk
        dS_out = Pm[..., None] * (dS2 + T(Qs) @ g)
    return y, SN, d_o, d_f, d_i, dS_out


@pytest.mark.parametrize("N,C", [(32, 8), (24, 4), (64, 64)])
def test_mid_frame_form_matches_oracle(N, C):
    r = np.random.default_rng(7 + N)
    B, H, dk, dv = 1, 2, 6, 5
    o = r.standard_normal((B, H, N, dk)); i = r.standard_normal((B, H, N, dv))
    f = 0.3 + 0.7 / (1 + np.exp(-r.standard_normal((B, H, N, dk))))
    dy = r.standard_normal(i.shape)
    S0 = r.standard_normal((B, H, dk, dv)); dSN = r.standard_normal((B, H, dk, dv))
    got = midframe_fwd_bwd(o, f, i, S0, dy, dSN, C)
    y_ref, SN_ref = ref.hgrn2_fwd(o, f, i, S0)
    want = (y_ref, SN_ref) + tuple(ref.hgrn2_bwd(o, f, i, S0, dy, dSN))
    for g, w in zip(got, want):
        np.testing.assert_allclose(g, w, rtol=1e-8, atol=1e-9)
