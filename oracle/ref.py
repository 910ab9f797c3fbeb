"""ctypes front end of the fp64 C oracle (``hgrn2_ref.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline / reference arm.  The CUDA package never imports it.

Every function takes and returns ``numpy.float64`` arrays in the layouts of the C
file: sequence tensors ``[B, H, N, d]``, states ``[B, H, d_k, d_v]``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hgrn2_ref.c")
_LIB = os.path.join(_HERE, "libhgrn2_ref.so")

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, OpenMP over the independent (b, h) units)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.hgrn2_ref_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().hgrn2_ref_num_threads())


_DP = ctypes.POINTER(ctypes.c_double)


def _in(x):
    if x is None:
        return None, ctypes.cast(None, _DP)
    a = np.ascontiguousarray(x, dtype=np.float64)
    return a, a.ctypes.data_as(_DP)


def _out(shape):
    a = np.empty(shape, dtype=np.float64)
    return a, a.ctypes.data_as(_DP)


def _check(rc, name):
    if rc != 0:
        raise RuntimeError(f"{name} failed with code {rc}")


def gla_fwd(q, k, v, a, S0=None):
    """Untied recurrence S_t = Diag(a_t) S_{t-1} + k_t^T v_t, y_t = q_t S_t.  Returns (y, S_N)."""
    B, H, N, dk = q.shape
    dv = v.shape[-1]
    q_, qp = _in(q); k_, kp = _in(k); v_, vp = _in(v); a_, ap = _in(a); s_, sp = _in(S0)
    y, yp = _out((B, H, N, dv)); SN, snp = _out((B, H, dk, dv))
    rc = _load().ref_gla_fwd(B, H, ctypes.c_long(N), dk, dv, qp, kp, vp, ap, sp, yp, snp)
    _check(rc, "ref_gla_fwd")
    return y, SN


def gla_bwd(q, k, v, a, S0, dy, dSN=None):
    """VJP of gla_fwd for L = <dy, y> + <dSN, S_N>.  Returns (dq, dk, dv, da, dS0)."""
    B, H, N, dk = q.shape
    dv = v.shape[-1]
    q_, qp = _in(q); k_, kp = _in(k); v_, vp = _in(v); a_, ap = _in(a); s_, sp = _in(S0)
    dy_, dyp = _in(dy); dsn_, dsnp = _in(dSN)
    dq, dqp = _out((B, H, N, dk)); dkk, dkp = _out((B, H, N, dk)); da, dap = _out((B, H, N, dk))
    dvv, dvp = _out((B, H, N, dv)); dS0, ds0p = _out((B, H, dk, dv))
    rc = _load().ref_gla_bwd(B, H, ctypes.c_long(N), dk, dv, qp, kp, vp, ap, sp, dyp, dsnp,
                             dqp, dkp, dvp, dap, ds0p)
    _check(rc, "ref_gla_bwd")
    return dq, dkk, dvv, da, dS0


def hgrn2_fwd(o, f, i, S0=None):
    """Eq. 3 with tied gates.  Returns (y, S_N)."""
    B, H, N, dk = o.shape
    dv = i.shape[-1]
    o_, op = _in(o); f_, fp = _in(f); i_, ip = _in(i); s_, sp = _in(S0)
    y, yp = _out((B, H, N, dv)); SN, snp = _out((B, H, dk, dv))
    rc = _load().ref_hgrn2_fwd(B, H, ctypes.c_long(N), dk, dv, op, fp, ip, sp, yp, snp)
    _check(rc, "ref_hgrn2_fwd")
    return y, SN


def hgrn2_bwd(o, f, i, S0, dy, dSN=None):
    """VJP of hgrn2_fwd.  Returns (d_o, d_f, d_i, dS0); d_f folds the decay and the 1-f paths."""
    B, H, N, dk = o.shape
    dv = i.shape[-1]
    o_, op = _in(o); f_, fp = _in(f); i_, ip = _in(i); s_, sp = _in(S0)
    dy_, dyp = _in(dy); dsn_, dsnp = _in(dSN)
    d_o, dop = _out((B, H, N, dk)); d_f, dfp = _out((B, H, N, dk))
    d_i, dip = _out((B, H, N, dv)); dS0, ds0p = _out((B, H, dk, dv))
    rc = _load().ref_hgrn2_bwd(B, H, ctypes.c_long(N), dk, dv, op, fp, ip, sp, dyp, dsnp,
                               dop, dfp, dip, ds0p)
    _check(rc, "ref_hgrn2_bwd")
    return d_o, d_f, d_i, dS0


def hgrn2_step(o, f, i, S):
    """One decode step.  o, f: [B, H, d_k]; i: [B, H, d_v]; S: [B, H, d_k, d_v] float64, updated IN PLACE.
    Returns y [B, H, d_v]."""
    B, H, dk = o.shape
    dv = i.shape[-1]
    if S.dtype != np.float64 or not S.flags["C_CONTIGUOUS"]:
        raise ValueError("S must be a contiguous float64 array (it is updated in place)")
    o_, op = _in(o); f_, fp = _in(f); i_, ip = _in(i)
    y, yp = _out((B, H, dv))
    rc = _load().ref_hgrn2_step(B, H, dk, dv, op, fp, ip, S.ctypes.data_as(_DP), yp)
    _check(rc, "ref_hgrn2_step")
    return y


def hgrn2_fwd_varlen(o, f, i, cu, S0=None):
    """Packed batch: o, f [H, T, d_k], i [H, T, d_v]; sequence b occupies rows cu[b]:cu[b+1] of every head and
    starts from S0[b] ([B, H, d_k, d_v], or zero).  No arithmetic of its own: every sequence goes through
    hgrn2_fwd (Eq. 3) separately.  Returns (y [H, T, d_v], S_N [B, H, d_k, d_v])."""
    H, T, dk = o.shape
    dv = i.shape[-1]
    B = len(cu) - 1
    y = np.zeros((H, T, dv), dtype=np.float64)
    SN = np.zeros((B, H, dk, dv), dtype=np.float64)
    for b in range(B):
        s, e = int(cu[b]), int(cu[b + 1])
        s0 = None if S0 is None else np.asarray(S0[b:b + 1], dtype=np.float64)
        if e == s:
            SN[b] = 0.0 if s0 is None else s0[0]
            continue
        yb, snb = hgrn2_fwd(o[None, :, s:e], f[None, :, s:e], i[None, :, s:e], s0)
        y[:, s:e] = yb[0]
        SN[b] = snb[0]
    return y, SN


def hgrn2_bwd_varlen(o, f, i, cu, S0, dy, dSN=None):
    """VJP of hgrn2_fwd_varlen, sequence by sequence through hgrn2_bwd.  Returns (d_o, d_f, d_i, dS0)."""
    H, T, dk = o.shape
    dv = i.shape[-1]
    B = len(cu) - 1
    d_o = np.zeros((H, T, dk), dtype=np.float64)
    d_f = np.zeros((H, T, dk), dtype=np.float64)
    d_i = np.zeros((H, T, dv), dtype=np.float64)
    dS0 = np.zeros((B, H, dk, dv), dtype=np.float64)
    for b in range(B):
        s, e = int(cu[b]), int(cu[b + 1])
        s0 = None if S0 is None else np.asarray(S0[b:b + 1], dtype=np.float64)
        dsn = None if dSN is None else np.asarray(dSN[b:b + 1], dtype=np.float64)
        if e == s:
            dS0[b] = 0.0 if dsn is None else dsn[0]
            continue
        a, c, d, g = hgrn2_bwd(o[None, :, s:e], f[None, :, s:e], i[None, :, s:e], s0, dy[None, :, s:e], dsn)
        d_o[:, s:e], d_f[:, s:e], d_i[:, s:e], dS0[b] = a[0], c[0], d[0], g[0]
    return d_o, d_f, d_i, dS0


def _sigmoid(x):
    return 1.0 / (1.0 + np.exp(-np.asarray(x, dtype=np.float64)))


def gates(zo, zf, zi, beta):
    """Eq. 1 / Eq. 2: o = sigmoid(zo), f = beta + (1 - beta) sigmoid(zf), i = zi sigmoid(zi) (SiLU).
    z* [B, H, N, d]; beta [H, d_k], broadcast over batch and time."""
    b = np.asarray(beta, dtype=np.float64)[None, :, None, :]
    zi = np.asarray(zi, dtype=np.float64)
    return _sigmoid(zo), b + (1.0 - b) * _sigmoid(zf), zi * _sigmoid(zi)


def hgrn2_fwd_gated(zo, zf, zi, beta, S0=None):
    """The gate activations followed by Eq. 3.  Returns (y, S_N)."""
    o, f, i = gates(zo, zf, zi, beta)
    return hgrn2_fwd(o, f, i, S0)


def hgrn2_bwd_gated(zo, zf, zi, beta, S0, dy, dSN=None):
    """VJP of hgrn2_fwd_gated: hgrn2_bwd, then the chain rule through the three activations.
    Returns (d_zo, d_zf, d_zi, d_beta [H, d_k], dS0)."""
    o, f, i = gates(zo, zf, zi, beta)
    d_o, d_f, d_i, dS0 = hgrn2_bwd(o, f, i, S0, dy, dSN)
    b = np.asarray(beta, dtype=np.float64)[None, :, None, :]
    g = _sigmoid(zf)
    zi = np.asarray(zi, dtype=np.float64)
    si = _sigmoid(zi)
    d_zo = d_o * o * (1.0 - o)
    d_zf = d_f * (1.0 - b) * g * (1.0 - g)
    d_zi = d_i * si * (1.0 + zi * (1.0 - si))
    d_beta = (d_f * (1.0 - g)).sum(axis=(0, 2))
    return d_zo, d_zf, d_zi, d_beta, dS0
