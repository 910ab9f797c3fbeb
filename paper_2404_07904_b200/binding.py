"""Thin Python binding of the C-ABI library (``include/hgrn2.h``): argument marshalling only.

Tensors are ``torch`` CUDA tensors used purely as device memory; every step of the
recurrence runs inside ``libhgrn2.so``.  There is no CPU or eager fallback: if the library
is missing or fails to load, importing this module's functions raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libhgrn2.so")

HGRN2_F32, HGRN2_BF16 = 0, 1
FLAG_FORCE_ALU = 1
FLAG_DEBUG_EXPIRE_WAITS = 0x80000000

STATUS_NAMES = {
    0: "HGRN2_OK", 1: "HGRN2_ERR_INVALID_ARG", 2: "HGRN2_ERR_UNSUPPORTED", 3: "HGRN2_ERR_ALIGNMENT",
    4: "HGRN2_ERR_WORKSPACE", 5: "HGRN2_ERR_CUDA", 6: "HGRN2_ERR_TIMEOUT", 7: "HGRN2_ERR_DOMAIN",
}

# Every symbol include/hgrn2.h declares.
EXPORTS = (
    "hgrn2_saved_bytes", "hgrn2_workspace_bytes", "hgrn2_fwd", "hgrn2_bwd", "hgrn2_step",
    "hgrn2_step_multi", "hgrn2_poll", "hgrn2_status_string", "hgrn2_chunk", "hgrn2_path", "hgrn2_bwd_static_scratch",
    "hgrn2_exact_path_units", "hgrn2_saved_bytes_varlen", "hgrn2_workspace_bytes_varlen", "hgrn2_fwd_varlen",
    "hgrn2_bwd_varlen", "hgrn2_span_summary_fwd", "hgrn2_span_summary_bwd", "hgrn2_span_compose", "hgrn2_saved_bytes_gated", "hgrn2_workspace_bytes_gated", "hgrn2_fwd_gated", "hgrn2_bwd_gated",
)
STATIC_SCRATCH_BYTES = 32 * 1024 * 1024


class Hgrn2Error(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {STATUS_NAMES.get(code, code)} ({status_string(code)})")


class Desc(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("H", ctypes.c_int32), ("N", ctypes.c_int32),
                ("dk", ctypes.c_int32), ("dv", ctypes.c_int32), ("io", ctypes.c_int32),
                ("chunk", ctypes.c_int32), ("flags", ctypes.c_uint32)]


_lib = None


def load() -> ctypes.CDLL:
    """Load libhgrn2.so (built in-tree by ``paper_2404_07904_b200.build``); raises if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2404_07904_b200.build` "
            "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, dp = ctypes.c_void_p, ctypes.POINTER(Desc)
    lib.hgrn2_saved_bytes.restype = ctypes.c_size_t
    lib.hgrn2_saved_bytes.argtypes = [dp]
    lib.hgrn2_workspace_bytes.restype = ctypes.c_size_t
    lib.hgrn2_workspace_bytes.argtypes = [dp]
    lib.hgrn2_chunk.restype = ctypes.c_int32
    lib.hgrn2_chunk.argtypes = [dp]
    lib.hgrn2_path.restype = ctypes.c_char_p
    lib.hgrn2_path.argtypes = [dp]
    lib.hgrn2_status_string.restype = ctypes.c_char_p
    lib.hgrn2_status_string.argtypes = [ctypes.c_int]
    lib.hgrn2_poll.restype = ctypes.c_int
    lib.hgrn2_poll.argtypes = [vp]
    lib.hgrn2_exact_path_units.restype = ctypes.c_int32
    lib.hgrn2_exact_path_units.argtypes = [vp]
    lib.hgrn2_fwd.restype = ctypes.c_int
    lib.hgrn2_fwd.argtypes = [dp] + [vp] * 9
    lib.hgrn2_bwd.restype = ctypes.c_int
    lib.hgrn2_bwd.argtypes = [dp] + [vp] * 13
    lib.hgrn2_saved_bytes_varlen.restype = ctypes.c_size_t
    lib.hgrn2_saved_bytes_varlen.argtypes = [dp]
    lib.hgrn2_workspace_bytes_varlen.restype = ctypes.c_size_t
    lib.hgrn2_workspace_bytes_varlen.argtypes = [dp]
    lib.hgrn2_fwd_varlen.restype = ctypes.c_int
    lib.hgrn2_fwd_varlen.argtypes = [dp] + [vp] * 10
    lib.hgrn2_bwd_varlen.restype = ctypes.c_int
    lib.hgrn2_bwd_varlen.argtypes = [dp] + [vp] * 14
    lib.hgrn2_span_summary_fwd.restype = ctypes.c_int
    lib.hgrn2_span_summary_fwd.argtypes = [dp] + [vp] * 6
    lib.hgrn2_span_summary_bwd.restype = ctypes.c_int
    lib.hgrn2_span_summary_bwd.argtypes = [dp] + [vp] * 7
    lib.hgrn2_span_compose.restype = ctypes.c_int
    lib.hgrn2_span_compose.argtypes = [dp, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32] + [vp] * 5
    lib.hgrn2_saved_bytes_gated.restype = ctypes.c_size_t
    lib.hgrn2_saved_bytes_gated.argtypes = [dp]
    lib.hgrn2_workspace_bytes_gated.restype = ctypes.c_size_t
    lib.hgrn2_workspace_bytes_gated.argtypes = [dp]
    lib.hgrn2_fwd_gated.restype = ctypes.c_int
    lib.hgrn2_fwd_gated.argtypes = [dp] + [vp] * 10
    lib.hgrn2_bwd_gated.restype = ctypes.c_int
    lib.hgrn2_bwd_gated.argtypes = [dp] + [vp] * 15
    lib.hgrn2_bwd_static_scratch.restype = ctypes.c_int
    lib.hgrn2_bwd_static_scratch.argtypes = [dp] + [vp] * 12
    lib.hgrn2_step.restype = ctypes.c_int
    lib.hgrn2_step.argtypes = [dp] + [vp] * 6
    lib.hgrn2_step_multi.restype = ctypes.c_int
    lib.hgrn2_step_multi.argtypes = [dp] + [vp] * 6
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load().hgrn2_status_string(int(code)).decode()


def _io_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return HGRN2_F32
    if t.dtype == torch.bfloat16:
        return HGRN2_BF16
    raise TypeError(f"unsupported I/O dtype {t.dtype}")


def make_desc(B, H, N, dk, dv, io, chunk=0, flags=0) -> Desc:
    return Desc(int(B), int(H), int(N), int(dk), int(dv), int(io), int(chunk), int(flags))


def saved_bytes(desc: Desc) -> int:
    return int(load().hgrn2_saved_bytes(ctypes.byref(desc)))


def workspace_bytes(desc: Desc) -> int:
    return int(load().hgrn2_workspace_bytes(ctypes.byref(desc)))


def chunk_of(desc: Desc) -> int:
    return int(load().hgrn2_chunk(ctypes.byref(desc)))


def path_of(desc: Desc) -> str:
    return load().hgrn2_path(ctypes.byref(desc)).decode()


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("the library takes device pointers: tensor is not on a CUDA device")
    if not t.is_contiguous():
        raise ValueError("tensors must be contiguous")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream: Optional[torch.cuda.Stream]):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check(code: int, what: str):
    if code != 0:
        raise Hgrn2Error(code, what)


def alloc_workspace(desc: Desc, device) -> torch.Tensor:
    n = workspace_bytes(desc)
    if n == 0:
        raise Hgrn2Error(2, "hgrn2_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=device)


def alloc_saved(desc: Desc, device) -> torch.Tensor:
    return torch.empty(max(saved_bytes(desc), 16), dtype=torch.uint8, device=device)


def hgrn2_fwd(o, f, i, S0=None, *, y=None, SN=None, saved=None, ws=None, want_final_state=True,
              save_for_backward=True, chunk=0, flags=0, stream=None):
    """Forward over [B, H, N, d] tensors.  Returns (y, SN, saved, ws, desc); buffers that are not passed in
    are allocated with torch (device memory only)."""
    B, H, N, dk = o.shape
    dv = i.shape[-1]
    desc = make_desc(B, H, N, dk, dv, _io_code(o), chunk, flags)
    dev = o.device
    if y is None:
        y = torch.empty((B, H, N, dv), dtype=o.dtype, device=dev)
    if SN is None and want_final_state:
        SN = torch.empty((B, H, dk, dv), dtype=torch.float32, device=dev)
    if saved is None and save_for_backward:
        saved = alloc_saved(desc, dev)
    if ws is None:
        ws = alloc_workspace(desc, dev)
    code = load().hgrn2_fwd(ctypes.byref(desc), _ptr(o), _ptr(f), _ptr(i), _ptr(S0), _ptr(y), _ptr(SN),
                            _ptr(saved), _ptr(ws), _stream(stream))
    _check(code, "hgrn2_fwd")
    return y, SN, saved, ws, desc


def hgrn2_bwd(o, f, i, S0, dy, dSN=None, saved=None, *, d_o=None, d_f=None, d_i=None, dS0=None, ws=None,
              want_dS0=True, chunk=0, flags=0, stream=None):
    """Backward of hgrn2_fwd.  Returns (d_o, d_f, d_i, dS0, ws)."""
    B, H, N, dk = o.shape
    dv = i.shape[-1]
    desc = make_desc(B, H, N, dk, dv, _io_code(o), chunk, flags)
    dev = o.device
    d_o = torch.empty_like(o) if d_o is None else d_o
    d_f = torch.empty_like(f) if d_f is None else d_f
    d_i = torch.empty_like(i) if d_i is None else d_i
    if dS0 is None and want_dS0:
        dS0 = torch.empty((B, H, dk, dv), dtype=torch.float32, device=dev)
    if ws is None:
        ws = alloc_workspace(desc, dev)
    code = load().hgrn2_bwd(ctypes.byref(desc), _ptr(o), _ptr(f), _ptr(i), _ptr(S0), _ptr(dy), _ptr(dSN),
                            _ptr(saved), _ptr(d_o), _ptr(d_f), _ptr(d_i), _ptr(dS0), _ptr(ws), _stream(stream))
    _check(code, "hgrn2_bwd")
    return d_o, d_f, d_i, dS0, ws


def hgrn2_fwd_varlen(o, f, i, cu_seqlens, S0=None, *, y=None, SN=None, saved=None, ws=None, want_final_state=True,
                     save_for_backward=True, chunk=0, flags=0, stream=None):
    """Forward over a packed batch: o, f [H, T, dk], i [H, T, dv]; cu_seqlens int32 [B + 1] on the device; states
    [B, H, dk, dv].  Returns (y, SN, saved, ws, desc)."""
    H, T, dk = o.shape
    dv = i.shape[-1]
    B = cu_seqlens.numel() - 1
    if cu_seqlens.dtype != torch.int32:
        raise TypeError("cu_seqlens must be int32")
    desc = make_desc(B, H, T, dk, dv, _io_code(o), chunk, flags)
    dev = o.device
    if y is None:
        y = torch.empty((H, T, dv), dtype=o.dtype, device=dev)
    if SN is None and want_final_state:
        SN = torch.empty((B, H, dk, dv), dtype=torch.float32, device=dev)
    lib = load()
    if saved is None and save_for_backward:
        saved = torch.empty(max(int(lib.hgrn2_saved_bytes_varlen(ctypes.byref(desc))), 16), dtype=torch.uint8, device=dev)
    if ws is None:
        ws = torch.empty(int(lib.hgrn2_workspace_bytes_varlen(ctypes.byref(desc))), dtype=torch.uint8, device=dev)
    code = lib.hgrn2_fwd_varlen(ctypes.byref(desc), _ptr(o), _ptr(f), _ptr(i), _ptr(cu_seqlens), _ptr(S0), _ptr(y),
                                _ptr(SN), _ptr(saved), _ptr(ws), _stream(stream))
    _check(code, "hgrn2_fwd_varlen")
    return y, SN, saved, ws, desc


def hgrn2_bwd_varlen(o, f, i, cu_seqlens, S0, dy, dSN=None, saved=None, *, d_o=None, d_f=None, d_i=None, dS0=None,
                     ws=None, want_dS0=True, chunk=0, flags=0, stream=None):
    """Backward of hgrn2_fwd_varlen.  Returns (d_o, d_f, d_i, dS0, ws)."""
    H, T, dk = o.shape
    dv = i.shape[-1]
    B = cu_seqlens.numel() - 1
    desc = make_desc(B, H, T, dk, dv, _io_code(o), chunk, flags)
    dev = o.device
    d_o = torch.empty_like(o) if d_o is None else d_o
    d_f = torch.empty_like(f) if d_f is None else d_f
    d_i = torch.empty_like(i) if d_i is None else d_i
    if dS0 is None and want_dS0:
        dS0 = torch.empty((B, H, dk, dv), dtype=torch.float32, device=dev)
    lib = load()
    if ws is None:
        ws = torch.empty(int(lib.hgrn2_workspace_bytes_varlen(ctypes.byref(desc))), dtype=torch.uint8, device=dev)
    code = lib.hgrn2_bwd_varlen(ctypes.byref(desc), _ptr(o), _ptr(f), _ptr(i), _ptr(cu_seqlens), _ptr(S0), _ptr(dy),
                                _ptr(dSN), _ptr(saved), _ptr(d_o), _ptr(d_f), _ptr(d_i), _ptr(dS0), _ptr(ws),
                                _stream(stream))
    _check(code, "hgrn2_bwd_varlen")
    return d_o, d_f, d_i, dS0, ws


def span_summary_fwd(f, i, *, ws=None, chunk=0, flags=0, stream=None):
    """A span's end state from a zero start state and its total decay: (S_loc [B,H,dk,dv], lam [B,H,dk])."""
    B, H, N, dk = f.shape
    dv = i.shape[-1]
    desc = make_desc(B, H, N, dk, dv, _io_code(f), chunk, flags)
    S_loc = torch.empty((B, H, dk, dv), dtype=torch.float32, device=f.device)
    lam = torch.empty((B, H, dk), dtype=torch.float32, device=f.device)
    ws = torch.empty(256, dtype=torch.uint8, device=f.device) if ws is None else ws
    _check(load().hgrn2_span_summary_fwd(ctypes.byref(desc), _ptr(f), _ptr(i), _ptr(S_loc), _ptr(lam), _ptr(ws),
                                         _stream(stream)), "hgrn2_span_summary_fwd")
    return S_loc, lam


def span_summary_bwd(o, f, dy, *, ws=None, chunk=0, flags=0, stream=None):
    """A span's state gradient at its start from a zero gradient at its end, and its total decay."""
    B, H, N, dk = o.shape
    dv = dy.shape[-1]
    desc = make_desc(B, H, N, dk, dv, _io_code(o), chunk, flags)
    G_loc = torch.empty((B, H, dk, dv), dtype=torch.float32, device=o.device)
    lam = torch.empty((B, H, dk), dtype=torch.float32, device=o.device)
    ws = torch.empty(256, dtype=torch.uint8, device=o.device) if ws is None else ws
    _check(load().hgrn2_span_summary_bwd(ctypes.byref(desc), _ptr(o), _ptr(f), _ptr(dy), _ptr(G_loc), _ptr(lam), _ptr(ws),
                                         _stream(stream)), "hgrn2_span_summary_bwd")
    return G_loc, lam


def span_compose(X_all, lam_all, r0, r1, reverse=False, init=None, *, stream=None):
    """Fold the spans r0 <= r < r1 (ascending, or descending when `reverse`) of X_all [R,B,H,dk,dv], lam_all [R,B,H,dk]
    onto `init` (None = zero): S <- Diag(lam[r]) S + X[r].  Returns [B,H,dk,dv] float32."""
    R, B, H, dk, dv = X_all.shape
    desc = make_desc(B, H, 0, dk, dv, HGRN2_F32)
    out = torch.empty((B, H, dk, dv), dtype=torch.float32, device=X_all.device)
    _check(load().hgrn2_span_compose(ctypes.byref(desc), int(r0), int(r1), int(bool(reverse)), _ptr(X_all), _ptr(lam_all),
                                     _ptr(init), _ptr(out), _stream(stream)), "hgrn2_span_compose")
    return out


def hgrn2_fwd_gated(zo, zf, zi, beta, S0=None, *, y=None, SN=None, saved=None, ws=None, want_final_state=True,
                    save_for_backward=True, chunk=0, flags=0, stream=None):
    """Forward from the pre-activations: o = sigmoid(zo), f = beta + (1 - beta) sigmoid(zf), i = silu(zi), then the
    recurrence.  zo, zf [B, H, N, dk], zi [B, H, N, dv], beta [H, dk] float32.  Returns (y, SN, saved, ws, desc)."""
    B, H, N, dk = zo.shape
    dv = zi.shape[-1]
    desc = make_desc(B, H, N, dk, dv, _io_code(zo), chunk, flags)
    dev = zo.device
    lib = load()
    if y is None:
        y = torch.empty((B, H, N, dv), dtype=zo.dtype, device=dev)
    if SN is None and want_final_state:
        SN = torch.empty((B, H, dk, dv), dtype=torch.float32, device=dev)
    if saved is None and save_for_backward:
        saved = torch.empty(max(int(lib.hgrn2_saved_bytes_gated(ctypes.byref(desc))), 16), dtype=torch.uint8, device=dev)
    if ws is None:
        ws = torch.empty(int(lib.hgrn2_workspace_bytes_gated(ctypes.byref(desc))), dtype=torch.uint8, device=dev)
    code = lib.hgrn2_fwd_gated(ctypes.byref(desc), _ptr(zo), _ptr(zf), _ptr(zi), _ptr(beta), _ptr(S0), _ptr(y), _ptr(SN),
                               _ptr(saved), _ptr(ws), _stream(stream))
    _check(code, "hgrn2_fwd_gated")
    return y, SN, saved, ws, desc


def hgrn2_bwd_gated(zo, zf, zi, beta, S0, dy, dSN=None, saved=None, *, d_zo=None, d_zf=None, d_zi=None, d_beta=None,
                    dS0=None, ws=None, want_dS0=True, want_d_beta=True, chunk=0, flags=0, stream=None):
    """Backward of hgrn2_fwd_gated.  Returns (d_zo, d_zf, d_zi, d_beta, dS0, ws)."""
    B, H, N, dk = zo.shape
    dv = zi.shape[-1]
    desc = make_desc(B, H, N, dk, dv, _io_code(zo), chunk, flags)
    dev = zo.device
    lib = load()
    d_zo = torch.empty_like(zo) if d_zo is None else d_zo
    d_zf = torch.empty_like(zf) if d_zf is None else d_zf
    d_zi = torch.empty_like(zi) if d_zi is None else d_zi
    if d_beta is None and want_d_beta:
        d_beta = torch.empty((H, dk), dtype=torch.float32, device=dev)
    if dS0 is None and want_dS0:
        dS0 = torch.empty((B, H, dk, dv), dtype=torch.float32, device=dev)
    if ws is None:
        ws = torch.empty(int(lib.hgrn2_workspace_bytes_gated(ctypes.byref(desc))), dtype=torch.uint8, device=dev)
    code = lib.hgrn2_bwd_gated(ctypes.byref(desc), _ptr(zo), _ptr(zf), _ptr(zi), _ptr(beta), _ptr(S0), _ptr(dy),
                               _ptr(dSN), _ptr(saved), _ptr(d_zo), _ptr(d_zf), _ptr(d_zi), _ptr(d_beta), _ptr(dS0),
                               _ptr(ws), _stream(stream))
    _check(code, "hgrn2_bwd_gated")
    return d_zo, d_zf, d_zi, d_beta, dS0, ws


def hgrn2_bwd_static_scratch(o, f, i, S0, dy, dSN, d_o, d_f, d_i, dS0=None, status_out=None, *, chunk=0, flags=0,
                             stream=None):
    """Backward for callers that may not allocate: every buffer, outputs included, is passed in, and the
    chunk-state scratch is the fixed array inside the library (problems whose states exceed
    STATIC_SCRATCH_BYTES raise HGRN2_ERR_WORKSPACE).  This wrapper allocates nothing either.  Calls that
    may overlap on the GPU share that array and must be serialised by the caller."""
    B, H, N, dk = o.shape
    dv = i.shape[-1]
    desc = make_desc(B, H, N, dk, dv, _io_code(o), chunk, flags)
    code = load().hgrn2_bwd_static_scratch(ctypes.byref(desc), _ptr(o), _ptr(f), _ptr(i), _ptr(S0), _ptr(dy),
                                           _ptr(dSN), _ptr(d_o), _ptr(d_f), _ptr(d_i), _ptr(dS0), _ptr(status_out),
                                           _stream(stream))
    _check(code, "hgrn2_bwd_static_scratch")
    return d_o, d_f, d_i, dS0


def hgrn2_step(o, f, i, S, *, y=None, stream=None):
    """One decode step on [B, H, d] gates; S [B, H, dk, dv] float32 is updated in place.  Returns y."""
    B, H, dk = o.shape
    dv = i.shape[-1]
    desc = make_desc(B, H, 1, dk, dv, _io_code(o))
    if y is None:
        y = torch.empty((B, H, dv), dtype=o.dtype, device=o.device)
    code = load().hgrn2_step(ctypes.byref(desc), _ptr(o), _ptr(f), _ptr(i), _ptr(S), _ptr(y), _stream(stream))
    _check(code, "hgrn2_step")
    return y


def hgrn2_step_multi(o, f, i, S, *, y=None, stream=None):
    """T successive decode steps in one launch on [B, H, T, d] gates; S [B, H, dk, dv] float32 is updated in
    place to the state after the last token.  Returns y [B, H, T, dv]."""
    B, H, T, dk = o.shape
    dv = i.shape[-1]
    desc = make_desc(B, H, T, dk, dv, _io_code(o))
    if y is None:
        y = torch.empty((B, H, T, dv), dtype=o.dtype, device=o.device)
    code = load().hgrn2_step_multi(ctypes.byref(desc), _ptr(o), _ptr(f), _ptr(i), _ptr(S), _ptr(y), _stream(stream))
    _check(code, "hgrn2_step_multi")
    return y


def exact_path_units(ws: torch.Tensor) -> int:
    """Unit passes the last tensor-core call using `ws` redid on the exact fp32 path (synchronise first)."""
    return int(load().hgrn2_exact_path_units(_ptr(ws)))


def hgrn2_poll(ws: torch.Tensor) -> int:
    """Device-side status of the last call that used `ws` (synchronise its stream first)."""
    return int(load().hgrn2_poll(_ptr(ws)))
