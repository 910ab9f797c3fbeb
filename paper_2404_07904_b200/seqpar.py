"""Sequence (context) parallelism around the library: one span of every sequence per rank.

Plumbing only: the arithmetic is in the library's span entry points (``hgrn2_span_summary_*``,
``hgrn2_span_compose``) and in ``hgrn2_fwd`` / ``hgrn2_bwd``; this module orders the calls and performs the one
collective the split needs, an all-gather of each rank's span summary (``d_k + d_k d_v`` floats per unit) with
``torch.distributed`` (NCCL on GPUs).  ``ops`` is the set of calls to use - by default the CUDA binding - so that
the ordering and the collective can be exercised on CPU ranks with stand-in calls.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


class CudaOps:
    """The library's calls on CUDA tensors."""

    def __init__(self):
        from . import binding
        self.b = binding

    def summary_fwd(self, f, i):
        return self.b.span_summary_fwd(f, i)

    def summary_bwd(self, o, f, dy):
        return self.b.span_summary_bwd(o, f, dy)

    def compose(self, X_all, lam_all, r0, r1, reverse, init):
        return self.b.span_compose(X_all, lam_all, r0, r1, reverse, init)

    def fwd(self, o, f, i, S0):
        y, SN, saved, ws, _ = self.b.hgrn2_fwd(o, f, i, S0)
        return y, (saved, ws)

    def bwd(self, o, f, i, S0, dy, dSN, ctx):
        saved, ws = ctx
        d_o, d_f, d_i, _, _ = self.b.hgrn2_bwd(o, f, i, S0, dy, dSN, saved, ws=ws, want_dS0=False)
        return d_o, d_f, d_i


def _all_gather(x, group):
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    if world == 1:
        return x.unsqueeze(0).contiguous()
    out = [torch.empty_like(x) for _ in range(world)]
    dist.all_gather(out, x.contiguous(), group=group)
    return torch.stack(out, dim=0)


def forward(o, f, i, S0=None, *, ops=None, group=None):
    """This rank's span of the forward.  o, f, i: the rank's own tokens [B, H, N_span, d]; S0: the sequences' initial
    state (the same tensor on every rank, or None).  Returns (y_span, S_N of the whole sequence, ctx for backward)."""
    ops = CudaOps() if ops is None else ops
    rank = dist.get_rank(group) if dist.is_initialized() else 0
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    S_loc, lam = ops.summary_fwd(f, i)
    X_all, lam_all = _all_gather(S_loc, group), _all_gather(lam, group)
    S_start = ops.compose(X_all, lam_all, 0, rank, False, S0)
    S_final = ops.compose(X_all, lam_all, 0, world, False, S0)
    y, inner = ops.fwd(o, f, i, S_start)
    return y, S_final, (S_start, lam_all, inner)


def backward(o, f, i, dy, dSN=None, *, ctx, ops=None, group=None):
    """This rank's span of the backward.  dSN: gradient with respect to the whole sequence's final state (the same
    tensor on every rank, or None).  Returns (d_o, d_f, d_i of the span, dS_0 of the whole sequence)."""
    ops = CudaOps() if ops is None else ops
    rank = dist.get_rank(group) if dist.is_initialized() else 0
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    S_start, lam_all, inner = ctx
    G_loc, _ = ops.summary_bwd(o, f, dy)
    G_all = _all_gather(G_loc, group)
    dS_end = ops.compose(G_all, lam_all, rank + 1, world, True, dSN)
    dS0 = ops.compose(G_all, lam_all, 0, world, True, dSN)
    d_o, d_f, d_i = ops.bwd(o, f, i, S_start, dy, dS_end, inner)
    return d_o, d_f, d_i, dS0
