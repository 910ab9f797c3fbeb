"""The allocation-free backward entry point, checked against the ordinary one.

`hgrn2_bwd_static_scratch` serves callers that cannot allocate device memory where they call the
library (a process whose memory pool already owns the whole GPU, a plug-in that is given tensors
but no allocator, a loop in which cudaMalloc's implicit synchronisation is not acceptable): it
keeps its chunk-state scratch in an array inside the library.  This file is collected last on
purpose, so that a run that stops at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2404_07904_b200 import binding, workloads as W
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def _reference(t, chunk):
    """Outputs of the existing entry points: hgrn2_fwd (saving its chunk states) then hgrn2_bwd."""
    _, _, saved, ws, _ = binding.hgrn2_fwd(t["o"], t["f"], t["i"], t["S0"], chunk=chunk)
    d_o, d_f, d_i, dS0, _ = binding.hgrn2_bwd(t["o"], t["f"], t["i"], t["S0"], t["dy"], t["dSN"], saved, ws=ws,
                                              chunk=chunk)
    torch.cuda.synchronize()
    return d_o, d_f, d_i, dS0


def _static(t, chunk):
    outs = [torch.empty_like(t["o"]), torch.empty_like(t["f"]), torch.empty_like(t["i"]),
            torch.empty((*t["o"].shape[:2], t["o"].shape[-1], t["i"].shape[-1]), dtype=torch.float32, device="cuda")]
    status = torch.full((64,), 7, dtype=torch.int32, device="cuda")
    binding.hgrn2_bwd_static_scratch(t["o"], t["f"], t["i"], t["S0"], t["dy"], t["dSN"], outs[0], outs[1], outs[2],
                                     outs[3], status, chunk=chunk)
    torch.cuda.synchronize()
    assert binding.hgrn2_poll(status) == 0
    return outs


@pytest.mark.parametrize("io", ["bf16", "f32"])
def test_two_calls_in_a_row_match_hgrn2_bwd(io):
    base = W.CONFIGS["lm_2048"] if io == "bf16" else W.CONFIGS["tiny_f32"]
    # two different problems back to back: the second call finds the first call's states in the array
    problems = [W.scaled(base, B=1, H=3, N=300, has_S0=True, has_dSN=True, seed=31),
                W.scaled(base, B=2, H=2, N=130, has_S0=False, has_dSN=True, seed=32)]
    for w in problems:
        t = G.to_dev(W.make_inputs(w), io)
        want = _reference(t, w.chunk)
        got = _static(t, w.chunk)
        for name, g, r in zip(("d_o", "d_f", "d_i", "dS0"), got, want):
            err = G.rel_err(g.float().cpu().numpy(), r.float().cpu().numpy())
            assert err <= G.TOL[io], (name, err)


def test_matches_the_oracle_and_serves_segmented_sequences():
    # few units: the sequences run as several segments, whose scratch also lives in the built-in array; outputs
    # against hgrn2_bwd and, for two units, against the fp64 oracle
    w = W.scaled(W.CONFIGS["long_16k"], B=1, H=4, N=2048, seed=33)
    d = binding.make_desc(w.B, w.H, w.N, w.dk, w.dv, binding.HGRN2_BF16)
    assert binding.workspace_bytes(d) - 256 <= binding.STATIC_SCRATCH_BYTES
    assert binding.workspace_bytes(d) > 256 + binding.saved_bytes(d) + w.B * w.H * w.dk * w.dv * 4, "segment scratch expected"
    inp = W.make_inputs(w)
    t = G.to_dev(inp, "bf16")
    want = _reference(t, w.chunk)
    got = _static(t, w.chunk)
    names = ("d_o", "d_f", "d_i", "dS0")
    for name, g, r in zip(names, got, want):
        assert G.rel_err(g.float().cpu().numpy(), r.float().cpu().numpy()) <= G.TOL["bf16"], name
    for (b, h), wu in G.oracle_fwd_bwd(inp, [(0, 0), (0, 3)]).items():
        gu = {name: g[b:b + 1, h:h + 1].float().cpu().numpy() for name, g in zip(names, got)}
        G.assert_close(gu, {k: wu[k] for k in names}, G.TOL["bf16"], f"static scratch vs oracle, unit {(b, h)}")


def test_rejects_problems_larger_than_the_array():
    # 8 x 16 heads x 32 chunks x 32 KB of bf16 states = 128 MB > 32 MB: refused on the host, nothing runs
    d = binding.make_desc(8, 16, 2048, 128, 128, binding.HGRN2_BF16)
    assert binding.workspace_bytes(d) - 256 > binding.STATIC_SCRATCH_BYTES
    x = torch.zeros(16, dtype=torch.bfloat16, device="cuda")      # never touched
    import ctypes
    p = ctypes.c_void_p(x.data_ptr())
    code = binding.load().hgrn2_bwd_static_scratch(ctypes.byref(d), p, p, p, None, p, None, p, p, p, None, None, None)
    assert code == 4
    bad = binding.make_desc(1, 1, 64, 48, 64, binding.HGRN2_BF16)
    assert binding.load().hgrn2_bwd_static_scratch(ctypes.byref(bad), p, p, p, None, p, None, p, p, p, None, None, None) == 2
