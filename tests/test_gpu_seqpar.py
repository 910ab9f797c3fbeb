"""GPU check of the sequence-parallel entry points on one GPU: the spans of R ranks are processed one after the
other (no kernel waits for another one), the all-gather is a stack, and the result must equal the oracle's on the
whole sequence.  Eq. 3 is linear in the state, so the spans need only their summaries (S_loc or G_loc, Lambda) of
each other.
"""
import numpy as np
import pytest
import torch

from paper_2404_07904_b200 import binding, workloads as W
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def _run_spans(inp, io, bounds, flags=0):
    t = G.to_dev(inp, io)
    R = len(bounds) - 1
    span = lambda k, r: t[k][:, :, bounds[r]:bounds[r + 1]].contiguous()
    # 1. every rank's forward summary, 2. the "all-gather"
    sums = [binding.span_summary_fwd(span("f", r), span("i", r), flags=flags) for r in range(R)]
    X_all = torch.stack([s[0] for s in sums]); lam_all = torch.stack([s[1] for s in sums])
    out = {k: [] for k in ("y", "d_o", "d_f", "d_i")}
    ctx = []
    for r in range(R):
        S_start = binding.span_compose(X_all, lam_all, 0, r, False, t["S0"])
        y, _, saved, ws, _ = binding.hgrn2_fwd(span("o", r), span("f", r), span("i", r), S_start, flags=flags)
        out["y"].append(y); ctx.append((S_start, saved, ws))
    SN = binding.span_compose(X_all, lam_all, 0, R, False, t["S0"])
    gs = [binding.span_summary_bwd(span("o", r), span("f", r), span("dy", r), flags=flags) for r in range(R)]
    G_all = torch.stack([g[0] for g in gs])
    for r in range(R):
        assert torch.equal(gs[r][1], sums[r][1]) or torch.allclose(gs[r][1], sums[r][1], rtol=1e-5, atol=0)
        dS_end = binding.span_compose(G_all, lam_all, r + 1, R, True, t["dSN"])
        S_start, saved, ws = ctx[r]
        d_o, d_f, d_i, _, _ = binding.hgrn2_bwd(span("o", r), span("f", r), span("i", r), S_start, span("dy", r), dS_end,
                                                saved, ws=ws, want_dS0=False, flags=flags)
        out["d_o"].append(d_o); out["d_f"].append(d_f); out["d_i"].append(d_i)
    dS0 = binding.span_compose(G_all, lam_all, 0, R, True, t["dSN"])
    torch.cuda.synchronize()
    got = {k: torch.cat(v, dim=2).float().cpu().numpy() for k, v in out.items()}
    got["SN"], got["dS0"] = SN.cpu().numpy(), dS0.cpu().numpy()
    return got


def test_three_spans_on_the_tensor_core_kernels():
    w = W.scaled(W.CONFIGS["lm_2048"], B=1, H=3, N=640, has_S0=True, has_dSN=True, seed=61)
    inp = W.make_inputs(w)
    got = _run_spans(inp, "bf16", [0, 256, 448, 640])           # whole chunks: the state-only tensor-core kernel
    G.assert_close(got, G.oracle_fwd_bwd(inp), 2e-2, "3 spans, bf16")


def test_ragged_spans_and_the_fp32_kernels():
    w = W.scaled(W.CONFIGS["lm_2048"], B=2, H=2, N=300, has_S0=True, has_dSN=True, seed=62)
    inp = W.make_inputs(w)
    got = _run_spans(inp, "bf16", [0, 100, 101, 300])           # not whole chunks: the plain summary loops
    G.assert_close(got, G.oracle_fwd_bwd(inp), 2e-2, "ragged spans, bf16")
    w = W.scaled(W.CONFIGS["tiny_f32"], B=1, H=2, N=150, has_S0=True, has_dSN=True, seed=63)
    inp = W.make_inputs(w)
    got = _run_spans(inp, "f32", [0, 64, 150])
    G.assert_close(got, G.oracle_fwd_bwd(inp), 1e-4, "spans, fp32")


def test_one_span_is_the_ordinary_call():
    w = W.scaled(W.CONFIGS["lm_2048"], B=1, H=2, N=128, has_S0=True, has_dSN=True, seed=64)
    inp = W.make_inputs(w)
    got = _run_spans(inp, "bf16", [0, 128])
    one = G.gpu_fwd_bwd(inp, "bf16")
    for k in ("y", "d_o", "d_f", "d_i"):
        np.testing.assert_array_equal(got[k], one[k])
    G.assert_close(got, G.oracle_fwd_bwd(inp), 2e-2, "one span")
