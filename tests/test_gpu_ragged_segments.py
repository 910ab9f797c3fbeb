"""GPU parity of few long sequences whose length is NOT a whole number of chunks on the default bf16 path.

With few (batch, head) units one CTA per unit would leave most SMs idle, so the launchers cut every sequence into
segments: a state-only pass per segment, a chaining step, then the full pass per segment from its start state
(Eq. 3 is linear in the state).  Here the segments have unequal length and the last one ends inside a chunk; they
run through the per-CTA geometry of the packed batches.  Everything is compared with the fp64 oracle on the whole
sequence, forward and backward.
"""
import numpy as np
import pytest
import torch

from paper_2404_07904_b200 import binding, workloads as W
from tests import gpu_util as G

pytestmark = pytest.mark.gpu

TOL = 2e-2


def _inputs(B, H, N, seed, gamma=0.9):
    w = W.scaled(W.CONFIGS["long_16k"], B=B, H=H, N=N, has_S0=True, has_dSN=True, seed=seed, gamma=gamma)
    d = binding.make_desc(B, H, N, 128, 128, binding.HGRN2_BF16)
    assert binding.path_of(d) == "tcgen05"
    # the plan is visible in the size queries: segment scratch, and the packed batches' slot numbering of the states
    assert binding.workspace_bytes(d) > 256 + binding.saved_bytes(d) + B * H * 128 * 128 * 4, "segments expected"
    assert binding.saved_bytes(d) > B * H * ((N + 63) // 64) * (128 * 128 * 2 + 2 * 128 * 4)
    return w, W.make_inputs(w)


@pytest.mark.parametrize("N", [5000, 1000, 513])
@pytest.mark.parametrize("use_saved", [True, False])
def test_ragged_sequences_in_segments(N, use_saved):
    # 5000 tokens: 8 segments of 10 chunks, the last one 520 tokens; 1000: 512 + 488; 513: 512 + a single token
    w, inp = _inputs(1, 4, N, seed=90 + N % 7)
    got = G.gpu_fwd_bwd(inp, "bf16", use_saved=use_saved)
    for (b, h), want in G.oracle_fwd_bwd(inp, [(0, 0), (0, 3)]).items():
        G.assert_close({k: got[k][b:b + 1, h:h + 1] for k in want}, want, TOL, f"N = {N}, unit {(b, h)}")


def test_saved_and_recreated_states_agree_bitwise():
    w, inp = _inputs(2, 2, 1100, seed=95)
    a = G.gpu_fwd_bwd(inp, "bf16", use_saved=True)
    b = G.gpu_fwd_bwd(inp, "bf16", use_saved=False)
    for k in a:
        np.testing.assert_array_equal(a[k], b[k])


def test_hard_forget_stretch_inside_one_ragged_segment():
    # 1100 tokens = segments of 512, 512, 76: the stretch sits in the second segment of unit (0, 1), which alone is redone
    w, inp = _inputs(1, 2, 1100, seed=96)
    inp["f"][0, 1, 600:660, 7] = W.round_to_bf16(np.float32(0.02))
    t = G.to_dev(inp, "bf16")
    y, SN, saved, ws, _ = binding.hgrn2_fwd(t["o"], t["f"], t["i"], t["S0"])
    torch.cuda.synchronize()
    assert binding.hgrn2_poll(ws) == 0 and binding.exact_path_units(ws) == 1
    d_o, d_f, d_i, dS0, ws = binding.hgrn2_bwd(t["o"], t["f"], t["i"], t["S0"], t["dy"], t["dSN"], saved, ws=ws)
    torch.cuda.synchronize()
    assert binding.hgrn2_poll(ws) == 0 and binding.exact_path_units(ws) == 1
    got = {k: v.float().cpu().numpy() for k, v in
           {"y": y, "SN": SN, "d_o": d_o, "d_f": d_f, "d_i": d_i, "dS0": dS0}.items()}
    G.assert_close(got, G.oracle_fwd_bwd(inp), TOL, "hard-forget stretch in a ragged segment")


def test_gated_entry_points_on_ragged_segments():
    from tests import test_gpu_gated as TG
    inp = TG._inputs(1, 2, 1000, 128, "bf16", seed=97, beta_lo=0.0, beta_hi=0.9, zf_shift=1.0, states=True)
    got, _ = TG._run(inp, "bf16", use_saved=True)
    G.assert_close(got, TG._oracle(inp), TOL, "gated, 1000 tokens in two segments")


@pytest.mark.parametrize("use_saved", [True, False])
def test_units_beyond_the_last_full_wave_with_ragged_sequences(use_saved):
    # more units than SMs and sequences that are not whole chunks: the full wave runs whole, the left-over units as
    # ragged segments; units on both sides of the split are compared
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    H = sms + 12
    w = W.scaled(W.CONFIGS["long_16k"], B=1, H=H, N=1000, has_S0=True, has_dSN=True, seed=98)
    d = binding.make_desc(1, H, 1000, 128, 128, binding.HGRN2_BF16)
    assert binding.workspace_bytes(d) > 256 + binding.saved_bytes(d) + H * 128 * 128 * 4, "segments expected"
    inp = W.make_inputs(w)
    inp["f"][0, H - 3, 600:660, 5] = W.round_to_bf16(np.float32(0.02))      # second segment of a left-over unit
    got = G.gpu_fwd_bwd(inp, "bf16", use_saved=use_saved)
    units = [(0, 0), (0, sms - 1), (0, sms), (0, H - 3), (0, H - 1)]
    for (b, h), want in G.oracle_fwd_bwd(inp, units).items():
        G.assert_close({k: got[k][b:b + 1, h:h + 1] for k in want}, want, TOL, f"unit {(b, h)}")
