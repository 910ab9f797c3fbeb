"""GPU parity on the whole closed interval f in [0, 1] for the library's default bf16 path.

The tensor-core kernels rescale their operands by in-chunk cumulative decay and can represent a pair of
factors only while the decay across half a chunk stays above 2^-100 per key dimension.  Units that leave
that range (hard-forget gates, f == 0) must be detected on the device and redone by the pairwise-safe fp32
routines inside the same call.  Every case here goes through the default dispatch (bf16, d_k = d_v = 128:
"tcgen05"), forward and backward, against the fp64 oracle at the bf16 tolerance; Eq. 3 is defined on all of
[0, 1] and Eq. 2 with a zero lower bound allows gates that stay near zero.
"""
import numpy as np
import pytest
import torch

from paper_2404_07904_b200 import binding, workloads as W
from oracle import ref
from tests import gpu_util as G

pytestmark = pytest.mark.gpu

TOL = 2e-2


def _base(B=1, H=2, N=320, seed=11, S0=True, dSN=True):
    w = W.scaled(W.CONFIGS["lm_2048"], B=B, H=H, N=N, has_S0=S0, has_dSN=dSN, seed=seed)
    d = binding.make_desc(w.B, w.H, w.N, w.dk, w.dv, binding.HGRN2_BF16)
    assert binding.path_of(d) == "tcgen05"
    return w, W.make_inputs(w)


def _run(inp, use_saved=True):
    """Forward + backward through the C ABI; returns outputs and the exact-path unit counts of the two calls."""
    t = G.to_dev(inp, "bf16")
    y, SN, saved, ws, _ = binding.hgrn2_fwd(t["o"], t["f"], t["i"], t["S0"])
    torch.cuda.synchronize()
    assert binding.hgrn2_poll(ws) == 0
    n_fwd = binding.exact_path_units(ws)
    d_o, d_f, d_i, dS0, ws = binding.hgrn2_bwd(t["o"], t["f"], t["i"], t["S0"], t["dy"], t["dSN"],
                                               saved if use_saved else None, ws=ws)
    torch.cuda.synchronize()
    assert binding.hgrn2_poll(ws) == 0
    n_bwd = binding.exact_path_units(ws)
    got = {"y": y, "SN": SN, "d_o": d_o, "d_f": d_f, "d_i": d_i, "dS0": dS0}
    return {k: v.float().cpu().numpy() for k, v in got.items()}, n_fwd, n_bwd


def test_f_zero_forward():
    # f == 0: y_t = (sum_k o_tk) i_t whatever S0 is, and S_N = 1 i_N^T
    w, inp = _base()
    inp["f"][:] = 0.0
    t = G.to_dev(inp, "bf16")
    y, SN, _, ws, _ = binding.hgrn2_fwd(t["o"], t["f"], t["i"], t["S0"], save_for_backward=False)
    torch.cuda.synchronize()
    assert binding.hgrn2_poll(ws) == 0
    assert binding.exact_path_units(ws) == w.B * w.H
    want = inp["o"].astype(np.float64).sum(-1, keepdims=True) * inp["i"].astype(np.float64)
    assert G.rel_err(y.float().cpu().numpy(), want) <= TOL
    y_ref, SN_ref = ref.hgrn2_fwd(inp["o"], inp["f"], inp["i"], inp["S0"])
    assert G.rel_err(y.float().cpu().numpy(), y_ref) <= TOL
    assert G.rel_err(SN.cpu().numpy(), SN_ref) <= TOL


def test_f_one_forward_backward():
    # f == 1: k = 0, the state never moves (y_t = o_t S_0); stays on the tensor-core kernels
    w, inp = _base()
    inp["f"][:] = 1.0
    got, n_fwd, n_bwd = _run(inp)
    assert n_fwd == 0 and n_bwd == 0
    G.assert_close(got, G.oracle_fwd_bwd(inp), TOL, "f == 1")


@pytest.mark.parametrize("use_saved", [True, False])
def test_f_constant_hard_forget(use_saved):
    # f == 0.05: 0.05^32 = 2^-138 is far below what one reference per half chunk can carry
    w, inp = _base()
    inp["f"][:] = W.round_to_bf16(np.full_like(inp["f"], 0.05))
    got, n_fwd, n_bwd = _run(inp, use_saved)
    assert n_fwd == w.B * w.H and n_bwd == w.B * w.H * (1 if use_saved else 2)
    G.assert_close(got, G.oracle_fwd_bwd(inp), TOL, "f == 0.05")


def test_sigmoid_gates_with_negative_bias():
    # Eq. 2 with a zero lower bound and pre-activations around -3: f = sigmoid(z), z ~ N(-3, 1)
    w, inp = _base(N=200, seed=12)
    rng = np.random.default_rng(99)
    z = rng.standard_normal(inp["f"].shape, dtype=np.float32) - np.float32(3.0)
    inp["f"] = W.round_to_bf16(1.0 / (1.0 + np.exp(-z)))
    got, n_fwd, n_bwd = _run(inp)
    assert n_fwd == w.B * w.H
    G.assert_close(got, G.oracle_fwd_bwd(inp), TOL, "sigmoid(N(-3,1))")


def test_a_few_hard_forget_dimensions():
    # ordinary gates except three key dimensions of one unit that stay near zero: that unit alone is redone
    w, inp = _base(B=1, H=3, N=256, seed=13)
    inp["f"][0, 1, :, [5, 64, 127]] = W.round_to_bf16(np.float32(0.02))
    got, n_fwd, n_bwd = _run(inp)
    assert n_fwd == 1 and n_bwd == 1
    G.assert_close(got, G.oracle_fwd_bwd(inp), TOL, "few hard-forget dims")


def test_hard_forget_stretch_inside_one_chunk_only():
    # a single stretch of 40 tokens with f = 0.01 in one key dimension, ragged length
    w, inp = _base(B=1, H=2, N=300, seed=14)
    inp["f"][0, 0, 100:140, 17] = W.round_to_bf16(np.float32(0.01))
    got, n_fwd, n_bwd = _run(inp)
    assert n_fwd == 1 and n_bwd == 1
    G.assert_close(got, G.oracle_fwd_bwd(inp), TOL, "hard-forget stretch")


def test_hard_forget_unit_among_segmented_sequences():
    # few units: every sequence runs as several segments (CTAs); the last segment to finish redoes the unit
    w = W.scaled(W.CONFIGS["long_16k"], B=1, H=4, N=2048, seed=79)
    d = binding.make_desc(w.B, w.H, w.N, w.dk, w.dv, binding.HGRN2_BF16)
    assert binding.workspace_bytes(d) > 256 + binding.saved_bytes(d) + w.H * 128 * 128 * 4, "segment scratch expected"
    inp = W.make_inputs(w)
    inp["f"][0, 2, 700:760, 3] = W.round_to_bf16(np.float32(0.03))       # inside one segment of unit 2
    for use_saved in (True, False):
        got, n_fwd, n_bwd = _run(inp, use_saved)
        assert n_fwd == 1 and n_bwd == (1 if use_saved else 2)
        want = G.oracle_fwd_bwd(inp, [(0, 2), (0, 3)])
        for (b, h), wu in want.items():
            G.assert_close({k: got[k][b:b + 1, h:h + 1] for k in wu}, wu, TOL, f"segmented unit {(b, h)}")


def test_hard_forget_units_in_full_wave_and_left_over_part():
    # more units than SMs: one flagged unit in the full wave of whole units, one among the left-over segmented units
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    H = sms + 3
    w = W.scaled(W.CONFIGS["long_16k"], B=1, H=H, N=1024, seed=80)
    inp = W.make_inputs(w)
    inp["f"][0, 7, 300:350, 100] = W.round_to_bf16(np.float32(0.02))
    inp["f"][0, H - 2, 10:60, 0] = W.round_to_bf16(np.float32(0.02))
    got, n_fwd, n_bwd = _run(inp)
    assert n_fwd == 2 and n_bwd == 2
    want = G.oracle_fwd_bwd(inp, [(0, 7), (0, 8), (0, H - 2), (0, H - 1)])
    for (b, h), wu in want.items():
        G.assert_close({k: got[k][b:b + 1, h:h + 1] for k in wu}, wu, TOL, f"unit {(b, h)}")


def test_decay_within_range_per_half_chunk_but_not_per_chunk():
    # f == 0.2 in a few key dimensions: 0.2^32 = 2^-74 per half chunk stays inside the operands' range (no exact path),
    # but the product of two such totals, 2^-149, is below fp32's range: the state rescaling between two chunks must
    # apply them one after the other (the accumulator it scales is as large as the first of them is small)
    w, inp = _base(B=1, H=2, N=300, seed=15)
    inp["f"][:, :, :, [0, 17, 64, 127]] = W.round_to_bf16(np.float32(0.2))
    for use_saved in (True, False):
        got, n_fwd, n_bwd = _run(inp, use_saved)
        assert n_fwd == 0 and n_bwd == 0
        G.assert_close(got, G.oracle_fwd_bwd(inp), TOL, "f == 0.2 in four key dimensions")
