"""GPU parity of the packed (variable-length) entry points against the fp64 oracle.

A packed batch holds B sequences of different lengths end to end in [H, T, d] tensors; the state is reset to each
sequence's own initial state at its boundary (Eq. 3 per sequence; linear cost in the tokens present, Section 1).
The oracle side loops over the sequences with the ordinary reference (no new arithmetic).
"""
import numpy as np
import pytest
import torch

from paper_2404_07904_b200 import binding, workloads as W
from oracle import ref
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def _packed_inputs(lengths, H, d, io, seed, gamma=0.9, with_states=True, pad_rows=0):
    """Seeded packed inputs (the recipe of workloads.make_inputs on a [1, H, T, d] problem)."""
    T = int(sum(lengths)) + pad_rows
    B = len(lengths)
    w = W.scaled(W.CONFIGS["lm_2048"], B=1, H=H, N=T, dk=d, dv=d, io=io, gamma=gamma, seed=seed)
    inp = W.make_inputs(w)
    out = {k: np.ascontiguousarray(inp[k][0]) for k in ("o", "f", "i", "dy")}
    rng = np.random.default_rng(seed + 1000)
    out["S0"] = (rng.standard_normal((B, H, d, d), dtype=np.float32) * np.float32(0.02)) if with_states else None
    out["dSN"] = (rng.standard_normal((B, H, d, d), dtype=np.float32) * np.float32(0.02)) if with_states else None
    out["cu"] = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    return out


def _run_gpu(inp, io, use_saved=True, flags=0):
    tdt = torch.float32 if io == "f32" else torch.bfloat16
    t = {k: torch.from_numpy(inp[k]).cuda().to(tdt) for k in ("o", "f", "i", "dy")}
    S0 = None if inp["S0"] is None else torch.from_numpy(inp["S0"]).cuda()
    dSN = None if inp["dSN"] is None else torch.from_numpy(inp["dSN"]).cuda()
    cu = torch.from_numpy(inp["cu"]).cuda()
    H, T, d = t["o"].shape
    ybuf, y = G.canary((H, T, d), tdt)
    y, SN, saved, ws, _ = binding.hgrn2_fwd_varlen(t["o"], t["f"], t["i"], cu, S0, y=y, flags=flags)
    bufs = {n: G.canary((H, T, d), tdt) for n in ("d_o", "d_f", "d_i")}
    d_o, d_f, d_i, dS0, ws = binding.hgrn2_bwd_varlen(t["o"], t["f"], t["i"], cu, S0, t["dy"], dSN,
                                                     saved if use_saved else None, d_o=bufs["d_o"][1],
                                                     d_f=bufs["d_f"][1], d_i=bufs["d_i"][1], ws=ws, flags=flags)
    torch.cuda.synchronize()
    assert binding.hgrn2_poll(ws) == 0
    assert G.canary_ok(ybuf) and all(G.canary_ok(b[0]) for b in bufs.values())
    got = {"y": y, "SN": SN, "d_o": d_o, "d_f": d_f, "d_i": d_i, "dS0": dS0}
    return {k: v.float().cpu().numpy() for k, v in got.items()}, ws


def _oracle(inp):
    y, SN = ref.hgrn2_fwd_varlen(inp["o"], inp["f"], inp["i"], inp["cu"], inp["S0"])
    d_o, d_f, d_i, dS0 = ref.hgrn2_bwd_varlen(inp["o"], inp["f"], inp["i"], inp["cu"], inp["S0"], inp["dy"], inp["dSN"])
    return {"y": y, "SN": SN, "d_o": d_o, "d_f": d_f, "d_i": d_i, "dS0": dS0}


def _mask_rows(arrs, cu, T):
    """Rows that belong to no sequence (after cu[-1]) are never written: leave them out of the comparison."""
    end = int(cu[-1])
    return {k: (v[:, :end] if v.ndim == 3 and v.shape[1] == T else v) for k, v in arrs.items()}


@pytest.mark.parametrize("with_states", [True, False])
def test_packed_bf16_lengths_1_63_64_65_1000_5000(with_states):
    lengths = [1, 63, 64, 65, 1000, 5000]
    inp = _packed_inputs(lengths, H=2, d=128, io="bf16", seed=21, with_states=with_states)
    d = binding.make_desc(len(lengths), 2, int(sum(lengths)), 128, 128, binding.HGRN2_BF16)
    assert binding.path_of(d) == "tcgen05"
    got, _ = _run_gpu(inp, "bf16")
    errs = G.assert_close(got, _oracle(inp), 2e-2, "packed bf16")
    print("packed bf16", {k: f"{v:.2e}" for k, v in errs.items()})
    got2, _ = _run_gpu(inp, "bf16", use_saved=False)
    for k in got:
        np.testing.assert_array_equal(got[k], got2[k])


def test_packed_bf16_empty_sequences_and_unused_tail_rows():
    # zero-length sequences pass their state through; rows after the last sequence are left alone
    lengths = [0, 130, 0, 64, 7, 0]
    inp = _packed_inputs(lengths, H=3, d=128, io="bf16", seed=22, pad_rows=37)
    T = inp["o"].shape[1]
    got, _ = _run_gpu(inp, "bf16")
    want = _oracle(inp)
    G.assert_close(_mask_rows(got, inp["cu"], T), _mask_rows(want, inp["cu"], T), 2e-2, "packed with empties")
    for b in (0, 2, 5):
        np.testing.assert_array_equal(got["SN"][b], inp["S0"][b])
        np.testing.assert_array_equal(got["dS0"][b], inp["dSN"][b])


def test_packed_equals_separate_calls_bitwise():
    # the packed call must give exactly what one ordinary call per sequence gives (same kernels, same order; a batch
    # this short is not cut into segments)
    lengths = [200, 64, 129]
    inp = _packed_inputs(lengths, H=2, d=128, io="bf16", seed=23)
    got, _ = _run_gpu(inp, "bf16")
    for b, (s, e) in enumerate(zip(inp["cu"][:-1], inp["cu"][1:])):
        sub = {k: np.ascontiguousarray(inp[k][None, :, s:e]) for k in ("o", "f", "i", "dy")}
        sub["S0"], sub["dSN"] = inp["S0"][b:b + 1], inp["dSN"][b:b + 1]
        one = G.gpu_fwd_bwd(sub, "bf16")
        for k in ("y", "d_o", "d_f", "d_i"):
            np.testing.assert_array_equal(got[k][:, s:e], one[k][0])
        np.testing.assert_array_equal(got["SN"][b], one["SN"][0])
        np.testing.assert_array_equal(got["dS0"][b], one["dS0"][0])


def test_packed_in_segments_equals_separate_calls():
    # few units and long enough to be cut into segments: y and the gradients are still bit-identical to separate calls
    # on whole-chunk sequences run the same way; the boundary states come out of the segment chaining (state-only
    # kernel) and agree within the bf16 tolerance
    lengths = [1100, 200, 700]
    inp = _packed_inputs(lengths, H=1, d=128, io="bf16", seed=28)
    got, _ = _run_gpu(inp, "bf16")
    want = _oracle(inp)
    G.assert_close(got, want, 2e-2, "packed in segments")
    b, (s, e) = 1, (int(inp["cu"][1]), int(inp["cu"][2]))               # the 200-token sequence: a single segment
    sub = {k: np.ascontiguousarray(inp[k][None, :, s:e]) for k in ("o", "f", "i", "dy")}
    sub["S0"], sub["dSN"] = inp["S0"][b:b + 1], inp["dSN"][b:b + 1]
    one = G.gpu_fwd_bwd(sub, "bf16")
    for k in ("y", "d_o", "d_f", "d_i"):
        np.testing.assert_array_equal(got[k][:, s:e], one[k][0])
    assert G.rel_err(got["SN"][b], one["SN"][0]) <= 2e-2
    assert G.rel_err(got["dS0"][b], one["dS0"][0]) <= 2e-2


def test_packed_hard_forget_sequence_takes_the_exact_path():
    lengths = [100, 300, 70]
    inp = _packed_inputs(lengths, H=2, d=128, io="bf16", seed=24)
    s = int(inp["cu"][1])
    inp["f"][1, s + 50:s + 120, 9] = W.round_to_bf16(np.float32(0.02))      # sequence 1, head 1
    got, ws = _run_gpu(inp, "bf16")
    assert binding.exact_path_units(ws) == 1
    G.assert_close(got, _oracle(inp), 2e-2, "packed, one hard-forget unit")


def test_packed_long_sequences_run_as_segments():
    # few units: every sequence is cut into segments on the device (its length is known only there); a hard-forget
    # stretch in a late segment of one sequence puts that segment alone on the exact path
    lengths = [3000, 0, 5000, 700]
    inp = _packed_inputs(lengths, H=2, d=128, io="bf16", seed=27)
    d = binding.make_desc(len(lengths), 2, int(sum(lengths)), 128, 128, binding.HGRN2_BF16)
    assert lib_ws_has_segments(d)
    s = int(inp["cu"][2])
    inp["f"][1, s + 4000:s + 4070, 11] = W.round_to_bf16(np.float32(0.02))
    got, ws = _run_gpu(inp, "bf16")
    assert binding.exact_path_units(ws) == 1
    G.assert_close(got, _oracle(inp), 2e-2, "packed long sequences")
    got2, _ = _run_gpu(inp, "bf16", use_saved=False)
    for k in got:
        np.testing.assert_array_equal(got[k], got2[k])


def lib_ws_has_segments(d):
    lib = binding.load()
    import ctypes
    ws = lib.hgrn2_workspace_bytes_varlen(ctypes.byref(d))
    saved = lib.hgrn2_saved_bytes_varlen(ctypes.byref(d))
    return ws > 256 + saved + 8 * d.B * d.H * 128 * 128 * 4          # room for eight segments per unit


@pytest.mark.parametrize("io,d,flags", [("f32", 64, 0), ("bf16", 128, binding.FLAG_FORCE_ALU)])
def test_packed_on_the_fp32_kernels(io, d, flags):
    lengths = [1, 33, 64, 90, 0, 17]
    inp = _packed_inputs(lengths, H=2, d=d, io=io, seed=25, gamma=0.5)
    got, _ = _run_gpu(inp, io, flags=flags)
    G.assert_close(got, _oracle(inp), G.TOL[io], f"packed {io}")
    got2, _ = _run_gpu(inp, io, use_saved=False, flags=flags)
    for k in got:
        np.testing.assert_array_equal(got[k], got2[k])


def test_malformed_offsets_are_reported_not_followed():
    inp = _packed_inputs([100, 100], H=1, d=128, io="bf16", seed=26, with_states=False)
    t = {k: torch.from_numpy(inp[k]).cuda().to(torch.bfloat16) for k in ("o", "f", "i")}
    cu = torch.tensor([0, 150, 400], dtype=torch.int32, device="cuda")       # second sequence runs past T = 200
    ybuf, y = G.canary((1, 200, 128), torch.bfloat16)
    y, SN, saved, ws, _ = binding.hgrn2_fwd_varlen(t["o"], t["f"], t["i"], cu, None, y=y)
    torch.cuda.synchronize()
    assert binding.hgrn2_poll(ws) == 1          # HGRN2_ERR_INVALID_ARG in the status word
    assert G.canary_ok(ybuf)
