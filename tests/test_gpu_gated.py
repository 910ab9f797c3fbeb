"""GPU parity of the gated entry points (Eq. 1 / Eq. 2 activations in front of the recurrence) against the oracle.

Inputs are the pre-activations zo, zf, zi (rounded once to the I/O type; both sides consume the rounded values)
and the per-channel lower bound beta; outputs y, S_N and the gradients with respect to the pre-activations, beta
and S_0.  The oracle applies the activations in fp64 and never rounds the gates.
"""
import numpy as np
import pytest
import torch

from paper_2404_07904_b200 import binding, workloads as W
from oracle import ref
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def _inputs(B, H, N, d, io, seed, beta_lo, beta_hi, zf_shift=0.0, states=True):
    rng = np.random.default_rng(seed)
    r = (lambda x: W.round_to_bf16(x)) if io == "bf16" else (lambda x: x.astype(np.float32))
    inp = {
        "zo": r(rng.standard_normal((B, H, N, d), dtype=np.float32)),
        "zf": r(rng.standard_normal((B, H, N, d), dtype=np.float32) + np.float32(zf_shift)),
        "zi": r(rng.standard_normal((B, H, N, d), dtype=np.float32)),
        "dy": r(rng.standard_normal((B, H, N, d), dtype=np.float32)),
        "beta": rng.uniform(beta_lo, beta_hi, (H, d)).astype(np.float32),
        "S0": (rng.standard_normal((B, H, d, d), dtype=np.float32) * np.float32(0.02)) if states else None,
        "dSN": (rng.standard_normal((B, H, d, d), dtype=np.float32) * np.float32(0.02)) if states else None,
    }
    return inp


def _run(inp, io, use_saved=True, flags=0):
    tdt = torch.float32 if io == "f32" else torch.bfloat16
    t = {k: torch.from_numpy(inp[k]).cuda().to(tdt) for k in ("zo", "zf", "zi", "dy")}
    beta = torch.from_numpy(inp["beta"]).cuda()
    S0 = None if inp["S0"] is None else torch.from_numpy(inp["S0"]).cuda()
    dSN = None if inp["dSN"] is None else torch.from_numpy(inp["dSN"]).cuda()
    shape = tuple(t["zo"].shape)
    ybuf, y = G.canary(shape, tdt)
    y, SN, saved, ws, _ = binding.hgrn2_fwd_gated(t["zo"], t["zf"], t["zi"], beta, S0, y=y, flags=flags)
    torch.cuda.synchronize()
    assert binding.hgrn2_poll(ws) == 0
    n_exact = binding.exact_path_units(ws)
    bufs = {n: G.canary(shape, tdt) for n in ("d_zo", "d_zf", "d_zi")}
    d_zo, d_zf, d_zi, d_beta, dS0, ws = binding.hgrn2_bwd_gated(
        t["zo"], t["zf"], t["zi"], beta, S0, t["dy"], dSN, saved if use_saved else None, d_zo=bufs["d_zo"][1],
        d_zf=bufs["d_zf"][1], d_zi=bufs["d_zi"][1], ws=ws, flags=flags)
    torch.cuda.synchronize()
    assert binding.hgrn2_poll(ws) == 0
    assert G.canary_ok(ybuf) and all(G.canary_ok(b[0]) for b in bufs.values())
    got = {"y": y, "SN": SN, "d_zo": d_zo, "d_zf": d_zf, "d_zi": d_zi, "d_beta": d_beta, "dS0": dS0}
    return {k: v.float().cpu().numpy() for k, v in got.items()}, n_exact


def _oracle(inp):
    y, SN = ref.hgrn2_fwd_gated(inp["zo"], inp["zf"], inp["zi"], inp["beta"], inp["S0"])
    d_zo, d_zf, d_zi, d_beta, dS0 = ref.hgrn2_bwd_gated(inp["zo"], inp["zf"], inp["zi"], inp["beta"], inp["S0"],
                                                        inp["dy"], inp["dSN"])
    return {"y": y, "SN": SN, "d_zo": d_zo, "d_zf": d_zf, "d_zi": d_zi, "d_beta": d_beta, "dS0": dS0}


@pytest.mark.parametrize("N", [64, 300])
def test_gated_bf16_default_path(N):
    inp = _inputs(2, 3, N, 128, "bf16", seed=40 + N, beta_lo=0.0, beta_hi=0.95)
    assert binding.path_of(binding.make_desc(2, 3, N, 128, 128, binding.HGRN2_BF16)) == "tcgen05"
    got, n_exact = _run(inp, "bf16")
    assert n_exact == 0
    errs = G.assert_close(got, _oracle(inp), 2e-2, f"gated bf16 N={N}")
    print("gated bf16", {k: f"{v:.2e}" for k, v in errs.items()})
    got2, _ = _run(inp, "bf16", use_saved=False)
    for k in got:
        np.testing.assert_array_equal(got[k], got2[k])


def test_gated_bf16_lower_bound_close_to_one_long_sequence():
    # beta = 0.99: f lies in [0.99, 1), where a bf16 f would have seven distinct values; the gates must not be
    # rounded on the way (the kernels are handed k = 1 - f, which bf16 resolves finely there)
    inp = _inputs(1, 4, 2048, 128, "bf16", seed=44, beta_lo=0.99, beta_hi=0.99)
    got, _ = _run(inp, "bf16")                  # few units: the sequences also run as segments
    G.assert_close(got, _oracle(inp), 2e-2, "gated, beta = 0.99, N = 2048")


def test_gated_bf16_hard_forget_gates_take_the_exact_path():
    # zero lower bound and pre-activations around -3 (f = sigmoid(zf) ~ 0.05): out of the operands' range
    inp = _inputs(1, 2, 200, 128, "bf16", seed=45, beta_lo=0.0, beta_hi=0.0, zf_shift=-3.0)
    got, n_exact = _run(inp, "bf16")
    assert n_exact == 2
    G.assert_close(got, _oracle(inp), 2e-2, "gated, hard-forget")


@pytest.mark.parametrize("io,d,flags,tol", [("f32", 64, 0, 1e-4), ("bf16", 128, binding.FLAG_FORCE_ALU, 2e-2)])
def test_gated_on_the_fp32_kernels(io, d, flags, tol):
    inp = _inputs(2, 2, 100, d, io, seed=46, beta_lo=0.0, beta_hi=0.9)
    got, _ = _run(inp, io, flags=flags)
    G.assert_close(got, _oracle(inp), tol, f"gated {io}")
    got2, _ = _run(inp, io, use_saved=False, flags=flags)
    for k in got:
        np.testing.assert_array_equal(got[k], got2[k])
