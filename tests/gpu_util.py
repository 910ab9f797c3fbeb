"""Helpers of the GPU parity tests: run the CUDA path through the binding, run the oracle, compare."""
import numpy as np
import torch

from oracle import ref
from paper_2404_07904_b200 import binding

TOL = {"f32": 1e-4, "bf16": 2e-2}      # max-norm relative error per output tensor


def rel_err(got, want):
    """max|got - want| / max|want| (an element-wise ratio is meaningless next to zeros)."""
    want = np.asarray(want, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    return float(np.abs(got - want).max() / max(float(np.abs(want).max()), 1e-30))


def to_dev(inp, io, dev="cuda"):
    tdt = torch.float32 if io == "f32" else torch.bfloat16
    out = {}
    for k, v in inp.items():
        if v is None:
            out[k] = None
        elif k in ("S0", "dSN"):
            out[k] = torch.from_numpy(v).to(dev)
        else:
            out[k] = torch.from_numpy(v).to(dev).to(tdt)     # exact: values are already representable
    return out


def canary(shape, dtype, dev="cuda", pad=64):
    """A tensor inside a larger buffer filled with a sentinel, to catch out-of-bounds writes."""
    n = int(np.prod(shape))
    buf = torch.full((n + 2 * pad,), 12345.0, dtype=dtype, device=dev)
    return buf, buf[pad:pad + n].view(*shape)


def canary_ok(buf, pad=64):
    return bool((buf[:pad] == 12345.0).all().item() and (buf[-pad:] == 12345.0).all().item())


def gpu_fwd_bwd(inp, io, chunk=0, flags=0, use_saved=True, check_canaries=True):
    t = to_dev(inp, io)
    B, H, N, dk = t["o"].shape
    dv = t["i"].shape[-1]
    tdt = t["o"].dtype
    bufs = {}
    outs = {}
    for name, shape, dt in (("y", (B, H, N, dv), tdt), ("SN", (B, H, dk, dv), torch.float32),
                            ("d_o", (B, H, N, dk), tdt), ("d_f", (B, H, N, dk), tdt),
                            ("d_i", (B, H, N, dv), tdt), ("dS0", (B, H, dk, dv), torch.float32)):
        bufs[name], outs[name] = canary(shape, dt)
    y, SN, saved, ws, desc = binding.hgrn2_fwd(t["o"], t["f"], t["i"], t["S0"], y=outs["y"], SN=outs["SN"],
                                               chunk=chunk, flags=flags)
    binding.hgrn2_bwd(t["o"], t["f"], t["i"], t["S0"], t["dy"], t["dSN"], saved if use_saved else None,
                      d_o=outs["d_o"], d_f=outs["d_f"], d_i=outs["d_i"], dS0=outs["dS0"], ws=ws,
                      chunk=chunk, flags=flags)
    torch.cuda.synchronize()
    assert binding.hgrn2_poll(ws) == 0
    if check_canaries:
        for name, b in bufs.items():
            assert canary_ok(b), f"out-of-bounds write next to {name}"
    return {k: v.float().cpu().numpy() for k, v in outs.items()}


def oracle_fwd_bwd(inp, units=None):
    """Oracle outputs; `units` = list of (b, h) to restrict to (each unit is independent)."""
    if units is None:
        y, SN = ref.hgrn2_fwd(inp["o"], inp["f"], inp["i"], inp["S0"])
        d_o, d_f, d_i, dS0 = ref.hgrn2_bwd(inp["o"], inp["f"], inp["i"], inp["S0"], inp["dy"], inp["dSN"])
        return {"y": y, "SN": SN, "d_o": d_o, "d_f": d_f, "d_i": d_i, "dS0": dS0}
    outs = {}
    for (b, h) in units:
        sub = {k: (None if v is None else v[b:b + 1, h:h + 1]) for k, v in inp.items()}
        outs[(b, h)] = oracle_fwd_bwd(sub)
    return outs


def assert_close(got, want, tol, what=""):
    errs = {k: rel_err(got[k], want[k]) for k in want}
    bad = {k: v for k, v in errs.items() if not (v <= tol)}
    assert not bad, f"{what}: rel errors {errs} exceed {tol}"
    return errs
