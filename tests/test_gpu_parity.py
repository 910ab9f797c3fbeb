"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle element by element.

Tolerances (max-norm relative error per output tensor): 1e-4 for float32 I/O, 2e-2 for bf16 I/O with
float32 state.  bf16 inputs are rounded once and both sides consume the rounded values.
"""
import numpy as np
import pytest
import torch

from paper_2404_07904_b200 import binding, workloads as W
from oracle import ref
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


# ---------------------------------------------------------------- decode step
@pytest.mark.parametrize("B,H,dk,dv,io", [(3, 2, 128, 128, "bf16"), (2, 3, 64, 64, "f32"), (1, 1, 16, 128, "f32"),
                                          (2, 1, 128, 16, "bf16"), (5, 4, 32, 64, "bf16"), (1, 2, 64, 32, "f32")])
def test_step_matches_oracle(B, H, dk, dv, io):
    w = W.scaled(W.CONFIGS["decode"], B=B, H=H, dk=dk, dv=dv, io=io)
    d = W.make_decode_inputs(w, steps=6)
    tdt = torch.float32 if io == "f32" else torch.bfloat16
    Sbuf, S = G.canary((B, H, dk, dv), torch.float32)
    S.copy_(torch.from_numpy(d["S0"]))
    S_ref = d["S0"].astype(np.float64)
    for t in range(6):
        o, f, i = (torch.from_numpy(d[k][t]).cuda().to(tdt) for k in ("o", "f", "i"))
        ybuf, y = G.canary((B, H, dv), tdt)
        binding.hgrn2_step(o, f, i, S, y=y)
        y_ref = ref.hgrn2_step(d["o"][t], d["f"][t], d["i"][t], S_ref)
        assert G.rel_err(y.float().cpu().numpy(), y_ref) <= G.TOL[io]
        assert G.canary_ok(ybuf)
    assert G.rel_err(S.cpu().numpy(), S_ref) <= 1e-5
    assert G.canary_ok(Sbuf)


def test_step_continues_prefill_state():
    # forward over N tokens, then decode steps from its S_N == forward over N + T tokens
    w = W.scaled(W.CONFIGS["lm_2048"], B=2, H=2, N=200, has_S0=True)
    inp = W.make_inputs(w)
    t = G.to_dev(inp, "bf16")
    m = 150
    _, Sm, _, ws, _ = binding.hgrn2_fwd(t["o"][:, :, :m].contiguous(), t["f"][:, :, :m].contiguous(),
                                        t["i"][:, :, :m].contiguous(), t["S0"], save_for_backward=False)
    ys = []
    for s in range(m, 200):
        ys.append(binding.hgrn2_step(t["o"][:, :, s].contiguous(), t["f"][:, :, s].contiguous(),
                                     t["i"][:, :, s].contiguous(), Sm))
    torch.cuda.synchronize()
    y_ref, SN_ref = ref.hgrn2_fwd(inp["o"], inp["f"], inp["i"], inp["S0"])
    got = torch.stack(ys, dim=2).float().cpu().numpy()
    assert G.rel_err(got, y_ref[:, :, m:]) <= 2e-2
    assert G.rel_err(Sm.cpu().numpy(), SN_ref) <= 2e-2


@pytest.mark.parametrize("B,H,d,io,T", [(3, 2, 128, "bf16", 7), (2, 3, 64, "f32", 5), (1, 1, 128, "f32", 1),
                                        (2, 2, 64, "bf16", 16)])
def test_step_multi_matches_oracle_and_single_steps(B, H, d, io, T):
    # T tokens in one launch: against the oracle's T single steps, and bit for bit against T calls of hgrn2_step
    w = W.scaled(W.CONFIGS["decode"], B=B, H=H, dk=d, dv=d, io=io)
    dd = W.make_decode_inputs(w, steps=T)
    tdt = torch.float32 if io == "f32" else torch.bfloat16
    seq = {k: torch.from_numpy(np.ascontiguousarray(np.moveaxis(dd[k], 0, 2))).cuda().to(tdt) for k in ("o", "f", "i")}
    Sbuf, S = G.canary((B, H, d, d), torch.float32)
    S.copy_(torch.from_numpy(dd["S0"]))
    ybuf, y = G.canary((B, H, T, d), tdt)
    binding.hgrn2_step_multi(seq["o"], seq["f"], seq["i"], S, y=y)
    S1 = torch.from_numpy(dd["S0"]).cuda()
    S_ref = dd["S0"].astype(np.float64)
    for t in range(T):
        y1 = binding.hgrn2_step(seq["o"][:, :, t].contiguous(), seq["f"][:, :, t].contiguous(),
                                seq["i"][:, :, t].contiguous(), S1)
        assert torch.equal(y1, y[:, :, t])
        y_ref = ref.hgrn2_step(dd["o"][t], dd["f"][t], dd["i"][t], S_ref)
        assert G.rel_err(y[:, :, t].float().cpu().numpy(), y_ref) <= G.TOL[io]
    assert torch.equal(S1, S)
    assert G.rel_err(S.cpu().numpy(), S_ref) <= 1e-5
    assert G.canary_ok(ybuf) and G.canary_ok(Sbuf)


def test_step_multi_continues_prefill_state():
    # forward over m tokens, then ONE multi-token step over the rest from its S_N == forward over all tokens
    w = W.scaled(W.CONFIGS["lm_2048"], B=2, H=2, N=200, has_S0=True)
    inp = W.make_inputs(w)
    t = G.to_dev(inp, "bf16")
    m = 150
    _, Sm, _, ws, _ = binding.hgrn2_fwd(t["o"][:, :, :m].contiguous(), t["f"][:, :, :m].contiguous(),
                                        t["i"][:, :, :m].contiguous(), t["S0"], save_for_backward=False)
    y = binding.hgrn2_step_multi(t["o"][:, :, m:].contiguous(), t["f"][:, :, m:].contiguous(),
                                 t["i"][:, :, m:].contiguous(), Sm)
    torch.cuda.synchronize()
    y_ref, SN_ref = ref.hgrn2_fwd(inp["o"], inp["f"], inp["i"], inp["S0"])
    assert G.rel_err(y.float().cpu().numpy(), y_ref[:, :, m:]) <= 2e-2
    assert G.rel_err(Sm.cpu().numpy(), SN_ref) <= 2e-2


# ---------------------------------------------------------------- config 1 and the fp32 path
def test_config1_tiny_f32():
    w = W.CONFIGS["tiny_f32"]
    inp = W.make_inputs(w)
    got = G.gpu_fwd_bwd(inp, "f32", chunk=w.chunk)
    errs = G.assert_close(got, G.oracle_fwd_bwd(inp), 1e-4, "config 1")
    print("config1 errs", errs)


@pytest.mark.parametrize("N", [1, 2, 63, 64, 65, 129])
@pytest.mark.parametrize("d,chunk", [(64, 0), (64, 16), (128, 0), (16, 32)])
def test_f32_shape_sweep(N, d, chunk):
    w = W.scaled(W.CONFIGS["tiny_f32"], B=2, H=1, N=N, dk=d, dv=d, has_S0=(N % 2 == 1), has_dSN=(N % 2 == 1),
                 seed=N + d, gamma=0.3)
    inp = W.make_inputs(w)
    got = G.gpu_fwd_bwd(inp, "f32", chunk=chunk)
    G.assert_close(got, G.oracle_fwd_bwd(inp), 1e-4, f"N={N} d={d} chunk={chunk}")


def test_f32_rectangular_state_and_recompute():
    w = W.scaled(W.CONFIGS["tiny_f32"], B=1, H=3, N=100, dk=32, dv=128, has_S0=True, has_dSN=True, seed=7)
    inp = W.make_inputs(w)
    want = G.oracle_fwd_bwd(inp)
    G.assert_close(G.gpu_fwd_bwd(inp, "f32"), want, 1e-4, "saved")
    G.assert_close(G.gpu_fwd_bwd(inp, "f32", use_saved=False), want, 1e-4, "recomputed")


def test_alu_path_bf16_io():
    w = W.scaled(W.CONFIGS["lm_2048"], B=1, H=2, N=300, has_S0=True, has_dSN=True)
    inp = W.make_inputs(w)
    got = G.gpu_fwd_bwd(inp, "bf16", flags=binding.FLAG_FORCE_ALU)
    G.assert_close(got, G.oracle_fwd_bwd(inp), 2e-2, "alu bf16")


def test_f_zero_and_f_one_forward():
    # f == 0: y_t = (sum_k o_tk) i_t whatever S0 is; f == 1: the state never moves.
    w = W.scaled(W.CONFIGS["tiny_f32"], N=70, has_S0=True)
    inp = W.make_inputs(w)
    for fv in (0.0, 1.0):
        inp["f"][:] = fv
        t = G.to_dev(inp, "f32")
        y, SN, _, ws, _ = binding.hgrn2_fwd(t["o"], t["f"], t["i"], t["S0"], save_for_backward=False)
        torch.cuda.synchronize()
        y_ref, SN_ref = ref.hgrn2_fwd(inp["o"], inp["f"], inp["i"], inp["S0"])
        assert G.rel_err(y.cpu().numpy(), y_ref) <= 1e-4
        assert G.rel_err(SN.cpu().numpy(), SN_ref) <= 1e-4


def test_empty_sequence_and_empty_batch():
    dev = "cuda"
    S0 = torch.randn(2, 2, 64, 64, device=dev)
    o = torch.empty(2, 2, 0, 64, device=dev); i = torch.empty(2, 2, 0, 64, device=dev)
    y, SN, saved, ws, _ = binding.hgrn2_fwd(o, o, i, S0)
    d_o, d_f, d_i, dS0, _ = binding.hgrn2_bwd(o, o, i, S0, i, S0, saved)
    torch.cuda.synchronize()
    assert torch.equal(SN, S0) and torch.equal(dS0, S0)
    o = torch.empty(0, 2, 8, 64, device=dev)
    binding.hgrn2_fwd(o, o, o, None)
    torch.cuda.synchronize()


@pytest.mark.parametrize("io,N,H", [("bf16", 200, 2), ("bf16", 1024, 3), ("f32", 100, 2)])
def test_every_call_starts_with_a_clean_status_word(io, N, H):
    # a stale error code in the workspace must not survive the next call: forward, backward with the saved
    # states, backward that recomputes them; whole units, segmented sequences (few units) and the fp32 path
    w = W.scaled(W.CONFIGS["lm_2048"], B=1, H=H, N=N, io=io, dk=128 if io == "bf16" else 64,
                 dv=128 if io == "bf16" else 64, seed=5)
    t = G.to_dev(W.make_inputs(w), io)
    y, SN, saved, ws, desc = binding.hgrn2_fwd(t["o"], t["f"], t["i"], None)
    torch.cuda.synchronize()
    stale = torch.tensor([6, 1], dtype=torch.int32, device="cuda").view(torch.uint8)
    for use_saved in (True, False):
        ws[:8] = stale
        binding.hgrn2_fwd(t["o"], t["f"], t["i"], None, y=y, saved=saved, ws=ws)
        torch.cuda.synchronize()
        assert binding.hgrn2_poll(ws) == 0
        ws[:8] = stale
        binding.hgrn2_bwd(t["o"], t["f"], t["i"], None, t["dy"], None, saved if use_saved else None, ws=ws)
        torch.cuda.synchronize()
        assert binding.hgrn2_poll(ws) == 0


def test_run_to_run_determinism():
    w = W.scaled(W.CONFIGS["lm_2048"], B=1, H=3, N=257, has_S0=True, has_dSN=True)
    inp = W.make_inputs(w)
    a = G.gpu_fwd_bwd(inp, "bf16")
    b = G.gpu_fwd_bwd(inp, "bf16")
    for k in a:
        np.testing.assert_array_equal(a[k], b[k])


# ---------------------------------------------------------------- the library's default path for the LM configs
def _check_units(inp, got, units, tol, what):
    want = G.oracle_fwd_bwd(inp, units)
    worst = {}
    for (b, h), wu in want.items():
        gu = {k: got[k][b:b + 1, h:h + 1] for k in wu}
        errs = G.assert_close(gu, wu, tol, f"{what} unit {(b, h)}")
        for k, v in errs.items():
            worst[k] = max(worst.get(k, 0.0), v)
    print(what, {k: f"{v:.2e}" for k, v in worst.items()})


@pytest.mark.parametrize("N", [1, 63, 64, 65, 200, 512])
def test_bf16_default_path_shape_sweep(N):
    w = W.scaled(W.CONFIGS["lm_2048"], B=2, H=2, N=N, has_S0=(N % 2 == 0), has_dSN=(N % 2 == 0), seed=50 + N)
    inp = W.make_inputs(w)
    got = G.gpu_fwd_bwd(inp, "bf16")
    G.assert_close(got, G.oracle_fwd_bwd(inp), 2e-2, f"bf16 N={N}")


@pytest.mark.parametrize("gamma", [0.0, 0.5, 0.9, 0.99])
def test_bf16_decay_sweep(gamma):
    w = W.scaled(W.CONFIGS["lm_2560"], B=1, H=3, N=640)
    inp = W.make_inputs(w, gamma=gamma)
    got = G.gpu_fwd_bwd(inp, "bf16")
    G.assert_close(got, G.oracle_fwd_bwd(inp), 2e-2, f"gamma={gamma}")


def test_bf16_recompute_matches_saved():
    w = W.scaled(W.CONFIGS["lm_2048"], B=1, H=2, N=400, has_S0=True, has_dSN=True)
    inp = W.make_inputs(w)
    a = G.gpu_fwd_bwd(inp, "bf16")
    b = G.gpu_fwd_bwd(inp, "bf16", use_saved=False)
    for k in a:
        np.testing.assert_array_equal(a[k], b[k])


def test_few_units_split_into_segments():
    # 4 units of 32 chunks: too few to fill the GPU, so each sequence runs as several segments chained through
    # their boundary states (forward) and boundary state gradients (backward); all outputs against the oracle
    w = W.scaled(W.CONFIGS["long_16k"], B=1, H=4, N=2048, seed=77)
    d = binding.make_desc(w.B, w.H, w.N, w.dk, w.dv, binding.HGRN2_BF16)
    assert binding.workspace_bytes(d) > 256 + binding.saved_bytes(d), "segment scratch expected in the workspace"
    inp = W.make_inputs(w)
    got = G.gpu_fwd_bwd(inp, "bf16")
    _check_units(inp, got, [(0, 0), (0, 3)], 2e-2, "segments")
    got2 = G.gpu_fwd_bwd(inp, "bf16", use_saved=False)
    for k in got:
        np.testing.assert_array_equal(got[k], got2[k])


def test_units_beyond_the_last_full_wave_are_split():
    # a few more units than SMs: the left-over units run as segments after the full wave; units from both
    # parts against the oracle, with initial state and final-state gradient so the slices' offsets are exercised
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    H = sms + 3
    w = W.scaled(W.CONFIGS["long_16k"], B=1, H=H, N=1024, seed=78)
    d = binding.make_desc(w.B, w.H, w.N, w.dk, w.dv, binding.HGRN2_BF16)
    assert binding.workspace_bytes(d) > 256 + binding.saved_bytes(d), "segment scratch expected in the workspace"
    inp = W.make_inputs(w)
    got = G.gpu_fwd_bwd(inp, "bf16")
    _check_units(inp, got, [(0, 0), (0, sms - 1), (0, sms), (0, H - 1)], 2e-2, "left-over units")
    got2 = G.gpu_fwd_bwd(inp, "bf16", use_saved=False)
    for k in got:
        np.testing.assert_array_equal(got[k], got2[k])


def test_config2_full_size_sampled_units():
    w = W.CONFIGS["lm_2048"]
    inp = W.make_inputs(w)
    got = G.gpu_fwd_bwd(inp, "bf16", check_canaries=True)
    _check_units(inp, got, [(0, 0), (3, 7), (7, 15)], 2e-2, "config 2")
    for k, v in got.items():
        assert np.isfinite(v).all(), k


def test_config3_long_context_sampled_units():
    w = W.CONFIGS["long_16k"]
    inp = W.make_inputs(w)
    got = G.gpu_fwd_bwd(inp, "bf16")
    _check_units(inp, got, [(0, 0), (1, 15)], 2e-2, "config 3")
    for k, v in got.items():
        assert np.isfinite(v).all(), k


@pytest.mark.parametrize("gamma", W.LM_2560_GAMMAS)
def test_config4_full_size_sampled_units(gamma):
    # the whole 8 x 20 batch: on a 148-SM GPU units 0..147 run as one wave of whole units and units 148..159 as
    # segments; units from both parts, next to the boundary and at both ends
    w = W.CONFIGS["lm_2560"]
    inp = W.make_inputs(w, gamma=gamma)
    got = G.gpu_fwd_bwd(inp, "bf16")
    _check_units(inp, got, [(0, 0), (7, 7), (7, 8), (7, 19)], 2e-2, f"config 4 gamma={gamma}")
    for k, v in got.items():
        assert np.isfinite(v).all(), k


def test_config5_decode_all_512_steps():
    # the full decode batch over all 512 consecutive one-token calls: every y_t of three sampled units and their
    # final states against the oracle's single steps (gates generated in blocks of 64 steps)
    w = W.CONFIGS["decode"]
    T, blk = w.N, 64
    units = [(0, 0), (100, 7), (255, 15)]
    S = None
    S_ref = {}
    worst = 0.0
    for b0 in range(0, T, blk):
        d = W.make_decode_inputs(w, steps=blk, seed=w.seed + 7 * (b0 // blk))
        if S is None:
            S = torch.from_numpy(d["S0"]).cuda()
            S_ref = {u: d["S0"][u[0]:u[0] + 1, u[1]:u[1] + 1].astype(np.float64) for u in units}
        dev = {k: torch.from_numpy(d[k]).cuda().to(torch.bfloat16) for k in ("o", "f", "i")}
        ys = torch.empty((blk, w.B, w.H, w.dv), dtype=torch.bfloat16, device="cuda")
        for t in range(blk):
            binding.hgrn2_step(dev["o"][t], dev["f"][t], dev["i"][t], S, y=ys[t])
        ys = ys.float().cpu().numpy()
        for t in range(blk):
            for (b, h) in units:
                y_ref = ref.hgrn2_step(d["o"][t][b:b + 1, h:h + 1], d["f"][t][b:b + 1, h:h + 1],
                                       d["i"][t][b:b + 1, h:h + 1], S_ref[(b, h)])
                err = G.rel_err(ys[t][b:b + 1, h:h + 1], y_ref)
                worst = max(worst, err)
                assert err <= 2e-2, (b0 + t, b, h, err)
    Sh = S.cpu().numpy()
    for (b, h) in units:
        assert G.rel_err(Sh[b:b + 1, h:h + 1], S_ref[(b, h)]) <= 1e-5
    print("config 5 worst y error over 512 steps", worst)


# ---------------------------------------------------------------- the kernels' time-out exit
def test_expired_waits_end_in_a_timeout_status_and_leave_the_context_usable():
    # With HGRN2_FLAG_DEBUG_EXPIRE_WAITS every device-side wait that has to wait gives up at once, so the product
    # kernels (unmodified) take their time-out exit: they must return, report HGRN2_ERR_TIMEOUT, write only
    # inside the caller's buffers, and the next ordinary call on the same workspace must be correct again.
    w = W.scaled(W.CONFIGS["lm_2048"], B=1, H=1, N=128, has_S0=True, has_dSN=True, seed=91)
    inp = W.make_inputs(w)
    t = G.to_dev(inp, "bf16")
    bufs = {}
    outs = {}
    for name, shape, dt in (("y", (1, 1, 128, 128), torch.bfloat16), ("SN", (1, 1, 128, 128), torch.float32),
                            ("d_o", (1, 1, 128, 128), torch.bfloat16), ("d_f", (1, 1, 128, 128), torch.bfloat16),
                            ("d_i", (1, 1, 128, 128), torch.bfloat16), ("dS0", (1, 1, 128, 128), torch.float32)):
        bufs[name], outs[name] = G.canary(shape, dt)
    y, SN, saved, ws, _ = binding.hgrn2_fwd(t["o"], t["f"], t["i"], t["S0"], y=outs["y"], SN=outs["SN"],
                                            flags=binding.FLAG_DEBUG_EXPIRE_WAITS)
    torch.cuda.synchronize()
    assert binding.hgrn2_poll(ws) == 6, "forward: HGRN2_ERR_TIMEOUT expected"
    # an ordinary forward fills `saved` properly for the backward under test
    binding.hgrn2_fwd(t["o"], t["f"], t["i"], t["S0"], y=outs["y"], SN=outs["SN"], saved=saved, ws=ws)
    torch.cuda.synchronize()
    assert binding.hgrn2_poll(ws) == 0
    binding.hgrn2_bwd(t["o"], t["f"], t["i"], t["S0"], t["dy"], t["dSN"], saved, d_o=outs["d_o"], d_f=outs["d_f"],
                      d_i=outs["d_i"], dS0=outs["dS0"], ws=ws, flags=binding.FLAG_DEBUG_EXPIRE_WAITS)
    torch.cuda.synchronize()
    assert binding.hgrn2_poll(ws) == 6, "backward: HGRN2_ERR_TIMEOUT expected"
    for name, b in bufs.items():
        assert G.canary_ok(b), f"out-of-bounds write next to {name}"
    # the same workspace and buffers, no flag: status clean again and every output right
    binding.hgrn2_bwd(t["o"], t["f"], t["i"], t["S0"], t["dy"], t["dSN"], saved, d_o=outs["d_o"], d_f=outs["d_f"],
                      d_i=outs["d_i"], dS0=outs["dS0"], ws=ws)
    torch.cuda.synchronize()
    assert binding.hgrn2_poll(ws) == 0
    got = {k: v.float().cpu().numpy() for k, v in outs.items()}
    G.assert_close(got, G.oracle_fwd_bwd(inp), 2e-2, "after the timed-out calls")
