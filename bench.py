#!/usr/bin/env python
"""Benchmark of the HGRN2 hot path on B200.

A step is one forward + one backward of the recurrence over the `lm_2048` workload (model
d = 2048: H = 16 heads of d_k = d_v = 128, B = 8 sequences of N = 2048 tokens, bf16 I/O, fp32
state).  The decode workload (`decode`: 256 x 16 states, one token per call, 512 consecutive
calls) is timed separately and reported in the same JSON line under "decode".

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

With N > 1 it runs one rank per GPU: either launched by torch.distributed.run, or - when started as a
plain `python bench.py --gpus N` - it starts its own ranks by re-executing itself under
torch.distributed.run on 127.0.0.1.  The (batch, head) units are independent, so every rank runs the
same per-GPU workload (weak scaling) and no collective touches the data path.

Timing.  The step loop is timed in batches of exactly K steps (CUDA events on the launching stream, a
barrier and a device synchronise on both sides, max over ranks); batches are repeated until at least
--min-seconds of device time have been spent, so that the SM clock is sampled under a sustained load, and
the MEDIAN batch is reported (`value`, `ms_per_step`; the spread is in `timing`).  `roofline.kernels` and the
dominant-kernel figures come from separate loops of one kernel alone (forward only, backward only), K launches
each, taken BEFORE the long step loop: a few milliseconds on a board that has not reached its power cap (boost
clock), whereas the step loop settles at the capped clock it reports; they also find different data in L2 than
the alternating step does.  So their sum is below the step's time, by the clock ratio and a few %.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL = {"hbm_gbs": 7700.0, "bf16_tflops": 2250.0}

# dram__bytes_read.sum + dram__bytes_write.sum per launch, copied from the ncu captures summarised under
# profiles/ (same workloads as timed here: lm_2048 and the full decode batch); nothing here measures traffic.
# None = the kernel has changed since its counters were taken.
NCU_TRAFFIC_BYTES = {"fwd": 201.41e6 + 154.02e6, "bwd": 406.96e6 + 170.88e6, "step": 271.60e6 + 212.48e6}
NCU_TRAFFIC_SOURCE = {"fwd": "profiles/tc_fwd_bwd_lm2048.md (captured 2026-11-30, kernels as of the two-read completion pass of the backward)",
                      "bwd": "profiles/tc_fwd_bwd_lm2048.md (captured 2026-11-30, kernels as of the two-read completion pass of the backward)",
                      "step": "profiles/step_kernel_decode.md"}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as fh:
            d = json.load(fh)
        return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ------------------------------------------------------------------------------------------------
# algorithmic work (what the method must move / compute, independent of the implementation)
# ------------------------------------------------------------------------------------------------
def train_bytes(w, esize=2):
    """fwd reads o, f, i and writes y; bwd reads o, f, i, dy and writes d_o, d_f, d_i: each once."""
    per_tensor = w.B * w.H * w.N * w.dk * esize
    return {"fwd": 4 * per_tensor, "bwd": 7 * per_tensor}


def train_flops(w, C=64):
    """Causal count of the chunked form per token-head (intra-chunk blocks counted (C+1)/2C)."""
    th = w.B * w.H * w.N
    fwd = 4 * w.dk * w.dv + 2 * w.dk * (C + 1)
    bwd = 8 * w.dk * w.dv + 5 * w.dk * (C + 1)
    return {"fwd": th * fwd, "bwd": th * bwd}


def decode_bytes(w, esize=2):
    units = w.B * w.H
    return units * (2 * w.dk * w.dv * 4 + (2 * w.dk + 2 * w.dv) * esize)


# ------------------------------------------------------------------------------------------------
# clocks sampling during the timed region
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    NAMES = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.samples = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) >= 6:
                self.samples.append(parts)

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        if self.thread is not None:
            self.thread.join(timeout=5)

    def summary(self):
        sm, mx, reasons = [], [], set()
        for p in self.samples:
            try:
                sm.append(float(p[0])); mx.append(float(p[1]))
            except ValueError:
                continue
            for name, val in zip(self.NAMES, p[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        hist = {}
        for v in sm:
            hist[str(int(v))] = hist.get(str(int(v)), 0) + 1
        return {"sm_mhz": statistics.median(sm), "sm_min_mhz": min(sm), "sm_max_mhz": max(mx),
                "reasons": sorted(reasons), "samples": len(sm), "sm_mhz_hist": hist}


# ------------------------------------------------------------------------------------------------
# the oracle arm (CPU): used for --impl reference and for the cpu_baseline object
# ------------------------------------------------------------------------------------------------
def oracle_sample_step(inp_units):
    from oracle import ref
    ref.hgrn2_fwd(inp_units["o"], inp_units["f"], inp_units["i"], inp_units["S0"])
    ref.hgrn2_bwd(inp_units["o"], inp_units["f"], inp_units["i"], inp_units["S0"], inp_units["dy"], inp_units["dSN"])


def oracle_sample_inputs(w, n_units):
    """The first n_units (b, h) units of the workload, as one [1, n_units, N, d] problem in fp64."""
    from paper_2404_07904_b200 import workloads as W
    small = W.scaled(w, B=1, H=n_units)
    inp = W.make_inputs(small)
    return {k: (None if v is None else v.astype(np.float64)) for k, v in inp.items()}


def time_oracle(w, steps, warmup, n_units):
    from oracle import ref
    ref.build()
    cores = ref.num_threads()
    inp = oracle_sample_inputs(w, n_units)
    for _ in range(warmup):
        oracle_sample_step(inp)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_sample_step(inp)
    dt = (time.perf_counter() - t0) / max(steps, 1)
    tokens = n_units * w.N / w.H          # a token spans all H heads
    return tokens / dt, dt, cores


def run_reference(args):
    from paper_2404_07904_b200 import workloads as W
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    w = W.CONFIGS["lm_2048"]
    from oracle import ref
    ref.build()
    n_units = max(1, min(ref.num_threads(), w.B * w.H))
    value, dt, cores = time_oracle(w, args.steps, args.warmup, n_units)
    sample = (f"{n_units} of {w.B * w.H} (batch, head) units of lm_2048 per step (N={w.N}, d_k=d_v={w.dk}), "
              f"fwd+bwd, fp64, scaled by tokens")
    line = {
        "impl": "reference", "metric": "HGRN2 layer fwd+bwd tokens/s", "value": value, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, None),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


def workload_config(w, path):
    return {"workload": w.name, "B": w.B, "H": w.H, "N": w.N, "d_k": w.dk, "d_v": w.dv, "d_model": w.H * w.dk,
            "io": w.io, "state": "f32", "gamma": w.gamma, "path": path,
            "l2": "inputs larger than L2 (each pass streams > 250 MB; no flush needed)"}


# ------------------------------------------------------------------------------------------------
# the CUDA arm
# ------------------------------------------------------------------------------------------------
def run_decode(args, binding, W, dev, rank, world, timed, max_over_ranks, peaks, peak_kind, bf):
    import torch
    # ---- decode: 512 consecutive one-token calls on the decode workload -------------------------
    wd = W.CONFIGS["decode"]
    T = args.decode_steps if args.decode_steps > 0 else wd.N
    blk = 64
    gates = {"o": [], "f": [], "i": []}
    S0 = None
    for b0 in range(0, T, blk):
        dd = W.make_decode_inputs(wd, steps=min(blk, T - b0), seed=wd.seed + 1000 * rank + 7 * (b0 // blk))
        if S0 is None:
            S0 = dd["S0"]
        for k in gates:
            gates[k].append(torch.from_numpy(dd[k]).to(bf))
    gates = {k: torch.cat(v, 0).to(dev) for k, v in gates.items()}
    S = torch.from_numpy(S0).to(dev)
    yd = torch.empty((T, wd.B, wd.H, wd.dv), dtype=bf, device=dev)

    def decode_all():
        for t in range(T):
            binding.hgrn2_step(gates["o"][t], gates["f"][t], gates["i"][t], S, y=yd[t])

    for t in range(min(8, T)):
        binding.hgrn2_step(gates["o"][t], gates["f"][t], gates["i"][t], S, y=yd[t])
    S.copy_(torch.from_numpy(S0))
    ms_dec = max_over_ranks(timed(decode_all, 1)) / T
    db = decode_bytes(wd)
    dec_gbps = db / (ms_dec * 1e-3) / 1e9
    decode = {"workload": wd.name, "B": wd.B, "H": wd.H, "steps": T, "us_per_step": ms_dec * 1e3,
              "value": dec_gbps, "unit": "GB/s", "tokens_per_s": world * wd.B / (ms_dec * 1e-3),
              "roofline": {"bound": "hbm", "kernel": "hgrn2_step", "achieved": dec_gbps, "peak": peaks["hbm_gbs"],
                           "unit": "GB/s", "frac": dec_gbps / peaks["hbm_gbs"], "traffic": NCU_TRAFFIC_BYTES["step"],
                           "peak_source": f"of {peak_kind}", "frac_nominal": dec_gbps / NOMINAL["hbm_gbs"]}}
    # ---- the same tokens, 8 per launch (hgrn2_step_multi): the state crosses HBM once per 8 tokens -------
    TM = 8
    if T >= TM:
        nl = T // TM
        seq = {k: gates[k][:nl * TM].reshape(nl, TM, wd.B, wd.H, -1).permute(0, 2, 3, 1, 4).contiguous() for k in gates}
        ym = torch.empty((nl, wd.B, wd.H, TM, wd.dv), dtype=bf, device=dev)
        S.copy_(torch.from_numpy(S0))

        def decode_multi():
            for l in range(nl):
                binding.hgrn2_step_multi(seq["o"][l], seq["f"][l], seq["i"][l], S, y=ym[l])

        binding.hgrn2_step_multi(seq["o"][0], seq["f"][0], seq["i"][0], S, y=ym[0])
        S.copy_(torch.from_numpy(S0))
        ms_l = max_over_ranks(timed(decode_multi, 1)) / nl
        if rank == 0:       # same arithmetic in the same order: identical to the one-token calls
            same = torch.equal(ym.permute(0, 3, 1, 2, 4).reshape(nl * TM, wd.B, wd.H, wd.dv), yd[:nl * TM])
            assert same, "multi-token step differs from single steps"
        gate_bytes = decode_bytes(wd) - 2 * wd.B * wd.H * wd.dk * wd.dv * 4
        mb = 2 * wd.B * wd.H * wd.dk * wd.dv * 4 + TM * gate_bytes
        decode["multi_token"] = {"tokens_per_launch": TM, "launches": nl, "us_per_launch": ms_l * 1e3,
                                 "us_per_token_step": ms_l * 1e3 / TM,
                                 "tokens_per_s": world * wd.B * TM / (ms_l * 1e-3),
                                 "achieved_GBps": mb / (ms_l * 1e-3) / 1e9,
                                 "algorithmic_bytes_per_launch": mb}
    # ---- longer bursts: hgrn2_step_multi against the prefill kernel used as a T-token step (hgrn2_fwd, saved = NULL)
    alts = []
    for TT in (8, 32, 64):
        if T < TT:
            continue
        seq = {k: gates[k][:TT].permute(1, 2, 0, 3).contiguous() for k in gates}
        yt = torch.empty((wd.B, wd.H, TT, wd.dv), dtype=bf, device=dev)
        S2 = torch.empty_like(S)
        desc_t = binding.make_desc(wd.B, wd.H, TT, wd.dk, wd.dv, binding.HGRN2_BF16)
        ws_t = binding.alloc_workspace(desc_t, dev)
        f_multi = lambda: binding.hgrn2_step_multi(seq["o"], seq["f"], seq["i"], S, y=yt)
        f_fwd = lambda: binding.hgrn2_fwd(seq["o"], seq["f"], seq["i"], S, y=yt, SN=S2, saved=None, ws=ws_t,
                                          save_for_backward=False)
        for fn in (f_multi, f_fwd):
            fn()
        nb = 5
        t_m = max_over_ranks(timed(f_multi, nb)) / nb
        t_f = max_over_ranks(timed(f_fwd, nb)) / nb
        alts.append({"tokens_per_launch": TT, "step_multi_us": t_m * 1e3, "fwd_as_step_us": t_f * 1e3})
    decode["multi_token_alternatives"] = alts
    if args.only == "decode" and rank == 0:
        print(json.dumps({"only": "decode", "decode": decode}), flush=True)
    return decode


def run_other_workloads(args, binding, W, dev, rank, timed, peaks, bf):
    """fwd + bwd on the long-context and the larger-layer workloads (reported, not the headline): same recipe,
    same calls, 10 timed steps each after 3 warm-ups.  Rank 0 only."""
    import torch
    out = []
    if rank != 0:
        return out
    # prefill_5000: few long sequences whose length is not a whole number of chunks (16 heads x 5000 tokens), the
    # recipe of long_16k at another shape
    for name, gamma in (("long_16k", None),) + tuple(("lm_2560", g) for g in W.LM_2560_GAMMAS) + (("prefill_5000", None),):
        w = W.scaled(W.CONFIGS["long_16k"], B=1, H=16, N=5000) if name == "prefill_5000" else W.CONFIGS[name]
        inp = W.make_inputs(w, gamma=gamma)
        t = {k: (None if v is None else torch.from_numpy(v).to(dev)) for k, v in inp.items()}
        o, f, i, dy = (t[k].to(bf) for k in ("o", "f", "i", "dy"))
        S0, dSN = t["S0"], t["dSN"]
        del inp, t
        desc = binding.make_desc(w.B, w.H, w.N, w.dk, w.dv, binding.HGRN2_BF16, w.chunk, 0)
        saved = binding.alloc_saved(desc, dev)
        ws = binding.alloc_workspace(desc, dev)
        y = torch.empty_like(i); d_o = torch.empty_like(o); d_f = torch.empty_like(o); d_i = torch.empty_like(i)
        SN = torch.empty((w.B, w.H, w.dk, w.dv), dtype=torch.float32, device=dev) if w.has_S0 else None
        dS0 = torch.empty_like(SN) if SN is not None else None

        def fwd():
            binding.hgrn2_fwd(o, f, i, S0, y=y, SN=SN, saved=saved, ws=ws, want_final_state=SN is not None)

        def bwd():
            binding.hgrn2_bwd(o, f, i, S0, dy, dSN, saved, d_o=d_o, d_f=d_f, d_i=d_i, dS0=dS0, ws=ws,
                              want_dS0=dS0 is not None)

        def step():
            fwd(); bwd()

        for _ in range(3):
            step()
        n = 10
        ms = timed(step, n) / n
        ms_f = timed(fwd, n) / n
        ms_b = timed(bwd, n) / n
        torch.cuda.synchronize()
        assert binding.hgrn2_poll(ws) == 0, f"device-side error on {name}"
        ab = train_bytes(w)
        state_bytes = 4 * w.B * w.H * w.dk * w.dv * 4 if w.has_S0 else 0
        t_hbm = (ab["fwd"] + ab["bwd"] + state_bytes) / (peaks["hbm_gbs"] * 1e9)
        out.append({"workload": name, "B": w.B, "H": w.H, "N": w.N, "gamma": w.gamma if gamma is None else gamma,
                    "units": w.B * w.H, "ms_per_step": ms, "fwd_ms": ms_f, "bwd_ms": ms_b,
                    "tokens_per_s": w.tokens / (ms * 1e-3), "frac_of_hbm_roofline": t_hbm * 1e3 / ms,
                    "frac_of_nominal_hbm_roofline": t_hbm * 1e3 / ms * peaks["hbm_gbs"] / NOMINAL["hbm_gbs"],
                    "exact_path_units": binding.exact_path_units(ws)})
        del o, f, i, dy, saved, ws, y, d_o, d_f, d_i
        torch.cuda.empty_cache()
    out.append(run_packed_mix(binding, W, dev, timed, peaks, bf))
    out.append(run_gated(binding, W, dev, timed, peaks, bf))
    return out


def run_gated(binding, W, dev, timed, peaks, bf):
    """lm_2048 through the gated entry points: pre-activations in, gradients of the pre-activations and of the lower
    bound out (Eq. 1 / Eq. 2 in front of the recurrence).  Algorithmic bytes: the same eleven tensor passes."""
    import torch
    w = W.CONFIGS["lm_2048"]
    rng = np.random.default_rng(11)
    shape = (w.B, w.H, w.N, w.dk)
    z = {k: torch.from_numpy(rng.standard_normal(shape, dtype=np.float32)).to(dev).to(bf) for k in ("zo", "zf", "zi", "dy")}
    beta = torch.full((w.H, w.dk), 0.9, dtype=torch.float32, device=dev)
    y, _, saved, ws, _ = binding.hgrn2_fwd_gated(z["zo"], z["zf"], z["zi"], beta, None, want_final_state=False)
    outs = [torch.empty_like(z["zo"]) for _ in range(3)]
    d_beta = torch.empty_like(beta)

    def fwd():
        binding.hgrn2_fwd_gated(z["zo"], z["zf"], z["zi"], beta, None, y=y, saved=saved, ws=ws, want_final_state=False)

    def bwd():
        binding.hgrn2_bwd_gated(z["zo"], z["zf"], z["zi"], beta, None, z["dy"], None, saved, d_zo=outs[0], d_zf=outs[1],
                                d_zi=outs[2], d_beta=d_beta, ws=ws, want_dS0=False)

    def step():
        fwd(); bwd()

    for _ in range(3):
        step()
    n = 20
    ms = timed(step, n) / n
    ms_f = timed(fwd, n) / n
    ms_b = timed(bwd, n) / n
    torch.cuda.synchronize()
    assert binding.hgrn2_poll(ws) == 0
    ab = train_bytes(w)
    t_hbm = (ab["fwd"] + ab["bwd"]) / (peaks["hbm_gbs"] * 1e9)
    return {"workload": "lm_2048_gated", "B": w.B, "H": w.H, "N": w.N, "beta": 0.9, "ms_per_step": ms, "fwd_ms": ms_f,
            "bwd_ms": ms_b, "tokens_per_s": w.tokens / (ms * 1e-3), "frac_of_hbm_roofline": t_hbm * 1e3 / ms,
            "exact_path_units": binding.exact_path_units(ws),
            "note": "tensor-core path: element-wise gate kernels in front (3 tensors in, 3 out) and behind (6 in, 3 out)"}


# A ragged batch as a long-context fine-tuning step would see it: 24 sequences between 256 and 4096 tokens
# (longest first), 16 heads of 128.  Timed packed (hgrn2_*_varlen) and padded to the longest (hgrn2_fwd/bwd).
PACKED_MIX_LENGTHS = (4096, 3072, 2048, 2048, 1536, 1024, 1024, 1024, 1024, 768, 768, 768, 512, 512, 512, 512,
                      384, 384, 256, 256, 256, 256, 256, 256)


def run_packed_mix(binding, W, dev, timed, peaks, bf):
    import torch
    lengths = PACKED_MIX_LENGTHS
    H, d, B, T, Nmax = 16, 128, len(lengths), int(sum(lengths)), max(lengths)
    w = W.scaled(W.CONFIGS["lm_2048"], B=1, H=H, N=T, seed=9)
    inp = W.make_inputs(w)
    pk = {k: torch.from_numpy(inp[k][0]).to(dev).to(bf) for k in ("o", "f", "i", "dy")}
    cu_h = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    cu = torch.from_numpy(cu_h).to(dev)
    # the padded equivalent: [B, H, Nmax, d] with neutral tokens (f = 1, o = i = dy = 0) after each sequence's end
    pad = {k: torch.zeros((B, H, Nmax, d), dtype=bf, device=dev) for k in pk}
    pad["f"].fill_(1.0)
    for b in range(B):
        s, e = int(cu_h[b]), int(cu_h[b + 1])
        for k in pk:
            pad[k][b, :, :e - s] = pk[k][:, s:e]
    res = {"workload": "packed_mix", "sequences": B, "H": H, "tokens": T, "longest": Nmax, "padded_tokens": B * Nmax}
    y, SN, saved, ws, _ = binding.hgrn2_fwd_varlen(pk["o"], pk["f"], pk["i"], cu, None, want_final_state=False)
    outs = [torch.empty_like(pk["o"]) for _ in range(3)]

    def step_packed():
        binding.hgrn2_fwd_varlen(pk["o"], pk["f"], pk["i"], cu, None, y=y, saved=saved, ws=ws, want_final_state=False)
        binding.hgrn2_bwd_varlen(pk["o"], pk["f"], pk["i"], cu, None, pk["dy"], None, saved, d_o=outs[0], d_f=outs[1],
                                 d_i=outs[2], ws=ws, want_dS0=False)

    for _ in range(3):
        step_packed()
    n = 10
    ms_p = timed(step_packed, n) / n
    torch.cuda.synchronize()
    assert binding.hgrn2_poll(ws) == 0
    y_packed = y.clone()
    del saved, ws, outs
    yp, _, saved2, ws2, _ = binding.hgrn2_fwd(pad["o"], pad["f"], pad["i"], None, want_final_state=False)
    outs2 = [torch.empty_like(pad["o"]) for _ in range(3)]

    def step_padded():
        binding.hgrn2_fwd(pad["o"], pad["f"], pad["i"], None, y=yp, saved=saved2, ws=ws2, want_final_state=False)
        binding.hgrn2_bwd(pad["o"], pad["f"], pad["i"], None, pad["dy"], None, saved2, d_o=outs2[0], d_f=outs2[1],
                          d_i=outs2[2], ws=ws2, want_dS0=False)

    for _ in range(3):
        step_padded()
    ms_d = timed(step_padded, n) / n
    torch.cuda.synchronize()
    assert binding.hgrn2_poll(ws2) == 0
    # both layouts must agree on the real tokens (padding with the neutral token is exact)
    s, e = int(cu_h[3]), int(cu_h[4])
    diff = (y_packed[:, s:e].float() - yp[3, :, :e - s].float()).abs().max() / yp[3, :, :e - s].float().abs().max()
    assert float(diff) < 1e-2, f"packed and padded results differ: {float(diff)}"
    bytes_real = 11 * H * T * d * 2
    res.update({"ms_per_step_packed": ms_p, "ms_per_step_padded": ms_d, "tokens_per_s_packed": T / (ms_p * 1e-3),
                "tokens_per_s_padded": T / (ms_d * 1e-3), "speedup_over_padded": ms_d / ms_p,
                "frac_of_hbm_roofline_packed": bytes_real / (peaks["hbm_gbs"] * 1e9) * 1e3 / ms_p})
    return res


def run_cuda(args):
    import torch
    import torch.distributed as dist
    from paper_2404_07904_b200 import binding, workloads as W
    import __graft_entry__ as entry

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but the launcher started {world} rank(s)")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback for the product path)")
    if rank == 0:
        entry.build()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
        dist.barrier()
    binding.load()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms):
        if world > 1:
            t = torch.tensor([ms], dtype=torch.float64, device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            return float(t.item())
        return ms

    peaks, peak_kind = load_peaks()
    w = W.CONFIGS["lm_2048"]
    # every rank holds its own batch of the same shape (weak scaling); a different seed per rank
    inp = W.make_inputs(w, seed=w.seed + 1000 * rank)
    bf = torch.bfloat16
    host = {k: torch.from_numpy(inp[k]).to(bf).pin_memory() for k in ("o", "f", "i", "dy")}
    d = {k: v.to(dev, non_blocking=True) for k, v in host.items()}
    desc = binding.make_desc(w.B, w.H, w.N, w.dk, w.dv, binding.HGRN2_BF16, w.chunk, 0)
    path = binding.path_of(desc)
    shape_k, shape_v = (w.B, w.H, w.N, w.dk), (w.B, w.H, w.N, w.dv)
    y = torch.empty(shape_v, dtype=bf, device=dev)
    d_o = torch.empty(shape_k, dtype=bf, device=dev)
    d_f = torch.empty(shape_k, dtype=bf, device=dev)
    d_i = torch.empty(shape_v, dtype=bf, device=dev)
    saved = binding.alloc_saved(desc, dev)
    ws = binding.alloc_workspace(desc, dev)
    host_out = {k: torch.empty_like(v, device="cpu").pin_memory() for k, v in (("y", y), ("d_o", d_o), ("d_f", d_f), ("d_i", d_i))}
    stream = torch.cuda.current_stream()

    def fwd():
        binding.hgrn2_fwd(d["o"], d["f"], d["i"], None, y=y, saved=saved, ws=ws, want_final_state=False)

    def bwd():
        binding.hgrn2_bwd(d["o"], d["f"], d["i"], None, d["dy"], None, saved, d_o=d_o, d_f=d_f, d_i=d_i, ws=ws,
                          want_dS0=False)

    def step():
        fwd(); bwd()

    # End to end from pinned host buffers: the batch is cut into slices of whole sequences (units are
    # independent); slice j+1 is uploaded and slice j-1 downloaded while slice j computes, on three streams,
    # so the two PCIe directions and the kernels overlap.  The timed region starts and ends on `stream`.
    n_slices = 4 if w.B % 4 == 0 else 1
    bs = w.B // n_slices
    s_up, s_dn = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    desc_s = binding.make_desc(bs, w.H, w.N, w.dk, w.dv, binding.HGRN2_BF16, w.chunk, 0)
    saved_s = binding.alloc_saved(desc_s, dev)
    ws_s = binding.alloc_workspace(desc_s, dev)
    outs = {"y": y, "d_o": d_o, "d_f": d_f, "d_i": d_i}

    def e2e_step():
        start = torch.cuda.Event(); start.record(stream)
        s_up.wait_event(start); s_dn.wait_event(start)
        ups, dones = [], []
        for j in range(n_slices):
            sl = slice(j * bs, (j + 1) * bs)
            with torch.cuda.stream(s_up):
                for k in ("o", "f", "i", "dy"):
                    d[k][sl].copy_(host[k][sl], non_blocking=True)
                ev = torch.cuda.Event(); ev.record(s_up); ups.append(ev)
        for j in range(n_slices):
            sl = slice(j * bs, (j + 1) * bs)
            stream.wait_event(ups[j])
            binding.hgrn2_fwd(d["o"][sl], d["f"][sl], d["i"][sl], None, y=y[sl], saved=saved_s, ws=ws_s,
                              want_final_state=False)
            binding.hgrn2_bwd(d["o"][sl], d["f"][sl], d["i"][sl], None, d["dy"][sl], None, saved_s, d_o=d_o[sl],
                              d_f=d_f[sl], d_i=d_i[sl], ws=ws_s, want_dS0=False)
            ev = torch.cuda.Event(); ev.record(stream); dones.append(ev)
            with torch.cuda.stream(s_dn):
                s_dn.wait_event(ev)
                for k, t in outs.items():
                    host_out[k][sl].copy_(t[sl], non_blocking=True)
        end = torch.cuda.Event(); end.record(s_dn)
        stream.wait_event(end)

    def timed(fn, n):
        """n calls between two events on the launching stream; ms for the n calls."""
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        for _ in range(n):
            fn()
        e1.record(stream)
        barrier()
        return e0.elapsed_time(e1)

    K, Wm = args.steps, max(args.warmup, 3)
    if args.only == "others":
        others = run_other_workloads(args, binding, W, dev, rank, timed, peaks, bf)
        if rank == 0:
            print(json.dumps({"only": "others", "other_workloads": others}), flush=True)
        return 0
    if args.only == "decode":
        run_decode(args, binding, W, dev, rank, world, timed, max_over_ranks, peaks, peak_kind, bf)
        return 0
    for _ in range(Wm):
        step()
    torch.cuda.synchronize()
    assert binding.hgrn2_poll(ws) == 0, "device-side error during warm-up"

    # isolated kernel loops, before the long step loop (see the module docstring)
    ms_fwd = max_over_ranks(timed(fwd, K))
    ms_bwd = max_over_ranks(timed(bwd, K))

    sampler = ClockSampler(torch.cuda.current_device() if "CUDA_VISIBLE_DEVICES" not in os.environ else local_rank)
    if rank == 0:
        sampler.start()
    # batches of exactly K steps until at least --min-seconds of device time; every rank takes the same number of
    # batches because the continue/stop decision is made on the max-over-ranks times
    batch_ms, spent = [], 0.0
    while True:
        batch_ms.append(max_over_ranks(timed(step, K)))
        spent += batch_ms[-1] * 1e-3
        if spent >= args.min_seconds or len(batch_ms) >= 100000:
            break
    if rank == 0:
        sampler.stop()
    clocks = sampler.summary()
    ms_total = statistics.median(batch_ms)
    for _ in range(2):
        e2e_step()
    torch.cuda.synchronize()
    # the sliced, overlapped path must deliver what the plain path does (slices of few units run split into
    # segments, so the comparison is up to rounding)
    y_e2e = host_out["y"].float()
    step()
    torch.cuda.synchronize()
    y_ref = y.float().cpu()
    e2e_err = float((y_e2e - y_ref).abs().max() / y_ref.abs().max())
    assert e2e_err < 1e-2, f"end-to-end path disagrees with the device-resident path: {e2e_err}"
    ms_e2e = max_over_ranks(timed(e2e_step, max(3, min(K, 10)))) / max(3, min(K, 10))
    assert binding.hgrn2_poll(ws) == 0, "device-side error during the timed region"
    assert binding.exact_path_units(ws) == 0, "the benchmark workload must stay on the tensor-core kernels"

    ms_step = ms_total / K
    tokens_per_step = world * w.tokens
    value = tokens_per_step / (ms_step * 1e-3)
    e2e_value = tokens_per_step / (ms_e2e * 1e-3)
    ab = train_bytes(w)
    fl = train_flops(w)
    kern = {}
    for name, ms in (("fwd", ms_fwd / K), ("bwd", ms_bwd / K)):
        kern[name] = {"ms": ms, "GBps": ab[name] / (ms * 1e-3) / 1e9, "TFLOPs": fl[name] / (ms * 1e-3) / 1e12,
                      "timed": "isolated loop of this kernel alone"}
    dom = "bwd" if kern["bwd"]["ms"] >= kern["fwd"]["ms"] else "fwd"
    # Roofline of a pass = the slower of its bytes at HBM bandwidth and its FLOPs at the dense bf16 rate.  Measured
    # peaks: the burst GEMM rate for a kernel timed alone, the sustained one for the seconds-long step loop.
    def bound_of(nbytes, flops, tf_key):
        t_h = nbytes / (peaks["hbm_gbs"] * 1e9)
        t_t = flops / (peaks[tf_key] * 1e12)
        t_hn = nbytes / (NOMINAL["hbm_gbs"] * 1e9)
        t_tn = flops / (NOMINAL["bf16_tflops"] * 1e12)
        return {"bound": "hbm" if t_h >= t_t else "tensor", "t_hbm_us": t_h * 1e6, "t_tensor_us": t_t * 1e6,
                "t_roof_us": max(t_h, t_t) * 1e6, "t_roof_nominal_us": max(t_hn, t_tn) * 1e6}
    rk = bound_of(ab[dom], fl[dom], "bf16_tflops")
    rs = bound_of(ab["fwd"] + ab["bwd"], fl["fwd"] + fl["bwd"], "bf16_tflops_sustained")
    sm_mhz = clocks.get("sm_mhz")
    roofline = {
        "bound": rk["bound"], "kernel": f"hgrn2_{dom} ({path})", "achieved": kern[dom]["GBps"], "peak": peaks["hbm_gbs"],
        "unit": "GB/s", "frac": kern[dom]["GBps"] / peaks["hbm_gbs"], "traffic": NCU_TRAFFIC_BYTES[dom],
        "traffic_source": NCU_TRAFFIC_SOURCE[dom],
        "peak_source": f"of {peak_kind}", "algorithmic_bytes_per_launch": ab[dom],
        "frac_nominal": kern[dom]["GBps"] / NOMINAL["hbm_gbs"], "timed": "isolated loop of the dominant kernel",
        "step": {"timed": "median batch of the fwd+bwd step loop (the line's value)", "bound": rs["bound"],
                 "t_hbm_us": rs["t_hbm_us"], "t_tensor_us": rs["t_tensor_us"],
                 "roofline_tokens_per_s": w.tokens / (rs["t_roof_us"] * 1e-6),
                 "frac": rs["t_roof_us"] * 1e-3 / ms_step, "frac_source": f"of {peak_kind}",
                 "frac_nominal": rs["t_roof_nominal_us"] * 1e-3 / ms_step,
                 "nominal": dict(NOMINAL),
                 "sm_mhz_median": sm_mhz,
                 "sm_cycles_per_step": (ms_step * 1e-3 * sm_mhz * 1e6) if sm_mhz else None},
        "kernels": kern,
    }
    timing = {"batches": len(batch_ms), "steps_per_batch": K, "seconds": spent,
              "ms_per_step_median": ms_step, "ms_per_step_min": min(batch_ms) / K, "ms_per_step_max": max(batch_ms) / K}

    if args.only == "train":
        if rank == 0:
            print(json.dumps({"only": "train", "ms_per_step": ms_step, "kernels": kern, "timing": timing,
                              "clocks": clocks}), flush=True)
        return 0
    decode = run_decode(args, binding, W, dev, rank, world, timed, max_over_ranks, peaks, peak_kind, bf)
    others = run_other_workloads(args, binding, W, dev, rank, timed, peaks, bf) if not args.skip_others else []

    if world > 1:
        dist.barrier()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    # ---- oracle on the host cores, bounded sample -------------------------------------------------
    from oracle import ref
    ref.build()
    cores = ref.num_threads()
    n_units = w.B * w.H                       # the whole workload per repetition
    _, probe_dt, cores = time_oracle(w, 1, 0, n_units)
    reps = int(min(12, max(2, round(12.0 / max(probe_dt, 1e-3)))))      # about 12 s of CPU work
    cpu_value, cpu_dt, cores = time_oracle(w, reps, 0, n_units)
    cpu_baseline = {"value": cpu_value, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                    "sample": f"all {n_units} (batch, head) units of lm_2048 (N={w.N}), fwd+bwd in fp64, "
                              f"{reps} timed repetitions of {cpu_dt:.2f} s after one untimed"}

    line = {
        "metric": "HGRN2 layer fwd+bwd tokens/s", "value": value, "unit": "tokens/s", "n_gpus": world,
        "steps": K, "warmup": Wm, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": workload_config(w, path),
        "roofline": roofline, "cpu_baseline": cpu_baseline, "decode": decode, "other_workloads": others,
        "e2e": {"value": e2e_value, "unit": "tokens/s", "ms_per_step": ms_e2e,
                "h2d_bytes_per_step": sum(v.numel() * v.element_size() for v in host.values()),
                "d2h_bytes_per_step": sum(v.numel() * v.element_size() for v in host_out.values())},
        "gpu_launches": 2 * K,
        "timing": timing,
        "clocks": clocks,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()
    return 0


def self_launch(argv, n):
    """Start n ranks of this script under torch.distributed.run on this node and return their exit code."""
    import socket
    sock = socket.socket()
    sock.bind(("127.0.0.1", 0))
    port = sock.getsockname()[1]
    sock.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "WARN")
    return subprocess.call(cmd, env=env)


def run_launch_check(args):
    """Stub arm for the launcher path (no GPU): the ranks rendezvous over gloo, take the barrier and the
    max-over-ranks reduction the CUDA arm uses for its timings, and rank 0 prints one JSON line."""
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    t = torch.tensor([100.0 + rank], dtype=torch.float64)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"impl": "launch-check", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                          "max_over_ranks": float(t.item())}), flush=True)
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference", "launch-check"])
    ap.add_argument("--min-seconds", type=float, default=2.0,
                    help="repeat the timed K-step batch until this much device time has been spent (median batch reported)")
    ap.add_argument("--only", default="all", choices=["all", "train", "decode", "others"],
                    help="restrict the run to one part (for profiling); the JSON line is printed for 'all' only")
    ap.add_argument("--decode-steps", type=int, default=0, help="decode calls to time (0 = the workload's 512)")
    ap.add_argument("--skip-others", action="store_true", help="do not time the long-context and larger-layer workloads")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)      # rank 0 alone works, with or without a launcher
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return self_launch(sys.argv[1:], args.gpus)
    if args.impl == "launch-check":
        return run_launch_check(args)
    return run_cuda(args)


if __name__ == "__main__":
    sys.exit(main())
