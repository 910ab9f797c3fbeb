"""Seeded random sweep of the default bf16 path against the oracle: shapes, lengths, lower bounds, states and, above
all, gate levels that sit near the limits of what the tensor-core operands can carry (key dimensions held at a
constant f between 0.03 and 1), where range and underflow mistakes show.  Eq. 3 is defined for every f in [0, 1];
each case checks every output, forward and backward, at the bf16 tolerance.
"""
import numpy as np
import pytest

from paper_2404_07904_b200 import workloads as W
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def _case(seed):
    rng = np.random.default_rng(seed)
    B, H = int(rng.integers(1, 4)), int(rng.integers(1, 5))
    N = int(rng.choice([1, 63, 65, 129, 200, 300, 512, 640, 1024, 2048]))
    gamma = float(rng.choice([0.0, 0.3, 0.9, 0.99]))
    states = bool(rng.integers(0, 2))
    w = W.scaled(W.CONFIGS["lm_2048"], B=B, H=H, N=N, has_S0=states, has_dSN=states, seed=seed, gamma=gamma)
    inp = W.make_inputs(w)
    mode = rng.choice(["as drawn", "constant columns", "stretches"])
    if mode == "constant columns":
        lo = float(rng.choice([0.03, 0.1, 0.2]))
        fc = np.exp(rng.uniform(np.log(lo), 0.0, (B, H, 1, 128))).astype(np.float32)
        pick = rng.uniform(0, 1, (B, H, 1, 128)) < 0.5
        inp["f"] = W.round_to_bf16(np.where(pick, fc, inp["f"]).astype(np.float32))
    elif mode == "stretches":
        for _ in range(int(rng.integers(1, 4))):
            b, h, c = int(rng.integers(0, B)), int(rng.integers(0, H)), int(rng.integers(0, 128))
            t0 = int(rng.integers(0, N))
            inp["f"][b, h, t0:t0 + int(rng.integers(1, 120)), c] = W.round_to_bf16(np.float32(rng.choice([0.01, 0.05, 0.2])))
    return inp, bool(rng.integers(0, 2)), f"seed {seed}: B{B} H{H} N{N} gamma {gamma} states {states}, {mode}"


@pytest.mark.parametrize("seed", range(100, 124))
def test_random_case_against_the_oracle(seed):
    inp, use_saved, what = _case(seed)
    got = G.gpu_fwd_bwd(inp, "bf16", use_saved=use_saved)
    B, H = inp["o"].shape[:2]
    units = sorted({(0, 0), (B - 1, H - 1), (B // 2, H // 2)})
    for (b, h), want in G.oracle_fwd_bwd(inp, units).items():
        G.assert_close({k: got[k][b:b + 1, h:h + 1] for k in want}, want, 2e-2, f"{what}, unit {(b, h)}")


@pytest.mark.parametrize("seed", range(200, 206))
def test_random_packed_batch_against_the_oracle(seed):
    from tests import test_gpu_varlen as TV
    rng = np.random.default_rng(seed)
    lengths = [int(rng.choice([0, 1, 30, 64, 65, 128, 200, 300, 700])) for _ in range(int(rng.integers(1, 6)))]
    if sum(lengths) == 0:
        lengths.append(70)
    inp = TV._packed_inputs(lengths, H=int(rng.integers(1, 4)), d=128, io="bf16", seed=seed,
                            gamma=float(rng.choice([0.0, 0.3, 0.9, 0.99])), with_states=bool(rng.integers(0, 2)),
                            pad_rows=int(rng.integers(0, 20)))
    T = inp["o"].shape[1]
    got, _ = TV._run_gpu(inp, "bf16", use_saved=bool(rng.integers(0, 2)))
    G.assert_close(TV._mask_rows(got, inp["cu"], T), TV._mask_rows(TV._oracle(inp), inp["cu"], T), 2e-2,
                   f"seed {seed}: lengths {lengths}")


@pytest.mark.parametrize("seed", range(300, 306))
def test_random_gated_case_against_the_oracle(seed):
    from tests import test_gpu_gated as TG
    rng = np.random.default_rng(seed)
    B, H = int(rng.integers(1, 4)), int(rng.integers(1, 4))
    N = int(rng.choice([5, 64, 129, 300, 511, 1024]))
    inp = TG._inputs(B, H, N, 128, "bf16", seed=seed, beta_lo=0.0, beta_hi=float(rng.choice([0.0, 0.9, 0.999])),
                     zf_shift=float(rng.choice([0.0, -2.0, 2.0])), states=bool(rng.integers(0, 2)))
    got, _ = TG._run(inp, "bf16", use_saved=bool(rng.integers(0, 2)))
    G.assert_close(got, TG._oracle(inp), 2e-2, f"seed {seed}: B{B} H{H} N{N}")
