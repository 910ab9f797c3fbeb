"""The seeded input recipes: determinism, distributions, bf16 rounding, unit sharding."""
import numpy as np
import pytest
import torch

from paper_2404_07904_b200 import workloads as W


def test_configs_match_the_paper_shapes():
    c = W.CONFIGS
    assert (c["tiny_f32"].B, c["tiny_f32"].H, c["tiny_f32"].N, c["tiny_f32"].dk, c["tiny_f32"].chunk) == (1, 2, 256, 64, 64)
    assert c["lm_2048"].H * c["lm_2048"].dk == 2048 and c["lm_2048"].N == 2048 and c["lm_2048"].B == 8
    assert c["long_16k"].N == 16384 and c["long_16k"].has_S0 and c["long_16k"].has_dSN and c["long_16k"].gamma == 0.99
    assert c["lm_2560"].H * c["lm_2560"].dk == 2560 and c["lm_2560"].N == 4096
    assert c["decode"].B == 256 and c["decode"].N == 512


def test_seeded_and_bounded():
    w = W.scaled(W.CONFIGS["lm_2048"], B=1, H=2, N=64)
    a, b = W.make_inputs(w), W.make_inputs(w)
    for k in a:
        if a[k] is not None:
            np.testing.assert_array_equal(a[k], b[k])
    assert a["S0"] is None and a["dSN"] is None
    f = a["f"]
    assert f.min() >= np.float32(0.9) - 1e-3 and f.max() <= 1.0
    assert abs(float(a["o"].std()) * np.sqrt(128) - 1) < 0.05
    c = W.make_inputs(w, seed=99)
    assert not np.array_equal(a["o"], c["o"])
    g0 = W.make_inputs(w, gamma=0.0)["f"]
    assert g0.min() < 0.2 and g0.min() > 0.0


def test_bf16_rounding_is_rne_and_matches_torch():
    x = np.random.default_rng(0).standard_normal(10000).astype(np.float32)
    x[:4] = [1.0, 1.00390625, 1.01171875, -0.0]          # exact, tie -> even, tie -> even, signed zero
    r = W.round_to_bf16(x)
    t = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(r, t)
    np.testing.assert_array_equal(W.round_to_bf16(r), r)
    bits = W.to_bf16_bits(r)
    back = (bits.astype(np.uint32) << 16).view(np.float32)
    np.testing.assert_array_equal(back, r)


def test_decode_inputs():
    w = W.scaled(W.CONFIGS["decode"], B=3, H=2)
    d = W.make_decode_inputs(w, steps=5)
    assert d["o"].shape == (5, 3, 2, 128) and d["i"].shape == (5, 3, 2, 128) and d["S0"].shape == (3, 2, 128, 128)
    assert abs(float(d["S0"].std()) - 0.02) < 0.002


@pytest.mark.parametrize("total,ws", [(128, 1), (128, 8), (10, 4), (3, 8), (0, 2)])
def test_shard_units_partition(total, ws):
    spans = [W.shard_units(total, ws, r) for r in range(ws)]
    assert sum(n for _, n in spans) == total
    pos = 0
    for s, n in spans:
        assert s == pos
        pos += n
    assert max(n for _, n in spans) - min(n for _, n in spans) <= 1


def test_lm_workloads_have_the_papers_layer_shapes():
    # the benchmark shapes come from the paper's table of model configurations (stored as a text fixture):
    # hidden dim = H * d_k, expand ratio = head dim = 128, training sequence length 2048
    import os
    rows = []
    with open(os.path.join(os.path.dirname(__file__), "golden", "model_configurations.txt")) as fh:
        for line in fh:
            if line.strip() and not line.startswith("#"):
                p = line.split()
                rows.append((float(p[0]), int(p[1]), int(p[2]), int(p[3])))
    by_hidden = {r[1]: r for r in rows}
    w = W.CONFIGS["lm_2048"]
    assert w.H * w.dk in by_hidden and w.dk == w.dv == by_hidden[w.H * w.dk][2] and w.N == by_hidden[w.H * w.dk][3]
    w = W.CONFIGS["lm_2560"]
    assert w.H * w.dk in by_hidden and w.dk == w.dv == by_hidden[w.H * w.dk][2]
    for name in ("long_16k", "decode"):
        assert W.CONFIGS[name].dk == W.CONFIGS[name].dv == 128
