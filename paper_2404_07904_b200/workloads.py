"""Seeded synthetic workloads shaped like the paper's language-model layers.

This module holds input recipes only: shapes, value distributions and the dtype
rounding of the inputs.  It contains none of the recurrence's arithmetic, so both
the CUDA path and the CPU oracle may be fed from it.

Recipe (numpy ``default_rng(seed)``, PCG64, ``standard_normal`` in float32, drawn in
the fixed order ``o, z, i, dy, S0, dSN``, each in its full shape):

* ``o, i``  = scale * N(0, 1)
* ``f``     = gamma + (1 - gamma) * sigmoid(z)       (Eq. 2: lower bound gamma plus a sigmoid residual)
* ``dy``    = N(0, 1) upstream gradient
* ``S0``    = 0.02 * N(0, 1) when the workload has an initial state, else absent
* ``dSN``   = 0.02 * N(0, 1) when the workload feeds a final-state gradient, else absent

With bf16 I/O the float32 draws are rounded once to bf16 (round to nearest even)
and returned as float32 arrays holding exactly representable values, so the GPU
and the oracle consume the same numbers and input quantisation is not counted as
error.  State tensors stay float32.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    N: int
    dk: int
    dv: int
    io: str                 # "f32" or "bf16"
    gamma: float
    scale: float
    has_S0: bool
    has_dSN: bool
    seed: int
    chunk: int = 0          # 0 = library default

    @property
    def units(self) -> int:
        return self.B * self.H

    @property
    def tokens(self) -> int:
        return self.B * self.N


_R = 1.0 / np.sqrt(128.0)

# The five configurations of the benchmark spec: tiny fp32, the 1B-model layer (hidden 2048, 16 heads,
# expand ratio 128, sequence 2048), the 16K long-context layer, the 2.9B-model layer
# (hidden 2560), and the decode batch.
CONFIGS: Dict[str, Workload] = {
    "tiny_f32":  Workload("tiny_f32", 1, 2, 256, 64, 64, "f32", 0.5, 1.0, False, False, 0, 64),
    "lm_2048":   Workload("lm_2048", 8, 16, 2048, 128, 128, "bf16", 0.9, _R, False, False, 1),
    "long_16k":  Workload("long_16k", 2, 16, 16384, 128, 128, "bf16", 0.99, _R, True, True, 2),
    "lm_2560":   Workload("lm_2560", 8, 20, 4096, 128, 128, "bf16", 0.9, _R, False, False, 3),
    "decode":    Workload("decode", 256, 16, 512, 128, 128, "bf16", 0.9, _R, True, False, 4),
}
LM_2560_GAMMAS = (0.0, 0.5, 0.9, 0.99)


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some fields replaced (used for reduced-size parity cases)."""
    return replace(w, **kw)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result is float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """The uint16 bit patterns of float32 values that are already bf16-representable."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def make_inputs(w: Workload, seed: Optional[int] = None, gamma: Optional[float] = None):
    """Training-shaped inputs: dict with o, f [B,H,N,dk]; i, dy [B,H,N,dv]; S0, dSN [B,H,dk,dv] or None."""
    rng = np.random.default_rng(w.seed if seed is None else seed)
    g = np.float32(w.gamma if gamma is None else gamma)
    sk = (w.B, w.H, w.N, w.dk)
    sv = (w.B, w.H, w.N, w.dv)
    ss = (w.B, w.H, w.dk, w.dv)
    sc = np.float32(w.scale)
    o = rng.standard_normal(sk, dtype=np.float32) * sc
    z = rng.standard_normal(sk, dtype=np.float32)
    f = g + (np.float32(1) - g) / (np.float32(1) + np.exp(-z))
    del z
    i = rng.standard_normal(sv, dtype=np.float32) * sc
    dy = rng.standard_normal(sv, dtype=np.float32)
    S0 = rng.standard_normal(ss, dtype=np.float32) * np.float32(0.02) if w.has_S0 else None
    dSN = rng.standard_normal(ss, dtype=np.float32) * np.float32(0.02) if w.has_dSN else None
    f = np.minimum(f, np.float32(1.0)).astype(np.float32)
    if w.io == "bf16":
        o, f, i, dy = (round_to_bf16(a) for a in (o, f, i, dy))
    return {"o": o, "f": f, "i": i, "dy": dy, "S0": S0, "dSN": dSN}


def make_decode_inputs(w: Workload, steps: Optional[int] = None, seed: Optional[int] = None):
    """Decode-shaped inputs: o, f [T,B,H,dk], i [T,B,H,dv] for T successive one-token calls, S0 [B,H,dk,dv]."""
    rng = np.random.default_rng(w.seed if seed is None else seed)
    T = w.N if steps is None else steps
    g = np.float32(w.gamma)
    sc = np.float32(w.scale)
    sk = (T, w.B, w.H, w.dk)
    sv = (T, w.B, w.H, w.dv)
    o = rng.standard_normal(sk, dtype=np.float32) * sc
    z = rng.standard_normal(sk, dtype=np.float32)
    f = np.minimum(g + (np.float32(1) - g) / (np.float32(1) + np.exp(-z)), np.float32(1.0)).astype(np.float32)
    del z
    i = rng.standard_normal(sv, dtype=np.float32) * sc
    S0 = rng.standard_normal((w.B, w.H, w.dk, w.dv), dtype=np.float32) * np.float32(0.02)
    if w.io == "bf16":
        o, f, i = (round_to_bf16(a) for a in (o, f, i))
    return {"o": o, "f": f, "i": i, "S0": S0}


def shard_units(total: int, world_size: int, rank: int):
    """Contiguous split of `total` independent units over ranks: (start, count)."""
    base, rem = divmod(total, world_size)
    start = rank * base + min(rank, rem)
    return start, base + (1 if rank < rem else 0)
