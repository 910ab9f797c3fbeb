"""The N > 1 path on CPU: two gloo ranks shard the independent (batch, head) units, each runs its shard
(the oracle stands in for the GPU kernels here), rank 0 gathers, and the result must equal the unsharded
run bit for bit; the max-over-ranks timing reduction of bench.py is exercised the same way."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    os.environ["OMP_NUM_THREADS"] = "2"
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2404_07904_b200 import workloads as W
    from oracle import ref
    w = W.scaled(W.CONFIGS["tiny_f32"], B=3, H=2, N=40, dk=16, dv=16, has_S0=True)
    inp = W.make_inputs(w)                      # same seed on every rank: the global problem
    units = w.B * w.H
    start, count = W.shard_units(units, world, rank)
    flat = {k: (None if v is None else v.reshape(units, 1, *v.shape[2:])) for k, v in inp.items()}
    sl = slice(start, start + count)
    y, SN = ref.hgrn2_fwd(flat["o"][sl], flat["f"][sl], flat["i"][sl], flat["S0"][sl])
    # gather shards on rank 0 (bench.py needs no data collective; this is only to check the sharding)
    gathered = [None] * world
    dist.gather_object((start, y), gathered if rank == 0 else None, dst=0)
    # max-over-ranks timing, as bench.py does with its event times
    t = torch.tensor([10.0 + rank], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    if rank == 0:
        full = np.concatenate([g[1] for g in sorted(gathered, key=lambda g: g[0])], axis=0)
        np.save(os.path.join(out_dir, "y.npy"), full)
        np.save(os.path.join(out_dir, "t.npy"), t.numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_unit_sharding_matches_single_process(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    from paper_2404_07904_b200 import workloads as W
    from oracle import ref
    w = W.scaled(W.CONFIGS["tiny_f32"], B=3, H=2, N=40, dk=16, dv=16, has_S0=True)
    inp = W.make_inputs(w)
    y, _ = ref.hgrn2_fwd(inp["o"], inp["f"], inp["i"], inp["S0"])
    got = np.load(tmp_path / "y.npy").reshape(y.shape)
    np.testing.assert_array_equal(got, y)
    assert float(np.load(tmp_path / "t.npy")[0]) == 11.0


def test_bench_starts_its_own_ranks():
    # `python bench.py --gpus 2` with no launcher around it must re-execute itself under torch.distributed.run
    # and print one JSON line from rank 0; driven here with the CPU stub arm (gloo)
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "launch-check",
                          "--steps", "3", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    assert lines[0]["n_gpus"] == 2 and lines[0]["max_over_ranks"] == 101.0 and lines[0]["steps"] == 3


# ---------------------------------------------------------------- sequence parallelism: ordering and collective on CPU
class _OracleOps:
    """Stand-ins for the library's span calls, built from the oracle (torch CPU tensors in and out), so that
    seqpar's call order and its all-gather can run on gloo ranks."""

    def __init__(self):
        from oracle import ref
        self.ref = ref

    @staticmethod
    def _np(x):
        return None if x is None else x.numpy().astype(np.float64)

    def summary_fwd(self, f, i):
        f_, i_ = self._np(f), self._np(i)
        _, S_loc = self.ref.hgrn2_fwd(np.zeros_like(f_), f_, i_, None)
        return torch.from_numpy(S_loc), torch.from_numpy(f_.prod(axis=2))

    def summary_bwd(self, o, f, dy):
        o_, f_, dy_ = self._np(o), self._np(f), self._np(dy)
        G_loc = self.ref.hgrn2_bwd(o_, f_, np.zeros_like(dy_), None, dy_, None)[3]      # dS_0 does not depend on i
        return torch.from_numpy(G_loc), torch.from_numpy(f_.prod(axis=2))

    def compose(self, X_all, lam_all, r0, r1, reverse, init):
        S = torch.zeros_like(X_all[0]) if init is None else init.clone()
        order = range(r1 - 1, r0 - 1, -1) if reverse else range(r0, r1)
        for r in order:
            S = lam_all[r].unsqueeze(-1) * S + X_all[r]
        return S

    def fwd(self, o, f, i, S0):
        y, _ = self.ref.hgrn2_fwd(self._np(o), self._np(f), self._np(i), self._np(S0))
        return torch.from_numpy(y), None

    def bwd(self, o, f, i, S0, dy, dSN, ctx):
        g = self.ref.hgrn2_bwd(self._np(o), self._np(f), self._np(i), self._np(S0), self._np(dy), self._np(dSN))
        return tuple(torch.from_numpy(x) for x in g[:3])


def _seqpar_worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    os.environ["OMP_NUM_THREADS"] = "2"
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2404_07904_b200 import seqpar, workloads as W
    w = W.scaled(W.CONFIGS["tiny_f32"], B=2, H=2, N=30, dk=8, dv=4, has_S0=True, has_dSN=True)
    inp = {k: (None if v is None else torch.from_numpy(v.astype(np.float64))) for k, v in W.make_inputs(w).items()}
    bounds = [0, 13, 30]                                    # spans of unequal length
    sl = slice(bounds[rank], bounds[rank + 1])
    o, f, i, dy = (inp[k][:, :, sl].contiguous() for k in ("o", "f", "i", "dy"))
    ops = _OracleOps()
    y, SN, ctx = seqpar.forward(o, f, i, inp["S0"], ops=ops)
    d_o, d_f, d_i, dS0 = seqpar.backward(o, f, i, dy, inp["dSN"], ctx=ctx, ops=ops)
    np.savez(os.path.join(out_dir, f"r{rank}.npz"), y=y.numpy(), SN=SN.numpy(), d_o=d_o.numpy(), d_f=d_f.numpy(),
             d_i=d_i.numpy(), dS0=dS0.numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_sequence_parallel_spans_match_the_whole_sequence(tmp_path):
    # two ranks, one span each: summary -> all-gather -> compose -> span forward / backward must give exactly the
    # whole-sequence results (fp64 stand-ins, so up to rounding), and every rank the same S_N and dS_0
    world = 2
    mp.spawn(_seqpar_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    from paper_2404_07904_b200 import workloads as W
    from oracle import ref
    w = W.scaled(W.CONFIGS["tiny_f32"], B=2, H=2, N=30, dk=8, dv=4, has_S0=True, has_dSN=True)
    inp = {k: (None if v is None else v.astype(np.float64)) for k, v in W.make_inputs(w).items()}
    y, SN = ref.hgrn2_fwd(inp["o"], inp["f"], inp["i"], inp["S0"])
    d_o, d_f, d_i, dS0 = ref.hgrn2_bwd(inp["o"], inp["f"], inp["i"], inp["S0"], inp["dy"], inp["dSN"])
    got = [np.load(tmp_path / f"r{r}.npz") for r in range(world)]
    for name, want in (("y", y), ("d_o", d_o), ("d_f", d_f), ("d_i", d_i)):
        full = np.concatenate([g[name] for g in got], axis=2)
        np.testing.assert_allclose(full, want, rtol=1e-10, atol=1e-12, err_msg=name)
    for g in got:
        np.testing.assert_allclose(g["SN"], SN, rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(g["dS0"], dS0, rtol=1e-10, atol=1e-12)
