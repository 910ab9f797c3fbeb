"""CPU checks of the boundary: the library loads, exports every declared symbol, and rejects
bad arguments on the host without launching anything (no GPU needed for any of this)."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as entry
from paper_2404_07904_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    entry.build()
    return binding.load()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "hgrn2.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hgrn2_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    syms = declared_symbols()
    assert set(binding.EXPORTS) <= set(syms)
    for s in syms:
        assert getattr(lib, s) is not None, s


def test_status_strings(lib):
    seen = {binding.status_string(c) for c in range(8)}
    assert len(seen) == 8 and "ok" in seen
    assert binding.status_string(99) == "unknown status"


def test_size_queries(lib):
    d = binding.make_desc(1, 2, 256, 64, 64, binding.HGRN2_F32, 64)
    assert binding.chunk_of(d) == 64 and binding.path_of(d) == "alu"
    assert binding.saved_bytes(d) == 1 * 2 * 4 * 64 * 64 * 4
    assert binding.workspace_bytes(d) == 256 + binding.saved_bytes(d)
    d = binding.make_desc(2, 3, 100, 128, 128, binding.HGRN2_F32, 0)
    C = binding.chunk_of(d)
    assert C in (16, 32, 64)
    assert binding.saved_bytes(d) == 2 * 3 * ((100 + C - 1) // C) * 128 * 128 * 4
    # unsupported shapes and chunks give 0
    assert binding.workspace_bytes(binding.make_desc(1, 1, 8, 48, 64, 0)) == 0
    assert binding.workspace_bytes(binding.make_desc(1, 1, 8, 64, 64, 0, chunk=7)) == 0
    assert binding.workspace_bytes(binding.make_desc(1, 1, 8, 64, 64, 5)) == 0
    assert binding.workspace_bytes(binding.make_desc(-1, 1, 8, 64, 64, 0)) == 0
    assert binding.path_of(binding.make_desc(1, 1, 8, 48, 64, 0)) == ""


def test_bf16_128_goes_to_tensor_cores_unless_forced(lib):
    d = binding.make_desc(8, 16, 2048, 128, 128, binding.HGRN2_BF16)
    forced = binding.make_desc(8, 16, 2048, 128, 128, binding.HGRN2_BF16, flags=binding.FLAG_FORCE_ALU)
    assert binding.path_of(forced) == "alu"
    assert binding.path_of(d) == "tcgen05"
    assert binding.chunk_of(d) == 64
    assert binding.saved_bytes(d) == 8 * 16 * 32 * (128 * 128 * 2 + 2 * 128 * 4)   # per chunk: bf16 state + decay totals
    assert binding.workspace_bytes(binding.make_desc(8, 16, 2048, 128, 128, binding.HGRN2_BF16, chunk=32)) == 0
    assert binding.path_of(binding.make_desc(1, 1, 64, 128, 64, binding.HGRN2_BF16)) == "alu"
    assert binding.path_of(binding.make_desc(1, 1, 64, 128, 128, binding.HGRN2_F32)) == "alu"


def _call_fwd(lib, d, ptrs):
    return lib.hgrn2_fwd(ctypes.byref(d), *[ctypes.c_void_p(p) for p in ptrs])


def test_host_side_argument_errors_launch_nothing(lib):
    d = binding.make_desc(1, 1, 8, 64, 64, binding.HGRN2_F32)
    ok = 0x1000  # never dereferenced: every call below is rejected on the host first
    # fwd args: o f i S0 y SN saved ws stream
    assert _call_fwd(lib, d, [0, ok, ok, 0, ok, 0, 0, ok, 0]) == 1            # NULL o
    assert _call_fwd(lib, d, [ok, ok, ok, 0, 0, 0, 0, ok, 0]) == 1            # NULL y
    assert _call_fwd(lib, d, [ok, ok, ok, 0, ok, 0, 0, 0, 0]) == 4            # no workspace
    assert _call_fwd(lib, d, [ok + 4, ok, ok, 0, ok, 0, 0, ok, 0]) == 3       # misaligned o
    assert _call_fwd(lib, d, [ok, ok, ok, ok + 8, ok, 0, 0, ok, 0]) == 3      # misaligned S0
    bad = binding.make_desc(1, 1, 8, 48, 64, binding.HGRN2_F32)
    assert _call_fwd(lib, bad, [ok] * 8 + [0]) == 2                           # unsupported dk
    bad = binding.make_desc(1, 1, 8, 64, 64, 3)
    assert _call_fwd(lib, bad, [ok] * 8 + [0]) == 1                           # bad dtype enum
    assert lib.hgrn2_fwd(None, *[ctypes.c_void_p(ok)] * 8, None) == 1         # NULL desc
    # bwd args: o f i S0 dy dSN saved d_o d_f d_i dS0 ws stream
    args = [ok, ok, ok, 0, ok, 0, 0, ok, ok, ok, 0, ok, 0]
    for hole in (0, 1, 2, 4, 7, 8, 9):
        a = list(args); a[hole] = 0
        assert lib.hgrn2_bwd(ctypes.byref(d), *[ctypes.c_void_p(p) for p in a]) == 1
    a = list(args); a[11] = 0
    assert lib.hgrn2_bwd(ctypes.byref(d), *[ctypes.c_void_p(p) for p in a]) == 4
    a = list(args); a[5] = ok + 2
    assert lib.hgrn2_bwd(ctypes.byref(d), *[ctypes.c_void_p(p) for p in a]) == 3
    # step args: o f i S y stream
    assert lib.hgrn2_step(ctypes.byref(d), *[ctypes.c_void_p(p) for p in [ok, ok, ok, 0, ok, 0]]) == 1
    assert lib.hgrn2_step(ctypes.byref(d), *[ctypes.c_void_p(p) for p in [ok, ok + 1, ok, ok, ok, 0]]) == 3
    # multi-token step: same arguments; N tokens; d_k = d_v in {64, 128} only
    assert lib.hgrn2_step_multi(ctypes.byref(d), *[ctypes.c_void_p(p) for p in [ok, ok, ok, 0, ok, 0]]) == 1
    assert lib.hgrn2_step_multi(ctypes.byref(d), *[ctypes.c_void_p(p) for p in [ok, ok + 1, ok, ok, ok, 0]]) == 3
    odd = binding.make_desc(1, 1, 4, 32, 64, binding.HGRN2_F32)
    assert lib.hgrn2_step_multi(ctypes.byref(odd), *[ctypes.c_void_p(p) for p in [ok, ok, ok, ok, ok, 0]]) == 2
    none = binding.make_desc(1, 1, 0, 64, 64, binding.HGRN2_F32)
    assert lib.hgrn2_step_multi(ctypes.byref(none), *[ctypes.c_void_p(0)] * 6) == 0      # no token: no-op
    assert lib.hgrn2_poll(None) == 1


def test_new_entry_points_reject_bad_arguments_on_the_host(lib):
    vp = ctypes.c_void_p
    ok = 0x1000  # never dereferenced
    d = binding.make_desc(2, 1, 100, 64, 64, binding.HGRN2_F32)
    # packed batches: args o f i cu S0 y SN saved ws stream
    call = lambda a: lib.hgrn2_fwd_varlen(ctypes.byref(d), *[vp(p) for p in a])
    assert call([ok, ok, ok, 0, 0, ok, 0, 0, ok, 0]) == 1                      # no offsets
    assert call([ok, ok, ok, ok + 2, 0, ok, 0, 0, ok, 0]) == 3                 # misaligned offsets
    assert call([ok, ok, ok, ok, 0, ok, 0, 0, 0, 0]) == 4                      # no workspace
    assert call([ok, 0, ok, ok, 0, ok, 0, 0, ok, 0]) == 1                      # NULL f
    bwd = [ok, ok, ok, ok, 0, ok, 0, 0, ok, ok, ok, 0, ok, 0]
    a = list(bwd); a[3] = 0
    assert lib.hgrn2_bwd_varlen(ctypes.byref(d), *[vp(p) for p in a]) == 1
    a = list(bwd); a[9] = 0
    assert lib.hgrn2_bwd_varlen(ctypes.byref(d), *[vp(p) for p in a]) == 1     # NULL d_f
    assert lib.hgrn2_saved_bytes_varlen(ctypes.byref(d)) == 1 * (100 // 64 + 2 + 1) * 64 * 64 * 4
    assert lib.hgrn2_workspace_bytes_varlen(ctypes.byref(binding.make_desc(2, 1, 100, 48, 64, 0))) == 0
    # gated: args zo zf zi beta S0 y SN saved ws stream
    call = lambda a: lib.hgrn2_fwd_gated(ctypes.byref(d), *[vp(p) for p in a])
    assert call([ok, ok, ok, 0, 0, ok, 0, 0, ok, 0]) == 1                      # no beta
    assert call([ok, ok, ok, ok + 4, 0, ok, 0, 0, ok, 0]) == 3                 # misaligned beta
    assert call([ok, ok, ok, ok, 0, ok, 0, 0, 0, 0]) == 4                      # no workspace
    gb = [ok, ok, ok, ok, 0, ok, 0, 0, ok, ok, ok, 0, 0, ok, 0]
    a = list(gb); a[10] = 0
    assert lib.hgrn2_bwd_gated(ctypes.byref(d), *[vp(p) for p in a]) == 1      # NULL d_zi
    tc = binding.make_desc(2, 3, 256, 128, 128, binding.HGRN2_BF16)
    assert lib.hgrn2_saved_bytes_gated(ctypes.byref(tc)) == 3 * 2 * 3 * 256 * 128 * 2 + binding.saved_bytes(tc)
    assert lib.hgrn2_saved_bytes_gated(ctypes.byref(d)) == binding.saved_bytes(d)
    # spans: summary args f i S_loc lam ws stream; compose args r0 r1 reverse X lam init out stream
    assert lib.hgrn2_span_summary_fwd(ctypes.byref(d), *[vp(p) for p in [ok, ok, 0, ok, ok, 0]]) == 1
    assert lib.hgrn2_span_summary_fwd(ctypes.byref(d), *[vp(p) for p in [ok, ok, ok, ok, 0, 0]]) == 4
    assert lib.hgrn2_span_summary_bwd(ctypes.byref(d), *[vp(p) for p in [ok, ok + 8, ok, ok, ok, ok, 0]]) == 3
    assert lib.hgrn2_span_compose(ctypes.byref(d), 2, 1, 0, vp(ok), vp(ok), None, vp(ok), None) == 1    # r1 < r0
    assert lib.hgrn2_span_compose(ctypes.byref(d), 0, 2, 0, vp(ok), vp(ok), None, None, None) == 1      # no output
    assert lib.hgrn2_span_compose(ctypes.byref(d), 0, 2, 0, None, vp(ok), None, vp(ok), None) == 1      # no summaries
    assert lib.hgrn2_exact_path_units(None) == -1


def test_binding_refuses_cpu_tensors(lib):
    import torch
    o = torch.zeros(1, 1, 4, 64)
    with pytest.raises(ValueError):
        binding._ptr(o)


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2404_07904_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, fn)).read()
                assert "oracle" not in text.replace("the oracle", "").replace("CPU oracle", ""), fn
