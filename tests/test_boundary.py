"""The C-ABI boundary without a GPU: the library loads, exports what include/gsa.h
declares, answers workspace queries and rejects bad arguments before any launch."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as entry
import paper_2409_07146_b200 as gsa
from paper_2409_07146_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    entry.build()
    return gsa.load_library()


def declared_symbols():
    """Every entry point declared in the public header and in the header of the development aids."""
    names = []
    for h in ("gsa.h", "gsa_dev.h"):
        text = open(os.path.join(ROOT, "include", h)).read()
        names += re.findall(r"GSA_API[^;(]*?\b(gsa_\w+)\s*\(", text)
    return names


def test_library_exports_every_declared_symbol(lib):
    names = declared_symbols()
    assert set(names) >= {"gsa_fwd", "gsa_bwd", "gsa_decode_step", "gsa_gate_cumsum",
                          "gsa_workspace_bytes", "gsa_status_string", "gsa_chunk_size"}
    for n in names:
        assert hasattr(lib, n), n
    assert set(gsa.exported_symbols()) == set(names)
    # the layer's interface is gsa.h alone: the self-tests and timing hooks live in gsa_dev.h
    public = open(os.path.join(ROOT, "include", "gsa.h")).read()
    assert "gsa_tc_selftest" not in public and "gsa_timing_begin" not in public and "gsa_wait_selftest" not in public


def test_chunk_and_workspace_queries(lib):
    p = gsa.Params(B=2, T=100, H=3, d_k=64, d_v=128, m=32, io="f32")
    assert gsa.gsa_chunk_size(p) == 64
    assert gsa.gsa_chunk_size(gsa.Params(1, 256, 1, 128, 128, 64, io="bf16")) == 128
    assert gsa.gsa_chunk_size(gsa.Params(1, 256, 1, 128, 128, 64, io="bf16", impl="simt")) == 64
    # 64-wide heads and 32 slots run on the tensor-core kernels too (bf16 io)
    assert gsa.gsa_chunk_size(gsa.Params(1, 256, 1, 64, 64, 32, io="bf16")) == 128
    assert gsa.gsa_chunk_size(gsa.Params(1, 256, 1, 64, 64, 32, io="f32")) == 64
    f, b = gsa.gsa_workspace_bytes(p, binding.GSA_WS_FWD), gsa.gsa_workspace_bytes(p, binding.GSA_WS_BWD)
    assert f > 0 and b > f and f % 256 == 0
    assert gsa.gsa_workspace_bytes(p, binding.GSA_WS_DECODE) == 0
    g = gsa.gsa_workspace_bytes(p, binding.GSA_WS_GATE)      # flags + G + I (fp32 kernels: no decayed rows)
    assert g % 256 == 0 and 2 * 4 * 2 * 100 * 3 * 32 <= g < f
    bad = gsa.Params(B=2, T=100, H=3, d_k=96, d_v=128, m=32)
    assert gsa.gsa_workspace_bytes(bad, binding.GSA_WS_FWD) == 0


def _call_fwd(lib, p, ptrs, ws=0x1000, ws_bytes=1 << 40):
    cp = p.c()
    return lib.gsa_fwd(ctypes.byref(cp), *[ctypes.c_void_p(x) for x in ptrs],
                       ctypes.c_void_p(ws), ws_bytes, None, None)


def test_validation_happens_before_any_launch(lib):
    ok = [0x1000] * 4 + [None, None] + [0x1000] + [None, None, None]  # q k v gate K0 V0 o ok KT VT
    good = gsa.Params(B=1, T=64, H=1, d_k=64, d_v=64, m=32, io="f32")
    S = binding
    # null / misaligned pointers
    for i in (0, 1, 2, 3, 6):
        ptrs = list(ok); ptrs[i] = None
        assert _call_fwd(lib, good, ptrs) == 1
        ptrs[i] = 0x1004
        assert _call_fwd(lib, good, ptrs) == 1
    # unsupported shapes / dtype combinations
    assert _call_fwd(lib, gsa.Params(1, 64, 1, 96, 64, 32, io="f32"), ok) == 2
    assert _call_fwd(lib, gsa.Params(1, 64, 1, 64, 64, 48, io="f32"), ok) == 2
    assert _call_fwd(lib, gsa.Params(1, 64, 1, 64, 64, 32, io="f32", impl="tc"), ok) == 2
    # the tensor-core kernels asked for by name on a shape they do not serve: an error, not the CUDA-core kernels
    assert _call_fwd(lib, gsa.Params(1, 64, 1, 64, 64, 48, io="bf16", impl="tc"), ok) == 2
    assert _call_fwd(lib, gsa.Params(1, 64, 1, 96, 64, 64, io="bf16", impl="tc"), ok) == 2
    # invalid sizes
    assert _call_fwd(lib, gsa.Params(1, 0, 1, 64, 64, 32, io="f32"), ok) == 1
    assert _call_fwd(lib, gsa.Params(0, 64, 1, 64, 64, 32, io="f32"), ok) == 1
    # a non-linearity outside gsa_act_t
    cp = good.c()
    cp.slot_act = 5
    assert lib.gsa_fwd(ctypes.byref(cp), *[ctypes.c_void_p(x) for x in ok], ctypes.c_void_p(0x1000), 1 << 40,
                       None, None) == 1
    assert _call_fwd(lib, gsa.Params(1, 64, 1, 64, 64, 32, io="f32", slot_act="relu2"), ok, ws=0) == 3
    # workspace: missing, misaligned, too small
    assert _call_fwd(lib, good, ok, ws=0) == 3
    assert _call_fwd(lib, good, ok, ws=0x1010) == 3
    assert _call_fwd(lib, good, ok, ws_bytes=16) == 3
    assert lib.gsa_status_string(3).decode().startswith("workspace")
    # decode and bwd validate the same way
    cp = good.c()
    assert lib.gsa_decode_step(ctypes.byref(cp), *([None] * 8)) == 1
    assert lib.gsa_bwd(ctypes.byref(cp), *([None] * 16), None, 0, None, None) == 1
    assert lib.gsa_fwd(None, *([None] * 10), None, 0, None, None) == 1
    # the saved-gate pair: validated like the plain calls; a missing or short block is a workspace error
    assert lib.gsa_fwd_save_gate(ctypes.byref(cp), *([None] * 10), None, 0, None, 0, None, None) == 1
    assert lib.gsa_bwd_saved_gate(ctypes.byref(cp), *([None] * 16), None, 0, None, 0, None, None) == 1
    okp = [ctypes.c_void_p(x) for x in ok]
    assert lib.gsa_fwd_save_gate(ctypes.byref(cp), *okp, None, 0, ctypes.c_void_p(0x1000), 1 << 40, None, None) == 3
    assert lib.gsa_fwd_save_gate(ctypes.byref(cp), *okp, ctypes.c_void_p(0x1000), 16, ctypes.c_void_p(0x1000), 1 << 40,
                                 None, None) == 3


def test_binding_refuses_cpu_tensors(lib):
    import torch
    p = gsa.Params(B=1, T=64, H=1, d_k=64, d_v=64, m=32, io="f32")
    q = torch.zeros(1, 64, 1, 64)
    with pytest.raises(TypeError, match="CUDA tensor"):
        gsa.gsa_decode_step(gsa.Params(1, 1, 1, 64, 64, 32, io="f32"), q[:, 0], q[:, 0], q[:, 0],
                            torch.zeros(1, 1, 32), torch.zeros(1, 1, 32, 64), torch.zeros(1, 1, 32, 64),
                            o=torch.zeros(1, 1, 64))
