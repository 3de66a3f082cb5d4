"""ctypes binding of libgsa.so: same names and argument order as include/gsa.h."""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libgsa.so")
_lib = None

GSA_F32, GSA_BF16 = 0, 1
GSA_GATE_A, GSA_GATE_LOG_A, GSA_GATE_LOGITS, GSA_GATE_ABC = 0, 1, 2, 3
GSA_IMPL_AUTO, GSA_IMPL_SIMT, GSA_IMPL_TC = 0, 1, 2
GSA_WS_FWD, GSA_WS_BWD, GSA_WS_DECODE, GSA_WS_GATE, GSA_WS_SHARD = 0, 1, 2, 3, 4

_IMPL = {"auto": GSA_IMPL_AUTO, "simt": GSA_IMPL_SIMT, "tc": GSA_IMPL_TC}
_ACT = {"softmax": 0, "none": 1, "relu": 2, "swish": 3, "relu2": 4}   # gsa_act_t


class GsaError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = load_library().gsa_status_string(code).decode()
        super().__init__(f"{where}: {msg} (status {code})")


class _CParams(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("T", ctypes.c_int32), ("H", ctypes.c_int32),
                ("d_k", ctypes.c_int32), ("d_v", ctypes.c_int32), ("m", ctypes.c_int32),
                ("io", ctypes.c_int32), ("gate_kind", ctypes.c_int32),
                ("scale", ctypes.c_float), ("impl", ctypes.c_int32), ("tau", ctypes.c_float),
                ("slot_act", ctypes.c_int32), ("tc_operands", ctypes.c_int32), ("fuse", ctypes.c_int32),
                ("gate_dtype", ctypes.c_int32), ("feature_map", ctypes.c_int32), ("gate_broadcast", ctypes.c_int32),
                ("nseq", ctypes.c_int32),
                ("cu_seqlens", ctypes.c_void_p)]


@dataclass(frozen=True)
class Params:
    """Mirror of gsa_params_t."""
    B: int
    T: int
    H: int
    d_k: int
    d_v: int
    m: int
    io: str = "bf16"          # "f32" | "bf16"
    gate_is_log: bool = False
    scale: float = 1.0
    impl: str = "auto"        # "auto" | "simt" | "tc"
    gate_is_logits: bool = False   # the gate tensor holds x, a = sigmoid(x)^(1/tau)
    tau: float = 8.0
    slot_act: str = "softmax"      # "softmax" | "none" | "relu" | "swish" | "relu2"
    tc_operands: str = "paired"    # "paired" | "single" (tensor-core kernels: derived operands as bf16 pairs or not)
    fuse: bool = False             # tensor-core kernels: pass 1 -> softmax -> pass 2 as one kernel where the shape allows (gsa_fuse_t)
    gate_bf16: bool = False        # the gate tensor is bfloat16 (log a or logits)
    feature_map: str = "none"      # "none" | "swish": q, k, v hold pre-activations, Swish applied by the library
    gate_is_abc: bool = False      # ABC (Eq. 3-4): the gate tensor holds score logits, no decay, cumulative-softmax writes
    gate_broadcast: bool = False   # data-independent decay: the gate tensor (and dgate) is one row [H, m]
    cu_seqlens: object = None      # packed sequences: int32 CUDA tensor of nseq + 1 offsets along T (kept alive by Params)

    def c(self) -> _CParams:
        return _CParams(self.B, self.T, self.H, self.d_k, self.d_v, self.m,
                        GSA_BF16 if self.io == "bf16" else GSA_F32,
                        GSA_GATE_ABC if self.gate_is_abc else (GSA_GATE_LOGITS if self.gate_is_logits else
                                                              (GSA_GATE_LOG_A if self.gate_is_log else GSA_GATE_A)),
                        float(self.scale), _IMPL[self.impl], float(self.tau), _ACT[self.slot_act],
                        0 if self.tc_operands == "paired" else 1, 1 if self.fuse else 0,
                        GSA_BF16 if self.gate_bf16 else GSA_F32, 1 if self.feature_map == "swish" else 0,
                        1 if self.gate_broadcast else 0,
                        0 if self.cu_seqlens is None else int(self.cu_seqlens.numel()) - 1,
                        None if self.cu_seqlens is None else self.cu_seqlens.data_ptr())

    @property
    def io_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.io == "bf16" else torch.float32

    @property
    def gate_torch_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.gate_bf16 else torch.float32

    def gate_shape(self, decode=False):
        if self.gate_broadcast:
            return (self.H, self.m)
        return (self.B, self.H, self.m) if decode else (self.B, self.T, self.H, self.m)


def lib_path() -> str:
    return _LIB_PATH


def exported_symbols():
    return ["gsa_chunk_size", "gsa_workspace_bytes", "gsa_status_string", "gsa_gate_cumsum",
            "gsa_fwd", "gsa_bwd", "gsa_decode_step", "gsa_tc_selftest", "gsa_timing_begin",
            "gsa_timing_end", "gsa_fwd_noalloc", "gsa_fwd_save_gate", "gsa_bwd_saved_gate", "gsa_release_streams",
            "gsa_wait_selftest", "gsa_shard_states", "gsa_shard_combine", "gsa_out_norm_fwd",
            "gsa_out_norm_workspace_bytes", "gsa_out_norm_bwd", "gsa_dev_pair_scans"]


def load_library():
    """Load libgsa.so; there is no fallback if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2409_07146_b200.build` "
            "(nvcc, sm_100a).  The GSA layer has no non-CUDA path.")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, sz, i32 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int32
    pp = ctypes.POINTER(_CParams)
    lib.gsa_chunk_size.argtypes = [pp]
    lib.gsa_chunk_size.restype = i32
    lib.gsa_workspace_bytes.argtypes = [pp, i32]
    lib.gsa_workspace_bytes.restype = sz
    lib.gsa_status_string.argtypes = [ctypes.c_int]
    lib.gsa_status_string.restype = ctypes.c_char_p
    lib.gsa_gate_cumsum.argtypes = [pp, vp, vp, vp, vp]
    lib.gsa_gate_cumsum.restype = ctypes.c_int
    lib.gsa_fwd.argtypes = [pp] + [vp] * 10 + [vp, sz, vp, vp]
    lib.gsa_fwd.restype = ctypes.c_int
    lib.gsa_bwd.argtypes = [pp] + [vp] * 16 + [vp, sz, vp, vp]
    lib.gsa_bwd.restype = ctypes.c_int
    lib.gsa_fwd_save_gate.argtypes = [pp] + [vp] * 10 + [vp, sz, vp, sz, vp, vp]
    lib.gsa_fwd_save_gate.restype = ctypes.c_int
    lib.gsa_bwd_saved_gate.argtypes = [pp] + [vp] * 16 + [vp, sz, vp, sz, vp, vp]
    lib.gsa_bwd_saved_gate.restype = ctypes.c_int
    lib.gsa_decode_step.argtypes = [pp] + [vp] * 8
    lib.gsa_decode_step.restype = ctypes.c_int
    lib.gsa_fwd_noalloc.argtypes = [pp] + [vp] * 10 + [vp, vp]
    lib.gsa_fwd_noalloc.restype = ctypes.c_int
    lib.gsa_timing_begin.argtypes = [i32]
    lib.gsa_timing_begin.restype = ctypes.c_int
    lib.gsa_timing_end.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_char_p), i32]
    lib.gsa_timing_end.restype = i32
    lib.gsa_tc_selftest.argtypes = [i32, vp, vp, vp, vp, vp]
    lib.gsa_tc_selftest.restype = ctypes.c_int
    lib.gsa_wait_selftest.argtypes = [ctypes.c_uint32, vp, vp, vp]
    lib.gsa_wait_selftest.restype = ctypes.c_int
    lib.gsa_dev_pair_scans.argtypes = [i32]
    lib.gsa_dev_pair_scans.restype = i32
    lib.gsa_shard_states.argtypes = [pp] + [vp] * 6 + [vp, sz, vp, vp]
    lib.gsa_shard_states.restype = ctypes.c_int
    lib.gsa_shard_combine.argtypes = [pp, i32, i32, i32, i32] + [vp] * 5 + [vp]
    lib.gsa_shard_combine.restype = ctypes.c_int
    lib.gsa_out_norm_fwd.argtypes = [pp, vp, vp, ctypes.c_float, vp, vp]
    lib.gsa_out_norm_fwd.restype = ctypes.c_int
    lib.gsa_out_norm_workspace_bytes.argtypes = [pp]
    lib.gsa_out_norm_workspace_bytes.restype = sz
    lib.gsa_out_norm_bwd.argtypes = [pp, vp, vp, vp, ctypes.c_float, vp, vp, vp, sz, vp]
    lib.gsa_out_norm_bwd.restype = ctypes.c_int
    lib.gsa_release_streams.argtypes = []
    lib.gsa_release_streams.restype = ctypes.c_int
    _lib = lib
    return lib


def _ptr(t, dtype=None, shape=None, name="tensor"):
    if t is None:
        return None
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name}: expected a CUDA tensor (the library has no CPU path)")
    if not t.is_contiguous():
        raise ValueError(f"{name}: must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name}: expected {dtype}, got {t.dtype}")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name}: expected shape {tuple(shape)}, got {tuple(t.shape)}")
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(code: int, where: str):
    if code != 0:
        raise GsaError(code, where)


def gsa_chunk_size(p: Params) -> int:
    cp = p.c()
    return int(load_library().gsa_chunk_size(ctypes.byref(cp)))


def gsa_workspace_bytes(p: Params, which: int) -> int:
    cp = p.c()
    return int(load_library().gsa_workspace_bytes(ctypes.byref(cp), which))


def _workspace(p: Params, which: int, ws, device):
    need = gsa_workspace_bytes(p, which)
    if ws is None:
        ws = torch.empty(max(need, 256), dtype=torch.uint8, device=device)
    return ws, ws.numel() * ws.element_size()


def gsa_gate_cumsum(p: Params, gate, G, I):
    shp = (p.B, p.T, p.H, p.m)
    cp = p.c()
    _check(load_library().gsa_gate_cumsum(
        ctypes.byref(cp), _ptr(gate, torch.float32, shp, "gate"), _ptr(G, torch.float32, shp, "G"),
        _ptr(I, torch.float32, shp, "I"), _stream()), "gsa_gate_cumsum")


def gate_block(p: Params, device):
    """A device block of gsa_workspace_bytes(p, GSA_WS_GATE) bytes for gsa_fwd(gate_save=...) and
    gsa_bwd(gate_saved=...)."""
    return torch.empty(gsa_workspace_bytes(p, GSA_WS_GATE), dtype=torch.uint8, device=device)


def gsa_fwd(p: Params, q, k, v, gate, K0=None, V0=None, o=None, ok_save=None, KT=None, VT=None,
            ws=None, dev_status=None, gate_save=None):
    """Enqueue the forward on the current stream.  `o` (and `ws`) are allocated with torch when
    not given.  With gate_save (see gate_block) the call is gsa_fwd_save_gate.  Returns o."""
    io = p.io_dtype
    qk, vv, mm = (p.B, p.T, p.H, p.d_k), (p.B, p.T, p.H, p.d_v), (p.B, p.T, p.H, p.m)
    sk, sv = (p.B, p.H, p.m, p.d_k), (p.B, p.H, p.m, p.d_v)
    if o is None:
        o = torch.empty(vv, dtype=io, device=q.device)
    ws, ws_bytes = _workspace(p, GSA_WS_FWD, ws, q.device)
    cp = p.c()
    head = (ctypes.byref(cp), _ptr(q, io, qk, "q"), _ptr(k, io, qk, "k"), _ptr(v, io, vv, "v"),
            _ptr(gate, p.gate_torch_dtype, p.gate_shape(), "gate"), _ptr(K0, torch.float32, sk, "K0"),
            _ptr(V0, torch.float32, sv, "V0"), _ptr(o, io, vv, "o"),
            _ptr(ok_save, torch.float32, mm, "ok_save"), _ptr(KT, torch.float32, sk, "KT"),
            _ptr(VT, torch.float32, sv, "VT"))
    tail = (_ptr(ws, None, None, "ws"), ws_bytes, _stream(), _ptr(dev_status, torch.int32, None, "dev_status"))
    if gate_save is None:
        _check(load_library().gsa_fwd(*head, *tail), "gsa_fwd")
    else:
        _check(load_library().gsa_fwd_save_gate(*head, _ptr(gate_save, None, None, "gate_save"),
                                                gate_save.numel() * gate_save.element_size(), *tail),
               "gsa_fwd_save_gate")
    return o


def gsa_bwd(p: Params, q, k, v, gate, dO, K0=None, V0=None, ok_saved=None, dKT=None, dVT=None,
            dq=None, dk=None, dv=None, dgate=None, dK0=None, dV0=None, ws=None, dev_status=None,
            gate_saved=None):
    """Enqueue the backward on the current stream.  With gate_saved (the block a forward with the
    same params and gate filled) the call is gsa_bwd_saved_gate.  Returns (dq, dk, dv, dgate)."""
    io = p.io_dtype
    qk, vv, mm = (p.B, p.T, p.H, p.d_k), (p.B, p.T, p.H, p.d_v), (p.B, p.T, p.H, p.m)
    sk, sv = (p.B, p.H, p.m, p.d_k), (p.B, p.H, p.m, p.d_v)
    dev = q.device
    dq = torch.empty(qk, dtype=io, device=dev) if dq is None else dq
    dk = torch.empty(qk, dtype=io, device=dev) if dk is None else dk
    dv = torch.empty(vv, dtype=io, device=dev) if dv is None else dv
    dgate = torch.empty(p.gate_shape(), dtype=torch.float32, device=dev) if dgate is None else dgate
    ws, ws_bytes = _workspace(p, GSA_WS_BWD, ws, dev)
    cp = p.c()
    head = (ctypes.byref(cp), _ptr(q, io, qk, "q"), _ptr(k, io, qk, "k"), _ptr(v, io, vv, "v"),
            _ptr(gate, p.gate_torch_dtype, p.gate_shape(), "gate"), _ptr(K0, torch.float32, sk, "K0"),
            _ptr(V0, torch.float32, sv, "V0"), _ptr(ok_saved, torch.float32, mm, "ok_saved"),
            _ptr(dO, io, vv, "dO"), _ptr(dKT, torch.float32, sk, "dKT"),
            _ptr(dVT, torch.float32, sv, "dVT"), _ptr(dq, io, qk, "dq"), _ptr(dk, io, qk, "dk"),
            _ptr(dv, io, vv, "dv"), _ptr(dgate, torch.float32, p.gate_shape(), "dgate"),
            _ptr(dK0, torch.float32, sk, "dK0"), _ptr(dV0, torch.float32, sv, "dV0"))
    tail = (_ptr(ws, None, None, "ws"), ws_bytes, _stream(), _ptr(dev_status, torch.int32, None, "dev_status"))
    if gate_saved is None:
        _check(load_library().gsa_bwd(*head, *tail), "gsa_bwd")
    else:
        _check(load_library().gsa_bwd_saved_gate(*head, _ptr(gate_saved, None, None, "gate_saved"),
                                                 gate_saved.numel() * gate_saved.element_size(), *tail),
               "gsa_bwd_saved_gate")
    return dq, dk, dv, dgate


def gsa_decode_step(p: Params, q, k, v, gate, Kstate, Vstate, o=None):
    """One recurrent step for p.B sequences; Kstate/Vstate are updated in place.  Returns o."""
    io = p.io_dtype
    qk, vv, mm = (p.B, p.H, p.d_k), (p.B, p.H, p.d_v), (p.B, p.H, p.m)
    if o is None:
        o = torch.empty(vv, dtype=io, device=q.device)
    cp = p.c()
    _check(load_library().gsa_decode_step(
        ctypes.byref(cp), _ptr(q, io, qk, "q"), _ptr(k, io, qk, "k"), _ptr(v, io, vv, "v"),
        _ptr(gate, p.gate_torch_dtype, p.gate_shape(decode=True), "gate"),
        _ptr(Kstate, torch.float32, (p.B, p.H, p.m, p.d_k), "Kstate"),
        _ptr(Vstate, torch.float32, (p.B, p.H, p.m, p.d_v), "Vstate"), _ptr(o, io, vv, "o"),
        _stream()), "gsa_decode_step")
    return o


def gsa_tc_selftest(mode: int, X, Y, dev_status=None):
    """Tensor-core building-block self-test: X, Y 128 x 128 bf16; returns D (fp32)."""
    n = 128 if (mode <= 1 or mode >= 4) else 64
    D = torch.zeros(128, n, dtype=torch.float32, device=X.device)
    _check(load_library().gsa_tc_selftest(
        mode, _ptr(X, torch.bfloat16, (128, 128), "X"), _ptr(Y, torch.bfloat16, (128, 128), "Y"),
        _ptr(D, torch.float32, None, "D"), _stream(), _ptr(dev_status, torch.int32, None, "dev_status")),
        "gsa_tc_selftest")
    return D


def gsa_wait_selftest(limit_us: int, dev_status, waited_us=None):
    """One CTA waits limit_us microseconds on an mbarrier that nothing signals, gives up and writes
    GSA_ERR_TIMEOUT to dev_status (int32 device tensor); waited_us (uint32/int32 device tensor, optional)
    receives the time it waited."""
    _check(load_library().gsa_wait_selftest(int(limit_us), _stream(), _ptr(dev_status, torch.int32, None, "dev_status"),
                                            _ptr(waited_us, torch.int32, None, "waited_us")), "gsa_wait_selftest")


def gsa_dev_pair_scans(enable: bool) -> bool:
    """Development switch: the backward's reversed scans as two pair kernels (True, the default) or as four
    single ones (False), for later gsa_bwd calls of this process.  Returns the previous setting."""
    return bool(load_library().gsa_dev_pair_scans(1 if enable else 0))


def gsa_shard_states(p: Params, k, v, gate, ws=None, dev_status=None):
    """End memories of a sequence shard run from empty memories, and the shard's log-decay.
    Returns (KT [B,H,m,d_k], VT [B,H,m,d_v], logdecay [B,H,m])."""
    io = p.io_dtype
    KT = torch.empty(p.B, p.H, p.m, p.d_k, dtype=torch.float32, device=k.device)
    VT = torch.empty(p.B, p.H, p.m, p.d_v, dtype=torch.float32, device=k.device)
    ld = torch.empty(p.B, p.H, p.m, dtype=torch.float32, device=k.device)
    ws, nbytes = _workspace(p, GSA_WS_SHARD, ws, k.device)
    cp = p.c()
    _check(load_library().gsa_shard_states(
        ctypes.byref(cp), _ptr(k, io, (p.B, p.T, p.H, p.d_k), "k"), _ptr(v, io, (p.B, p.T, p.H, p.d_v), "v"),
        _ptr(gate, torch.float32, (p.B, p.T, p.H, p.m), "gate"), _ptr(KT), _ptr(VT), _ptr(ld),
        _ptr(ws, torch.uint8, None, "ws"), nbytes, _stream(), _ptr(dev_status, torch.int32, None, "dev_status")),
        "gsa_shard_states")
    return KT, VT, ld


def gsa_shard_combine(p: Params, d: int, rank: int, logdecay_all, local_all, S0=None, reverse=False, want_final=False):
    """From the gathered shard results (logdecay_all [R,B,H,m], local_all [R,B,H,m,d], rank order) to the
    memories entering shard `rank` (and, with want_final, those leaving the last / first shard)."""
    R = logdecay_all.shape[0]
    start = torch.empty(p.B, p.H, p.m, d, dtype=torch.float32, device=local_all.device)
    final = torch.empty_like(start) if want_final else None
    cp = p.c()
    _check(load_library().gsa_shard_combine(
        ctypes.byref(cp), d, R, rank, 1 if reverse else 0,
        _ptr(logdecay_all, torch.float32, (R, p.B, p.H, p.m), "logdecay_all"),
        _ptr(local_all, torch.float32, (R, p.B, p.H, p.m, d), "local_all"),
        _ptr(S0, torch.float32, (p.B, p.H, p.m, d), "S0"), _ptr(start), _ptr(final), _stream()), "gsa_shard_combine")
    return (start, final) if want_final else start


def gsa_out_norm_fwd(p: Params, o, weight=None, eps=1e-6, y=None):
    """y = weight * Swish(o) / sqrt(mean(Swish(o)^2) + eps) over the H d_v values of every token."""
    io = p.io_dtype
    shp = (p.B, p.T, p.H, p.d_v)
    if y is None:
        y = torch.empty(shp, dtype=io, device=o.device)
    cp = p.c()
    _check(load_library().gsa_out_norm_fwd(ctypes.byref(cp), _ptr(o, io, shp, "o"),
                                           _ptr(weight, torch.float32, (p.H * p.d_v,), "weight"), float(eps),
                                           _ptr(y, io, shp, "y"), _stream()), "gsa_out_norm_fwd")
    return y


def gsa_out_norm_bwd(p: Params, o, dy, weight=None, eps=1e-6, want_dweight=True):
    """Gradients of gsa_out_norm_fwd: returns (d_o, dweight or None)."""
    io = p.io_dtype
    shp = (p.B, p.T, p.H, p.d_v)
    d_o = torch.empty(shp, dtype=io, device=o.device)
    dw = torch.empty(p.H * p.d_v, dtype=torch.float32, device=o.device) if want_dweight else None
    cp = p.c()
    nbytes = int(load_library().gsa_out_norm_workspace_bytes(ctypes.byref(cp))) if want_dweight else 0
    ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=o.device)
    _check(load_library().gsa_out_norm_bwd(ctypes.byref(cp), _ptr(o, io, shp, "o"), _ptr(dy, io, shp, "dy"),
                                           _ptr(weight, torch.float32, (p.H * p.d_v,), "weight"), float(eps),
                                           _ptr(d_o, io, shp, "d_o"), _ptr(dw), _ptr(ws), nbytes, _stream()), "gsa_out_norm_bwd")
    return d_o, dw


def gsa_release_streams():
    """Destroy the calling thread's internal streams and events on the current device."""
    _check(load_library().gsa_release_streams(), "gsa_release_streams")


def gsa_timing_begin(capacity: int = 4096):
    _check(load_library().gsa_timing_begin(capacity), "gsa_timing_begin")


def gsa_timing_end(capacity: int = 4096):
    """Returns [(label, milliseconds)] of the kernels timed since gsa_timing_begin."""
    ms = (ctypes.c_float * capacity)()
    labels = (ctypes.c_char_p * capacity)()
    n = load_library().gsa_timing_end(ms, labels, capacity)
    if n < 0:
        raise RuntimeError("gsa_timing_end failed")
    return [(labels[i].decode(), float(ms[i])) for i in range(n)]


GSA_NOALLOC_MAX_WORKSPACE_BYTES = 32 << 20   # mirror of the macro in include/gsa.h


def gsa_fwd_noalloc(p: Params, q, k, v, gate, o, K0=None, V0=None, ok_save=None, KT=None, VT=None,
                    dev_status=None):
    """gsa_fwd for callers that cannot allocate device memory: the scratch is a fixed array
    inside the library (32 MiB per GPU), so the caller passes inputs and outputs only -- `o`
    must be given, nothing is allocated here either.  Calls that overlap on the GPU share
    that array and race; shapes that need more scratch raise GsaError (workspace)."""
    io = p.io_dtype
    qk, vv, mm = (p.B, p.T, p.H, p.d_k), (p.B, p.T, p.H, p.d_v), (p.B, p.T, p.H, p.m)
    sk, sv = (p.B, p.H, p.m, p.d_k), (p.B, p.H, p.m, p.d_v)
    cp = p.c()
    _check(load_library().gsa_fwd_noalloc(
        ctypes.byref(cp), _ptr(q, io, qk, "q"), _ptr(k, io, qk, "k"), _ptr(v, io, vv, "v"),
        _ptr(gate, p.gate_torch_dtype, p.gate_shape(), "gate"), _ptr(K0, torch.float32, sk, "K0"),
        _ptr(V0, torch.float32, sv, "V0"), _ptr(o, io, vv, "o"),
        _ptr(ok_save, torch.float32, mm, "ok_save"), _ptr(KT, torch.float32, sk, "KT"),
        _ptr(VT, torch.float32, sv, "VT"), _stream(),
        _ptr(dev_status, torch.int32, None, "dev_status")), "gsa_fwd_noalloc")
    return o
